"""CPU oracle of the INT8 SSD layer: test infrastructure, never imported by the CUDA path."""
