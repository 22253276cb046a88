"""B200 (sm_100a) INT8 State Space Duality layer: Python front end of libssdi8.

`paper_2608_21952_b200.inputs` (seeded synthetic workloads) imports without the
CUDA library; everything else lives in `paper_2608_21952_b200.binding`, which
loads the C-ABI library and fails loudly if it is missing.
"""
__all__ = ["inputs", "binding", "build"]
