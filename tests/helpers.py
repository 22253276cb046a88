"""Shared test helpers: small workloads and dequantisation (no method arithmetic
beyond multiplying an int8 code by its step size)."""
import numpy as np

from paper_2608_21952_b200.inputs import SSDConfig, make_prefill

TINY = SSDConfig("tiny", 2, 32, 4, 8, 16, 2, 8, 0.05, 20.0, 11)
TWO_BLOCK = SSDConfig("two_block", 1, 256, 2, 8, 16, 1, 128, 0.05, 20.0, 12)


def dequant(cfg, q):
    """int8 codes times step sizes, fp64."""
    xh = q["xq"].astype(np.float64) * q["s_x"].astype(np.float64).reshape(cfg.nheads, cfg.headdim)
    Bh = q["Bq"].astype(np.float64) * q["s_B"].astype(np.float64)[:, None]
    Ch = q["Cq"].astype(np.float64) * q["s_C"].astype(np.float64)[:, None]
    return xh, Bh, Ch


def rms(a):
    return float(np.sqrt(np.mean(np.asarray(a, np.float64) ** 2)))


def group_of(cfg, h):
    return h // (cfg.nheads // cfg.ngroups)
