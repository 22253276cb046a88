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


# ---- boundary-aware comparison of integer codes with the plain fp64 definition -------------------
# A code produced in binary32 (the library's operation-by-operation arithmetic) may differ from the
# code of the fp64 definition only where the fp64 pre-rounding value v sits next to the rounding
# boundary m + 1/2 between the two codes.  `rel` is the relative error the binary32 chain can carry:
#   Q(X_scaled), Eq. 3:  four binary32 operations (6e-8 each), one exp32 (2e-7, pinned against libm)
#     whose argument fsub(cs_last, cs_i) is rounded (6e-8 |arg|, |arg| < 8 wherever the code is not 0)
#     -> below 1.0e-6; the comparison uses 4e-6.
#   Q(State), Eq. 4:  fdiv(1, s_h) and one fmul -> 1.2e-7; the comparison uses 4e-6.
#   Mq (per-row Eq. 1 of the masked operand):  the numerator carries up to 15 per-token decays
#     (15 exp32 + 14 fmul = 3.84e-6) or two exp32 with rounded arguments (< 3e-6) plus three fmul; the
#     row maximum it is divided by carries the same; fdiv and two fmul on top: below 8.1e-6; the
#     comparison uses 1e-5.
WINDOW_ABS = 1e-6


def census(code, v, rel):
    """code: integer codes under test; v: fp64 pre-rounding values of the definition.
    Returns (differing fraction, largest |code - rint(v)|, number of differing entries outside the
    window rel |v| + 1e-6 around a rounding boundary)."""
    v = np.asarray(v, np.float64)
    want = np.clip(np.rint(v), -127, 127)
    diff = np.asarray(code, np.float64) - want
    bad = diff != 0
    if not bad.any():
        return 0.0, 0, 0
    vb = v[bad]
    dist = np.abs(np.abs(vb - np.floor(vb)) - 0.5)        # distance of v to the nearest m + 1/2
    outside = int(np.count_nonzero(dist > rel * np.abs(vb) + WINDOW_ABS))
    return float(bad.mean()), int(np.abs(diff).max()), outside


def half_neighbours(a, b):
    """True where the binary16 values a and b (given as float64) are equal or adjacent."""
    a16 = np.asarray(a, np.float64).astype(np.float16)
    b16 = np.asarray(b, np.float64).astype(np.float16)
    up = np.nextafter(a16, np.float16(np.inf))
    dn = np.nextafter(a16, np.float16(-np.inf))
    return (a16 == b16) | (up == b16) | (dn == b16)
