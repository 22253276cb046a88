"""ctypes front end of the CPU oracle (test infrastructure).

Only tests, the smoke check and the CPU-baseline leg of the benchmark import
this module.  It takes and returns numpy arrays and forwards to the functions
of ssdi8_oracle.cpp; it contains no arithmetic of its own beyond dtype casts.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())


class Dims(C.Structure):
    _fields_ = [(k, C.c_int32) for k in
                ("batch", "seqlen", "nheads", "headdim", "dstate", "ngroups", "chunk")]


class Taps(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in
                ("cs", "acc_cb", "CBq", "Xsq", "acc_st", "loc", "prev", "hq",
                 "acc_off", "rowmax", "Mq", "acc_diag")]


def dims_of(cfg) -> Dims:
    return Dims(cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim, cfg.dstate, cfg.ngroups, cfg.chunk)


def _p(a):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _i8(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int8)


def num_threads() -> int:
    return int(_lib.orc_num_threads())


def round_half(v):
    """Round-to-nearest-even to IEEE binary16, returned as float64 (the oracle's own routine)."""
    v = np.ascontiguousarray(v, np.float64)
    _lib.orc_round_half.restype = C.c_double
    _lib.orc_round_half.argtypes = [C.c_double]
    return np.array([_lib.orc_round_half(float(x)) for x in v.ravel()]).reshape(v.shape)


def exp32(x):
    x = _f32(x)
    out = np.empty_like(x)
    _lib.orc_exp32(_p(x), _p(out), C.c_int64(x.size))
    return out


def quantize(v, R, Ch, I, scale=None, mode=1, want_out=True):
    """Eq. 1 on the view v[R][Ch][I]; returns (q int8 of v's shape or None, scale[Ch])."""
    v = _f32(v)
    assert v.size == R * Ch * I
    scale = np.zeros(Ch, np.float32) if scale is None else _f32(scale).copy()
    out = np.empty(v.shape, np.int8) if want_out else None
    _lib.orc_quantize(_p(v), C.c_int64(R), C.c_int64(Ch), C.c_int64(I), _p(scale),
                      C.c_int(mode), _p(out))
    return out, scale


def ssd_recurrence(cfg, x, B, Cm, dt, A, D=None, corr=None, init=None):
    d = dims_of(cfg)
    x, B, Cm, dt, A, D, corr, init = map(_f64, (x, B, Cm, dt, A, D, corr, init))
    y = np.empty((cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim), np.float64)
    fin = np.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), np.float64)
    _lib.orc_ssd_recurrence(C.byref(d), _p(x), _p(B), _p(Cm), _p(dt), _p(A), _p(D), _p(corr),
                            _p(init), _p(y), _p(fin))
    return y, fin


def ssd_chunked(cfg, x, B, Cm, dt, A, D=None, corr=None, init=None):
    d = dims_of(cfg)
    x, B, Cm, dt, A, D, corr, init = map(_f64, (x, B, Cm, dt, A, D, corr, init))
    y = np.empty((cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim), np.float64)
    fin = np.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), np.float64)
    _lib.orc_ssd_chunked(C.byref(d), _p(x), _p(B), _p(Cm), _p(dt), _p(A), _p(D), _p(corr),
                         _p(init), _p(y), _p(fin))
    return y, fin


def chunk_cumsum(cfg, dt, A):
    d = dims_of(cfg)
    dt, A = _f32(dt), _f32(A)
    cs = np.empty((cfg.batch, cfg.nheads, cfg.nchunks, cfg.chunk), np.float32)
    _lib.orc_chunk_cumsum(C.byref(d), _p(dt), _p(A), _p(cs))
    return cs


def chunk_decay(cfg, cs):
    d = dims_of(cfg)
    cs = _f32(cs)
    g = np.empty((cfg.batch, cfg.nheads, cfg.nchunks), np.float32)
    _lib.orc_chunk_decay(C.byref(d), _p(cs), _p(g))
    return g


def chunk_bmm(cfg, Cq, Bq, s_C, s_B, s_cb):
    d = dims_of(cfg)
    shp = (cfg.batch, cfg.nchunks, cfg.ngroups, cfg.chunk, cfg.chunk)
    acc = np.empty(shp, np.int32)
    cbq = np.empty(shp, np.int8) if s_cb is not None else None
    _lib.orc_chunk_bmm(C.byref(d), _p(_i8(Cq)), _p(_i8(Bq)), _p(_f32(s_C)), _p(_f32(s_B)),
                       _p(_f32(s_cb)), _p(acc), _p(cbq))
    return acc, cbq


def chunk_state(cfg, xq, Bq, s_x, s_xs, s_B, dt, cs):
    d = dims_of(cfg)
    xsq = np.empty((cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim), np.int8)
    shp = (cfg.batch, cfg.nchunks, cfg.nheads, cfg.headdim, cfg.dstate)
    acc = np.empty(shp, np.int32)
    loc = np.empty(shp, np.float32)
    _lib.orc_chunk_state(C.byref(d), _p(_i8(xq)), _p(_i8(Bq)), _p(_f32(s_x)), _p(_f32(s_xs)),
                         _p(_f32(s_B)), _p(_f32(dt)), _p(_f32(cs)), _p(xsq), _p(acc), _p(loc))
    return xsq, acc, loc


def state_passing(cfg, loc, gamma, init=None, s_h=None):
    d = dims_of(cfg)
    shp = (cfg.batch, cfg.nchunks, cfg.nheads, cfg.headdim, cfg.dstate)
    loc = _f32(loc)
    prev = np.empty(shp, np.float32)
    fin = np.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), np.float32)
    hq = np.empty(shp, np.int8) if s_h is not None else None
    _lib.orc_state_passing(C.byref(d), _p(loc), _p(_f32(gamma)), _p(_f32(init)), _p(_f32(s_h)),
                           _p(prev), _p(fin), _p(hq))
    return prev, fin, hq


def calibrate(cfg, xq, Bq, Cq, s_x, s_B, s_C, dt, A, init=None):
    d = dims_of(cfg)
    s_xs = np.empty(cfg.channels, np.float32)
    s_cb = np.empty(cfg.ngroups, np.float32)
    s_h = np.empty(cfg.channels, np.float32)
    _lib.orc_calibrate(C.byref(d), _p(_i8(xq)), _p(_i8(Bq)), _p(_i8(Cq)), _p(_f32(s_x)),
                       _p(_f32(s_B)), _p(_f32(s_C)), _p(_f32(dt)), _p(_f32(A)), _p(_f32(init)),
                       _p(s_xs), _p(s_cb), _p(s_h))
    return s_xs, s_cb, s_h


TAP_SPECS = {
    # name: (shape function, dtype)
    "cs": (lambda c: (c.batch, c.nheads, c.nchunks, c.chunk), np.float32),
    "acc_cb": (lambda c: (c.batch, c.nchunks, c.ngroups, c.chunk, c.chunk), np.int32),
    "CBq": (lambda c: (c.batch, c.nchunks, c.ngroups, c.chunk, c.chunk), np.int8),
    "Xsq": (lambda c: (c.batch, c.seqlen, c.nheads, c.headdim), np.int8),
    "acc_st": (lambda c: (c.batch, c.nchunks, c.nheads, c.headdim, c.dstate), np.int32),
    "loc": (lambda c: (c.batch, c.nchunks, c.nheads, c.headdim, c.dstate), np.float32),
    "prev": (lambda c: (c.batch, c.nchunks, c.nheads, c.headdim, c.dstate), np.float32),
    "hq": (lambda c: (c.batch, c.nchunks, c.nheads, c.headdim, c.dstate), np.int8),
    "acc_off": (lambda c: (c.batch, c.seqlen, c.nheads, c.headdim), np.int32),
    "rowmax": (lambda c: (c.batch, c.seqlen, c.nheads), np.float32),
    "Mq": (lambda c: (c.batch, c.nchunks, c.nheads, c.chunk, c.chunk), np.int8),
    "acc_diag": (lambda c: (c.batch, c.seqlen, c.nheads, c.headdim), np.int32),
}


FLAG_INT8_STATE = 2
FLAG_FP16_OPERAND = 1   # the paper's FP16 ChunkScan2 operand (no per-row re-quantisation)


def state_passing_int8(cfg, acc_st, gamma, init, s_xs, s_B, s_h):
    """Eq. 4 + Eq. 7: persistent INT8 states with the fixed-point decay.  Returns (hq int8, final fp32)."""
    d = dims_of(cfg)
    shp = (cfg.batch, cfg.nchunks, cfg.nheads, cfg.headdim, cfg.dstate)
    acc = np.ascontiguousarray(acc_st, dtype=np.int32)
    hq = np.empty(shp, np.int8)
    fin = np.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), np.float32)
    _lib.orc_state_passing_int8(C.byref(d), _p(acc), _p(_f32(gamma)), _p(_f32(init)), _p(_f32(s_xs)),
                                _p(_f32(s_B)), _p(_f32(s_h)), _p(hq), _p(fin))
    return hq, fin


def ssdi8_fwd(cfg, xq, Bq, Cq, s_x, s_B, s_C, dt, A, D, corr, s_xs, s_cb, s_h, init=None,
              taps=(), flags=0):
    """L2 forward.  Returns (y fp64, final fp32, {tap name: array})."""
    d = dims_of(cfg)
    y = np.empty((cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim), np.float64)
    fin = np.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), np.float32)
    t = Taps()
    out = {}
    for name in taps:
        shp, dt_ = TAP_SPECS[name]
        out[name] = np.zeros(shp(cfg), dt_)
        setattr(t, name, out[name].ctypes.data)
    _lib.orc_ssdi8_fwd(C.byref(d), _p(_i8(xq)), _p(_i8(Bq)), _p(_i8(Cq)), _p(_f32(s_x)),
                       _p(_f32(s_B)), _p(_f32(s_C)), _p(_f32(dt)), _p(_f32(A)), _p(_f32(D)),
                       _p(_f32(corr)), _p(_f32(s_xs)), _p(_f32(s_cb)), _p(_f32(s_h)),
                       _p(_f32(init)), _p(y), _p(fin), C.byref(t), C.c_uint32(flags))
    return y, fin, out


def ssd_step(cfg, xq, s_x, Bq, s_B, Cq, s_C, dt, A, D, corr, state):
    """L3: updates `state` (fp64, [b,H,P,N]) in place, returns y fp64 [b,H,P]."""
    d = dims_of(cfg)
    assert state.dtype == np.float64 and state.flags["C_CONTIGUOUS"]
    y = np.empty((cfg.batch, cfg.nheads, cfg.headdim), np.float64)
    _lib.orc_ssd_step(C.byref(d), _p(_i8(xq)), _p(_f32(s_x)), _p(_i8(Bq)), _p(_f32(s_B)),
                      _p(_i8(Cq)), _p(_f32(s_C)), _p(_f32(dt)), _p(_f32(A)), _p(_f32(D)),
                      _p(_f32(corr)), _p(state), _p(y))
    return y


def mean_correction(Y, Yq, eta):
    Y, Yq = _f64(Y), _f64(Yq)
    rows, Ch = Y.shape
    c = np.empty(Ch, np.float64)
    _lib.orc_mean_correction(_p(Y), _p(Yq), C.c_int64(rows), C.c_int64(Ch), C.c_double(eta), _p(c))
    return c


def prepare_quantized(cfg, t, init=None):
    """Quantises a generated fp32 layer input (Eq. 1: x per channel, B and C per
    group) and calibrates the internal step sizes.  Returns a dict with every
    array the L2 forward takes."""
    T = cfg.tokens
    xq, s_x = quantize(t["x"], T, cfg.channels, 1, mode=1)
    Bq, s_B = quantize(t["B"], T, cfg.ngroups, cfg.dstate, mode=1)
    Cq, s_C = quantize(t["C"], T, cfg.ngroups, cfg.dstate, mode=1)
    s_xs, s_cb, s_h = calibrate(cfg, xq, Bq, Cq, s_x, s_B, s_C, t["dt"], t["A"], init)
    return dict(xq=xq, Bq=Bq, Cq=Cq, s_x=s_x, s_B=s_B, s_C=s_C, dt=t["dt"], A=t["A"], D=t["D"],
                s_xs=s_xs, s_cb=s_cb, s_h=s_h, init=init)


# ---------------------------------------------------------------------------- plain definitions
def chunk_state_plain(cfg, xq, s_x, s_xs, dt, cs):
    """Eq. 3 from its definition in fp64.  Returns (v = X_scaled / s_xs as float64, its code int8)."""
    d = dims_of(cfg)
    shp = (cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim)
    v = np.empty(shp, np.float64)
    code = np.empty(shp, np.int8)
    _lib.orc_chunk_state_plain(C.byref(d), _p(_i8(xq)), _p(_f32(s_x)), _p(_f32(s_xs)), _p(_f32(dt)),
                               _p(_f32(cs)), _p(v), _p(code))
    return v, code


def state_codes_plain(cfg, S, s_h):
    """Eq. 4 from its definition in fp64: (v = State / s_h as float64, its code int8); S [b,c,H,P,N]."""
    d = dims_of(cfg)
    S = _f32(S)
    v = np.empty(S.shape, np.float64)
    code = np.empty(S.shape, np.int8)
    _lib.orc_state_codes_plain(C.byref(d), _p(S), _p(_f32(s_h)), _p(v), _p(code))
    return v, code


def chunk_scan_plain(cfg, xq, Cq, CBq, hq, s_x, s_C, s_cb, s_h, dt, cs, D=None, corr=None, flags=0,
                     want_operand=True):
    """Algorithm 2 modules 5 and 6 from their definitions in fp64 (one libm exp per element).
    Returns y and a dict with M (real masked operand [b,c,H,Q,Q]), sM [b,L,H] and Mq (int8 mode)."""
    d = dims_of(cfg)
    b, L, H, P, Q, c = cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim, cfg.chunk, cfg.nchunks
    y = np.empty((b, L, H, P), np.float64)
    out = {}
    if want_operand:
        out["M"] = np.empty((b, c, H, Q, Q), np.float64)
        if not (flags & FLAG_FP16_OPERAND):
            out["sM"] = np.empty((b, L, H), np.float64)
            out["Mq"] = np.empty((b, c, H, Q, Q), np.int8)
    _lib.orc_chunk_scan_plain(C.byref(d), _p(_i8(xq)), _p(_i8(Cq)), _p(_i8(CBq)), _p(_i8(hq)),
                              _p(_f32(s_x)), _p(_f32(s_C)), _p(_f32(s_cb)), _p(_f32(s_h)), _p(_f32(dt)),
                              _p(_f32(cs)), _p(_f32(D)), _p(_f32(corr)), _p(out.get("M")),
                              _p(out.get("sM")), _p(out.get("Mq")), _p(y), C.c_uint32(flags))
    return y, out


def ssdi8_fwd_plain(cfg, xq, Bq, Cq, s_x, s_B, s_C, dt, A, D, corr, s_xs, s_cb, s_h, init=None, flags=0):
    """The whole forward from the plain definitions (fp64 throughout).  Returns (y, final) float64."""
    d = dims_of(cfg)
    y = np.empty((cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim), np.float64)
    fin = np.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), np.float64)
    _lib.orc_ssdi8_fwd_plain(C.byref(d), _p(_i8(xq)), _p(_i8(Bq)), _p(_i8(Cq)), _p(_f32(s_x)),
                             _p(_f32(s_B)), _p(_f32(s_C)), _p(_f32(dt)), _p(_f32(A)), _p(_f32(D)),
                             _p(_f32(corr)), _p(_f32(s_xs)), _p(_f32(s_cb)), _p(_f32(s_h)),
                             _p(_f32(init)), _p(y), _p(fin), C.c_uint32(flags))
    return y, fin


def prop1_mse(cfg, x, dt, cs):
    """Proposition 1 diagnostic: (per-element MSE of Q(X_scaled), per-element MSE of Q(X) (.) LUT_state,
    zero fraction of Q(X_scaled), the second error summed over the l axis of a chunk as in the proof)."""
    d = dims_of(cfg)
    out = np.empty(4, np.float64)
    _lib.orc_prop1_mse(C.byref(d), _p(_f32(x)), _p(_f32(dt)), _p(_f32(cs)), _p(out))
    return tuple(float(v) for v in out)


def chunk_scan_fp16_operand(cfg, xq, Cq, CBq, hq, s_x, s_C, s_cb, s_h, dt, cs, D=None, corr=None):
    """The binary32-defined FP16 operand of orc_chunk_scan (flags bit 0) and its y: (y, M16 [b,c,H,Q,Q])."""
    d = dims_of(cfg)
    b, L, H, P, Q, c = cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim, cfg.chunk, cfg.nchunks
    y = np.empty((b, L, H, P), np.float64)
    m16 = np.empty((b, c, H, Q, Q), np.float64)
    _lib.orc_chunk_scan(C.byref(d), _p(_i8(xq)), _p(_i8(Cq)), _p(_i8(CBq)), _p(_i8(hq)), _p(_f32(s_x)),
                        _p(_f32(s_C)), _p(_f32(s_cb)), _p(_f32(s_h)), _p(_f32(dt)), _p(_f32(cs)),
                        _p(_f32(D)), _p(_f32(corr)), None, None, None, None, _p(y),
                        C.c_uint32(FLAG_FP16_OPERAND), _p(m16))
    return y, m16


def softplus_dt(dt_raw, bias=None, plain=False):
    """dt = softplus(dt_raw + bias[h]) (Algorithm 2 module 1), dt_raw [..., H] -> float32.  plain=True:
    the libm definition in fp64; otherwise the library's operation-by-operation binary64 sequence."""
    x = _f32(dt_raw)
    H = x.shape[-1]
    out = np.empty_like(x)
    fn = _lib.orc_softplus_dt_plain if plain else _lib.orc_softplus_dt
    fn(_p(x), _p(_f32(bias)), C.c_int64(x.size // H), C.c_int64(H), _p(out))
    return out
