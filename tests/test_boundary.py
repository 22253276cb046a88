"""Host-side checks of the C-ABI boundary: the library loads, exports every symbol the
header declares, and rejects bad arguments with error codes before touching a device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2608_21952_b200 import build
    return C.CDLL(build.build())


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ssdi8.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ssdi8_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    syms = declared_symbols()
    assert {"ssdi8_quantize_act", "ssdi8_chunk_scan_fwd", "ssdi8_state_passing", "ssdi8_ssd_step",
            "ssdi8_workspace_bytes", "ssdi8_status_string", "ssdi8_calibrate"} <= set(syms)
    for s in syms:
        assert hasattr(lib, s), s


def test_binding_names_match_header():
    from paper_2608_21952_b200 import binding
    for s in declared_symbols():
        assert callable(getattr(binding, s)), s


def test_status_strings(lib):
    lib.ssdi8_status_string.restype = C.c_char_p
    seen = set()
    for code in range(0, -9, -1):
        s = lib.ssdi8_status_string(code)
        assert s and s != b"unknown status"
        seen.add(s)
    assert len(seen) == 9
    assert lib.ssdi8_status_string(-99) == b"unknown status"


def test_workspace_bytes_and_shape_rules():
    from paper_2608_21952_b200 import binding as bd
    from paper_2608_21952_b200.inputs import CONFIGS
    for name in ("cfg0", "cfg1", "cfg2", "cfg3"):
        cfg = CONFIGS[name]
        n = bd.ssdi8_workspace_bytes(bd.dims_of(cfg))
        nst = cfg.batch * cfg.nchunks * cfg.nheads * cfg.headdim * cfg.dstate
        assert n >= 5 * nst and n % 256 == 0
    bad = [CONFIGS["cfg0"].replace(headdim=32), CONFIGS["cfg0"].replace(dstate=96),
           CONFIGS["cfg0"].replace(chunk=48), CONFIGS["cfg0"].replace(seqlen=500),
           CONFIGS["cfg0"].replace(nheads=4, ngroups=3), CONFIGS["cfg0"].replace(batch=0)]
    for cfg in bad:
        assert bd.ssdi8_workspace_bytes(bd.dims_of(cfg)) == 0


def test_host_side_argument_errors():
    """Null pointers, bad shapes, bad alignment and short workspaces are rejected on the host,
    before any CUDA call, so these run without a device."""
    from paper_2608_21952_b200 import binding as bd
    from paper_2608_21952_b200.inputs import CONFIGS
    L = bd._lib
    d = bd.dims_of(CONFIGS["cfg0"])
    a = bd.FwdArgs()
    assert L.ssdi8_chunk_scan_fwd(None, None, 0, None, 0, None) == bd.ERR_NULL
    assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), 0, None, 0, None) == bd.ERR_NULL
    assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), 1, None, 0, None) == bd.ERR_NULL   # bit 0: FP16 operand, valid
    assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), (1 << 2) | (1 << 3), None, 0, None) == bd.ERR_UNSUPPORTED
    assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), 1 << 13, None, 0, None) == bd.ERR_UNSUPPORTED
    dbad = bd.dims_of(CONFIGS["cfg0"].replace(chunk=32))
    assert L.ssdi8_chunk_scan_fwd(C.byref(dbad), C.byref(a), 0, None, 0, None) == bd.ERR_SHAPE
    for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "s_xs", "s_cb", "s_h", "y"):
        setattr(a, k, 4096)
    a.xq = 4096 + 4
    assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), 0, 4096, 1 << 30, None) == bd.ERR_ALIGN
    a.xq = 4096
    for k in ("s_x", "s_xs", "s_h", "corr"):   # per-channel vectors: read 16 bytes at a time
        setattr(a, k, 4096 + 4)
        assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), 0, 4096, 1 << 30, None) == bd.ERR_ALIGN, k
        setattr(a, k, 4096 if k != "corr" else None)
    assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), 0, 4096 + 16, 1 << 30, None) == bd.ERR_ALIGN
    assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), 0, 4096, 16, None) == bd.ERR_WORKSPACE
    # quantiser
    assert L.ssdi8_quantize_act(None, 1, 4, 1, None, 0, None, None) == bd.ERR_NULL
    assert L.ssdi8_quantize_act(4096, 1, 4, 1, 4096, 7, 4096, None) == bd.ERR_UNSUPPORTED
    assert L.ssdi8_quantize_act(4096, 1, 6, 1, 4096, 0, 4096, None) == bd.ERR_SHAPE
    assert L.ssdi8_quantize_act(4096, 1, 4, 3, 4096, 0, 4096, None) == bd.ERR_SHAPE
    assert L.ssdi8_quantize_act(4100, 1, 4, 1, 4096, 0, 4096, None) == bd.ERR_ALIGN
    assert L.ssdi8_quantize_act(4096, 1, 4, 1, 4096, 0, None, None) == bd.ERR_NULL
    # state passing, step
    assert L.ssdi8_state_passing(C.byref(d), None, None, None, None, None, None, None, None) == bd.ERR_NULL
    assert L.ssdi8_state_passing(C.byref(d), 4096, 4096, None, None, None, 4096, None, None) == bd.ERR_NULL
    assert L.ssdi8_state_passing(C.byref(d), 4100, 4096, None, None, None, None, None, None) == bd.ERR_ALIGN
    assert L.ssdi8_ssd_step(C.byref(d), *([None] * 13)) == bd.ERR_NULL
    dstep = bd.dims_of(CONFIGS["cfg4"].replace(headdim=48))
    assert L.ssdi8_ssd_step(C.byref(dstep), *([4096] * 12), None) == bd.ERR_SHAPE


def test_binding_raises_on_error_code():
    from paper_2608_21952_b200 import binding as bd
    with pytest.raises(bd.SSDi8Error) as e:
        bd._check(bd.ERR_SHAPE, "x")
    assert e.value.code == bd.ERR_SHAPE and "dimensions" in str(e.value)


def test_reciprocal_fast_path_of_the_quantiser_is_exact():
    """The quantiser kernels replace fdiv(v, alpha) by fmul(v, frcp(alpha)) for every element whose
    product lies farther than 6e-5 from a rounding boundary k + 1/2 and divide for the rest.  Checked
    here in numpy binary32 on values placed on and next to the boundaries: outside the guard band
    both roundings give the same code, and the band catches every element where they differ."""
    import numpy as np
    rng = np.random.default_rng(5)
    alpha = np.concatenate([rng.uniform(1e-3, 10, 2000), 10.0 ** rng.uniform(-29, 29, 2000)]).astype(np.float32)
    k = rng.integers(-128, 128, (alpha.size, 512)).astype(np.float64) + 0.5
    off = rng.choice([0.0, 1e-7, -1e-7, 1e-6, -1e-6, 1e-5, -1e-5, 5e-5, -5e-5, 1e-4, 0.3], k.shape)
    v = ((k + off) * alpha[:, None].astype(np.float64)).astype(np.float32)
    v[:, :64] = (rng.standard_normal((alpha.size, 64)) * 60).astype(np.float32) * alpha[:, None]
    a = np.broadcast_to(alpha[:, None], v.shape)
    d = np.clip(np.rint(v / a), -127, 127)                       # float32 division, rne, saturate
    rcp = (np.float32(1.0) / alpha).astype(np.float32)
    t = np.clip(v * rcp[:, None], np.float32(-127), np.float32(127)).astype(np.float32)
    kf = np.rint(t)
    e = np.abs(t - kf)
    fast = e <= np.float32(0.49994)
    assert np.array_equal(kf[fast], d[fast])
    assert 0.2 < fast.mean() < 1.0 and (~fast).sum() > 1000      # both paths exercised


def test_zero_row_bound_of_the_fused_state_kernel_is_exact():
    """The fused ChunkState kernel stores row i of Q(X_scaled) as zeros, without the arithmetic,
    when fmul(fmul(127, rxm), |LUT_state[i]|) < 1/2, rxm being the largest |s_x / s_xs| of the
    channels it covers.  Checked here in numpy binary32, every code x in [-127, 127] against
    channel ratios up to rxm and LUT values placed on both sides of the threshold: where the bound
    holds every code of Eq. 3, rne(fmul(fmul(x, rx), lut)), is zero; and the bound is not vacuous."""
    import numpy as np
    rng = np.random.default_rng(11)
    x = np.arange(-127, 128, dtype=np.float32)
    n_dead = n_live_nonzero = 0
    for _ in range(100):
        rx = (10.0 ** rng.uniform(-3, 3, 64)).astype(np.float32)
        rxm = np.float32(np.abs(rx).max())
        b127 = np.float32(127.0) * rxm
        # LUT values around the threshold 0.5 / b127, of both signs, plus far smaller and larger ones
        thr = 0.5 / float(b127)
        lut = np.concatenate([thr * (1 + rng.uniform(-1e-3, 1e-3, 200)), thr * (1 + rng.uniform(-1e-6, 1e-6, 200)),
                              thr * 10.0 ** rng.uniform(-6, 1, 100), [0.0, thr]]).astype(np.float32)
        lut *= rng.choice(np.float32([1, -1]), lut.shape)
        dead = (b127 * np.abs(lut)).astype(np.float32) < np.float32(0.5)
        xr = (x[:, None] * rx[None, :]).astype(np.float32)                     # fmul(x, rx)
        v = (xr[None, :, :] * lut[:, None, None]).astype(np.float32)           # fmul(., lut)
        code = np.clip(np.rint(v), -127, 127)
        assert not code[dead].any()
        n_dead += int(dead.sum())
        n_live_nonzero += int((np.abs(code[~dead]).max(axis=(1, 2)) > 0).sum())
    assert n_dead > 10000 and n_live_nonzero > 10000


def test_host_side_argument_errors_of_the_layer_and_entry_calls():
    """The one-call layer entries and the entry quantiser validate on the host before any CUDA
    call: these checks run without a device."""
    from paper_2608_21952_b200 import binding as bd
    from paper_2608_21952_b200.inputs import CONFIGS
    L = bd._lib
    d = bd.dims_of(CONFIGS["cfg0"])
    a = bd.LayerArgs()
    for fn in (L.ssdi8_layer_fwd, L.ssdi8_layer_fwd_host):
        assert fn(None, None, None, 0, 0, None) == bd.ERR_NULL
        assert fn(C.byref(d), C.byref(a), 4096, 1 << 40, 0, None) == bd.ERR_NULL          # no tensors
    for k in ("x", "B", "C", "dt", "A", "s_x", "s_B", "s_C", "s_xs", "s_cb", "s_h", "y"):
        setattr(a, k, 4096)
    for fn, size in ((L.ssdi8_layer_fwd, L.ssdi8_layer_fwd_workspace_bytes),
                     (L.ssdi8_layer_fwd_host, L.ssdi8_layer_fwd_host_scratch_bytes)):
        need = size(C.byref(d), 0)
        assert need > 0
        assert fn(C.byref(d), C.byref(a), 4096, need - 1, 0, None) == bd.ERR_WORKSPACE
        assert fn(C.byref(d), C.byref(a), 4096 + 8, need, 0, None) == bd.ERR_ALIGN
        assert fn(C.byref(d), C.byref(a), 4096, need, 1 << 13, None) == bd.ERR_UNSUPPORTED
        if fn is L.ssdi8_layer_fwd:   # device tensors are read 16 bytes at a time: refused before anything is enqueued
            for k in ("x", "B", "C"):
                setattr(a, k, 4096 + 4)
                assert fn(C.byref(d), C.byref(a), 4096, need, 0, None) == bd.ERR_ALIGN
                setattr(a, k, 4096)
        assert size(C.byref(d), 1) == need                     # the FP16 operand needs no scratch of its own
        bad = bd.dims_of(CONFIGS["cfg0"].replace(chunk=48))
        assert size(C.byref(bad), 0) == 0
        assert fn(C.byref(bad), C.byref(a), 4096, 1 << 40, 0, None) == bd.ERR_SHAPE
    q = L.ssdi8_quantize_entry
    assert q(None, 0, 16, 64, 1, 16, 4096, 4096, 4096, 4096, 4096, 4096, None) == bd.ERR_NULL
    assert q(4096, 3, 16, 64, 1, 16, 4096, 4096, 4096, 4096, 4096, 4096, None) == bd.ERR_UNSUPPORTED
    assert q(4096, 0, 16, 62, 1, 16, 4096, 4096, 4096, 4096, 4096, 4096, None) == bd.ERR_SHAPE
    assert q(4096 + 4, 0, 16, 64, 1, 16, 4096, 4096, 4096, 4096, 4096, 4096, None) == bd.ERR_ALIGN
