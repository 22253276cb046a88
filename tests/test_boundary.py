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
    assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), 1, None, 0, None) == bd.ERR_UNSUPPORTED
    assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), 1 << 13, None, 0, None) == bd.ERR_UNSUPPORTED
    dbad = bd.dims_of(CONFIGS["cfg0"].replace(chunk=32))
    assert L.ssdi8_chunk_scan_fwd(C.byref(dbad), C.byref(a), 0, None, 0, None) == bd.ERR_SHAPE
    for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "s_xs", "s_cb", "s_h", "y"):
        setattr(a, k, 4096)
    a.xq = 4096 + 4
    assert L.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), 0, 4096, 1 << 30, None) == bd.ERR_ALIGN
    a.xq = 4096
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
