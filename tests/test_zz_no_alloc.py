"""The forward entry point that allocates nothing (ssdi8_chunk_scan_fwd_static).

It serves callers that cannot give the library a workspace: processes whose device memory is
fully assigned at start-up, and latency-critical loops that must never call cudaMalloc or
cudaFree.  Its scratch is a fixed array inside the library, shared by all calls and never
cleared, so this test calls it twice in a row (the second call sees the first call's leftovers)
and compares each result with the ordinary entry point on a caller-owned workspace.  The file
name makes pytest collect it last, so a run that stops at the first failure has already run
every other test; it also passes when run alone in a fresh process.
"""
import ctypes as C

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2608_21952_b200 import inputs
from paper_2608_21952_b200.inputs import CONFIGS, SSDConfig


def test_static_entry_rejects_what_does_not_fit_on_the_host():
    """Size and argument checks happen before any CUDA call, so they run without a device."""
    from paper_2608_21952_b200 import binding as bd
    L = bd._lib
    a = bd.FwdArgs()
    big = bd.dims_of(CONFIGS["cfg2"])
    assert bd.ssdi8_workspace_bytes(big) > bd.STATIC_WORKSPACE_BYTES
    assert L.ssdi8_chunk_scan_fwd_static(C.byref(big), C.byref(a), 0, None) == bd.ERR_WORKSPACE
    assert L.ssdi8_chunk_scan_fwd_static(None, None, 0, None) == bd.ERR_NULL
    bad = bd.dims_of(CONFIGS["cfg0"].replace(chunk=48))
    assert L.ssdi8_chunk_scan_fwd_static(C.byref(bad), C.byref(a), 0, None) == bd.ERR_SHAPE
    assert L.ssdi8_chunk_scan_fwd_static(C.byref(big), C.byref(a), 1 << 13, None) == bd.ERR_UNSUPPORTED
    for name in ("cfg0", "cfg1"):
        assert bd.ssdi8_workspace_bytes(bd.dims_of(CONFIGS[name])) <= bd.STATIC_WORKSPACE_BYTES


@pytest.mark.gpu
def test_static_entry_matches_workspace_entry_twice_in_a_row():
    import torch
    from paper_2608_21952_b200 import binding as bd
    import gpu_harness as gh

    results = []
    # two different workloads back to back: the second call runs on the first call's leftovers
    for cfg in (CONFIGS["cfg0"], SSDConfig("static_b", 1, 512, 6, 64, 128, 2, 128, 0.02, 20.0, 51)):
        t = inputs.make_prefill(cfg)
        q = orc.prepare_quantized(cfg, t)
        dims = bd.dims_of(cfg)
        dv = {k: gh.dev(q[k]) for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "D", "s_xs",
                                         "s_cb", "s_h")}
        outs = []
        for static in (False, True):
            y = torch.full((cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim), float("nan"), device="cuda")
            fin = torch.full((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), float("nan"), device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            args = bd.make_fwd_args(y=y, final_state=fin, status=status, **dv)
            if static:
                bd.ssdi8_chunk_scan_fwd_static(dims, args)
            else:
                bd.ssdi8_chunk_scan_fwd(dims, args, bd.alloc_workspace(dims))
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            outs.append((y.cpu().numpy(), fin.cpu().numpy()))
        (y_ws, fin_ws), (y_st, fin_st) = outs
        # same kernels on the same inputs: identical bits, well inside the 1e-3 * RMS bar of the
        # parity tests
        assert np.array_equal(fin_st, fin_ws)
        assert np.abs(y_st - y_ws).max() <= 1e-3 * float(np.sqrt(np.mean(y_ws.astype(np.float64) ** 2)))
        assert np.array_equal(y_st, y_ws)
        results.append(y_st)
    assert all(np.all(np.isfinite(r)) for r in results)

    # one flagged mode through the same scratch: the paper's persistent INT8 states (Eq. 4, 7)
    cfg = CONFIGS["cfg0"]
    t = inputs.make_prefill(cfg)
    q = orc.prepare_quantized(cfg, t)
    dims = bd.dims_of(cfg)
    dv = {k: gh.dev(q[k]) for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "D", "s_xs", "s_cb", "s_h")}
    outs = []
    for static in (False, True):
        y = torch.full((cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim), float("nan"), device="cuda")
        fin = torch.full((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), float("nan"), device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        args = bd.make_fwd_args(y=y, final_state=fin, status=status, **dv)
        if static:
            bd.ssdi8_chunk_scan_fwd_static(dims, args, flags=bd.FLAG_INT8_STATE)
        else:
            bd.ssdi8_chunk_scan_fwd(dims, args, bd.alloc_workspace(dims), flags=bd.FLAG_INT8_STATE)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        outs.append((y.cpu().numpy(), fin.cpu().numpy()))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])

    with pytest.raises(bd.SSDi8Error) as e:
        big = CONFIGS["cfg2"]
        bd.ssdi8_chunk_scan_fwd_static(bd.dims_of(big), bd.FwdArgs())
    assert e.value.code == bd.ERR_WORKSPACE
