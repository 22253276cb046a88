"""Eq. 8 on the device: corr = eta * channel-wise mean of (y_ref - y_q), against the oracle."""
import ctypes as C

import numpy as np
import pytest

from oracle import oracle as orc


def test_host_side_argument_errors():
    from paper_2608_21952_b200 import binding as bd
    L = bd._lib
    assert bd.ssdi8_mean_correction_workspace_bytes(64) == 8 * 256 * 64
    assert bd.ssdi8_mean_correction_workspace_bytes(0) == 0
    assert L.ssdi8_mean_correction(None, None, 4, 4, C.c_float(0.15), None, None, 0, None) == bd.ERR_NULL
    assert L.ssdi8_mean_correction(4096, 4096, 4, 6, C.c_float(0.15), 4096, 4096, 1 << 20, None) == bd.ERR_SHAPE
    assert L.ssdi8_mean_correction(4096, 4096, 0, 8, C.c_float(0.15), 4096, 4096, 1 << 20, None) == bd.ERR_SHAPE
    assert L.ssdi8_mean_correction(4100, 4096, 4, 8, C.c_float(0.15), 4096, 4096, 1 << 20, None) == bd.ERR_ALIGN
    assert L.ssdi8_mean_correction(4096, 4096, 4, 8, C.c_float(0.15), 4096, 4096, 16, None) == bd.ERR_WORKSPACE


@pytest.mark.gpu
@pytest.mark.parametrize("R,Ch", [(512, 256), (37, 8), (16384, 5120), (1, 4)])
def test_mean_correction_matches_oracle(R, Ch):
    import torch
    from paper_2608_21952_b200 import binding as bd
    rng = np.random.default_rng(R + Ch)
    y = rng.standard_normal((R, Ch)).astype(np.float32) * 3
    yq = (y + 0.05 * rng.standard_normal((R, Ch)) + np.linspace(-0.3, 0.3, Ch)).astype(np.float32)
    ref = orc.mean_correction(y, yq, 0.15)
    dy, dq = torch.from_numpy(y).cuda(), torch.from_numpy(yq).cuda()
    corr = torch.empty(Ch, device="cuda")
    ws = torch.empty(bd.ssdi8_mean_correction_workspace_bytes(Ch), dtype=torch.uint8, device="cuda")
    bd.ssdi8_mean_correction(dy, dq, R, Ch, 0.15, corr, ws)
    torch.cuda.synchronize()
    got = corr.cpu().numpy().astype(np.float64)
    assert np.abs(got - ref).max() <= 1e-6 * max(1.0, np.abs(ref).max())
    # deterministic: a second run gives the same bits
    corr2 = torch.empty(Ch, device="cuda")
    bd.ssdi8_mean_correction(dy, dq, R, Ch, 0.15, corr2, ws)
    torch.cuda.synchronize()
    assert torch.equal(corr, corr2)


@pytest.mark.gpu
def test_estimated_correction_reduces_the_channel_mean_error_of_the_layer():
    """End to end on cfg0: estimate c from the fp64 dual form on the unquantised inputs and the
    SSDi8 output, apply it in the layer epilogue, and check every channel's mean error shrinks by eta."""
    import torch
    import gpu_harness as gh
    from paper_2608_21952_b200 import binding as bd, inputs
    cfg = inputs.CONFIGS["cfg0"]
    t = inputs.make_prefill(cfg)
    q = orc.prepare_quantized(cfg, t)
    y_fp, _ = orc.ssd_chunked(cfg, t["x"], t["B"], t["C"], t["dt"], t["A"], t["D"])
    y0, _, _ = gh.gpu_fwd(cfg, q, taps=())
    R, Ch = cfg.tokens, cfg.channels
    corr = torch.empty(Ch, device="cuda")
    ws = torch.empty(bd.ssdi8_mean_correction_workspace_bytes(Ch), dtype=torch.uint8, device="cuda")
    bd.ssdi8_mean_correction(gh.dev(y_fp.astype(np.float32).reshape(R, Ch)), gh.dev(y0.reshape(R, Ch)), R, Ch, 0.15,
                             corr, ws)
    torch.cuda.synchronize()
    c = corr.cpu().numpy()
    y1, _, _ = gh.gpu_fwd(cfg, q, corr=c, taps=())
    e0 = (y_fp - y0).reshape(R, Ch).mean(0)
    e1 = (y_fp - y1).reshape(R, Ch).mean(0)
    assert np.allclose(e1, 0.85 * e0, rtol=1e-3, atol=1e-6 * np.abs(e0).max() + 1e-7)
