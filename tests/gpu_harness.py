"""Runs the CUDA path through its C-ABI binding and returns numpy arrays (tests only)."""
import numpy as np
import torch

from paper_2608_21952_b200 import binding as bd

TAP_NAMES = ("cs", "acc_cb", "CBq", "Xsq", "acc_st", "loc", "prev", "hq", "acc_off", "rowmax", "Mq",
             "acc_diag")
_NP2T = {np.float32: torch.float32, np.int32: torch.int32, np.int8: torch.int8}


def dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


def tap_shapes(cfg):
    b, L, H, P, N, G, Q, c = (cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim, cfg.dstate, cfg.ngroups,
                              cfg.chunk, cfg.nchunks)
    return {
        "cs": ((b, H, c, Q), np.float32), "acc_cb": ((b, c, G, Q, Q), np.int32),
        "CBq": ((b, c, G, Q, Q), np.int8), "Xsq": ((b, L, H, P), np.int8),
        "acc_st": ((b, c, H, P, N), np.int32), "loc": ((b, c, H, P, N), np.float32),
        "prev": ((b, c, H, P, N), np.float32), "hq": ((b, c, H, P, N), np.int8),
        "acc_off": ((b, L, H, P), np.int32), "rowmax": ((b, L, H), np.float32),
        "Mq": ((b, c, H, Q, Q), np.int8), "acc_diag": ((b, L, H, P), np.int32),
    }


def gpu_fwd(cfg, q, corr=None, taps=TAP_NAMES, D="use", flags=0, dt_bias=None):
    """q: dict with xq,Bq,Cq,s_x,s_B,s_C,dt,A,D,s_xs,s_cb,s_h,init (numpy).  Returns y, final, taps."""
    dims = bd.dims_of(cfg)
    t = {k: dev(q[k]) for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "s_xs", "s_cb", "s_h")}
    t["D"] = dev(q["D"]) if D == "use" else None
    t["corr"] = dev(corr)
    if dt_bias is not None:
        t["dt_bias"] = dev(dt_bias)
    t["init_state"] = dev(q.get("init"))
    y = torch.full((cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim), float("nan"), device="cuda")
    fin = torch.full((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tp = {}
    shapes = tap_shapes(cfg)
    for name in taps:
        shp, dt_ = shapes[name]
        tp["tap_" + name] = torch.zeros(shp, dtype=_NP2T[dt_], device="cuda")
    ws = bd.alloc_workspace(dims, flags=flags)
    args = bd.make_fwd_args(y=y, final_state=fin, status=status, **t, **tp)
    bd.ssdi8_chunk_scan_fwd(dims, args, ws, flags=flags)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return y.cpu().numpy(), fin.cpu().numpy(), {k[4:]: v.cpu().numpy() for k, v in tp.items()}


def gpu_quantize(v, R, Ch, I, scale=None, mode=1, want_out=True):
    vin = dev(np.asarray(v, np.float32))
    s = torch.zeros(Ch, device="cuda") if scale is None else dev(np.asarray(scale, np.float32))
    out = torch.empty(vin.shape, dtype=torch.int8, device="cuda") if want_out else None
    bd.ssdi8_quantize_act(vin, R, Ch, I, s, mode, out)
    torch.cuda.synchronize()
    return (out.cpu().numpy() if want_out else None), s.cpu().numpy()
