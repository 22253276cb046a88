"""Parity of the CUDA path (through the C-ABI) with the CPU oracle on seeded inputs.

Bar: bit-exact on every int8 tensor and int32 accumulator and on the fp32 tensors that
are defined operation by operation (cs, loc, states); max-abs error <= 1e-3 * RMS on
the fp32 output y and on the final state.
"""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2608_21952_b200 import inputs
from paper_2608_21952_b200.inputs import CONFIGS, SSDConfig
from helpers import census, half_neighbours, rms

pytestmark = pytest.mark.gpu

Y_TOL = 1e-3  # max-abs error relative to the RMS of the reference output


def _harness():
    import gpu_harness
    return gpu_harness


def _causal(cfg):
    return np.tril(np.ones((cfg.chunk, cfg.chunk), bool))


def check_fwd(cfg, init=None, corr=None, use_D=True, mutate=None):
    gh = _harness()
    t = inputs.make_prefill(cfg)
    if mutate is not None:
        mutate(t)
    q = orc.prepare_quantized(cfg, t, init)
    y_ref, fin_ref, ref = orc.ssdi8_fwd(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"],
                                        q["dt"], q["A"], q["D"] if use_D else None, corr, q["s_xs"],
                                        q["s_cb"], q["s_h"], init, taps=gh.TAP_NAMES)
    y, fin, got = gh.gpu_fwd(cfg, q, corr=corr, D="use" if use_D else None)
    tril = _causal(cfg)
    for name in ("cs", "Xsq", "acc_st", "loc", "prev", "hq", "acc_off", "rowmax", "Mq", "acc_diag"):
        assert np.array_equal(got[name], ref[name]), name
    for name in ("acc_cb", "CBq"):  # only the causal half is defined
        assert np.array_equal(got[name][..., tril], ref[name][..., tril]), name
    assert np.array_equal(fin, fin_ref)
    assert np.abs(y - y_ref).max() <= Y_TOL * rms(y_ref)
    return y, y_ref


SMALL = [
    CONFIGS["cfg0"],
    SSDConfig("g2_n64_q128", 2, 256, 4, 64, 64, 2, 128, 0.02, 20.0, 21),
    SSDConfig("n128_q256", 1, 512, 3, 64, 128, 1, 256, 0.02, 20.0, 22),
    SSDConfig("g4_q64", 2, 128, 8, 64, 128, 4, 64, 0.02, 20.0, 23),
    SSDConfig("one_chunk", 1, 128, 2, 64, 64, 1, 128, 0.02, 20.0, 24),
]


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
def test_fwd_all_taps_bit_exact(cfg):
    check_fwd(cfg)


def test_fwd_with_init_state_and_correction():
    cfg = SMALL[1]
    init = inputs.make_init_state(cfg, 0.5)
    corr = (0.05 * np.random.default_rng(3).standard_normal(cfg.channels)).astype(np.float32)
    check_fwd(cfg, init=init, corr=corr)


def test_fwd_without_skip_weight():
    check_fwd(SMALL[0], use_D=False)


def test_fwd_cfg1_full():
    check_fwd(CONFIGS["cfg1"])


def _scale_A(f):
    def m(t):
        t["A"] = (t["A"] * np.float32(f)).astype(np.float32)
    return m


def _growing_head(t):
    """Head 1 grows instead of decaying (A > 0, outside the model's range but inside the
    interface's): the cumulative sums are not monotone there."""
    t["A"] = t["A"].copy()
    t["A"][1] = np.float32(0.25)


def _mixed_sign_dt(t):
    """dt of both signs: cs wanders, so no ordering of the decay factors may be assumed."""
    t["dt"] = (t["dt"] * np.where(np.random.default_rng(9).random(t["dt"].shape) < 0.3, -1, 1)).astype(np.float32)


@pytest.mark.parametrize("cfg", [SMALL[1], SMALL[2]], ids=lambda c: c.name)
@pytest.mark.parametrize("regime", ["slow", "fast", "very_fast", "growing", "mixed_dt"])
def test_fwd_decay_regimes_bit_exact(cfg, regime):
    """The masked operand skips sub-blocks that cannot matter; the skipping must decide no bit
    whether almost nothing decays (every sub-block of a row matters), almost everything does
    (only the row's own sub-block survives), or the decay is not monotone (the walk may not stop early)."""
    mutate = {"slow": _scale_A(0.01), "fast": _scale_A(8.0), "very_fast": _scale_A(200.0),
              "growing": _growing_head, "mixed_dt": _mixed_sign_dt}[regime]
    check_fwd(cfg, mutate=mutate)


def test_fwd_degenerate_inputs():
    """dt = 0 (every decay exactly 1, nothing enters the state) and x = 0 (all-zero rows of
    the masked operand) run through the same path."""
    gh = _harness()
    cfg = SMALL[0]
    t = inputs.make_prefill(cfg)
    for case in ("dt0", "x0"):
        tt = dict(t)
        if case == "dt0":
            tt["dt"] = np.zeros_like(t["dt"])
        else:
            tt["x"] = np.zeros_like(t["x"])
        q = orc.prepare_quantized(cfg, tt)
        y_ref, fin_ref, ref = orc.ssdi8_fwd(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"],
                                            q["dt"], q["A"], q["D"], None, q["s_xs"], q["s_cb"], q["s_h"],
                                            None, taps=("Mq", "rowmax", "hq", "Xsq"))
        y, fin, got = gh.gpu_fwd(cfg, q, taps=("Mq", "rowmax", "hq", "Xsq"))
        for name in ("Mq", "rowmax", "hq", "Xsq"):
            assert np.array_equal(got[name], ref[name]), (case, name)
        assert np.array_equal(fin, fin_ref)
        assert np.abs(y - y_ref).max() <= Y_TOL * max(rms(y_ref), 1e-30)


def _sampled_problem(cfg, t, pairs):
    """Scales for a full-size workload without running the oracle on all of it: Eq. 1 on the
    whole input tensors, internal step sizes calibrated by the oracle on the sampled
    (batch, head) pairs and reused for the other heads (any positive step size is a valid
    static scale; codes beyond it saturate)."""
    T = cfg.tokens
    xq, s_x = orc.quantize(t["x"], T, cfg.channels, 1, mode=1)
    Bq, s_B = orc.quantize(t["B"], T, cfg.ngroups, cfg.dstate, mode=1)
    Cq, s_C = orc.quantize(t["C"], T, cfg.ngroups, cfg.dstate, mode=1)
    P = cfg.headdim
    hpg = cfg.nheads // cfg.ngroups
    one = cfg.replace(batch=1, nheads=1, ngroups=1)
    per_head = {}
    for (b, h) in pairs:
        g = h // hpg
        sub = _slice(cfg, b, h, xq, Bq, Cq, s_x, s_B, s_C, t)
        s_xs, s_cb, s_h = orc.calibrate(one, sub["xq"], sub["Bq"], sub["Cq"], sub["s_x"], sub["s_B"],
                                        sub["s_C"], sub["dt"], sub["A"])
        per_head[h] = (s_xs, s_h, g, s_cb)
    hs = sorted(per_head)
    s_xs = np.empty(cfg.channels, np.float32); s_h = np.empty(cfg.channels, np.float32)
    s_cb = np.ones(cfg.ngroups, np.float32)
    for h in range(cfg.nheads):
        src = per_head[hs[h % len(hs)]]
        ratio = s_x[h * P:(h + 1) * P] / s_x[hs[h % len(hs)] * P:(hs[h % len(hs)] + 1) * P]
        s_xs[h * P:(h + 1) * P] = src[0] * ratio
        s_h[h * P:(h + 1) * P] = src[1] * ratio
    for g in range(cfg.ngroups):
        c = [v[3][0] for v in per_head.values() if v[2] == g]
        s_cb[g] = max(c) if c else max(v[3][0] for v in per_head.values())
    return dict(xq=xq, Bq=Bq, Cq=Cq, s_x=s_x, s_B=s_B, s_C=s_C, dt=t["dt"], A=t["A"], D=t["D"],
                s_xs=s_xs.astype(np.float32), s_cb=s_cb, s_h=s_h.astype(np.float32), init=None)


def _slice(cfg, b, h, xq, Bq, Cq, s_x, s_B, s_C, t, extra=None):
    P = cfg.headdim
    g = h // (cfg.nheads // cfg.ngroups)
    d = dict(xq=xq[b:b + 1, :, h:h + 1], Bq=Bq[b:b + 1, :, g:g + 1], Cq=Cq[b:b + 1, :, g:g + 1],
             s_x=s_x[h * P:(h + 1) * P], s_B=s_B[g:g + 1], s_C=s_C[g:g + 1],
             dt=t["dt"][b:b + 1, :, h:h + 1], A=t["A"][h:h + 1], D=t["D"][h:h + 1])
    if extra:
        d.update(s_xs=extra["s_xs"][h * P:(h + 1) * P], s_cb=extra["s_cb"][g:g + 1],
                 s_h=extra["s_h"][h * P:(h + 1) * P])
    return {k: np.ascontiguousarray(v) for k, v in d.items()}


# chunks of 128 and of 64 tokens with about 20 tiles per CTA of the persistent scan kernel, so that its
# rings (4, 8 deep) wrap several times in the one-tile-per-chunk geometry as well
DEEP = {
    "deep_q128": SSDConfig("deep_q128", 2, 4096, 48, 64, 64, 2, 128, 0.01, 50.0, 51),
    "deep_q64": SSDConfig("deep_q64", 2, 2048, 48, 64, 128, 4, 64, 0.01, 50.0, 52),
}


@pytest.mark.parametrize("flags", [0, 1], ids=["int8_operand", "fp16_operand"])
@pytest.mark.parametrize("name,npairs", [("cfg2", 4), ("cfg3", 3), ("deep_q128", 3), ("deep_q64", 3)])
def test_fwd_full_size_sampled(name, npairs, flags):
    """Full-size workloads in the launch configuration the benchmark times (no taps); the
    oracle recomputes sampled (batch, head) pairs one by one.  flags = 1: the paper's FP16
    ChunkScan2 operand on both sides."""
    gh = _harness()
    cfg = CONFIGS[name] if name in CONFIGS else DEEP[name]
    t = inputs.make_prefill(cfg)
    rng = np.random.default_rng(100 + cfg.seed)
    pairs = [(0, 0), (cfg.batch - 1, cfg.nheads - 1)]
    while len(pairs) < npairs:
        pr = (int(rng.integers(cfg.batch)), int(rng.integers(cfg.nheads)))
        if pr not in pairs:
            pairs.append(pr)
    q = _sampled_problem(cfg, t, pairs)
    y, fin, _ = gh.gpu_fwd(cfg, q, taps=(), flags=flags)
    assert np.all(np.isfinite(y)) and np.all(np.isfinite(fin))
    one = cfg.replace(batch=1, nheads=1, ngroups=1)
    for (b, h) in pairs:
        s = _slice(cfg, b, h, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], t, extra=q)
        y_ref, fin_ref, _ = orc.ssdi8_fwd(one, s["xq"], s["Bq"], s["Cq"], s["s_x"], s["s_B"], s["s_C"],
                                          s["dt"], s["A"], s["D"], None, s["s_xs"], s["s_cb"], s["s_h"],
                                          flags=flags)
        assert np.array_equal(fin[b, h], fin_ref[0, 0]), (b, h)
        assert np.abs(y[b, :, h] - y_ref[0, :, 0]).max() <= Y_TOL * rms(y_ref), (b, h)


@pytest.mark.parametrize("name,npairs", [("cfg2", 3), ("cfg3", 3)])
def test_layer_fwd_full_size_sampled(name, npairs):
    """The call the benchmark's step makes (ssdi8_layer_fwd: fp32 x, B, C in, the three Eq. 1
    quantisers as one launch, side streams inside) at full size; the oracle quantises the whole
    tensors and recomputes sampled (batch, head) pairs one by one."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    cfg = CONFIGS[name]
    t = inputs.make_prefill(cfg)
    rng = np.random.default_rng(200 + cfg.seed)
    pairs = [(0, 0), (cfg.batch - 1, cfg.nheads - 1)]
    while len(pairs) < npairs:
        pr = (int(rng.integers(cfg.batch)), int(rng.integers(cfg.nheads)))
        if pr not in pairs:
            pairs.append(pr)
    q = _sampled_problem(cfg, t, pairs)
    dims = bd.dims_of(cfg)
    dv = {k: gh.dev(q[k]) for k in ("s_x", "s_B", "s_C", "s_xs", "s_cb", "s_h", "A", "D")}
    dv.update({k: gh.dev(t[k]) for k in ("x", "B", "C", "dt")})
    y = torch.empty(t["x"].shape, device="cuda")
    fin = torch.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = bd.make_layer_args(y=y, final_state=fin, status=status, **dv)
    ws = torch.empty(bd.ssdi8_layer_fwd_workspace_bytes(dims, 0), dtype=torch.uint8, device="cuda")
    y_h = fin_h = None
    for rep in range(2):   # the second call finds the first one's contents in the workspace
        y.fill_(float("nan")); fin.fill_(float("nan"))
        bd.ssdi8_layer_fwd(dims, args, ws, 0)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        if rep == 0:
            y_h, fin_h = y.cpu().numpy(), fin.cpu().numpy()
        else:
            assert np.array_equal(y.cpu().numpy(), y_h) and np.array_equal(fin.cpu().numpy(), fin_h)
    assert np.all(np.isfinite(y_h)) and np.all(np.isfinite(fin_h))
    one = cfg.replace(batch=1, nheads=1, ngroups=1)
    for (b, h) in pairs:
        s = _slice(cfg, b, h, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], t, extra=q)
        y_ref, fin_ref, _ = orc.ssdi8_fwd(one, s["xq"], s["Bq"], s["Cq"], s["s_x"], s["s_B"], s["s_C"],
                                          s["dt"], s["A"], s["D"], None, s["s_xs"], s["s_cb"], s["s_h"])
        assert np.array_equal(fin_h[b, h], fin_ref[0, 0]), (b, h)
        assert np.abs(y_h[b, :, h] - y_ref[0, :, 0]).max() <= Y_TOL * rms(y_ref), (b, h)



# --------------------------------------------------------------------------- against the plain definitions
PLAIN_CASES = {
    "cfg0": (CONFIGS["cfg0"], None), "cfg1": (CONFIGS["cfg1"], None),
    "slow": (SMALL[1], _scale_A(0.01)), "fast": (SMALL[2], _scale_A(8.0)), "very_fast": (SMALL[1], _scale_A(200.0)),
}


@pytest.mark.parametrize("case", list(PLAIN_CASES))
def test_fwd_boundary_aware_against_the_plain_definitions(case, capsys):
    """The GPU's integer tensors against the fp64 definitions (libm exp, no sub-blocks): a code
    equals round(v) of the fp64 value v, or is its neighbour with v inside the derived window around
    the rounding boundary between the two; the row maxima within 1e-5; y against the y of the plain
    definitions on the same integer inputs as a relative L2 distance."""
    gh = _harness()
    cfg, mutate = PLAIN_CASES[case]
    t = inputs.make_prefill(cfg)
    if mutate is not None:
        mutate(t)
    init = inputs.make_init_state(cfg, 0.3)
    q = orc.prepare_quantized(cfg, t, init)
    y, fin, got = gh.gpu_fwd(cfg, q)
    rep = {}
    v, _ = orc.chunk_state_plain(cfg, q["xq"], q["s_x"], q["s_xs"], q["dt"], got["cs"])
    rep["Xsq"], worst, outside = census(got["Xsq"], v, 4e-6)
    assert worst <= 1 and outside == 0
    v, _ = orc.state_codes_plain(cfg, got["prev"], q["s_h"])
    rep["hq"], worst, outside = census(got["hq"], v, 4e-6)
    assert worst <= 1 and outside == 0
    y_plain, out = orc.chunk_scan_plain(cfg, q["xq"], q["Cq"], got["CBq"] * _causal(cfg), got["hq"], q["s_x"], q["s_C"],
                                        q["s_cb"], q["s_h"], q["dt"], got["cs"], q["D"], None)
    b, c, Q, H = cfg.batch, cfg.nchunks, cfg.chunk, cfg.nheads
    sM = out["sM"].reshape(b, c, Q, H).transpose(0, 1, 3, 2)[..., None]
    # the library treats a row whose largest |CBq dt_j exp(cs_i - cs_j)| is below 1e-30 as a zero row
    # (and exponentials below e^-80 as zero); Eq. 1 taken literally would still spread such a row over
    # the 8-bit range.  Those rows (they contribute less than 1e-30 to y) must be all-zero codes.
    rm = got["rowmax"].reshape(b, c, Q, H).transpose(0, 1, 3, 2)                 # [b,c,H,Q]
    flushed = rm < 1e-30
    assert np.all(got["Mq"][flushed] == 0)
    rep["flushed_rows"] = float(flushed.mean())
    keep = ~flushed
    rep["Mq"], worst, outside = census(got["Mq"][keep], (out["M"] / sM)[keep], 1e-5)
    assert worst <= 1 and outside == 0
    hg = np.arange(H) // (H // cfg.ngroups)
    rowmax = got["rowmax"].astype(np.float64) * q["s_cb"].astype(np.float64)[hg][None, None, :]
    amax = np.abs(out["M"]).max(-1).transpose(0, 1, 3, 2).reshape(b, c * Q, H)
    live = got["rowmax"] >= 1e-30
    assert np.allclose(rowmax[live], amax[live], rtol=1e-5, atol=0) and np.all(amax[~live] < 4e-30)
    rep["y_rel_l2"] = float(np.sqrt(((y - y_plain) ** 2).sum() / (y_plain ** 2).sum()))
    assert rep["y_rel_l2"] < 1e-3
    # the whole forward from the plain definitions alone (no tensor of the GPU run enters it)
    y_ind, fin_ind = orc.ssdi8_fwd_plain(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], q["dt"], q["A"],
                                         q["D"], None, q["s_xs"], q["s_cb"], q["s_h"], init)
    rep["y_rel_l2_independent"] = float(np.sqrt(((y - y_ind) ** 2).sum() / (y_ind ** 2).sum()))
    rep["final_rel_l2_independent"] = float(np.sqrt(((fin - fin_ind) ** 2).sum() / (fin_ind ** 2).sum()))
    assert rep["y_rel_l2_independent"] < 5e-3 and rep["final_rel_l2_independent"] < 5e-3
    with capsys.disabled():
        print(f"\n[GPU vs plain, {case}] " + ", ".join(f"{k} {v:.2e}" for k, v in rep.items()))


# --------------------------------------------------------------------------- the benchmark's own problem, every pair
@pytest.mark.parametrize("name,flags", [("cfg2", 0), ("cfg2", 2), ("cfg2", 1), ("cfg3", 0)],
                         ids=["cfg2", "cfg2_int8_state", "cfg2_fp16_operand", "cfg3"])
def test_fwd_full_size_all_pairs(name, flags):
    """Exactly what the benchmark runs: Eq. 1 on the whole tensors, internal step sizes from
    ssdi8_calibrate on the whole tensors (compared bit for bit with the oracle's calibration), then
    ssdi8_layer_fwd without taps; the oracle recomputes EVERY (batch, head) pair, one batch element
    at a time.  Final state bit for bit, y within the tolerance per pair."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    cfg = CONFIGS[name]
    t = inputs.make_prefill(cfg)
    T = cfg.tokens
    dims = bd.dims_of(cfg)
    dv = {k: gh.dev(t[k]) for k in ("x", "B", "C", "dt", "A", "D")}
    i8 = lambda k: torch.empty(t[k].shape, dtype=torch.int8, device="cuda")
    xq, Bq, Cq = i8("x"), i8("B"), i8("C")
    z = lambda n: torch.empty(n, device="cuda")
    s_x, s_B, s_C = z(cfg.channels), z(cfg.ngroups), z(cfg.ngroups)
    s_xs, s_cb, s_h = z(cfg.channels), z(cfg.ngroups), z(cfg.channels)
    bd.ssdi8_quantize_act(dv["x"], T, cfg.channels, 1, s_x, 1, xq)
    bd.ssdi8_quantize_act(dv["B"], T, cfg.ngroups, cfg.dstate, s_B, 1, Bq)
    bd.ssdi8_quantize_act(dv["C"], T, cfg.ngroups, cfg.dstate, s_C, 1, Cq)
    ws = bd.alloc_workspace(dims)
    cal = bd.make_fwd_args(xq=xq, Bq=Bq, Cq=Cq, s_x=s_x, s_B=s_B, s_C=s_C, dt=dv["dt"], A=dv["A"])
    bd.ssdi8_calibrate(dims, cal, s_xs, s_cb, s_h, ws)
    torch.cuda.synchronize()
    q = orc.prepare_quantized(cfg, t)
    for k, g in (("xq", xq), ("Bq", Bq), ("Cq", Cq), ("s_x", s_x), ("s_B", s_B), ("s_C", s_C), ("s_xs", s_xs),
                 ("s_cb", s_cb), ("s_h", s_h)):
        assert np.array_equal(g.cpu().numpy(), q[k]), k
    del ws, xq, Bq, Cq
    td = torch.float16 if flags & 1 else torch.float32
    yflag = bd.FLAG_Y_FP16 if flags & 1 else 0     # the paper's operand with the paper's output format
    y = torch.full(t["x"].shape, float("nan"), dtype=td, device="cuda")
    fin = torch.full((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = bd.make_layer_args(x=dv["x"], B=dv["B"], C=dv["C"], dt=dv["dt"], A=dv["A"], D=dv["D"], s_x=s_x, s_B=s_B,
                              s_C=s_C, s_xs=s_xs, s_cb=s_cb, s_h=s_h, y=y, final_state=fin, status=status)
    lws = torch.empty(bd.ssdi8_layer_fwd_workspace_bytes(dims, flags | yflag), dtype=torch.uint8, device="cuda")
    bd.ssdi8_layer_fwd(dims, args, lws, flags | yflag)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    y_h, fin_h = y.float().cpu().numpy(), fin.cpu().numpy()
    del y, lws
    one = cfg.replace(batch=1)
    worst = 0.0
    for b in range(cfg.batch):
        sl = lambda a: np.ascontiguousarray(a[b:b + 1])
        y_ref, fin_ref, _ = orc.ssdi8_fwd(one, sl(q["xq"]), sl(q["Bq"]), sl(q["Cq"]), q["s_x"], q["s_B"], q["s_C"],
                                          sl(q["dt"]), q["A"], q["D"], None, q["s_xs"], q["s_cb"], q["s_h"], flags=flags)
        assert np.array_equal(fin_h[b], fin_ref[0]), b
        pair_rms = np.sqrt((y_ref[0] ** 2).mean(axis=(0, 2)))                       # [H]
        err = np.abs(y_h[b] - y_ref[0])
        if flags & 1:   # fp16 y: half a unit in the last place of each element on top
            err = np.maximum(err - 1.01 * 2.0 ** -11 * np.abs(y_ref[0]), 0.0)
        pair_err = err.max(axis=(0, 2))
        assert np.all(pair_err <= Y_TOL * pair_rms), (b, int(np.argmax(pair_err / pair_rms)))
        worst = max(worst, float((pair_err / pair_rms).max()))
    print(f"{name} flags={flags}: worst pair max|dy|/rms = {worst:.2e} over {cfg.batch * cfg.nheads} pairs")

# --------------------------------------------------------------------------- softplus of the raw time step
@pytest.mark.parametrize("with_bias", [True, False])
def test_fwd_from_the_raw_time_step(with_bias):
    """SSDI8_FLAG_DT_SOFTPLUS: ChunkCumsum starts from dt = softplus(dt_raw + dt_bias) (Algorithm 2 module 1).
    The oracle applies its own softplus and runs the forward on the positive time step; every tap,
    the final state and y must agree as in the default mode."""
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    cfg = SMALL[1]
    t = inputs.make_prefill(cfg)
    rng = np.random.default_rng(77)
    raw = rng.normal(-3.0, 1.0, t["dt"].shape).astype(np.float32)
    raw[0, :4, 0] = [60.0, -60.0, 0.0, -100.0]              # both tails and the middle of the softplus
    bias = rng.normal(0.0, 0.3, cfg.nheads).astype(np.float32) if with_bias else None
    t["dt"] = orc.softplus_dt(raw, bias)
    q = orc.prepare_quantized(cfg, t)
    y_ref, fin_ref, ref = orc.ssdi8_fwd(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], q["dt"], q["A"],
                                        q["D"], None, q["s_xs"], q["s_cb"], q["s_h"], None, taps=gh.TAP_NAMES)
    qg = dict(q)
    qg["dt"] = raw
    y, fin, got = gh.gpu_fwd(cfg, qg, flags=bd.FLAG_DT_SOFTPLUS, dt_bias=bias)
    tril = _causal(cfg)
    for name in ("cs", "Xsq", "acc_st", "loc", "prev", "hq", "acc_off", "rowmax", "Mq", "acc_diag"):
        assert np.array_equal(got[name], ref[name]), name
    assert np.array_equal(got["CBq"][..., tril], ref["CBq"][..., tril])
    assert np.array_equal(fin, fin_ref)
    assert np.abs(y - y_ref).max() <= Y_TOL * rms(y_ref)


def test_softplus_dt_entry_point_bit_exact():
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    rng = np.random.default_rng(78)
    H = 80
    raw = np.concatenate([rng.normal(-3, 1.5, (30000, H)), rng.uniform(-95, 95, (3000, H))]).astype(np.float32)
    bias = rng.normal(0, 0.5, H).astype(np.float32)
    for b in (bias, None):
        want = orc.softplus_dt(raw, b)
        d_raw = gh.dev(raw)
        out = torch.empty_like(d_raw)
        bd.ssdi8_softplus_dt(d_raw, gh.dev(b), raw.shape[0], H, out)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy(), want)
        # and against the libm definition: the same binary32 value in all but a handful of elements
        plain = orc.softplus_dt(raw, b, plain=True)
        assert np.mean(out.cpu().numpy() != plain) < 1e-5


# --------------------------------------------------------------------------- persistent INT8 states (Eq. 4, 7)
@pytest.mark.parametrize("cfg", [SMALL[0], SMALL[1], SMALL[2]], ids=lambda c: c.name)
def test_fwd_int8_state_mode_bit_exact(cfg):
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    t = inputs.make_prefill(cfg)
    init = inputs.make_init_state(cfg, 0.3)
    q = orc.prepare_quantized(cfg, t, init)
    names = ("cs", "Xsq", "acc_st", "hq", "acc_off", "rowmax", "Mq", "acc_diag")
    y_ref, fin_ref, ref = orc.ssdi8_fwd(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], q["dt"],
                                        q["A"], q["D"], None, q["s_xs"], q["s_cb"], q["s_h"], init, taps=names,
                                        flags=orc.FLAG_INT8_STATE)
    y, fin, got = gh.gpu_fwd(cfg, q, taps=names, flags=bd.FLAG_INT8_STATE)
    for name in names:
        assert np.array_equal(got[name], ref[name]), name
    assert np.array_equal(fin, fin_ref)
    assert np.abs(y - y_ref).max() <= Y_TOL * rms(y_ref)


def test_int8_state_flag_needs_the_fused_state_kernel():
    from paper_2608_21952_b200 import binding as bd
    a = bd.FwdArgs()
    d = bd.dims_of(SMALL[0])
    import ctypes as C
    rc = bd._lib.ssdi8_chunk_scan_fwd(C.byref(d), C.byref(a), bd.FLAG_INT8_STATE | bd.PHASE_CHUNK_STATE, None, 0, None)
    assert rc == bd.ERR_UNSUPPORTED


# --------------------------------------------------------------------------- quantiser
@pytest.mark.parametrize("R,Ch,I", [(512, 256, 1), (37, 8, 1), (1000, 5120, 1), (512, 1, 64),
                                    (333, 8, 128), (4, 4, 4), (1, 4, 1)])
def test_quantizer_bit_exact(R, Ch, I):
    gh = _harness()
    rng = np.random.default_rng(R + Ch + I)
    v = (rng.standard_normal((R, Ch, I)) * rng.uniform(0.05, 40, (1, Ch, 1))).astype(np.float32)
    v[:, Ch // 2, :] = 0 if Ch > 1 else v[:, 0, :]
    q_ref, s_ref = orc.quantize(v, R, Ch, I, mode=1)
    q, s = gh.gpu_quantize(v, R, Ch, I, mode=1)
    assert np.array_equal(s, s_ref) and np.array_equal(q, q_ref)
    # static mode with a step size that saturates part of the tensor
    st = (s_ref * 0.5).astype(np.float32)
    q_ref, _ = orc.quantize(v, R, Ch, I, scale=st, mode=0)
    q, s2 = gh.gpu_quantize(v, R, Ch, I, scale=st, mode=0)
    assert np.array_equal(q, q_ref) and np.array_equal(s2, st)
    # observe mode keeps the running maximum and writes nothing else
    _, s_obs_ref = orc.quantize(v * 0.5, R, Ch, I, scale=s_ref, mode=2, want_out=False)
    _, s_obs = gh.gpu_quantize(v * 0.5, R, Ch, I, scale=s_ref, mode=2, want_out=False)
    assert np.array_equal(s_obs, s_obs_ref) and np.array_equal(s_obs, s_ref)
    _, s_obs_ref = orc.quantize(v * 3, R, Ch, I, scale=s_ref, mode=2, want_out=False)
    _, s_obs = gh.gpu_quantize(v * 3, R, Ch, I, scale=s_ref, mode=2, want_out=False)
    assert np.array_equal(s_obs, s_obs_ref)


def test_quantizer_empty_input_is_a_no_op():
    import torch
    from paper_2608_21952_b200 import binding as bd
    x = torch.zeros(16, device="cuda"); s = torch.ones(4, device="cuda")
    o = torch.full((16,), 5, dtype=torch.int8, device="cuda")
    bd.ssdi8_quantize_act(x, 0, 4, 1, s, 0, o)
    torch.cuda.synchronize()
    assert bool((o == 5).all())


def test_entry_quantizer_empty_input_is_a_no_op():
    import torch
    from paper_2608_21952_b200 import binding as bd
    x = torch.zeros(64, dtype=torch.bfloat16, device="cuda"); s = torch.ones(16, device="cuda")
    o = torch.full((64,), 5, dtype=torch.int8, device="cuda")
    bd.ssdi8_quantize_entry(x, 0, 16, 1, 16, s, s, s, o, o, o)
    torch.cuda.synchronize()
    assert bool((o == 5).all())


def test_quantizer_full_size_x_and_bc():
    gh = _harness()
    cfg = CONFIGS["cfg2"]
    t = inputs.make_prefill(cfg)
    for key, Ch, I in (("x", cfg.channels, 1), ("B", cfg.ngroups, cfg.dstate)):
        q_ref, s_ref = orc.quantize(t[key], cfg.tokens, Ch, I, mode=1)
        q, s = gh.gpu_quantize(t[key], cfg.tokens, Ch, I, mode=1)
        assert np.array_equal(s, s_ref) and np.array_equal(q, q_ref)


@pytest.mark.parametrize("dtype", ["float32", "float16", "bfloat16"])
@pytest.mark.parametrize("T,H,P,G,N", [(333, 3, 8, 1, 16), (1000, 4, 64, 2, 64), (4096, 24, 64, 1, 128)])
def test_entry_quantizer_bit_exact(dtype, T, H, P, G, N):
    """xBC [T][D + 2GN] in one pass == the Eq. 1 oracle on its three slices (static step sizes)."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    D, GN = H * P, G * N
    rng = np.random.default_rng([T, D, GN])
    xBC = (rng.standard_normal((T, D + 2 * GN)) * rng.uniform(0.05, 20, (1, D + 2 * GN))).astype(np.float32)
    td = getattr(torch, dtype)
    dv = torch.from_numpy(xBC).to(td).cuda()
    v = dv.float().cpu().numpy()          # the values the kernel sees (the widening is exact)
    s_x = (np.abs(v[:, :D]).max(0) / 200).astype(np.float32)     # saturates part of every channel
    s_x[D // 2] = 1.0
    s_B = rng.uniform(0.01, 0.2, G).astype(np.float32)
    s_C = rng.uniform(0.01, 0.2, G).astype(np.float32)
    xq = torch.empty((T, D), dtype=torch.int8, device="cuda")
    Bq = torch.empty((T, GN), dtype=torch.int8, device="cuda")
    Cq = torch.empty((T, GN), dtype=torch.int8, device="cuda")
    bd.ssdi8_quantize_entry(dv, T, D, G, N, torch.from_numpy(s_x).cuda(), torch.from_numpy(s_B).cuda(),
                            torch.from_numpy(s_C).cuda(), xq, Bq, Cq)
    torch.cuda.synchronize()
    x_ref, _ = orc.quantize(np.ascontiguousarray(v[:, :D]), T, D, 1, scale=s_x, mode=0)
    B_ref, _ = orc.quantize(np.ascontiguousarray(v[:, D:D + GN]), T, G, N, scale=s_B, mode=0)
    C_ref, _ = orc.quantize(np.ascontiguousarray(v[:, D + GN:]), T, G, N, scale=s_C, mode=0)
    assert np.array_equal(xq.cpu().numpy(), x_ref)
    assert np.array_equal(Bq.cpu().numpy(), B_ref)
    assert np.array_equal(Cq.cpu().numpy(), C_ref)
    assert np.abs(x_ref).max() == 127


# --------------------------------------------------------------------------- calibration
@pytest.mark.parametrize("cfg", SMALL[:3], ids=lambda c: c.name)
def test_calibrate_bit_exact(cfg):
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    t = inputs.make_prefill(cfg)
    init = inputs.make_init_state(cfg, 0.3)
    q = orc.prepare_quantized(cfg, t, init)
    dims = bd.dims_of(cfg)
    dv = {k: gh.dev(q[k]) for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A")}
    args = bd.make_fwd_args(init_state=gh.dev(init), **dv)
    s_xs = torch.empty(cfg.channels, device="cuda"); s_cb = torch.empty(cfg.ngroups, device="cuda")
    s_h = torch.empty(cfg.channels, device="cuda")
    ws = bd.alloc_workspace(dims)
    bd.ssdi8_calibrate(dims, args, s_xs, s_cb, s_h, ws)
    torch.cuda.synchronize()
    assert np.array_equal(s_xs.cpu().numpy(), q["s_xs"])
    assert np.array_equal(s_cb.cpu().numpy(), q["s_cb"])
    assert np.array_equal(s_h.cpu().numpy(), q["s_h"])


# --------------------------------------------------------------------------- state passing
@pytest.mark.parametrize("alias", [False, True])
def test_state_passing_standalone(alias):
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    cfg = SSDConfig("sp", 2, 6 * 64, 3, 64, 128, 1, 64, 0, 1, 31)
    rng = np.random.default_rng(31)
    shp = (cfg.batch, cfg.nchunks, cfg.nheads, cfg.headdim, cfg.dstate)
    loc = rng.standard_normal(shp).astype(np.float32)
    gamma = rng.uniform(0.0, 1.0, (cfg.batch, cfg.nheads, cfg.nchunks)).astype(np.float32)
    init = rng.standard_normal(shp[:1] + shp[2:]).astype(np.float32)
    s_h = rng.uniform(0.01, 0.05, cfg.channels).astype(np.float32)
    prev_ref, fin_ref, hq_ref = orc.state_passing(cfg, loc, gamma, init, s_h)
    dloc = gh.dev(loc)
    prev = dloc if alias else torch.empty_like(dloc)
    fin = torch.empty(shp[:1] + shp[2:], device="cuda")
    hq = torch.empty(shp, dtype=torch.int8, device="cuda")
    bd.ssdi8_state_passing(bd.dims_of(cfg), dloc, gh.dev(gamma), gh.dev(init), prev, fin, hq, gh.dev(s_h))
    torch.cuda.synchronize()
    assert np.array_equal(prev.cpu().numpy(), prev_ref)
    assert np.array_equal(fin.cpu().numpy(), fin_ref)
    assert np.array_equal(hq.cpu().numpy(), hq_ref)


# --------------------------------------------------------------------------- decode step
def _decode_case(cfg, steps):
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    prm = inputs.make_decode_params(cfg)
    raw = [inputs.make_decode_step(cfg, s) for s in range(steps)]
    # static scales over all steps (Eq. 1, observe mode)
    s_x = np.zeros(cfg.channels, np.float32); s_B = np.zeros(cfg.ngroups, np.float32)
    s_C = np.zeros(cfg.ngroups, np.float32)
    for r in raw:
        _, s_x = orc.quantize(r["x"], cfg.batch, cfg.channels, 1, scale=s_x, mode=2, want_out=False)
        _, s_B = orc.quantize(r["B"], cfg.batch, cfg.ngroups, cfg.dstate, scale=s_B, mode=2, want_out=False)
        _, s_C = orc.quantize(r["C"], cfg.batch, cfg.ngroups, cfg.dstate, scale=s_C, mode=2, want_out=False)
    corr = np.linspace(-0.2, 0.2, cfg.channels).astype(np.float32)
    st_ref = np.zeros((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate))
    state = torch.zeros(st_ref.shape, device="cuda")
    y = torch.empty((cfg.batch, cfg.nheads, cfg.headdim), device="cuda")
    dims = bd.dims_of(cfg)
    d = {k: gh.dev(v) for k, v in dict(s_x=s_x, s_B=s_B, s_C=s_C, A=prm["A"], D=prm["D"], corr=corr).items()}
    worst = 0.0
    for r in raw:
        xq, _ = orc.quantize(r["x"], cfg.batch, cfg.channels, 1, scale=s_x, mode=0)
        Bq, _ = orc.quantize(r["B"], cfg.batch, cfg.ngroups, cfg.dstate, scale=s_B, mode=0)
        Cq, _ = orc.quantize(r["C"], cfg.batch, cfg.ngroups, cfg.dstate, scale=s_C, mode=0)
        y_ref = orc.ssd_step(cfg, xq, s_x, Bq, s_B, Cq, s_C, r["dt"], prm["A"], prm["D"], corr, st_ref)
        bd.ssdi8_ssd_step(dims, gh.dev(xq), d["s_x"], gh.dev(Bq), d["s_B"], gh.dev(Cq), d["s_C"],
                          gh.dev(r["dt"]), d["A"], d["D"], d["corr"], state, y)
        worst = max(worst, np.abs(y.cpu().numpy() - y_ref).max() / rms(y_ref))
    assert worst <= Y_TOL
    got = state.cpu().numpy()
    assert np.abs(got - st_ref).max() <= Y_TOL * rms(st_ref)


def test_step_256_tokens_small_batch():
    _decode_case(CONFIGS["cfg4"].replace(batch=2, nheads=8), 256)


def test_step_n64_groups():
    _decode_case(SSDConfig("dec64", 3, 1, 4, 64, 64, 2, 64, 0.02, 20.0, 41, decode_steps=16), 16)


def test_step_full_size_batch():
    _decode_case(CONFIGS["cfg4"], 8)


def test_step_full_size_batch_all_256_steps():
    """cfg4 as specified: batch 64, 256 steps; y of every step and the state after the last one."""
    _decode_case(CONFIGS["cfg4"], 256)


# --------------------------------------------------------------------------- host-buffer entry point
@pytest.mark.parametrize("batch", [3, 1])
@pytest.mark.parametrize("flags", [0, 2])
def test_layer_fwd_host_matches_the_device_path_bit_for_bit(flags, batch):
    """ssdi8_layer_fwd_host (pinned host tensors in, pipelined per batch element) == Eq. 1 quantiser +
    ssdi8_chunk_scan_fwd on the whole batch, and the oracle agrees with both; twice in a row
    (the second call reuses the side streams and both scratch stages)."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    cfg = SSDConfig("host_b", batch, 256, 4, 64, 64, 2, 128, 0.02, 20.0, 31)   # odd batch: both stages, ragged; 1: one stage
    t = inputs.make_prefill(cfg)
    init = inputs.make_init_state(cfg, 0.3)
    q = orc.prepare_quantized(cfg, t, init)
    y_ref, fin_ref, _ = orc.ssdi8_fwd(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], q["dt"],
                                      q["A"], q["D"], None, q["s_xs"], q["s_cb"], q["s_h"], init, flags=flags)
    q["init"] = init
    y_dev, fin_dev, _ = gh.gpu_fwd(cfg, q, taps=(), flags=flags)
    dims = bd.dims_of(cfg)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    host = {k: pin(t[k]) for k in ("x", "B", "C", "dt")}
    y = torch.empty(t["x"].shape).pin_memory()
    fin = torch.empty(init.shape).pin_memory()
    status = torch.full((1,), -99, dtype=torch.int32).pin_memory()
    dv = {k: gh.dev(q[k]) for k in ("s_x", "s_B", "s_C", "s_xs", "s_cb", "s_h", "A", "D")}
    args = bd.make_host_args(y=y, final_state=fin, status=status, init_state=gh.dev(init), **host, **dv)
    scratch = torch.empty(bd.ssdi8_layer_fwd_host_scratch_bytes(dims, flags), dtype=torch.uint8, device="cuda")
    for rep in range(2):
        y.fill_(float("nan")); fin.fill_(float("nan"))
        bd.ssdi8_layer_fwd_host(dims, args, scratch, flags)
        torch.cuda.synchronize()
        assert int(status[0]) == 0
        assert np.array_equal(fin.numpy(), fin_ref)
        assert np.abs(y.numpy() - y_ref).max() <= Y_TOL * rms(y_ref)
        assert np.array_equal(y.numpy(), y_dev) and np.array_equal(fin.numpy(), fin_dev)


@pytest.mark.parametrize("flags", [0, 1, 3], ids=["default", "fp16_operand", "fp16_operand_int8_state"])
@pytest.mark.parametrize("cfg", [SMALL[1], SMALL[3]], ids=lambda c: c.name)
def test_layer_fwd_matches_the_separate_calls_bit_for_bit(cfg, flags):
    """ssdi8_layer_fwd (fp32 device tensors in, side-stream overlap inside) == three quantiser calls +
    ssdi8_chunk_scan_fwd; run three times in a row on the same workspace."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    t = inputs.make_prefill(cfg)
    q = orc.prepare_quantized(cfg, t)
    y_dev, fin_dev, _ = gh.gpu_fwd(cfg, q, taps=(), flags=flags)
    dims = bd.dims_of(cfg)
    dv = {k: gh.dev(q[k]) for k in ("s_x", "s_B", "s_C", "s_xs", "s_cb", "s_h", "A", "D")}
    dv.update({k: gh.dev(t[k]) for k in ("x", "B", "C", "dt")})
    y = torch.empty(t["x"].shape, device="cuda")
    fin = torch.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = bd.make_layer_args(y=y, final_state=fin, status=status, **dv)
    ws = torch.empty(bd.ssdi8_layer_fwd_workspace_bytes(dims, flags), dtype=torch.uint8, device="cuda")
    for rep in range(3):
        y.fill_(float("nan")); fin.fill_(float("nan"))
        bd.ssdi8_layer_fwd(dims, args, ws, flags)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert np.array_equal(y.cpu().numpy(), y_dev) and np.array_equal(fin.cpu().numpy(), fin_dev)


def test_layer_fwd_back_to_back_on_one_workspace_with_alternating_inputs():
    """The kernels of consecutive calls overlap at their edges (programmatic dependent launch: a kernel may be
    scheduled while its predecessor drains, and ChunkBMM runs beside the state kernel), and all calls share
    one workspace.  Forty calls without a synchronisation in between, alternating between two inputs and two
    outputs: every call must still produce what the same call produces alone."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    cfg = SSDConfig("b2b", 2, 1024, 24, 64, 128, 2, 256, 0.02, 20.0, 61)
    dims = bd.dims_of(cfg)
    sets = []
    for seed in (61, 62):
        t = inputs.make_prefill(cfg.replace(seed=seed))
        q = orc.prepare_quantized(cfg, t)
        dv = {k: gh.dev(q[k]) for k in ("s_x", "s_B", "s_C", "s_xs", "s_cb", "s_h", "A", "D")}
        dv.update({k: gh.dev(t[k]) for k in ("x", "B", "C", "dt")})
        y = torch.empty(t["x"].shape, device="cuda")
        fin = torch.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        sets.append(dict(args=bd.make_layer_args(y=y, final_state=fin, status=status, **dv), y=y, fin=fin, status=status))
    ws = torch.empty(bd.ssdi8_layer_fwd_workspace_bytes(dims), dtype=torch.uint8, device="cuda")
    ref = []
    for s_ in sets:   # each call alone
        bd.ssdi8_layer_fwd(dims, s_["args"], ws)
        torch.cuda.synchronize()
        ref.append((s_["y"].clone(), s_["fin"].clone()))
        s_["y"].fill_(float("nan")); s_["fin"].fill_(float("nan"))
    for i in range(40):
        bd.ssdi8_layer_fwd(dims, sets[i & 1]["args"], ws)
    torch.cuda.synchronize()
    for s_, (y0, f0) in zip(sets, ref):
        assert int(s_["status"].item()) == 0
        assert torch.equal(s_["y"], y0) and torch.equal(s_["fin"], f0)
    # and Algorithm 2 alone (ssdi8_chunk_scan_fwd) the same way, on the int8 tensors of the first input
    t = inputs.make_prefill(cfg.replace(seed=61))
    q = orc.prepare_quantized(cfg, t)
    y_a, fin_a, _ = gh.gpu_fwd(cfg, q, taps=())
    dq = {k: gh.dev(q[k]) for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "D", "s_xs", "s_cb", "s_h")}
    y = torch.empty(t["x"].shape, device="cuda")
    fin = torch.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), device="cuda")
    args = bd.make_fwd_args(y=y, final_state=fin, **dq)
    ws2 = bd.alloc_workspace(dims)
    for i in range(40):
        bd.ssdi8_chunk_scan_fwd(dims, args, ws2)
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy(), y_a) and np.array_equal(fin.cpu().numpy(), fin_a)


def test_layer_fwd_and_decode_steps_replay_from_a_cuda_graph():
    """The library's calls are stream work only (no allocation, no synchronisation, no host read of a device
    value), so a caller can capture them into a CUDA graph and replay it: the layer forward (five kernels
    chained by programmatic dependent launch) and a run of decode steps, each replayed on new input values
    written into the captured buffers, must equal the same calls made directly."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    cfg = SSDConfig("graph", 2, 512, 6, 64, 128, 2, 128, 0.02, 20.0, 71)
    dims = bd.dims_of(cfg)
    data = []
    for seed in (71, 72):
        t = inputs.make_prefill(cfg.replace(seed=seed))
        data.append({k: gh.dev(t[k]) for k in ("x", "B", "C", "dt")})
    t = inputs.make_prefill(cfg)
    q = orc.prepare_quantized(cfg, t)
    dv = {k: gh.dev(q[k]) for k in ("s_x", "s_B", "s_C", "s_xs", "s_cb", "s_h", "A", "D")}
    buf = {k: torch.empty_like(v) for k, v in data[0].items()}       # the captured input buffers
    y = torch.empty(t["x"].shape, device="cuda")
    fin = torch.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = bd.make_layer_args(y=y, final_state=fin, status=status, **dv, **buf)
    ws = torch.empty(bd.ssdi8_layer_fwd_workspace_bytes(dims), dtype=torch.uint8, device="cuda")
    ref = []
    for dset in data:   # direct calls
        for k in buf:
            buf[k].copy_(dset[k])
        bd.ssdi8_layer_fwd(dims, args, ws)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref.append((y.clone(), fin.clone()))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):   # (torch asks for a warm-up on a side stream before a capture)
        bd.ssdi8_layer_fwd(dims, args, ws)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        bd.ssdi8_layer_fwd(dims, args, ws)
    for rep in range(3):
        for dset, (y0, f0) in zip(data, ref):
            for k in buf:
                buf[k].copy_(dset[k])
            y.fill_(float("nan")); fin.fill_(float("nan"))
            g.replay()
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert torch.equal(y, y0) and torch.equal(fin, f0)

    # decode: four steps per graph, the state carried in place from replay to replay
    dc = CONFIGS["cfg4"].replace(batch=4, nheads=8)
    ddims = bd.dims_of(dc)
    prm = inputs.make_decode_params(dc)
    nsteps = 12
    raw = [inputs.make_decode_step(dc, s_) for s_ in range(nsteps)]
    s_x = np.zeros(dc.channels, np.float32); s_B = np.zeros(dc.ngroups, np.float32); s_C = np.zeros(dc.ngroups, np.float32)
    for r in raw:
        _, s_x = orc.quantize(r["x"], dc.batch, dc.channels, 1, scale=s_x, mode=2, want_out=False)
        _, s_B = orc.quantize(r["B"], dc.batch, dc.ngroups, dc.dstate, scale=s_B, mode=2, want_out=False)
        _, s_C = orc.quantize(r["C"], dc.batch, dc.ngroups, dc.dstate, scale=s_C, mode=2, want_out=False)
    codes = []
    for r in raw:
        codes.append(dict(xq=gh.dev(orc.quantize(r["x"], dc.batch, dc.channels, 1, scale=s_x, mode=0)[0]),
                          Bq=gh.dev(orc.quantize(r["B"], dc.batch, dc.ngroups, dc.dstate, scale=s_B, mode=0)[0]),
                          Cq=gh.dev(orc.quantize(r["C"], dc.batch, dc.ngroups, dc.dstate, scale=s_C, mode=0)[0]),
                          dt=gh.dev(r["dt"])))
    d = {k: gh.dev(v) for k, v in dict(s_x=s_x, s_B=s_B, s_C=s_C, A=prm["A"], D=prm["D"]).items()}
    shape_state = (dc.batch, dc.nheads, dc.headdim, dc.dstate)

    def step(c, state, yy):
        bd.ssdi8_ssd_step(ddims, c["xq"], d["s_x"], c["Bq"], d["s_B"], c["Cq"], d["s_C"], c["dt"], d["A"], d["D"], None,
                          state, yy)

    state_ref = torch.zeros(shape_state, device="cuda")
    y_ref = [torch.empty((dc.batch, dc.nheads, dc.headdim), device="cuda") for _ in range(nsteps)]
    for i in range(nsteps):
        step(codes[i], state_ref, y_ref[i])
    torch.cuda.synchronize()
    slots = [{k: torch.empty_like(v) for k, v in codes[0].items()} for _ in range(4)]
    ys = [torch.empty_like(y_ref[0]) for _ in range(4)]
    state = torch.zeros(shape_state, device="cuda")
    with torch.cuda.stream(side):
        side.wait_stream(torch.cuda.current_stream())
        warm = torch.zeros(shape_state, device="cuda")
        for j in range(4):
            for k in slots[j]:
                slots[j][k].copy_(codes[j][k])
            step(slots[j], warm, ys[j])
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g2 = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g2):
        for j in range(4):
            step(slots[j], state, ys[j])
    state.zero_()
    for i0 in range(0, nsteps, 4):
        for j in range(4):
            for k in slots[j]:
                slots[j][k].copy_(codes[i0 + j][k])
        g2.replay()
        torch.cuda.synchronize()
        for j in range(4):
            assert torch.equal(ys[j], y_ref[i0 + j])
    assert torch.equal(state, state_ref)


def test_layer_fwd_host_rejects_a_short_scratch():
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    cfg = SMALL[0]
    dims = bd.dims_of(cfg)
    z = torch.zeros(16).pin_memory()
    d = gh.dev(np.zeros(16, np.float32))
    args = bd.make_host_args(x=z, B=z, C=z, dt=z, y=z, A=d, s_x=d, s_B=d, s_C=d, s_xs=d, s_cb=d, s_h=d)
    scratch = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(bd.SSDi8Error) as e:
        bd.ssdi8_layer_fwd_host(dims, args, scratch)
    assert e.value.code == bd.ERR_WORKSPACE


# --------------------------------------------------------------------------- 16-bit y
@pytest.mark.parametrize("fmt", ["float16", "bfloat16"])
@pytest.mark.parametrize("cfg", [SMALL[0], SMALL[1], SMALL[3]], ids=lambda c: c.name)
def test_fwd_16_bit_y(cfg, fmt):
    """SSDI8_FLAG_Y_FP16 / _BF16: y leaves the epilogue rounded to nearest even into the 16-bit
    format.  Checked two ways: bit for bit against the kernel's own binary32 y converted by the
    library routine, and against the oracle's y within the fp32 tolerance plus half a 16-bit ulp."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    t = inputs.make_prefill(cfg)
    q = orc.prepare_quantized(cfg, t)
    y_ref, fin_ref, _ = orc.ssdi8_fwd(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], q["dt"],
                                      q["A"], q["D"], None, q["s_xs"], q["s_cb"], q["s_h"], None)
    y32, fin32, _ = gh.gpu_fwd(cfg, q, taps=())
    td = getattr(torch, fmt)
    flag = bd.FLAG_Y_FP16 if fmt == "float16" else bd.FLAG_Y_BF16
    dims = bd.dims_of(cfg)
    dv = {k: gh.dev(q[k]) for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "D", "s_xs", "s_cb", "s_h")}
    y16 = torch.full(t["x"].shape, float("nan"), dtype=td, device="cuda")
    fin = torch.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = bd.make_fwd_args(y=y16, final_state=fin, status=status, **dv)
    bd.ssdi8_chunk_scan_fwd(dims, args, bd.alloc_workspace(dims), flags=flag)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(fin.cpu().numpy(), fin32)
    want = torch.from_numpy(y32).to(td)
    assert torch.equal(y16.cpu().view(torch.int16), want.view(torch.int16))
    half_ulp = 2.0 ** -11 if fmt == "float16" else 2.0 ** -8
    err = np.abs(y16.float().cpu().numpy() - y_ref)
    assert np.all(err <= Y_TOL * rms(y_ref) + 1.01 * half_ulp * np.abs(y_ref) + 1e-7)


def test_16_bit_y_flags_are_exclusive_and_without_taps():
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    cfg = SMALL[0]
    t = inputs.make_prefill(cfg)
    q = orc.prepare_quantized(cfg, t)
    dims = bd.dims_of(cfg)
    dv = {k: gh.dev(q[k]) for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "D", "s_xs", "s_cb", "s_h")}
    y16 = torch.empty(t["x"].shape, dtype=torch.float16, device="cuda")
    ws = bd.alloc_workspace(dims)
    with pytest.raises(bd.SSDi8Error) as e:
        bd.ssdi8_chunk_scan_fwd(dims, bd.make_fwd_args(y=y16, **dv), ws, flags=bd.FLAG_Y_FP16 | bd.FLAG_Y_BF16)
    assert e.value.code == bd.ERR_UNSUPPORTED
    tap = torch.zeros((cfg.batch, cfg.seqlen, cfg.nheads), device="cuda")
    with pytest.raises(bd.SSDi8Error) as e:
        bd.ssdi8_chunk_scan_fwd(dims, bd.make_fwd_args(y=y16, tap_rowmax=tap, **dv), ws, flags=bd.FLAG_Y_FP16)
    assert e.value.code == bd.ERR_UNSUPPORTED
    torch.cuda.synchronize()



@pytest.mark.parametrize("fmt", ["float16", "bfloat16"])
@pytest.mark.parametrize("operand", [0, 1], ids=["int8_operand", "fp16_operand"])
def test_fwd_16_bit_y_with_correction_and_init_state(operand, fmt):
    """The mean-correction vector (Eq. 8) and an initial state together with 16-bit y, for both operand
    formats of ChunkScan2: the 16-bit y is the kernel's own binary32 y of the same call rounded to
    nearest even, and that binary32 y agrees with the oracle."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    cfg = SMALL[2]
    t = inputs.make_prefill(cfg)
    init = inputs.make_init_state(cfg, 0.3)
    q = orc.prepare_quantized(cfg, t, init)
    corr = (0.05 * np.random.default_rng(5).standard_normal(cfg.channels)).astype(np.float32)
    y_ref, fin_ref, _ = orc.ssdi8_fwd(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], q["dt"],
                                      q["A"], q["D"], corr, q["s_xs"], q["s_cb"], q["s_h"], init, flags=operand)
    y32, fin32, _ = gh.gpu_fwd(cfg, q, corr=corr, taps=(), flags=operand)
    assert np.array_equal(fin32, fin_ref)
    assert np.abs(y32 - y_ref).max() <= Y_TOL * rms(y_ref)
    td = getattr(torch, fmt)
    flag = operand | (bd.FLAG_Y_FP16 if fmt == "float16" else bd.FLAG_Y_BF16)
    dims = bd.dims_of(cfg)
    dv = {k: gh.dev(q[k]) for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "D", "s_xs", "s_cb", "s_h")}
    y16 = torch.full(t["x"].shape, float("nan"), dtype=td, device="cuda")
    fin = torch.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = bd.make_fwd_args(y=y16, final_state=fin, status=status, corr=gh.dev(corr), init_state=gh.dev(init), **dv)
    bd.ssdi8_chunk_scan_fwd(dims, args, bd.alloc_workspace(dims, flags=flag), flags=flag)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(fin.cpu().numpy(), fin32)
    want = torch.from_numpy(y32).to(td)
    assert torch.equal(y16.cpu().view(torch.int16), want.view(torch.int16))

# --------------------------------------------------------------------------- the paper's FP16 ChunkScan2 operand
@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
def test_fwd_fp16_operand_against_the_oracle_mode(cfg):
    """SSDI8_FLAG_FP16_OPERAND: the masked operand in FP16 in tensor memory, kind::f16 MMA.  y within
    the fp32 tolerance of the oracle's FP16-operand mode (the operand is formed in binary32 before its
    rounding to FP16, the oracle forms it in binary64: single FP16 ulps may differ); the states, which
    this mode does not touch, bit for bit."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    gh = _harness()
    t = inputs.make_prefill(cfg)
    init = inputs.make_init_state(cfg, 0.3)
    q = orc.prepare_quantized(cfg, t, init)
    y_ref, fin_ref, _ = orc.ssdi8_fwd(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], q["dt"],
                                      q["A"], q["D"], None, q["s_xs"], q["s_cb"], q["s_h"], init,
                                      flags=orc.FLAG_FP16_OPERAND)
    dims = bd.dims_of(cfg)
    dv = {k: gh.dev(q[k]) for k in ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "D", "s_xs", "s_cb", "s_h")}
    y = torch.full(t["x"].shape, float("nan"), device="cuda")
    fin = torch.empty(init.shape, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = bd.make_fwd_args(y=y, final_state=fin, status=status, init_state=gh.dev(init), **dv)
    ws = bd.alloc_workspace(dims, flags=bd.FLAG_FP16_OPERAND)
    for rep in range(2):
        y.fill_(float("nan"))
        bd.ssdi8_chunk_scan_fwd(dims, args, ws, flags=bd.FLAG_FP16_OPERAND)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert np.array_equal(fin.cpu().numpy(), fin_ref)
        err = np.abs(y.cpu().numpy() - y_ref).max()
        assert err <= Y_TOL * rms(y_ref), err / rms(y_ref)
    # with the paper's output format as well
    y16 = torch.full(t["x"].shape, float("nan"), dtype=torch.float16, device="cuda")
    args16 = bd.make_fwd_args(y=y16, final_state=fin, status=status, init_state=gh.dev(init), **dv)
    bd.ssdi8_chunk_scan_fwd(dims, args16, ws, flags=bd.FLAG_FP16_OPERAND | bd.FLAG_Y_FP16)
    torch.cuda.synchronize()
    assert torch.equal(y16.cpu().view(torch.int16), y.cpu().half().view(torch.int16))


@pytest.mark.parametrize("G", [1, 8])
def test_layer_fwd_host_with_head_range_slices(G):
    """A batch element whose x exceeds 96 MB is cut into head ranges by the host entry (strided
    copies, offset step-size vectors, per-range groups): the result must equal the whole-batch
    device call bit for bit.  Scales come from the library's own calibration (parity of every
    kernel with the oracle is established by the tests above)."""
    import torch
    from paper_2608_21952_b200 import binding as bd
    cfg = SSDConfig("host_wide", 2, 4096, 128, 64, 64, G, 256, 0.01, 50.0, 41)   # 134 MB of x per element
    t = inputs.make_prefill(cfg)
    init = inputs.make_init_state(cfg, 0.2)
    dims = bd.dims_of(cfg)
    dv = {k: torch.from_numpy(t[k]).cuda() for k in ("x", "B", "C", "dt", "A", "D")}
    dinit = torch.from_numpy(init).cuda()
    T = cfg.tokens
    i8 = lambda k: torch.empty(t[k].shape, dtype=torch.int8, device="cuda")
    xq, Bq, Cq = i8("x"), i8("B"), i8("C")
    z = lambda n: torch.empty(n, device="cuda")
    s_x, s_B, s_C = z(cfg.channels), z(cfg.ngroups), z(cfg.ngroups)
    s_xs, s_cb, s_h = z(cfg.channels), z(cfg.ngroups), z(cfg.channels)
    bd.ssdi8_quantize_act(dv["x"], T, cfg.channels, 1, s_x, 1, xq)
    bd.ssdi8_quantize_act(dv["B"], T, cfg.ngroups, cfg.dstate, s_B, 1, Bq)
    bd.ssdi8_quantize_act(dv["C"], T, cfg.ngroups, cfg.dstate, s_C, 1, Cq)
    ws = bd.alloc_workspace(dims)
    cal = bd.make_fwd_args(xq=xq, Bq=Bq, Cq=Cq, s_x=s_x, s_B=s_B, s_C=s_C, dt=dv["dt"], A=dv["A"], init_state=dinit)
    bd.ssdi8_calibrate(dims, cal, s_xs, s_cb, s_h, ws)
    scales = dict(s_x=s_x, s_B=s_B, s_C=s_C, s_xs=s_xs, s_cb=s_cb, s_h=s_h, A=dv["A"], D=dv["D"])
    # whole-batch device call
    y_d = torch.empty(t["x"].shape, device="cuda")
    fin_d = torch.empty(init.shape, device="cuda")
    st_d = torch.zeros(1, dtype=torch.int32, device="cuda")
    a_d = bd.make_layer_args(x=dv["x"], B=dv["B"], C=dv["C"], dt=dv["dt"], init_state=dinit, y=y_d,
                             final_state=fin_d, status=st_d, **scales)
    lws = torch.empty(bd.ssdi8_layer_fwd_workspace_bytes(dims), dtype=torch.uint8, device="cuda")
    bd.ssdi8_layer_fwd(dims, a_d, lws)
    # host call: two head ranges per batch element
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    host = {k: pin(t[k]) for k in ("x", "B", "C", "dt")}
    y_h = torch.full(t["x"].shape, float("nan")).pin_memory()
    fin_h = torch.full(init.shape, float("nan")).pin_memory()
    st_h = torch.full((1,), -99, dtype=torch.int32).pin_memory()
    a_h = bd.make_host_args(y=y_h, final_state=fin_h, status=st_h, init_state=dinit, **host, **scales)
    need = bd.ssdi8_layer_fwd_host_scratch_bytes(dims)
    # sized for half of the heads: well below the need of the same element at half the length, uncut
    uncut = bd.ssdi8_layer_fwd_host_scratch_bytes(bd.dims_of(cfg.replace(seqlen=2048, nheads=64, ngroups=max(1, G // 2))))
    assert need < 2.2 * uncut
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
    bd.ssdi8_layer_fwd_host(dims, a_h, scratch)
    torch.cuda.synchronize()
    assert int(st_d.item()) == 0 and int(st_h[0]) == 0
    assert torch.equal(y_h, y_d.cpu()) and torch.equal(fin_h, fin_d.cpu())
