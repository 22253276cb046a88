"""The oracle's plain definitions (fp64, libm, one exponential per element) and how far the
binary32 operation-by-operation form used for bit-exact comparison may be from them.

Pins of the plain functions: special cases that reduce to an integer matrix product (numpy), the
unquantised dual form within the quantisation noise, Eq. 1's half-step bound per row, the numpy
restatements with float16.  Census: every code of the binary32 form equals the plain code or is its
neighbour with the fp64 value inside a derived window around the rounding boundary."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2608_21952_b200 import inputs
from paper_2608_21952_b200.inputs import CONFIGS
from helpers import TINY, TWO_BLOCK, census, dequant, half_neighbours, rms

ALL_TAPS = tuple(orc.TAP_SPECS)


def _case(cfg, init=None, corr=None, flags=0, taps=ALL_TAPS):
    t = inputs.make_prefill(cfg)
    q = orc.prepare_quantized(cfg, t, init)
    y, fin, tp = orc.ssdi8_fwd(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], q["dt"], q["A"],
                               q["D"], corr, q["s_xs"], q["s_cb"], q["s_h"], init, taps=taps, flags=flags)
    return t, q, y, fin, tp


def _plain_scan(cfg, q, tp, corr=None, flags=0):
    return orc.chunk_scan_plain(cfg, q["xq"], q["Cq"], tp["CBq"], tp["hq"], q["s_x"], q["s_C"], q["s_cb"],
                                q["s_h"], q["dt"], tp["cs"], q["D"], corr, flags=flags)


# --------------------------------------------------------------------------- pins of the plain functions
def test_plain_scan_without_decay_is_an_integer_matrix_product():
    """A = 0 makes every decay 1 and dt = 1/4 keeps every product exact: with trivial step sizes the
    FP16-operand ChunkScan2 is tril(CBq)/4 times xq and ChunkScan1 is Cq times hq, both integer
    matrix products that numpy evaluates exactly."""
    cfg = TINY
    rng = np.random.default_rng(21)
    b, L, H, P, N, G, Q, c = (cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim, cfg.dstate, cfg.ngroups,
                              cfg.chunk, cfg.nchunks)
    xq = rng.integers(-127, 128, (b, L, H, P)).astype(np.int8)
    Cq = rng.integers(-127, 128, (b, L, G, N)).astype(np.int8)
    CBq = rng.integers(-127, 128, (b, c, G, Q, Q)).astype(np.int8)
    hq = rng.integers(-127, 128, (b, c, H, P, N)).astype(np.int8)
    one_d, one_g = np.ones(H * P, np.float32), np.ones(G, np.float32)
    dt = np.full((b, L, H), 0.25, np.float32)
    cs = np.zeros((b, H, c, Q), np.float32)
    D = rng.integers(-3, 4, H).astype(np.float32)
    y, out = orc.chunk_scan_plain(cfg, xq, Cq, CBq, hq, one_d, one_g, one_g, one_d, dt, cs, D, None,
                                  flags=orc.FLAG_FP16_OPERAND)
    hg = np.arange(H) // (H // G)
    x5 = xq.astype(np.int64).reshape(b, c, Q, H, P)
    off = np.einsum("bcihn,bchpn->bcihp", Cq.astype(np.int64).reshape(b, c, Q, G, N)[:, :, :, hg], hq.astype(np.int64))
    diag = np.einsum("bchij,bcjhp->bcihp", np.tril(CBq.astype(np.int64))[:, :, hg], x5)
    want = off + diag / 4.0 + D[None, None, None, :, None] * x5
    assert np.array_equal(y, want.reshape(b, L, H, P))
    assert np.array_equal(out["M"], np.tril(CBq.astype(np.float64))[:, :, hg] / 4.0)


@pytest.mark.parametrize("cfg", [TINY, TWO_BLOCK, CONFIGS["cfg0"]], ids=lambda c: c.name)
def test_plain_scan_against_numpy(cfg):
    """M = s_cb CBq dt_j exp(cs_i - cs_j) on j <= i, Eq. 1 per row, and the output sum, restated with
    numpy broadcasting."""
    corr = np.linspace(-0.2, 0.2, cfg.channels).astype(np.float32)
    t, q, y_spec, fin, tp = _case(cfg, corr=corr)
    y, out = _plain_scan(cfg, q, tp, corr)
    b, c, Q, H, P, N, G = cfg.batch, cfg.nchunks, cfg.chunk, cfg.nheads, cfg.headdim, cfg.dstate, cfg.ngroups
    hg = np.arange(H) // (H // G)
    cs = tp["cs"].astype(np.float64).transpose(0, 2, 1, 3)                      # [b,c,H,Q]
    dt = q["dt"].astype(np.float64).reshape(b, c, Q, H).transpose(0, 1, 3, 2)    # [b,c,H,Q]
    tril = np.tril(np.ones((Q, Q), bool))
    with np.errstate(over="ignore"):
        lut = np.where(tril, np.exp(cs[..., :, None] - cs[..., None, :]), 0.0) * dt[..., None, :]
    M = q["s_cb"].astype(np.float64)[hg][None, None, :, None, None] * tp["CBq"].astype(np.float64)[:, :, hg] * lut
    assert np.allclose(out["M"], M, rtol=1e-13, atol=0)
    amax = np.abs(M).max(-1)
    sM = np.where(amax == 0, 1.0, amax / 127.0)
    assert np.allclose(out["sM"].reshape(b, c, Q, H).transpose(0, 1, 3, 2), sM, rtol=1e-13)
    # Eq. 1 per row: half a step, extreme element at +-127, nothing above the diagonal
    assert np.all(np.abs(out["Mq"] * sM[..., None] - M) <= 0.5 * sM[..., None] * (1 + 1e-12))
    assert np.all(np.abs(out["Mq"].astype(int)).max(-1)[amax > 0] == 127)
    assert np.all(np.triu(out["Mq"], 1) == 0)
    s_x = q["s_x"].astype(np.float64).reshape(H, P); s_h = q["s_h"].astype(np.float64).reshape(H, P)
    x5 = q["xq"].astype(np.float64).reshape(b, c, Q, H, P)
    diag = np.einsum("bchij,bcjhp->bcihp", out["Mq"].astype(np.float64), x5) * sM.transpose(0, 1, 3, 2)[..., None] * s_x
    Cq = q["Cq"].astype(np.float64).reshape(b, c, Q, G, N)[:, :, :, hg]
    off = np.einsum("bcihn,bchpn->bcihp", Cq, tp["hq"].astype(np.float64)) * np.exp(cs).transpose(0, 1, 3, 2)[..., None] \
        * q["s_C"].astype(np.float64)[hg][None, None, None, :, None] * s_h
    want = off + diag + q["D"].astype(np.float64)[None, None, None, :, None] * s_x * x5 + corr.reshape(H, P)
    assert np.abs(y - want.reshape(y.shape)).max() <= 1e-12 * rms(want)


@pytest.mark.parametrize("cfg", [TINY, TWO_BLOCK], ids=lambda c: c.name)
def test_plain_fp16_operand_against_numpy_half_arithmetic(cfg):
    """Section 4.2's ChunkScan2: y_diag = s_x sum_j half(s_cb CBq dt_j exp(cs_i - cs_j)) xq[j], the
    rounding done here by numpy's float16."""
    t, q, y8, fin, tp = _case(cfg)
    y16, out = _plain_scan(cfg, q, tp, flags=orc.FLAG_FP16_OPERAND)
    b, c, Q, H, P, G = cfg.batch, cfg.nchunks, cfg.chunk, cfg.nheads, cfg.headdim, cfg.ngroups
    hg = np.arange(H) // (H // G)
    s_x = q["s_x"].astype(np.float64).reshape(H, P)
    cs = tp["cs"].astype(np.float64); dt = q["dt"].astype(np.float64).reshape(b, c, Q, H)
    xq = q["xq"].astype(np.float64).reshape(b, c, Q, H, P)
    tril = np.tril(np.ones((Q, Q), bool))
    y_int8_plain, out8 = _plain_scan(cfg, q, tp)
    diag8 = np.einsum("bchij,bcjhp->bcihp", out8["Mq"].astype(np.float64), xq) \
        * out8["sM"].reshape(b, c, Q, H)[..., None] * s_x
    diag16 = np.zeros((b, c, Q, H, P))
    for bi in range(b):
        for k in range(c):
            for h in range(H):
                lut = dt[bi, k, :, h][None, :] * np.exp(cs[bi, h, k][:, None] - cs[bi, h, k][None, :])
                m = float(q["s_cb"][hg[h]]) * tp["CBq"][bi, k, hg[h]].astype(np.float64) * lut
                with np.errstate(over="ignore"):
                    m16 = np.where(tril, m, 0.0).astype(np.float16).astype(np.float64)
                diag16[bi, k, :, h, :] = (m16 @ xq[bi, k, :, h, :]) * s_x[h][None, :]
    want = y_int8_plain - diag8.reshape(y16.shape) + diag16.reshape(y16.shape)
    assert np.abs(y16 - want).max() <= 1e-9 * rms(want)


@pytest.mark.parametrize("cfg", [TINY, TWO_BLOCK, CONFIGS["cfg0"]], ids=lambda c: c.name)
@pytest.mark.parametrize("flags", [0, orc.FLAG_FP16_OPERAND], ids=["int8_operand", "fp16_operand"])
def test_plain_forward_close_to_unquantised_dual_form(cfg, flags):
    """The forward built from the plain definitions alone stays within the quantisation noise of
    Algorithm 2 in fp64 on the same dequantised inputs (a wrong index or a dropped factor is O(1))."""
    rng = np.random.default_rng(3)
    init = (0.1 * rng.standard_normal((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate))).astype(np.float32)
    corr = (0.01 * rng.standard_normal(cfg.channels)).astype(np.float32)
    t = inputs.make_prefill(cfg)
    q = orc.prepare_quantized(cfg, t, init)
    y, fin = orc.ssdi8_fwd_plain(cfg, q["xq"], q["Bq"], q["Cq"], q["s_x"], q["s_B"], q["s_C"], q["dt"], q["A"],
                                 q["D"], corr, q["s_xs"], q["s_cb"], q["s_h"], init, flags=flags)
    xh, Bh, Ch = dequant(cfg, q)
    y1, f1 = orc.ssd_chunked(cfg, xh, Bh, Ch, t["dt"], t["A"], t["D"], corr, init)
    assert np.sqrt(((y - y1) ** 2).sum() / (y1 ** 2).sum()) < 3e-2
    assert np.sqrt(((fin - f1) ** 2).sum() / (f1 ** 2).sum()) < 5e-2


def test_plain_chunk_state_and_state_codes_are_eq1_on_the_real_tensors():
    cfg = CONFIGS["cfg0"]
    t, q, y, fin, tp = _case(cfg)
    v, code = orc.chunk_state_plain(cfg, q["xq"], q["s_x"], q["s_xs"], q["dt"], tp["cs"])
    b, c, Q, H, P = cfg.batch, cfg.nchunks, cfg.chunk, cfg.nheads, cfg.headdim
    cs = tp["cs"].astype(np.float64)
    dt = q["dt"].astype(np.float64).reshape(b, c, Q, H)
    lut = dt * np.exp(cs[..., -1:] - cs).transpose(0, 2, 3, 1)
    real = q["xq"].astype(np.float64).reshape(b, c, Q, H, P) * q["s_x"].astype(np.float64).reshape(H, P) * lut[..., None]
    s_xs = q["s_xs"].astype(np.float64).reshape(H, P)
    assert np.allclose(v.reshape(real.shape) * s_xs, real, rtol=1e-13, atol=0)
    assert np.array_equal(code, np.clip(np.rint(v), -127, 127).astype(np.int8))
    assert np.abs(code.astype(int)).max() == 127           # s_xs was calibrated on this tensor
    vh, ch = orc.state_codes_plain(cfg, tp["prev"], q["s_h"])
    assert np.allclose(vh * q["s_h"].astype(np.float64).reshape(H, P)[None, None, :, :, None], tp["prev"], rtol=1e-13)
    assert np.array_equal(ch, np.clip(np.rint(vh), -127, 127).astype(np.int8))


# --------------------------------------------------------------------------- census: binary32 form vs plain form
CENSUS_CASES = [TINY, TWO_BLOCK, CONFIGS["cfg0"], CONFIGS["cfg1"]]


@pytest.mark.parametrize("cfg", CENSUS_CASES, ids=lambda c: c.name)
def test_census_binary32_codes_against_plain_definitions(cfg, capsys):
    """Each stage is fed the same inputs on both sides (the integer tensors of the stage before are
    exact, so nothing is forced that could differ)."""
    rng = np.random.default_rng(17)
    init = (0.1 * rng.standard_normal((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate))).astype(np.float32)
    t, q, y_spec, fin, tp = _case(cfg, init=init)
    report = {}
    # Q(X_scaled), Eq. 3
    v, _ = orc.chunk_state_plain(cfg, q["xq"], q["s_x"], q["s_xs"], q["dt"], tp["cs"])
    frac, worst, outside = census(tp["Xsq"], v, 4e-6)
    assert worst <= 1 and outside == 0
    report["Xsq"] = frac
    # Q(State), Eq. 4
    v, _ = orc.state_codes_plain(cfg, tp["prev"], q["s_h"])
    frac, worst, outside = census(tp["hq"], v, 4e-6)
    assert worst <= 1 and outside == 0
    report["hq"] = frac
    # per-row Eq. 1 of the masked operand
    y_plain, out = _plain_scan(cfg, q, tp)
    b, c, Q, H = cfg.batch, cfg.nchunks, cfg.chunk, cfg.nheads
    sM = out["sM"].reshape(b, c, Q, H).transpose(0, 1, 3, 2)[..., None]          # [b,c,H,Q,1]
    frac, worst, outside = census(tp["Mq"], out["M"] / sM, 1e-5)
    assert worst <= 1 and outside == 0
    report["Mq"] = frac
    hg = np.arange(H) // (H // cfg.ngroups)
    rowmax = tp["rowmax"].astype(np.float64) * q["s_cb"].astype(np.float64)[hg][None, None, :]
    amax = np.abs(out["M"]).max(-1).transpose(0, 1, 3, 2).reshape(b, c * Q, H)
    assert np.allclose(rowmax, amax, rtol=1e-5, atol=1e-36)
    # FP16 operand: equal or adjacent binary16 values
    y16_spec, m16_spec = orc.chunk_scan_fp16_operand(cfg, q["xq"], q["Cq"], tp["CBq"], tp["hq"], q["s_x"], q["s_C"],
                                                     q["s_cb"], q["s_h"], q["dt"], tp["cs"], q["D"])
    with np.errstate(over="ignore"):
        m16_plain = out["M"].astype(np.float16).astype(np.float64)
    assert np.all(half_neighbours(m16_plain, m16_spec))
    report["M16"] = float((m16_plain != m16_spec).mean())
    # outputs: the few neighbouring codes move y by a small multiple of one step of one term
    y16_plain, _ = orc.chunk_scan_plain(cfg, q["xq"], q["Cq"], tp["CBq"], tp["hq"], q["s_x"], q["s_C"], q["s_cb"],
                                        q["s_h"], q["dt"], tp["cs"], q["D"], None, flags=orc.FLAG_FP16_OPERAND,
                                        want_operand=False)
    report["y_rel_l2"] = float(np.sqrt(((y_spec - y_plain) ** 2).sum() / (y_plain ** 2).sum()))
    report["y16_rel_l2"] = float(np.sqrt(((y16_spec - y16_plain) ** 2).sum() / (y16_plain ** 2).sum()))
    assert report["y_rel_l2"] < 1e-3 and report["y16_rel_l2"] < 1e-4
    with capsys.disabled():
        print(f"\n[census {cfg.name}] differing fraction " +
              ", ".join(f"{k} {v:.2e}" for k, v in report.items()))


def test_prop1_mse_of_the_reformulation_does_not_exceed_the_alternative(capsys):
    """Proposition 1 (Appendix A) with the two quantities as its proof defines them: the error of
    Q(X_scaled) as an expectation per element (Step 2), the error of Q(X) (.) LUT_state as a squared
    norm over the l axis (Step 3).  On the synthetic workloads the first does not exceed the second;
    Q(X_scaled) is mostly zeros (Section 4.2).  Per element on both sides the order is the other way
    round on these inputs (LUT_state spans many orders of magnitude within a chunk, so an error that is
    scaled by it afterwards is small wherever it is small); both figures are printed."""
    for name in ("cfg0", "cfg1"):
        cfg = CONFIGS[name]
        t = inputs.make_prefill(cfg)
        cs = orc.chunk_cumsum(cfg, t["dt"], t["A"])
        mse_scaled, mse_x_elem, zeros, mse_x_vec = orc.prop1_mse(cfg, t["x"], t["dt"], cs)
        assert 0 < mse_scaled <= mse_x_vec
        assert zeros > 0.5
        with capsys.disabled():
            print(f"\n[prop1 {name}] MSE Q(X_scaled) {mse_scaled:.3e} per element; Q(X)(.)LUT {mse_x_elem:.3e} per "
                  f"element, {mse_x_vec:.3e} per l-vector; zero codes {zeros:.3f}")


def test_prop1_mse_against_numpy():
    cfg = TINY
    t = inputs.make_prefill(cfg)
    cs = orc.chunk_cumsum(cfg, t["dt"], t["A"])
    got = orc.prop1_mse(cfg, t["x"], t["dt"], cs)
    b, c, Q, H, P = cfg.batch, cfg.nchunks, cfg.chunk, cfg.nheads, cfg.headdim
    c64 = cs.astype(np.float64)
    lut = (t["dt"].astype(np.float64).reshape(b, c, Q, H) * np.exp(c64[..., -1:] - c64).transpose(0, 2, 3, 1))[..., None]
    x = t["x"].astype(np.float64).reshape(b, c, Q, H, P)
    yv = x * lut
    sx = np.abs(x).max((0, 1, 2)) / 127; sy = np.abs(yv).max((0, 1, 2)) / 127
    qy = np.clip(np.rint(yv / sy), -127, 127); qx = np.clip(np.rint(x / sx), -127, 127)
    e2 = (sx * qx * lut - yv) ** 2
    want = (((sy * qy - yv) ** 2).mean(), e2.mean(), (qy == 0).mean(), e2.sum(2).mean())
    assert np.allclose(got, want, rtol=1e-12)


# --------------------------------------------------------------------------- softplus of the raw time step
def test_softplus_dt_against_numpy_and_its_limits():
    """Algorithm 2 module 1 starts from dt = softplus(dt_raw + bias).  The plain function is libm's; the
    operation-by-operation binary64 sequence agrees with numpy.logaddexp(0, v) to a few 1e-16 before the
    rounding to binary32, so that the two binary32 results differ (by one unit) in fewer than one element
    in a million; large |v| reduce to v and to exp(v)."""
    rng = np.random.default_rng(31)
    H = 6
    raw = np.concatenate([rng.normal(-3, 1.5, (40000, H)), rng.uniform(-90, 90, (20000, H)),
                          np.array([[0, -0.0, 1e-30, -1e-30, 50, -50]] * 2)]).astype(np.float32)
    bias = rng.normal(0, 0.5, H).astype(np.float32)
    v = (raw + bias).astype(np.float64)                       # binary32 sum, widened
    want64 = np.logaddexp(0.0, v)
    plain = orc.softplus_dt(raw, bias, plain=True)
    spec = orc.softplus_dt(raw, bias)
    assert np.mean(plain != want64.astype(np.float32)) < 1e-6
    assert np.mean(plain != spec) < 1e-6
    assert np.mean(spec != want64.astype(np.float32)) < 1e-6
    normal = want64 > 1.2e-38                                  # (binary32 subnormals round more coarsely)
    assert np.all(np.abs(spec.astype(np.float64) - want64)[normal] <= 6.0e-8 * want64[normal])
    assert np.all(spec[normal] > 0)
    big = orc.softplus_dt(np.array([[60.0, -60.0]], np.float32))
    assert big[0, 0] == np.float32(60.0) and abs(float(big[0, 1]) / np.exp(-60.0) - 1) < 1e-6
    assert orc.softplus_dt(np.zeros((1, 1), np.float32))[0, 0] == np.float32(np.log(2.0))
    # without a bias the raw value is used as it is
    assert np.array_equal(orc.softplus_dt(raw, None), orc.softplus_dt(raw, np.zeros(H, np.float32)))
