#!/usr/bin/env python
"""Benchmark of the B200 INT8 SSD layer (SSDi8 hot path).

One step = one pass of the whole hot path over one batch of seeded synthetic input:
Eq. 1 quantisation of fp32 x, B, C with static step sizes (one launch), then the
layer forward (ChunkCumsum, ChunkBMM, fused ChunkState+StatePassing, ChunkScan)
from int8 x, B, C to the fp32 output y and the final state.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

N > 1: one rank per GPU under torch.distributed.run (started by the caller, or by this
script itself when WORLD_SIZE is not in the environment).  The layer shards over
(batch, head) with no exchange, so every rank runs the same workload on its own
GPU (weak scaling, no data-path collective); the time is the maximum over ranks.

The K timed steps are repeated as rounds (each bracketed by a barrier and a device
synchronisation) until at least half a second has been timed; `ms_per_step` is the median
round, so that the clock record covers hundreds of samples.  Every timed call carries a
status word that must read 0 after its round, and after the timed loop the output and final
state of the last step are compared with the CPU oracle (`parity`); a failure exits non-zero.

Prints ONE JSON line.  `--impl reference` times the CPU oracle (as it stands) on
the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2608_21952_b200 import inputs  # noqa: E402

METRIC = "int8_ssd_layer_tokens_per_s"
UNIT = "tokens/s"
# Paper's own figure for this metric and workload, derived from its block-latency table
# (SSD module of block 55, Mamba-2 2.7B, batch 8, L = 2048: 4.481 ms on an RTX A5000):
# 16384 tokens / 4.481 ms.  Another machine's number: context, not the target.
PAPER_TOKENS_PER_S = {"cfg2": 16384 / 4.481e-3}
# Figures read from ncu captures (a number taken under a profiler is never a bench value; these are
# byte counts and a pipe utilisation, which do not depend on the clock): DRAM bytes per launch
# (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel and of the decode step kernel,
# and the tensor-pipe active share of the scan kernel, each with the summary file it comes from.
NCU_SCAN = {"cfg2": {"traffic": 435.5e6, "tensor_active_pct": 8.8,
                     "source": "profiles/chunk_scan_cfg2_ncu_full.md"}}
NCU_TRAFFIC_BYTES_DECODE = 276.6e6  # ssd_step_kernel at cfg4: profiles/launch_list_bench_cfg2.md
INT8_NOMINAL_TOPS = 4500.0          # dense INT8 figure of the B200 data sheet
MIN_TIMED_SECONDS = 0.5


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


def scan_algorithmic_bytes(cfg) -> int:
    """Bytes the chunk-scan kernel must move per launch: int8 x and fp32 y once per
    (token, head), the int8 state once per (chunk, head), C and the causal half of CBq once
    per (chunk, group), dt and cs once per (token, head)."""
    T, H, P, N, G, Q, c = cfg.tokens, cfg.nheads, cfg.headdim, cfg.dstate, cfg.ngroups, cfg.chunk, cfg.nchunks
    per_token_head = P * 1 + P * 4 + 4 + 4
    state = cfg.batch * c * H * P * N
    group = T * G * N + cfg.batch * c * G * (Q * (Q + 1) // 2)
    return T * H * per_token_head + state + group


def layer_ideal_bytes(cfg) -> int:
    """Bytes Algorithm 2 must move from the int8 tensors to y if nothing were written and read back:
    int8 x, B, C and fp32 dt in, fp32 y and the final state out."""
    T = cfg.tokens
    return (T * cfg.channels + 2 * T * cfg.ngroups * cfg.dstate + T * cfg.nheads * 4 +
            T * cfg.channels * 4 + cfg.batch * cfg.channels * cfg.dstate * 4)


def scan_mma_ops(cfg) -> float:
    """Integer operations (2 per multiply-accumulate) of the MMAs the scan kernel issues: per 128-row
    tile C h over N and the masked operand times x over the columns up to the tile's last row."""
    TM = min(cfg.chunk, 128)
    ntpu = cfg.chunk // TM
    per_unit = sum(2.0 * TM * cfg.headdim * (cfg.dstate + (it + 1) * TM) for it in range(ntpu))
    return per_unit * cfg.batch * cfg.nchunks * cfg.nheads


def step_algorithmic_bytes(cfg) -> int:
    """Bytes one whole step must move if nothing were re-read: fp32 x, B, C in, dt in,
    fp32 y and final state out."""
    T = cfg.tokens
    return (T * cfg.channels * 4 + 2 * T * cfg.ngroups * cfg.dstate * 4 + T * cfg.nheads * 4 +
            T * cfg.channels * 4 + cfg.batch * cfg.channels * cfg.dstate * 4)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while a region runs."""
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
               0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index: int):
        self.samples, self.reasons, self._stop, self.ok = [], set(), threading.Event(), False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.max_mhz = None
        self.t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                m = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if m & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.ok:
            self.t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self.ok:
            self.t.join()

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(statistics.median(self.samples)), "sm_max_mhz": float(self.max_mhz),
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(cfg, seconds: float):
    """Times the oracle (quantiser + SSDi8 forward) on the whole workload if that fits the
    time budget, else on the first heads of batch element 0, and scales by the number of
    (batch, head) pairs (they are independent)."""
    from oracle import oracle as orc
    cores = max(1, len(os.sched_getaffinity(0)))
    # ~1e9 inner-loop operations per second per core on the plain oracle loops
    per_pair = cfg.seqlen * cfg.headdim * (2 * cfg.dstate + cfg.chunk / 2 + cfg.chunk * cfg.dstate / (2.0 * cfg.headdim))
    pairs_total = cfg.batch * cfg.nheads
    fit = int(seconds * 1e9 * cores / per_pair)
    if fit >= pairs_total:
        sub, npairs = cfg, pairs_total
        tt = inputs.make_prefill(cfg)
    else:
        nh = max(1, min(fit, cfg.nheads // cfg.ngroups))
        sub, npairs = cfg.replace(batch=1, nheads=nh, ngroups=1), nh
        if cfg.tokens * cfg.channels <= (1 << 27):
            t = inputs.make_prefill(cfg)
            tt = dict(x=np.ascontiguousarray(t["x"][:1, :, :nh]), B=np.ascontiguousarray(t["B"][:1, :, :1]),
                      C=np.ascontiguousarray(t["C"][:1, :, :1]), dt=np.ascontiguousarray(t["dt"][:1, :, :nh]),
                      A=t["A"][:nh], D=t["D"][:nh])
        else:  # very large workloads: draw the sample's own tensors with the same recipe
            tt = inputs.make_prefill(sub)
    q = orc.prepare_quantized(sub, tt)  # static scales, untimed (as on the GPU)
    t0 = time.perf_counter()
    xq, _ = orc.quantize(tt["x"], sub.tokens, sub.channels, 1, scale=q["s_x"], mode=0)
    Bq, _ = orc.quantize(tt["B"], sub.tokens, sub.ngroups, sub.dstate, scale=q["s_B"], mode=0)
    Cq, _ = orc.quantize(tt["C"], sub.tokens, sub.ngroups, sub.dstate, scale=q["s_C"], mode=0)
    orc.ssdi8_fwd(sub, xq, Bq, Cq, q["s_x"], q["s_B"], q["s_C"], tt["dt"], tt["A"], tt["D"], None,
                  q["s_xs"], q["s_cb"], q["s_h"])
    el = time.perf_counter() - t0
    est_full = el * pairs_total / npairs
    return {"value": cfg.tokens / est_full, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"{npairs} of {pairs_total} (batch, head) pairs of {cfg.name} (quantiser + SSDi8 "
                      f"forward, {el:.2f} s of CPU wall time), scaled by pair count"}, el


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = inputs.CONFIGS[args.workload]
    budget = 8.0
    for _ in range(args.warmup):
        oracle_sample(cfg, budget)
    vals, secs = [], []
    for _ in range(args.steps):
        cb, el = oracle_sample(cfg, budget)
        vals.append(cb["value"]); secs.append(el)
    value = float(len(vals) / sum(1.0 / v for v in vals))  # total work / total time
    cb["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * cfg.tokens / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(cfg, 1),
            "cpu_baseline": cb,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(cfg, n_gpus):
    return {"workload": f"{cfg.name}: Mamba-2 SSD layer forward, batch {cfg.batch} x seqlen {cfg.seqlen}, "
                        f"{cfg.nheads} heads x headdim {cfg.headdim}, d_state {cfg.dstate}, "
                        f"ngroups {cfg.ngroups}, chunk {cfg.chunk}",
            "batch": cfg.batch, "seqlen": cfg.seqlen, "nheads": cfg.nheads, "headdim": cfg.headdim,
            "dstate": cfg.dstate, "ngroups": cfg.ngroups, "chunk": cfg.chunk,
            "tokens_per_step_per_gpu": cfg.tokens, "parallelism": f"batch-sharded replicas x{n_gpus}, no collective",
            "l2": "each step touches more bytes than the 126 MB L2 (fp32 x in and fp32 y out alone exceed it)"
                  if 8 * cfg.tokens * cfg.channels > 126e6 else "L2 flushed between steps by a 256 MB write",
            "scales": "static: Eq. 1 on the synthetic tensors, internal scales by ssdi8_calibrate, untimed"}


# ----------------------------------------------------------------------------- GPU leg
class Layer:
    """Device buffers and calls of one workload (all arithmetic inside libssdi8)."""

    def __init__(self, cfg, torch, bd):
        self.cfg, self.torch, self.bd = cfg, torch, bd
        self.dims = bd.dims_of(cfg)
        t = self.t = inputs.make_prefill(cfg)
        self.host = {k: torch.from_numpy(t[k]).pin_memory() for k in ("x", "B", "C", "dt")}
        self.f = {k: v.cuda(non_blocking=True) for k, v in self.host.items()}
        self.A = torch.from_numpy(t["A"]).cuda(); self.D = torch.from_numpy(t["D"]).cuda()
        i8 = lambda k: torch.empty(t[k].shape, dtype=torch.int8, device="cuda")
        self.xq, self.Bq, self.Cq = i8("x"), i8("B"), i8("C")
        z = lambda n: torch.empty(n, device="cuda")
        self.s_x, self.s_B, self.s_C = z(cfg.channels), z(cfg.ngroups), z(cfg.ngroups)
        self.s_xs, self.s_cb, self.s_h = z(cfg.channels), z(cfg.ngroups), z(cfg.channels)
        self.y = torch.empty(t["x"].shape, device="cuda")
        self.fin = torch.empty((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), device="cuda")
        self.y_host = torch.empty(t["x"].shape).pin_memory()
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")   # written by a kernel whose wait ran out
        self.ws = bd.alloc_workspace(self.dims)
        self.args = bd.make_fwd_args(xq=self.xq, Bq=self.Bq, Cq=self.Cq, s_x=self.s_x, s_B=self.s_B,
                                     s_C=self.s_C, dt=self.f["dt"], A=self.A, D=self.D, s_xs=self.s_xs,
                                     s_cb=self.s_cb, s_h=self.s_h, y=self.y, final_state=self.fin,
                                     status=self.status)
        # static calibration (untimed)
        self.quantize(mode=1)
        bd.ssdi8_calibrate(self.dims, self.args, self.s_xs, self.s_cb, self.s_h, self.ws)
        torch.cuda.synchronize()
        self.flush = None
        self.host_args = None
        self.layer_args = None
        if 8 * cfg.tokens * cfg.channels <= 126e6:
            self.flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def quantize(self, mode=0):
        c, bd = self.cfg, self.bd
        bd.ssdi8_quantize_act(self.f["x"], c.tokens, c.channels, 1, self.s_x, mode, self.xq)
        bd.ssdi8_quantize_act(self.f["B"], c.tokens, c.ngroups, c.dstate, self.s_B, mode, self.Bq)
        bd.ssdi8_quantize_act(self.f["C"], c.tokens, c.ngroups, c.dstate, self.s_C, mode, self.Cq)

    def fwd(self, flags=0):
        self.bd.ssdi8_chunk_scan_fwd(self.dims, self.args, self.ws, flags=flags)

    def step(self):
        """One pass of the hot path through the one-call entry point: the three Eq. 1 quantisers and
        the layer forward (inside, ChunkCumsum runs beside the quantisers and ChunkBMM beside the state kernel)."""
        if self.layer_args is None:
            bd, torch = self.bd, self.torch
            self.layer_ws = torch.empty(bd.ssdi8_layer_fwd_workspace_bytes(self.dims), dtype=torch.uint8,
                                        device="cuda")
            self.layer_args = bd.make_layer_args(
                x=self.f["x"], B=self.f["B"], C=self.f["C"], dt=self.f["dt"], A=self.A, D=self.D,
                s_x=self.s_x, s_B=self.s_B, s_C=self.s_C, s_xs=self.s_xs, s_cb=self.s_cb, s_h=self.s_h,
                y=self.y, final_state=self.fin, status=self.status)
        self.bd.ssdi8_layer_fwd(self.dims, self.layer_args, self.layer_ws)

    def step_separate(self):
        self.quantize(0)
        self.fwd()

    def entry_fused_ms(self, iters):
        """Device time of the one-launch entry quantiser on a bf16 xBC tensor of this workload's
        shape (the form a Mamba-2 block hands over); reported beside the step, not part of it."""
        c, torch = self.cfg, self.torch
        xbc = torch.cat([self.f["x"].reshape(c.tokens, -1), self.f["B"].reshape(c.tokens, -1),
                         self.f["C"].reshape(c.tokens, -1)], dim=1).to(torch.bfloat16).contiguous()
        fn = lambda: self.bd.ssdi8_quantize_entry(xbc, c.tokens, c.channels, c.ngroups, c.dstate, self.s_x,
                                                  self.s_B, self.s_C, self.xq, self.Bq, self.Cq)
        fn(); torch.cuda.synchronize()
        ms = self.timed(fn, iters)
        self.quantize(0)
        return ms

    LAUNCHES_PER_STEP = 5  # quantisers (one launch), cumsum, BMM, fused chunk state / state passing, chunk scan

    def e2e_step(self):
        """The same step through the host-buffer entry point of the C-ABI: pinned fp32 x, B, C, dt in,
        fp32 y out, copies pipelined against the kernels batch element by batch element."""
        if self.host_args is None:
            bd, torch = self.bd, self.torch
            self.host_scratch = torch.empty(bd.ssdi8_layer_fwd_host_scratch_bytes(self.dims), dtype=torch.uint8,
                                            device="cuda")
            self.host_status = torch.zeros(1, dtype=torch.int32).pin_memory()
            self.host_args = bd.make_host_args(
                x=self.host["x"], B=self.host["B"], C=self.host["C"], dt=self.host["dt"], A=self.A, D=self.D,
                s_x=self.s_x, s_B=self.s_B, s_C=self.s_C, s_xs=self.s_xs, s_cb=self.s_cb, s_h=self.s_h,
                y=self.y_host, status=self.host_status)
        self.bd.ssdi8_layer_fwd_host(self.dims, self.host_args, self.host_scratch)

    def h2d_bytes(self):
        return sum(v.numel() * v.element_size() for v in self.host.values())

    def d2h_bytes(self):
        return self.y_host.numel() * self.y_host.element_size()

    def check_status(self, where):
        """The status word of the timed calls: non-zero means a bounded wait of a kernel ran out and
        the launch finished with undefined results, which must never be timed as a success."""
        self.torch.cuda.synchronize()
        code = int(self.status.item())
        if self.host_args is not None:
            code = code or int(self.host_status[0])
        if code != 0:
            raise RuntimeError(f"{where}: device status word = {code} ({self.bd.ssdi8_status_string(code)})")

    def timed(self, fn, iters):
        """Average device time of fn in ms (CUDA events on the current stream); the L2 flush
        of small workloads sits outside the event pairs."""
        torch = self.torch
        if self.flush is None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(iters):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / iters
        tot = 0.0
        evs = []
        for _ in range(iters):
            self.flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        for e0, e1 in evs:
            tot += e0.elapsed_time(e1)
        return tot / iters

    def timed_rounds(self, fn, iters, min_seconds, where, barrier=None, reduce=None, max_rounds=4000):
        """Rounds of `iters` calls, each bracketed by a barrier and a device synchronisation, until
        `min_seconds` have been timed (at least 3 rounds).  Returns (median, min, max, rounds) of the
        per-call time in ms; with several ranks every round's time is the slowest rank's, so all
        ranks take the same decisions."""
        per_call, total = [], 0.0
        while (total < min_seconds * 1e3 or len(per_call) < 3) and len(per_call) < max_rounds:
            if barrier is not None:
                barrier()
            ms = self.timed(fn, iters)
            if reduce is not None:
                ms = reduce(ms)
            self.check_status(where)
            per_call.append(ms)
            total += ms * iters
        return float(statistics.median(per_call)), float(min(per_call)), float(max(per_call)), len(per_call)


def parity_check(layer, npairs=8):
    """The output and final state the GPU holds after its last step against the CPU oracle, which
    quantises and calibrates the whole tensors itself (nothing of the GPU run enters the oracle):
    step sizes bit for bit, then `npairs` random (batch, head) pairs (all pairs of small workloads)
    recomputed one by one, final state bit for bit and y within 1e-3 of the pair's RMS."""
    from oracle import oracle as orc
    cfg, t = layer.cfg, layer.t
    layer.torch.cuda.synchronize()
    q = orc.prepare_quantized(cfg, t)
    g = lambda v: v.cpu().numpy()
    scales_ok = all(np.array_equal(g(getattr(layer, k)), q[k]) for k in ("s_x", "s_B", "s_C", "s_xs", "s_cb", "s_h"))
    y, fin = g(layer.y), g(layer.fin)
    total = cfg.batch * cfg.nheads
    rng = np.random.default_rng(1000 + cfg.seed)
    if total <= 32:
        pairs = [(b, h) for b in range(cfg.batch) for h in range(cfg.nheads)]
    else:
        pairs = [(int(v) // cfg.nheads, int(v) % cfg.nheads) for v in rng.choice(total, size=npairs, replace=False)]
    one = cfg.replace(batch=1, nheads=1, ngroups=1)
    P, hpg = cfg.headdim, cfg.nheads // cfg.ngroups
    worst, fin_ok = 0.0, True
    for (b, h) in pairs:
        gi = h // hpg
        c_ = np.ascontiguousarray
        y_ref, fin_ref, _ = orc.ssdi8_fwd(
            one, c_(q["xq"][b:b + 1, :, h:h + 1]), c_(q["Bq"][b:b + 1, :, gi:gi + 1]), c_(q["Cq"][b:b + 1, :, gi:gi + 1]),
            q["s_x"][h * P:(h + 1) * P], q["s_B"][gi:gi + 1], q["s_C"][gi:gi + 1], c_(t["dt"][b:b + 1, :, h:h + 1]),
            t["A"][h:h + 1], t["D"][h:h + 1], None, q["s_xs"][h * P:(h + 1) * P], q["s_cb"][gi:gi + 1],
            q["s_h"][h * P:(h + 1) * P])
        fin_ok = fin_ok and np.array_equal(fin[b, h], fin_ref[0, 0])
        rms = float(np.sqrt((y_ref ** 2).mean()))
        worst = max(worst, float(np.abs(y[b, :, h] - y_ref[0, :, 0]).max()) / max(rms, 1e-30))
    ok = bool(scales_ok and fin_ok and worst <= 1e-3)
    return {"pairs": len(pairs), "of": total, "max_err_over_rms": worst, "final_state_bit_exact": bool(fin_ok),
            "step_sizes_bit_exact": bool(scales_ok), "status": 0, "ok": ok}


def run_decode(torch, bd, steps=256, warmup=8):
    """Recurrent-mode decode at 2.7B shapes (batch 64, 256 steps): tokens/s and HBM fractions of the step kernel."""
    cfg = inputs.CONFIGS["cfg4"]
    dims = bd.dims_of(cfg)
    prm = inputs.make_decode_params(cfg)
    st = inputs.make_decode_step(cfg, 0)
    g = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    x, B, C, dt = g(st["x"]), g(st["B"]), g(st["C"]), g(st["dt"])
    xq = torch.empty(x.shape, dtype=torch.int8, device="cuda"); Bq = torch.empty(B.shape, dtype=torch.int8, device="cuda")
    Cq = torch.empty(C.shape, dtype=torch.int8, device="cuda")
    s_x, s_B, s_C = torch.empty(cfg.channels, device="cuda"), torch.empty(1, device="cuda"), torch.empty(1, device="cuda")
    bd.ssdi8_quantize_act(x, cfg.batch, cfg.channels, 1, s_x, 1, xq)
    bd.ssdi8_quantize_act(B, cfg.batch, 1, cfg.dstate, s_B, 1, Bq)
    bd.ssdi8_quantize_act(C, cfg.batch, 1, cfg.dstate, s_C, 1, Cq)
    state = torch.zeros((cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), device="cuda")
    y = torch.empty((cfg.batch, cfg.nheads, cfg.headdim), device="cuda")
    A, D = g(prm["A"]), g(prm["D"])
    call = lambda: bd.ssdi8_ssd_step(dims, xq, s_x, Bq, s_B, Cq, s_C, dt, A, D, None, state, y)
    for _ in range(warmup):
        call()
    per = []
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            call()
        e1.record()
        torch.cuda.synchronize()
        per.append(e0.elapsed_time(e1) / steps)
    ms = float(statistics.median(per))
    nbytes = 2 * state.numel() * 4 + xq.numel() + Bq.numel() + Cq.numel() + dt.numel() * 4 + y.numel() * 4
    peaks = measured_peaks()
    gbs = nbytes / (ms * 1e-3) / 1e9
    dram_gbs = NCU_TRAFFIC_BYTES_DECODE / (ms * 1e-3) / 1e9
    return {"workload": "cfg4: decode step, batch 64, 80 heads x 64, d_state 128 (state 168 MB > L2)",
            "tokens_per_s": cfg.batch / (ms * 1e-3), "ms_per_step": ms, "steps": steps, "rounds": len(per),
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
                         "algorithmic_bytes": nbytes, "traffic": NCU_TRAFFIC_BYTES_DECODE,
                         "dram_frac": dram_gbs / peaks["hbm_gbs"],
                         "note": "frac counts the algorithmic bytes (state read and written once per step); "
                                 "dram_frac the DRAM bytes of an ncu capture (part of the state written by one "
                                 "step is still in L2 when the next step reads it)"}}


def measure_int8_peak(torch, bd):
    """Dense tcgen05.mma.kind::i8 throughput of this device: best single launch (about 1 ms) and a
    back-to-back loop of about 0.3 s, CUDA events on the launching stream."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bd.ssdi8_int8_mma_peak(2048, status)
    torch.cuda.synchronize()
    best = 0.0
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); ops = bd.ssdi8_int8_mma_peak(16384, status); e1.record()
        torch.cuda.synchronize()
        best = max(best, ops / (e0.elapsed_time(e1) * 1e-3) / 1e12)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = 256
    e0.record()
    for _ in range(n):
        ops = bd.ssdi8_int8_mma_peak(16384, status)
    e1.record()
    torch.cuda.synchronize()
    sustained = n * ops / (e0.elapsed_time(e1) * 1e-3) / 1e12
    if int(status.item()) != 0:
        raise RuntimeError("int8 MMA loop: a bounded wait ran out")
    return {"burst_tops": best, "sustained_tops": sustained,
            "how": "ssdi8_int8_mma_peak: one CTA per SM, M 128 x N 256 x K 32 MMAs on operands resident in shared memory"}


def measure_workload(cfg, torch, bd, steps, warmup, min_seconds, peaks, int8_peak, full, barrier=None, reduce=None,
                     clock_index=0):
    """Times one workload.  full = the headline workload (every leg); otherwise the short record of the
    `workloads` list.  Returns (record, layer)."""
    layer = Layer(cfg, torch, bd)
    for _ in range(warmup):
        if layer.flush is not None:
            layer.flush.fill_(1)
        layer.step()
    layer.check_status("warm-up")
    with ClockSampler(clock_index) as clk:
        ms, ms_min, ms_max, rounds = layer.timed_rounds(layer.step, steps, min_seconds, "timed steps", barrier, reduce)
    it = max(5, min(steps, 20))
    rec = {"workload": cfg.name, "tokens_per_step": cfg.tokens, "ms_per_step": ms, "ms_per_step_min": ms_min,
           "ms_per_step_max": ms_max, "rounds": rounds, "steps_per_round": steps,
           "tokens_per_s": cfg.tokens / (ms * 1e-3), "clocks": clk.summary()}
    if reduce is not None and not full:
        return rec, layer
    sec = min_seconds / 5
    layer_only, _, _, _ = layer.timed_rounds(lambda: layer.fwd(0), it, sec, "layer only")
    scan_ms, _, _, _ = layer.timed_rounds(lambda: layer.fwd(bd.PHASE_SCAN), it, sec, "chunk scan")
    alg = scan_algorithmic_bytes(cfg)
    scan_gbs = alg / (scan_ms * 1e-3) / 1e9
    ideal = layer_ideal_bytes(cfg)
    tops = scan_mma_ops(cfg) / (scan_ms * 1e-3) / 1e12
    rec.update({
        "layer_only_ms": layer_only, "layer_only_tokens_per_s": cfg.tokens / (layer_only * 1e-3),
        "layer_only_hbm": {"ideal_bytes": ideal, "achieved_gbs": ideal / (layer_only * 1e-3) / 1e9,
                           "frac": ideal / (layer_only * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "chunk_scan_ms": scan_ms,
        "chunk_scan_hbm": {"algorithmic_bytes": alg, "achieved_gbs": scan_gbs, "frac": scan_gbs / peaks["hbm_gbs"]},
        "chunk_scan_int8": {"mma_ops": scan_mma_ops(cfg), "achieved_tops": tops,
                            "frac_of_measured": tops / int8_peak["sustained_tops"] if int8_peak else None,
                            "frac_of_4.5POPS": tops / INT8_NOMINAL_TOPS},
        "launch_bound": bool(8 * cfg.tokens * cfg.channels <= 126e6)})
    return rec, layer


def spawn_ranks(n):
    """`python bench.py --gpus N` without a launcher: start N ranks under torch.distributed.run."""
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2608_21952_b200 import binding as bd

    from paper_2608_21952_b200 import ranks
    world, rank, local = ranks.env_world()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    cfg = inputs.CONFIGS[args.workload]
    peaks = measured_peaks()
    int8_peak = None   # measured after the timed steps: half a second of dense MMAs runs into the power cap

    def barrier():
        ranks.barrier()
        torch.cuda.synchronize()

    reduce = (lambda v: ranks.max_over_ranks(v, "cuda")) if world > 1 else None
    head, layer = measure_workload(cfg, torch, bd, args.steps, args.warmup,
                                   0.0 if args.quick else MIN_TIMED_SECONDS, peaks, int8_peak,
                                   full=not args.quick, barrier=barrier, reduce=reduce, clock_index=local)
    ms = head["ms_per_step"]
    value = ranks.whole_job_tokens_per_s(cfg.tokens, world, ms)
    if rank == 0 and not args.quick:
        int8_peak = measure_int8_peak(torch, bd)
        head["chunk_scan_int8"]["frac_of_measured"] = head["chunk_scan_int8"]["achieved_tops"] / int8_peak["sustained_tops"]
        time.sleep(1.0)   # let the package cool before the remaining legs

    if args.quick:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
                              "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "quick": True,
                              "config": workload_config(cfg, world), "clocks": head["clocks"]}))
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # parity of what was just timed: y and the final state of the last step against the CPU oracle
    layer.step()
    parity = parity_check(layer) if rank == 0 else None

    # end to end: pinned host fp32 inputs -> device, the step, fp32 y -> pinned host
    for _ in range(2):
        layer.e2e_step()
    ms_e2e, _, _, e2e_rounds = layer.timed_rounds(layer.e2e_step, max(3, min(args.steps, 10)), 0.3, "end to end",
                                                  barrier, reduce)

    line = None
    if rank == 0:
        it = max(5, min(args.steps, 20))
        sec = MIN_TIMED_SECONDS / 5
        t_of = lambda fn, where: layer.timed_rounds(fn, it, sec, where)[0]
        # per-module device time (CUDA events around partial runs of the same call)
        phases = {"quantize": lambda: layer.quantize(0), "cumsum": lambda: layer.fwd(bd.PHASE_CUMSUM),
                  "bmm": lambda: layer.fwd(bd.PHASE_BMM),
                  "chunk_state_passing": lambda: layer.fwd(bd.PHASE_CHUNK_STATE | bd.PHASE_STATE_PASSING),
                  "chunk_state_passing_int8_state":
                      lambda: layer.fwd(bd.PHASE_CHUNK_STATE | bd.PHASE_STATE_PASSING | bd.FLAG_INT8_STATE)}
        layer.step(); torch.cuda.synchronize()
        kernel_ms = {k: t_of(fn, k) for k, fn in phases.items()}
        layer.fwd(bd.PHASE_CHUNK_STATE | bd.PHASE_STATE_PASSING); torch.cuda.synchronize()   # fp32-state hq back in the workspace
        kernel_ms["chunk_scan"] = head["chunk_scan_ms"]
        dom = max((k for k in kernel_ms if k not in ("quantize", "chunk_state_passing_int8_state")), key=lambda k: kernel_ms[k])
        entry_ms = layer.entry_fused_ms(it)
        ms_separate = t_of(layer.step_separate, "separate calls")
        # the scan kernel with the paper's 16-bit output format (beside the step, which keeps fp32 y)
        y16 = torch.empty(layer.y.shape, dtype=torch.bfloat16, device="cuda")
        args16 = bd.make_fwd_args(**{**layer.args._keepalive, "y": y16})
        scan16 = lambda: bd.ssdi8_chunk_scan_fwd(layer.dims, args16, layer.ws, flags=bd.PHASE_SCAN | bd.FLAG_Y_BF16)
        scan16(); torch.cuda.synchronize()
        kernel_ms["chunk_scan_bf16_y"] = t_of(scan16, "chunk scan, bf16 y")
        # the paper's own ChunkScan2: FP16 masked operand (kind::f16 MMA) and FP16 y
        y_h = torch.empty(layer.y.shape, dtype=torch.float16, device="cuda")
        args_h = bd.make_fwd_args(**{**layer.args._keepalive, "y": y_h})
        fl_h = bd.PHASE_SCAN | bd.FLAG_FP16_OPERAND | bd.FLAG_Y_FP16
        ws_h = bd.alloc_workspace(layer.dims, flags=bd.FLAG_FP16_OPERAND)
        bd.ssdi8_chunk_scan_fwd(layer.dims, args_h, ws_h, flags=bd.FLAG_FP16_OPERAND | bd.FLAG_Y_FP16)
        torch.cuda.synchronize()
        scan_h = lambda: bd.ssdi8_chunk_scan_fwd(layer.dims, args_h, ws_h, flags=fl_h)
        kernel_ms["chunk_scan_fp16_operand_fp16_y"] = t_of(scan_h, "chunk scan, FP16 operand")
        del y16, y_h, ws_h
        ncu = NCU_SCAN.get(cfg.name, {})
        roofline = {"bound": "hbm", "kernel": "chunk_scan", "achieved": head["chunk_scan_hbm"]["achieved_gbs"],
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": head["chunk_scan_hbm"]["frac"],
                    "peak_source": peaks["source"], "algorithmic_bytes": head["chunk_scan_hbm"]["algorithmic_bytes"],
                    "launch_ms": kernel_ms["chunk_scan"], "traffic": ncu.get("traffic"),
                    "traffic_source": ncu.get("source"), "slowest_module": dom,
                    "limiter": "instruction issue of the CUDA cores that build the int8 masked operand and the "
                               "fp32 output around the MMAs (neither DRAM nor the tensor pipe is saturated); "
                               "HBM is the roof the bytes of this kernel set"}
        roofline_tensor = dict(head["chunk_scan_int8"])
        roofline_tensor.update({"int8_tops_measured": int8_peak, "tensor_active_pct": ncu.get("tensor_active_pct"),
                                "tensor_active_source": ncu.get("source")})
        step_gbs = step_algorithmic_bytes(cfg) / (ms * 1e-3) / 1e9
        layer_h2d, layer_d2h = layer.h2d_bytes(), layer.d2h_bytes()
        decode = run_decode(torch, bd) if world == 1 else None
        cpu_baseline, _ = oracle_sample(cfg, 20.0) if world == 1 else (None, 0)
        # the other workloads, one after the other on this GPU (single-GPU runs only)
        workloads = [{k: v for k, v in head.items()}]
        if world == 1 and not args.no_workloads:
            del layer
            torch.cuda.empty_cache()
            for name in ("cfg0", "cfg1", "cfg2", "cfg3"):
                if name == cfg.name:
                    continue
                rec, lay = measure_workload(inputs.CONFIGS[name], torch, bd, args.steps, args.warmup,
                                            MIN_TIMED_SECONDS / 2, peaks, int8_peak, full=True)
                lay.step()
                rec["parity"] = parity_check(lay)
                workloads.append(rec)
                del lay
                torch.cuda.empty_cache()
            workloads.sort(key=lambda r: r["workload"])
        paper = PAPER_TOKENS_PER_S.get(cfg.name)
        config = workload_config(cfg, world)
        config["value_is"] = ("tokens/s of the whole step: the Eq. 1 quantisers of fp32 x, B, C (one launch) plus "
                              "Algorithm 2; layer_only_* is Algorithm 2 alone from the int8 tensors")
        config["timing"] = (f"median of {head['rounds']} rounds of {args.steps} steps, each round bracketed by a "
                            f"barrier and a device synchronisation, at least {MIN_TIMED_SECONDS} s timed in all")
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms, "ms_per_step_min": head["ms_per_step_min"],
                "ms_per_step_max": head["ms_per_step_max"], "rounds": head["rounds"],
                "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "s8",
                "data": "synthetic", "config": config,
                "clocks": head["clocks"],
                "e2e": {"value": ranks.whole_job_tokens_per_s(cfg.tokens, world, ms_e2e), "unit": UNIT,
                        "h2d_bytes_per_step": layer_h2d, "d2h_bytes_per_step": layer_d2h,
                        "ms_per_step": ms_e2e, "rounds": e2e_rounds,
                        "api": "ssdi8_layer_fwd_host (pinned host buffers; copies pipelined per batch element)"},
                "gpu_launches": Layer.LAUNCHES_PER_STEP * args.steps * head["rounds"],
                "gpu_launches_per_step": Layer.LAUNCHES_PER_STEP,
                "parity": parity,
                "roofline": roofline,
                "roofline_tensor": roofline_tensor,
                "int8_tops_measured": int8_peak["sustained_tops"] if int8_peak else None,
                "step_hbm": {"algorithmic_bytes": step_algorithmic_bytes(cfg), "achieved_gbs": step_gbs,
                             "frac_of_peak": step_gbs / peaks["hbm_gbs"]},
                "kernel_ms": kernel_ms,
                "ms_per_step_separate_calls_one_stream": ms_separate,
                "entry_quantizer_bf16_xBC_one_launch_ms": entry_ms,
                "layer_only_ms": head["layer_only_ms"],
                "layer_only_tokens_per_s": world * cfg.tokens / (head["layer_only_ms"] * 1e-3),
                "layer_only_hbm": head["layer_only_hbm"],
                "workloads": workloads,
                "decode": decode, "cpu_baseline": cpu_baseline,
                "paper_context": ({"tokens_per_s": paper, "hardware": "RTX A5000",
                                   "source": "the paper's block-latency table: SSD module of block 55, Mamba-2 2.7B, "
                                             "batch 8, L = 2048, 4.481 ms; another machine, context only"}
                                  if paper else None)}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line))
        bad = [w["workload"] for w in line["workloads"] if w.get("parity") and not w["parity"]["ok"]]
        if not line["parity"]["ok"] or bad:
            sys.stderr.write(f"parity failed: headline {line['parity']}, workloads {bad}\n")
            sys.exit(1)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg0", "cfg1", "cfg2", "cfg3"])
    ap.add_argument("--quick", action="store_true",
                    help="timed steps only: skip the end-to-end, per-module, decode and CPU legs (profiling runs)")
    ap.add_argument("--no-workloads", action="store_true", help="skip the list of the other workloads")
    ap.add_argument("--decode-only", action="store_true",
                    help="the cfg4 decode leg alone on one GPU (profiling runs of the step kernel)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(spawn_ranks(args.gpus))
    if args.decode_only:
        import torch
        from paper_2608_21952_b200 import binding as bd
        torch.cuda.set_device(0)
        print(json.dumps(run_decode(torch, bd, steps=args.steps, warmup=max(args.warmup, 3))))
        return
    if args.impl == "reference":
        if args.steps > 5:
            args.steps = 5  # each step is seconds of CPU work; keep the run within minutes
        args.warmup = min(args.warmup, 1)
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
