#!/usr/bin/env python
"""Benchmark of the B200 INT8 SSD layer (SSDi8 hot path).

One step = one pass of the whole hot path over one batch of seeded synthetic input:
Eq. 1 quantisation of fp32 x, B, C with static step sizes (3 launches), then the
layer forward (ChunkCumsum, ChunkBMM, fused ChunkState+StatePassing, ChunkScan)
from int8 x, B, C to the fp32 output y and the final state.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

N > 1: launched by torch.distributed.run, one rank per GPU.  The layer shards over
(batch, head) with no exchange, so every rank runs the same workload on its own
GPU (weak scaling, no data-path collective); the time is the maximum over ranks.

Prints ONE JSON line.  `--impl reference` times the CPU oracle (as it stands) on
the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
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
# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum
# of one ncu capture; see profiles/).  None until a capture of that workload exists.
NCU_TRAFFIC_BYTES = {"cfg2": 441.5e6}  # profiles/chunk_scan_cfg2_ncu_full.md
NCU_TRAFFIC_BYTES_DECODE = 279.6e6  # ssd_step_kernel at cfg4: profiles/ssd_step_cfg4_and_quant_jobs_cfg2_ncu.md


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
        t = inputs.make_prefill(cfg)
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
        self.ws = bd.alloc_workspace(self.dims)
        self.args = bd.make_fwd_args(xq=self.xq, Bq=self.Bq, Cq=self.Cq, s_x=self.s_x, s_B=self.s_B,
                                     s_C=self.s_C, dt=self.f["dt"], A=self.A, D=self.D, s_xs=self.s_xs,
                                     s_cb=self.s_cb, s_h=self.s_h, y=self.y, final_state=self.fin)
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
        the layer forward (inside, the modules that do not need xq run under the quantiser of x)."""
        if self.layer_args is None:
            bd, torch = self.bd, self.torch
            self.layer_ws = torch.empty(bd.ssdi8_layer_fwd_workspace_bytes(self.dims), dtype=torch.uint8,
                                        device="cuda")
            self.layer_args = bd.make_layer_args(
                x=self.f["x"], B=self.f["B"], C=self.f["C"], dt=self.f["dt"], A=self.A, D=self.D,
                s_x=self.s_x, s_B=self.s_B, s_C=self.s_C, s_xs=self.s_xs, s_cb=self.s_cb, s_h=self.s_h,
                y=self.y, final_state=self.fin)
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


def run_decode(torch, bd, steps=64, warmup=8):
    """Recurrent-mode decode at 2.7B shapes (batch 64): tokens/s and HBM fraction of the step kernel."""
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
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    nbytes = 2 * state.numel() * 4 + xq.numel() + Bq.numel() + Cq.numel() + dt.numel() * 4 + y.numel() * 4
    peaks = measured_peaks()
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"workload": "cfg4: decode step, batch 64, 80 heads x 64, d_state 128 (state 168 MB > L2)",
            "tokens_per_s": cfg.batch / (ms * 1e-3), "ms_per_step": ms, "steps": steps,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
                         "traffic": NCU_TRAFFIC_BYTES_DECODE}}


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
    layer = Layer(cfg, torch, bd)

    def barrier():
        ranks.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        if layer.flush is not None:
            layer.flush.fill_(1)
        layer.step()
    barrier()
    with ClockSampler(local) as clk:
        ms = layer.timed(layer.step, args.steps)
        torch.cuda.synchronize()
    barrier()
    ms = ranks.max_over_ranks(ms, "cuda")
    value = ranks.whole_job_tokens_per_s(cfg.tokens, world, ms)

    if args.quick:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
                              "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "quick": True,
                              "config": workload_config(cfg, world), "clocks": clk.summary()}))
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # end to end: pinned host fp32 inputs -> device, the step, fp32 y -> pinned host
    for _ in range(2):
        layer.e2e_step()
    barrier()
    ms_e2e = layer.timed(layer.e2e_step, max(3, min(args.steps, 10)))
    barrier()
    ms_e2e = ranks.max_over_ranks(ms_e2e, "cuda")

    line = None
    if rank == 0:
        peaks = measured_peaks()
        # per-module device time (CUDA events around partial runs of the same call)
        phases = {"quantize": lambda: layer.quantize(0), "cumsum": lambda: layer.fwd(bd.PHASE_CUMSUM),
                  "bmm": lambda: layer.fwd(bd.PHASE_BMM),
                  "chunk_state_passing": lambda: layer.fwd(bd.PHASE_CHUNK_STATE | bd.PHASE_STATE_PASSING),
                  "chunk_scan": lambda: layer.fwd(bd.PHASE_SCAN)}
        layer.step(); torch.cuda.synchronize()
        kernel_ms = {k: layer.timed(fn, max(5, min(args.steps, 20))) for k, fn in phases.items()}
        dom = max((k for k in kernel_ms if k != "quantize"), key=lambda k: kernel_ms[k])
        # Algorithm 2 alone, from the int8 tensors to y and the final state (one ssdi8_chunk_scan_fwd call)
        layer_only_ms = layer.timed(lambda: layer.fwd(0), max(5, min(args.steps, 20)))
        entry_ms = layer.entry_fused_ms(max(5, min(args.steps, 20)))
        ms_separate = layer.timed(layer.step_separate, max(5, min(args.steps, 20)))
        # the scan kernel with the paper's 16-bit output format (beside the step, which keeps fp32 y)
        y16 = torch.empty(layer.y.shape, dtype=torch.bfloat16, device="cuda")
        args16 = bd.make_fwd_args(**{**layer.args._keepalive, "y": y16})
        scan16 = lambda: bd.ssdi8_chunk_scan_fwd(layer.dims, args16, layer.ws, flags=bd.PHASE_SCAN | bd.FLAG_Y_BF16)
        scan16(); torch.cuda.synchronize()
        kernel_ms["chunk_scan_bf16_y"] = layer.timed(scan16, max(5, min(args.steps, 20)))
        # the paper's own ChunkScan2: FP16 masked operand (kind::f16 MMA) and FP16 y
        y_h = torch.empty(layer.y.shape, dtype=torch.float16, device="cuda")
        args_h = bd.make_fwd_args(**{**layer.args._keepalive, "y": y_h})
        fl_h = bd.PHASE_SCAN | bd.FLAG_FP16_OPERAND | bd.FLAG_Y_FP16
        ws_h = bd.alloc_workspace(layer.dims, flags=bd.FLAG_FP16_OPERAND)
        layer.fwd_into = lambda: bd.ssdi8_chunk_scan_fwd(layer.dims, args_h, ws_h, flags=bd.FLAG_FP16_OPERAND | bd.FLAG_Y_FP16)
        layer.fwd_into(); torch.cuda.synchronize()
        scan_h = lambda: bd.ssdi8_chunk_scan_fwd(layer.dims, args_h, ws_h, flags=fl_h)
        kernel_ms["chunk_scan_fp16_operand_fp16_y"] = layer.timed(scan_h, max(5, min(args.steps, 20)))
        alg = scan_algorithmic_bytes(cfg)
        scan_gbs = alg / (kernel_ms["chunk_scan"] * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": "chunk_scan", "achieved": scan_gbs, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": scan_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
                    "algorithmic_bytes": alg, "launch_ms": kernel_ms["chunk_scan"],
                    "traffic": NCU_TRAFFIC_BYTES.get(cfg.name), "slowest_module": dom}
        step_gbs = step_algorithmic_bytes(cfg) / (ms * 1e-3) / 1e9
        decode = run_decode(torch, bd) if world == 1 else None
        cpu_baseline, _ = oracle_sample(cfg, 20.0) if world == 1 else (None, 0)
        paper = PAPER_TOKENS_PER_S.get(cfg.name)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": (value / paper) if (paper and world == 1) else None, "dtype": "s8",
                "data": "synthetic", "config": workload_config(cfg, world),
                "clocks": clk.summary(),
                "e2e": {"value": ranks.whole_job_tokens_per_s(cfg.tokens, world, ms_e2e), "unit": UNIT,
                        "h2d_bytes_per_step": layer.h2d_bytes(), "d2h_bytes_per_step": layer.d2h_bytes(),
                        "ms_per_step": ms_e2e, "api": "ssdi8_layer_fwd_host (pinned host buffers; copies pipelined per batch element)"},
                "gpu_launches": Layer.LAUNCHES_PER_STEP * args.steps,
                "roofline": roofline,
                "step_hbm": {"algorithmic_bytes": step_algorithmic_bytes(cfg), "achieved_gbs": step_gbs,
                             "frac_of_peak": step_gbs / peaks["hbm_gbs"]},
                "kernel_ms": kernel_ms,
                "ms_per_step_separate_calls_one_stream": ms_separate,
                "entry_quantizer_bf16_xBC_one_launch_ms": entry_ms,
                "layer_only_ms": layer_only_ms,
                "layer_only_tokens_per_s": world * cfg.tokens / (layer_only_ms * 1e-3),
                "decode": decode, "cpu_baseline": cpu_baseline}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg0", "cfg1", "cfg2", "cfg3"])
    ap.add_argument("--quick", action="store_true",
                    help="timed steps only: skip the end-to-end, per-module, decode and CPU legs (profiling runs)")
    ap.add_argument("--decode-only", action="store_true",
                    help="the cfg4 decode leg alone on one GPU (profiling runs of the step kernel)")
    args = ap.parse_args()
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
