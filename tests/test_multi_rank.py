"""N > 1 path of the benchmark on CPU: two gloo ranks, barrier, MAX-over-ranks timing, whole-job
aggregation and batch sharding (the layer needs no data-path collective)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_21952_b200 import ranks


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(world),
                      RANK=str(rank), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert ranks.env_world() == (world, rank, rank)
        ranks.barrier()
        ms = ranks.max_over_ranks(1.0 + rank)            # rank 1 is the slow one
        value = ranks.whole_job_tokens_per_s(1000, world, ms)
        lo, hi = ranks.shard_of_batch(5, world, rank)
        ranks.barrier()
        out.put((rank, ms, value, lo, hi))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_time_as_the_slowest_and_sum_their_tokens():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    ps = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in ps:
        p.start()
    res = sorted(q.get(timeout=120) for _ in ps)
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [2.0, 2.0]               # MAX over ranks on every rank
    assert all(abs(r[2] - 2 * 1000 / 2e-3) < 1e-6 for r in res)
    assert [(r[3], r[4]) for r in res] == [(0, 3), (3, 5)]  # disjoint cover of the batch


def test_single_process_defaults():
    assert ranks.max_over_ranks(3.5) == 3.5
    assert ranks.shard_of_batch(8, 1, 0) == (0, 8)
    covered = []
    for r in range(3):
        covered += list(range(*ranks.shard_of_batch(8, 3, r)))
    assert covered == list(range(8))


def test_bench_starts_its_own_ranks_when_no_launcher_did(monkeypatch):
    """`python bench.py --gpus N` with no WORLD_SIZE in the environment re-executes itself under
    torch.distributed.run with N ranks on 127.0.0.1 and hands on its own arguments."""
    import sys
    import bench
    seen = {}
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: seen.setdefault("cmd", cmd) and 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "7"])
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    try:
        bench.main()
    except SystemExit as e:
        assert e.code == 0
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "7"] and cmd[-5].endswith("bench.py")
