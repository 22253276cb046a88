"""Host-side logic of the multi-GPU benchmark: one process per GPU, no data-path collective.

The SSD layer is independent across (batch, head) pairs, so N GPUs run N batch shards with no
exchange (replicas: weak scaling).  The only collectives are the barrier that brackets the timed
region and the MAX reduction of the per-rank device times.  Works on any backend (`nccl` on
GPUs, `gloo` in the CPU tests).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(world_size, rank, local_rank) from the torchrun environment (1, 0, 0 when absent)."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(ms: float, device="cpu") -> float:
    """Slowest rank's time: the job is as fast as its slowest shard."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank: int, world: int, ms: float) -> float:
    """Aggregate throughput of `world` replicas that each process `tokens_per_rank` in `ms`."""
    return world * tokens_per_rank / (ms * 1e-3)


def shard_of_batch(global_batch: int, world: int, rank: int):
    """[start, stop) of the batch rows rank `rank` owns when one global batch is split
    (strong-scaling use of the same independence; remainder rows go to the first ranks)."""
    base, rem = divmod(global_batch, world)
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)
