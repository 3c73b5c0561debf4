"""Host-side plumbing of multi-GPU runs: replicas only.

Scenes are independent (own KV cache, own bitmaps), so N GPUs run N independent batches of
scenes and no data crosses between them.  What the ranks share is bookkeeping: which seed a
rank draws its scenes from, the step time of the slowest rank (the job's time) and the
job-wide throughput.  The collective is a single scalar all-reduce outside the timed region;
it works on any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


def rank_and_world() -> tuple:
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def replica_seed_shift(rank: int) -> int:
    """Every rank draws different scenes from the same recipe."""
    return int(rank)


def max_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    """The slowest rank's time: the job is done when every replica is."""
    _, world = rank_and_world()
    if world == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    _, world = rank_and_world()
    if world == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_this_rank: float, ms_this_rank: float, device: Optional[torch.device] = None) -> tuple:
    """(units of all ranks per second, job milliseconds) with time = max over ranks."""
    ms = max_over_ranks(ms_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / (ms * 1e-3), ms


def barrier() -> None:
    _, world = rank_and_world()
    if world > 1:
        dist.barrier()
