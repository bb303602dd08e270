"""Rank plumbing for `bench.py --gpus N`: the path does not shard across GPUs, so N ranks are N
independent replicas; this module only reduces their timings and work counts."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def dist_env() -> tuple[int, int, int]:
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) without one."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_seed(base_seed: int, rank: int) -> int:
    """Each replica works on its own synthetic layer."""
    return base_seed + 100 * rank


def barrier(world: int) -> None:
    if world > 1:
        dist.barrier()


def max_over_ranks(value: float, world: int, device) -> float:
    """The job's time is the slowest replica's."""
    if world == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device) -> float:
    """The job's work is the sum of the replicas' work."""
    if world == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(work_local: float, ms_local: float, world: int, device) -> tuple[float, float]:
    """(whole-job work per second, ms of the slowest replica)."""
    ms = max_over_ranks(ms_local, world, device)
    work = sum_over_ranks(work_local, world, device)
    return work / (ms * 1e-3), ms
