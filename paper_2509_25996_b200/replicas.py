"""Throughput of N independent replicas (one process per GPU).

The AdamS step has no exchange between groups, matrices or GPUs, so several GPUs only ever run
independent replicas (or disjoint shards) of it.  The one thing the ranks share is the clock: the job
takes as long as its slowest rank.  These helpers hold that bookkeeping; they move one scalar through
`torch.distributed` (NCCL on GPUs, gloo on CPUs) outside any timed region.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def world_size() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def max_over_ranks(value: float, device="cpu") -> float:
    """The largest `value` any rank holds (the value itself without a process group)."""
    if world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank_per_step: int, steps: int, local_ms: float, device="cpu"):
    """(units per second summed over all ranks, ms of the slowest rank) for `steps` steps that took
    `local_ms` on this rank.  Every rank processes the same number of units per step (weak scaling)."""
    ms = max_over_ranks(local_ms, device)
    return world_size() * units_per_rank_per_step * steps / (ms * 1e-3), ms
