"""Sharding of independent units (images / video clips) over ranks.

PACT reads nothing across requests, so a batch is split by image with no exchange on the data
path; the only communication is bookkeeping (max of the per-rank step time, sum of the units).
These helpers hold that host-side logic so that it can be exercised with the gloo backend on CPU.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_units(n_units: int, rank: int, world: int) -> range:
    """Contiguous, balanced share of units 0..n_units-1 for `rank` (first ranks take the remainder)."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    base, rem = divmod(n_units, world)
    start = rank * base + min(rank, rem)
    return range(start, start + base + (1 if rank < rem else 0))


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the synthetic workload a rank generates (weak scaling: one workload per rank)."""
    return base_seed + 100 * rank


def max_over_ranks(value: float, device="cpu") -> float:
    """Slowest rank's value (the job's step time); identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_this_rank: float, seconds_this_rank: float, device="cpu") -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    return sum_over_ranks(units_this_rank, device) / max_over_ranks(seconds_this_rank, device)
