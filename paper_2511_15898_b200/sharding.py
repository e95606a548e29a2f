"""Batch sharding across ranks (one process per GPU).

Instances are independent, so the N-GPU path is pure batch sharding: every rank owns a
contiguous slice of the batch, runs gr_solve / gr_verify on it, and the results stay on the
rank that owns the rows.  There is no data-path collective; the only communication is the
barrier around a timed region and the max-over-ranks of its duration.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_range(batch: int, world: int, rank: int) -> Tuple[int, int]:
    """[lo, hi) of the instances rank `rank` owns: contiguous, sizes differ by at most one."""
    if world < 1 or not (0 <= rank < world) or batch < 0:
        raise ValueError("bad sharding arguments")
    base, extra = divmod(batch, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` over all ranks (the slowest rank's time); a no-op without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: int, seconds_this_rank: float, device="cpu") -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    return world * units_per_rank / max_over_ranks(seconds_this_rank, device)
