"""Sharding of a batch of sequences over ranks (one process per GPU).

Sequences are independent in the verify-and-feedback step, so rank r of W takes a contiguous
block of sequences and no data crosses ranks on the path.  The only reductions are for reporting:
the slowest rank's time and the number of positions all ranks processed.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_range(B: int, rank: int, world: int) -> Tuple[int, int]:
    """Half-open range [b0, b1) of the sequences of rank ``rank``; sizes differ by at most one."""
    if world < 1 or not (0 <= rank < world) or B < 0:
        raise ValueError("bad rank/world/B")
    base, rem = divmod(B, world)
    b0 = rank * base + min(rank, rem)
    return b0, b0 + base + (1 if rank < rem else 0)


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """Largest ``value`` over all ranks (the step time of the job is the slowest rank's)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: str = "cpu") -> float:
    """Sum of ``value`` over all ranks (units processed by the whole job)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
