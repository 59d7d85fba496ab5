"""How the hot path spreads over several GPUs: by independent units, with no exchange.

A "unit" is one layer's cache (or one stream of a ragged batch): score, select, compact and
attention of a unit touch nothing of another unit, so rank r simply owns units
r, r + world, r + 2*world, ... and the only communication is the max-over-ranks of the timing.
"""
from __future__ import annotations

from typing import List


def units_for_rank(n_units: int, rank: int, world: int) -> List[int]:
    """Round-robin ownership of independent units; every unit has exactly one owner."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    return list(range(rank, n_units, world))


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's value (a no-op without an initialised process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
