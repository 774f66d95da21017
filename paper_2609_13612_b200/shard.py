"""Host-side partition of the work units for more than one GPU.

A unit is a (batch, kv head) pair: a kv head with its g query heads is independent of every other
unit in forward and backward (dK/dV reduce only inside the unit), so ranks need no exchange step.
"""
from __future__ import annotations

from typing import List, Tuple


def units(B: int, Hkv: int) -> List[Tuple[int, int]]:
    return [(b, h) for b in range(B) for h in range(Hkv)]


def shard_units(B: int, Hkv: int, world: int, rank: int) -> List[Tuple[int, int]]:
    """Round-robin assignment of units to ranks."""
    assert 0 <= rank < world
    return units(B, Hkv)[rank::world]


def aggregate_throughput(units_done_per_rank: List[float], max_time_s: float) -> float:
    """Whole-job throughput: everything all ranks processed over the slowest rank's time."""
    return sum(units_done_per_rank) / max_time_s
