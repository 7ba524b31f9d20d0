"""Host-side partition of a job over several GPUs (one process per GPU).

Packets evolve independently, so a job of `units` buckets (or packets) is split
into contiguous ranges, one per rank; the only cross-rank quantity is the sum of
the per-replica squared drift sums.
"""
from __future__ import annotations


def shard_range(units: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous range [lo, hi) of `units` owned by `rank`; sizes differ by at most one."""
    if world <= 0 or not 0 <= rank < world:
        raise ValueError("bad rank/world")
    base, extra = divmod(units, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)
