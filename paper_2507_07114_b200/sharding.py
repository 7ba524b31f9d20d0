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


def packet_range_config(total_elems: int, packet_elems: int, rank: int, world: int) -> dict:
    """One bucket simulated by `world` GPUs, each a contiguous packet range for all W workers.

    Returns the keyword arguments that describe rank's range to lossy_init (`n`, `shard_packet0`,
    `bucket_packets`) plus the element offset `e0` of the range inside the bucket's arrays.
    """
    K = (total_elems + packet_elems - 1) // packet_elems
    lo, hi = shard_range(K, rank, world)
    e0, e1 = min(total_elems, lo * packet_elems), min(total_elems, hi * packet_elems)   # a rank may get nothing
    return {"n": e1 - e0, "shard_packet0": lo, "bucket_packets": K, "e0": e0}
