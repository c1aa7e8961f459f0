"""Batch sharding for multi-GPU runs.  Every sequence of a round is independent through all steps, so N
ranks split the batch into contiguous ranges and run the same single-GPU path with no data-path collective;
the caller concatenates the outputs in rank order."""
from __future__ import annotations


def shard_range(batch: int, rank: int, world: int) -> tuple[int, int]:
    """Sequences [lo, hi) that `rank` of `world` owns; sizes differ by at most one, earlier ranks larger."""
    if world < 1 or not (0 <= rank < world) or batch < 0:
        raise ValueError("bad shard arguments")
    base, rem = divmod(batch, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
