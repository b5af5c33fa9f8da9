"""Batch sharding over ranks.

Requests are independent (Eq. 8-10 never couple two images), so N GPUs run N copies of the
single-GPU path on disjoint slices of the batch and no collective sits on the data path.
"""
from __future__ import annotations

from typing import Tuple


def shard_range(batch: int, rank: int, world: int) -> Tuple[int, int]:
    """Half-open range [lo, hi) of requests owned by `rank`: contiguous, sizes differ by at most one."""
    if world <= 0 or not (0 <= rank < world) or batch < 0:
        raise ValueError("bad shard arguments")
    base, extra = divmod(batch, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return lo, hi
