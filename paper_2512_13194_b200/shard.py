"""Batch partition across GPUs.  Sequences are independent, so a rank verifies a
contiguous slice of the batch and passes the slice's first global index as
``b_first``; no data-path collective is needed and results do not depend on the split."""
from __future__ import annotations

from typing import Tuple


def shard_range(B: int, rank: int, world_size: int) -> Tuple[int, int]:
    """-> (first, count): contiguous, sizes differ by at most one, earlier ranks larger."""
    if world_size < 1 or not 0 <= rank < world_size or B < 0:
        raise ValueError("bad rank / world_size / B")
    base, extra = divmod(B, world_size)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)
