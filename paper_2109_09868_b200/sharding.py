"""Splitting a batch of groups over ranks.

Every group is an independent problem (its own queries, mask and predictions),
so a batch shards over GPUs by contiguous blocks of groups with no exchange
step: each rank encodes / locates / decodes its block and the results are
concatenated in rank order.
"""
from __future__ import annotations

from typing import Tuple


def shard_groups(G: int, world_size: int, rank: int) -> Tuple[int, int]:
    """(first group, number of groups) of `rank`'s contiguous block; block sizes
    differ by at most one and earlier ranks get the larger blocks."""
    if world_size < 1 or not (0 <= rank < world_size) or G < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(G, world_size)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)
