"""Batch sharding across GPUs.

Every call of the library treats sequences independently, so a batch is split
into contiguous ranges of sequences, one per rank, with NO collective on the
data path.  Ranges are balanced by the number of cached tokens (decode cost is
proportional to it).  The Philox list index stays global through ``list_base``,
so a sharded batch draws exactly the keep sets of the unsharded one.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def shard_batch(lens: Sequence[int], world: int) -> List[Tuple[int, int]]:
    """Contiguous [begin, end) ranges, one per rank, with near-equal sums of ``lens``.
    Every rank gets at least one sequence when ``len(lens) >= world``."""
    B = len(lens)
    if world <= 0:
        raise ValueError("world must be positive")
    if B <= world:      # one sequence per rank, the last ranks idle
        return [(min(r, B), min(r + 1, B)) for r in range(world)]
    total = float(sum(int(x) for x in lens))
    ranges = []
    begin = 0
    acc = 0.0
    for r in range(world):
        remaining_ranks = world - r
        if r == world - 1:
            end = B
        else:
            target = total * (r + 1) / world
            end = begin
            # leave at least one sequence for each later rank
            limit = B - (remaining_ranks - 1)
            while end < limit and (end == begin or acc + int(lens[end]) / 2.0 <= target):
                acc += int(lens[end])
                end += 1
            if B < world:
                end = min(end, B)
        ranges.append((begin, end))
        begin = end
    return ranges


def list_base(rank_range: Tuple[int, int], G: int) -> int:
    """Global index of the first eviction list of a rank's shard."""
    return rank_range[0] * G
