"""Sharding of a batch of positions over GPUs (the data-parallel axis of the training step).

Positions are independent through tree building, reward and the accepted path; Eq. 9-10
couple only the m positions of one group.  A batch therefore splits over ranks in whole
groups with no collective on the data path: every rank runs the three calls on its own
positions and the throughputs add.
"""
from __future__ import annotations


def shard_positions(B: int, m: int, world: int):
    """Split B positions (B a multiple of the group size m) over `world` ranks in whole groups.

    Ranks own consecutive blocks; the B / m groups are dealt as evenly as possible and the
    first (B / m) % world ranks take one extra group.  Returns a list of (first position,
    number of positions) per rank; a rank may get (first, 0) when there are fewer groups
    than ranks."""
    if B < 0 or m < 1 or world < 1 or B % m != 0:
        raise ValueError("B must be a non-negative multiple of m; world and m at least 1")
    groups = B // m
    base, extra = divmod(groups, world)
    out, first = [], 0
    for r in range(world):
        n = (base + (1 if r < extra else 0)) * m
        out.append((first, n))
        first += n
    return out
