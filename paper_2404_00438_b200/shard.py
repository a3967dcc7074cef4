"""Coordinate sharding of a parameter set across GPUs (one process per GPU).

Every coordinate of a Distributed-Lion step is independent of every other one
(Algorithm 1 is element-wise; the vote is across workers, not across
coordinates), so a model can be cut into contiguous coordinate slabs, one per
rank, each holding its slab of ALL N workers' state.  A rank then runs the
ordinary single-GPU calls on its slab and no data-path collective is needed.
This module only computes the cut; it holds no optimizer arithmetic.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple

ALIGN = 128


@dataclass
class Piece:
    global_offset: int      # arena index in the unsharded layout
    local_offset: int       # arena index in this rank's layout (multiple of ALIGN)
    numel: int


@dataclass
class Shard:
    rank: int
    world: int
    pieces: List[Piece]
    d_pad: int              # length of this rank's arenas

    @property
    def segments(self) -> List[Tuple[int, int]]:
        """Segment table of this rank's slab, ready for ``dlion_init``."""
        return [(p.local_offset, p.numel) for p in self.pieces] or [(0, 0)]

    @property
    def d(self) -> int:
        return sum(p.numel for p in self.pieces)


def _cuts(segments: Sequence[Tuple[int, int]], world: int) -> List[int]:
    """Cut points in 'parameter index' space (0..D), each falling on a segment
    boundary or on a multiple of ALIGN inside a segment."""
    total = sum(n for _, n in segments)
    cuts = [0]
    for r in range(1, world):
        target = total * r // world
        acc = 0
        cut = total
        for _, n in segments:
            if target < acc + n:
                inside = (target - acc) // ALIGN * ALIGN
                cut = acc + inside
                break
            acc += n
        cuts.append(max(cut, cuts[-1]))
    cuts.append(total)
    return cuts


def shard_segments(segments: Sequence[Tuple[int, int]], rank: int, world: int) -> Shard:
    """The slab of ``rank`` when ``segments`` is split across ``world`` ranks."""
    if not 0 <= rank < world:
        raise ValueError("rank out of range")
    cuts = _cuts(segments, world)
    lo, hi = cuts[rank], cuts[rank + 1]
    pieces, acc, local = [], 0, 0
    for off, n in segments:
        a, b = max(lo, acc), min(hi, acc + n)
        if a < b:
            pieces.append(Piece(off + (a - acc), local, b - a))
            local += (b - a + ALIGN - 1) // ALIGN * ALIGN
        acc += n
    return Shard(rank, world, pieces, max(local, ALIGN))
