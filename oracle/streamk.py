"""CPU oracle (test infrastructure, never on the product path) for the k-split of the tail wave.

The paper's method is the remap of tile ids; it has no counterpart for splitting a tile along
k, so this file pins the library's own definition (stated in the C header) by plain
enumeration: every k-block position is assigned to a unit one by one, and the segments are
read off that assignment.  No arithmetic is shared with the library.
"""

from __future__ import annotations

from typing import List, Tuple

FULL, CONTRIB, OWNER = 0, 1, 2
MIN_RANGE = 4   # a unit's range is at least this many k-blocks, else fewer units share the tail
MAX_PIECES = 8  # pieces per tile: the storing unit adds the others one after the other


def tail(T: int, units: int, kblocks: int) -> Tuple[int, int]:
    """(number of tail slots, units sharing them): the remainder R = T mod units, each of its tiles cut into
    f = units // R equal pieces (at least MIN_RANGE k-blocks each, at most MAX_PIECES); nothing when f < 2."""
    R = T % units
    if R == 0:
        return 0, units
    f = min(units // R, kblocks // MIN_RANGE, MAX_PIECES)
    if f < 2:
        return 0, units
    return R, R * f


def plan(T: int, units: int, kblocks: int):
    """(first_slot, segments): segments[u] = [(slot, k0, k1, kind), ...] in walking order (highest slot first)."""
    tiles, share = tail(T, units, kblocks)
    first = T - tiles
    W = tiles * kblocks
    owner_of_pos: List[int] = []
    if tiles:
        begins = [u * W // share for u in range(share + 1)]
        u = 0
        for p in range(W):                      # one position at a time
            while not (begins[u] <= p < begins[u + 1]):
                u += 1
            owner_of_pos.append(u)
    segs = [[] for _ in range(units)]
    for j in range(tiles):                      # tail slot j: which units hold which of its k-blocks
        row = owner_of_pos[j * kblocks:(j + 1) * kblocks]
        kb = 0
        while kb < kblocks:
            u = row[kb]
            end = kb
            while end < kblocks and row[end] == u:
                end += 1
            if kb == 0 and end == kblocks:
                kind = FULL
            elif end == kblocks:
                kind = OWNER
            else:
                kind = CONTRIB
            segs[u].append((first + j, kb, end, kind))
            kb = end
    for u in range(units):
        segs[u].sort(key=lambda s: -s[0])
    return first, segs
