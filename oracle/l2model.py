"""LRU model of operand-panel reuse in L2 for a tiled GEMM run under a tile order.

TEST INFRASTRUCTURE, and a MODEL: it predicts the ordering and sign of the effect of a
swizzle on L2 hit rate and DRAM reads, not the hardware counter.  It is the counterpart of
the paper's qualitative argument (tiles in one row of C share rows of A, tiles in one
column share columns of B, so co-scheduling them raises the hit rate of the L2 they share).

Model: `units` persistent workers; in round r worker u runs slot r*units + u.  The tiles of
a round advance through the K dimension in lockstep, one 64-wide k-block at a time; each
tile reads its A chunk (tile_m x 64 bf16) and its B chunk (64 x tile_n bf16).  Chunks live
in an LRU cache of `capacity` bytes; a read that finds its chunk is a hit.  After a round,
the C tiles written by it are inserted as pollution.  With `halves=2` there are two caches
of capacity/2, and the tiles of each worker go to the cache of that worker's half.

Known gaps against the hardware: concurrent misses to one chunk count as one miss, address
hashing and set conflicts are ignored, rounds are not really in lockstep.
"""

from __future__ import annotations

from collections import OrderedDict
from typing import Callable, Dict, Optional, Sequence


class _LRU:
    def __init__(self, capacity: int):
        self.capacity = capacity
        self.used = 0
        self.d: "OrderedDict[tuple, int]" = OrderedDict()

    def touch(self, key, size: int) -> bool:
        """Returns True on a hit.  On a miss the chunk is inserted, evicting the least recent."""
        if key in self.d:
            self.d.move_to_end(key)
            return True
        self.d[key] = size
        self.used += size
        while self.used > self.capacity and self.d:
            _, s = self.d.popitem(last=False)
            self.used -= s
        return False


def simulate(perm: Sequence[int], Tm: int, Tn: int, K: int, tile_m: int, tile_n: int, units: int,
             capacity: int, halves: int = 1, half_of_unit: Optional[Callable[[int], int]] = None,
             out_bytes_per_elem: int = 2, slots_of_unit: Optional[Callable[[int], Sequence[int]]] = None) -> Dict[str, float]:
    """Hit rate and DRAM read bytes of the operand stream.

    perm[s] = tile at slot s.  By default unit u runs slots u, u+units, ...; `slots_of_unit`
    overrides that (used for die-pinned schedules).  `half_of_unit(u)` names the cache a unit
    uses when halves == 2 (default: u % 2).
    """
    assert len(perm) == Tm * Tn
    kblocks = -(-K // 64)
    a_chunk, b_chunk = tile_m * 64 * 2, tile_n * 64 * 2
    c_tile = tile_m * tile_n * out_bytes_per_elem
    caches = [_LRU(capacity // halves) for _ in range(halves)]
    if half_of_unit is None:
        half_of_unit = (lambda u: u % 2)
    if slots_of_unit is None:
        queues = [list(range(u, len(perm), units)) for u in range(units)]
    else:
        queues = [list(slots_of_unit(u)) for u in range(units)]
    rounds = max(len(q) for q in queues) if queues else 0
    read = hit = 0
    for r in range(rounds):
        active = [(u, perm[q[r]]) for u, q in enumerate(queues) if r < len(q)]
        for kb in range(kblocks):
            for (u, t) in active:
                cache = caches[half_of_unit(u) if halves > 1 else 0]
                tm, tn = divmod(t, Tn)
                read += a_chunk + b_chunk
                if cache.touch(("A", tm, kb), a_chunk):
                    hit += a_chunk
                if cache.touch(("B", tn, kb), b_chunk):
                    hit += b_chunk
        for (u, t) in active:
            caches[half_of_unit(u) if halves > 1 else 0].touch(("C", t), c_tile)
    return {"read_bytes": float(read), "hit_bytes": float(hit), "hit_rate": hit / read if read else 0.0,
            "dram_read_bytes": float(read - hit)}


def simulate_two_level(perm: Sequence[int], Tm: int, Tn: int, K: int, tile_m: int, tile_n: int, units: int,
                       capacity_per_half: int, k_alternate: bool = False, out_bytes_per_elem: int = 2,
                       die_of_unit: Optional[Callable[[int], int]] = None,
                       slots_of_unit: Optional[Callable[[int], Sequence[int]]] = None) -> Dict[str, float]:
    """The same lockstep model over the two-level structure the probes found on B200: two L2 halves, every address homed
    on one of them (half of every chunk on each), an SM's request looked up first in the half of its own die and, when the
    line is homed on the other die and misses there, in the home half; DRAM is read only when the home misses; both
    halves keep a copy.  So data read from both dies occupies both halves (capacity is not pooled) but costs DRAM once.

    `k_alternate`: odd rounds walk the k-blocks in descending order (SP_FLAG_K_ALTERNATE).  `die_of_unit(u)` names the
    die of unit u (default u % 2: the hardware places consecutive CTA pairs on alternating halves only roughly; the
    model needs just an even spread).  Written C tiles go to their home half.  Same known gaps as `simulate`.
    """
    assert len(perm) == Tm * Tn
    kblocks = -(-K // 64)
    a_half, b_half = tile_m * 64 * 2 // 2, tile_n * 64 * 2 // 2           # bytes of the part of a chunk homed on one die
    c_half = tile_m * tile_n * out_bytes_per_elem // 2
    caches = [_LRU(capacity_per_half), _LRU(capacity_per_half)]
    if die_of_unit is None:
        die_of_unit = (lambda u: u % 2)
    if slots_of_unit is None:
        queues = [list(range(u, len(perm), units)) for u in range(units)]
    else:
        queues = [list(slots_of_unit(u)) for u in range(units)]
    rounds = max(len(q) for q in queues) if queues else 0
    stat = {"read": 0, "dram": 0}

    def request(d: int, key: tuple, size: int) -> None:
        for home in (0, 1):
            stat["read"] += size
            k2 = key + (home,)
            if caches[d].touch(k2, size):
                continue
            if home != d and caches[home].touch(k2, size):
                continue
            stat["dram"] += size

    for r in range(rounds):
        active = [(u, perm[q[r]]) for u, q in enumerate(queues) if r < len(q)]
        ks = range(kblocks - 1, -1, -1) if (k_alternate and r % 2) else range(kblocks)
        for kb in ks:
            for (u, t) in active:
                tm, tn = divmod(t, Tn)
                request(die_of_unit(u), ("A", tm, kb), a_half)
                request(die_of_unit(u), ("B", tn, kb), b_half)
        for (u, t) in active:
            for home in (0, 1):
                caches[home].touch(("C", t, home), c_half)
    read, dram = stat["read"], stat["dram"]
    return {"read_bytes": float(read), "hit_bytes": float(read - dram), "hit_rate": (read - dram) / read if read else 0.0,
            "dram_read_bytes": float(dram)}
