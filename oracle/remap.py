"""Remap oracle: every tile-order permutation written out by plain enumeration.

TEST INFRASTRUCTURE.  Nothing here is shared with the CUDA library.

Vocabulary (paper, GEMM case study in the appendix): the output matrix C (M x N) is cut
into Tm x Tn tiles; a logical tile id is ``t = tm * Tn + tn`` (the row-major
decomposition the paper's hardware-unaware listing uses: pid_m = pid // Tn,
pid_n = pid % Tn).  A *swizzle* recomputes the id of each block: ``pid = f(pid)``.
Here ``perm[s] = t`` says "the block issued at slot s works on tile t" -- the same
direction as the paper's formula (hardware id in, logical id out).  A remap is only
valid if it is a bijection on [0, T); the paper counts non-bijective maps as broken.

Each function below returns the permutation as a Python list and is written as the
nested loops of the definition, not as a closed form.
"""

from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

# scheme numbers: the values of the C enum the library's header declares
ROW_MAJOR, COL_MAJOR, GROUP_M, GROUP_N, MORTON, HILBERT, XCD, DIE_SPLIT, CUSTOM, HILBERT_RECT = range(10)


class NotBijective(ValueError):
    """The requested remap does not hit every tile id exactly once."""


def ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def grid(M: int, N: int, tile_m: int, tile_n: int) -> Tuple[int, int]:
    """Tm, Tn: number of tile rows / tile columns covering an M x N output."""
    if M <= 0 or N <= 0 or tile_m <= 0 or tile_n <= 0:
        raise ValueError("sizes must be positive")
    return ceil_div(M, tile_m), ceil_div(N, tile_n)


def is_bijection(perm: Sequence[int], T: int) -> bool:
    if len(perm) != T:
        return False
    seen = [False] * T
    for t in perm:
        if not (0 <= t < T) or seen[t]:
            return False
        seen[t] = True
    return True


# ----------------------------------------------------------------------------------
# plain orders
# ----------------------------------------------------------------------------------
def row_major(Tm: int, Tn: int) -> List[int]:
    """Identity: the paper's hardware-unaware order (tile rows outer, columns inner)."""
    out = []
    for tm in range(Tm):
        for tn in range(Tn):
            out.append(tm * Tn + tn)
    return out


def col_major(Tm: int, Tn: int) -> List[int]:
    out = []
    for tn in range(Tn):
        for tm in range(Tm):
            out.append(tm * Tn + tn)
    return out


def group_m(Tm: int, Tn: int, G: int, serpentine: bool = False) -> List[int]:
    """Supertiles of G tile rows: bands of G rows; inside a band walk the columns,
    and inside a column walk the band's rows.  The last band may have fewer rows.
    With ``serpentine`` every second band walks its columns from the far end back."""
    if G < 1:
        raise ValueError("group must be >= 1")
    out = []
    for band, first in enumerate(range(0, Tm, G)):
        cols = range(Tn)
        if serpentine and band % 2 == 1:
            cols = reversed(range(Tn))
        for tn in cols:
            for tm in range(first, min(first + G, Tm)):
                out.append(tm * Tn + tn)
    return out


def group_n(Tm: int, Tn: int, G: int, serpentine: bool = False) -> List[int]:
    """Supertiles of G tile columns: the transpose of ``group_m``."""
    if G < 1:
        raise ValueError("group must be >= 1")
    out = []
    for band, first in enumerate(range(0, Tn, G)):
        rows = range(Tm)
        if serpentine and band % 2 == 1:
            rows = reversed(range(Tm))
        for tm in rows:
            for tn in range(first, min(first + G, Tn)):
                out.append(tm * Tn + tn)
    return out


# ----------------------------------------------------------------------------------
# space-filling curves on the enclosing power-of-two square, cells outside dropped
# ----------------------------------------------------------------------------------
def _enclosing_order(Tm: int, Tn: int) -> int:
    k = 0
    while (1 << k) < max(Tm, Tn):
        k += 1
    return k


def hilbert_cells(k: int) -> List[Tuple[int, int]]:
    """H_k as a list of (x, y), built geometrically from four copies of H_{k-1}:
    a transposed copy in the lower-left quadrant, two upright copies in the two upper
    quadrants, and an anti-transposed copy in the lower-right quadrant.  Starts at
    (0,0), ends at (2^k - 1, 0); consecutive cells are unit steps."""
    cells = [(0, 0)]
    for level in range(1, k + 1):
        h = 1 << (level - 1)
        q0 = [(y, x) for (x, y) in cells]
        q1 = [(x, y + h) for (x, y) in cells]
        q2 = [(x + h, y + h) for (x, y) in cells]
        q3 = [(2 * h - 1 - y, h - 1 - x) for (x, y) in cells]
        cells = q0 + q1 + q2 + q3
    return cells


def morton_cells(k: int) -> List[Tuple[int, int]]:
    """Z-order over a 2^k square: x takes the even bits of the index, y the odd bits."""
    cells = []
    for z in range(1 << (2 * k)):
        x = 0
        y = 0
        for b in range(k):
            x |= ((z >> (2 * b)) & 1) << b
            y |= ((z >> (2 * b + 1)) & 1) << b
        cells.append((x, y))
    return cells


def _curve(Tm: int, Tn: int, cells: List[Tuple[int, int]]) -> List[int]:
    # the long side of the grid is walked by y
    out = []
    for (x, y) in cells:
        tm, tn = (y, x) if Tm >= Tn else (x, y)
        if tm < Tm and tn < Tn:
            out.append(tm * Tn + tn)
    return out


def hilbert(Tm: int, Tn: int) -> List[int]:
    return _curve(Tm, Tn, hilbert_cells(_enclosing_order(Tm, Tn)))


def morton(Tm: int, Tn: int) -> List[int]:
    return _curve(Tm, Tn, morton_cells(_enclosing_order(Tm, Tn)))


# ----------------------------------------------------------------------------------
# the paper's formula (appendix listing for GEMM): chiplet-aware transposition
# ----------------------------------------------------------------------------------
def hilbert_rect_cells(width: int, height: int) -> List[Tuple[int, int]]:
    """Generalised Hilbert curve over a width x height rectangle: the cells (x, y) in visiting order.

    Not in the paper.  The construction is the "generalized Hilbert curve" for rectangles of arbitrary size that Jakub
    Cerveny published (2018, with a reference implementation under the BSD 2-clause licence); it is restated here from
    its rules, as a work list of oriented rectangles.  An oriented rectangle has a corner, a unit direction `along` with
    a length (the side the curve runs along, entering at the corner and leaving at the far end of that side) and a unit
    direction `across` with a length:

      * one cell thick (either way): walk it;
      * more than 1.5 times as long as thick: cut it in two along its length;
      * else three parts: a first strip of the thickness, walked across-wise; the rest, walked along; and the first
        strip's other half, walked back across-wise towards the exit corner.

    Halves are floor(length / 2) when the direction points the positive way and ceil(length / 2) when it points the
    negative way (the rule is "floor of the signed half"); a cut that would leave an odd first piece of a side longer
    than 2 is moved by one, so that pieces meet at even offsets and steps stay unit steps where parity allows."""
    def half(length: int, direction: Tuple[int, int]) -> int:
        positive = direction[0] + direction[1] > 0
        return length // 2 if positive else (length + 1) // 2

    def evened(piece: int, whole: int) -> int:
        return piece + 1 if (piece % 2 == 1 and whole > 2) else piece

    out: List[Tuple[int, int]] = []
    x_dir, y_dir = (1, 0), (0, 1)
    first = ((0, 0), x_dir, width, y_dir, height) if width >= height else ((0, 0), y_dir, height, x_dir, width)
    todo = [first]                                   # last in, first out: parts are pushed in reverse visiting order
    while todo:
        (cx, cy), along, la, across, lc = todo.pop()
        if lc == 1 or la == 1:
            step, n = (along, la) if lc == 1 else (across, lc)
            out.extend((cx + i * step[0], cy + i * step[1]) for i in range(n))
            continue
        back = (-along[0], -along[1])
        if 2 * la > 3 * lc:
            cut = evened(half(la, along), la)
            todo.append(((cx + cut * along[0], cy + cut * along[1]), along, la - cut, across, lc))
            todo.append(((cx, cy), along, cut, across, lc))
            continue
        strip = evened(half(lc, across), lc)         # thickness of the first and third part
        near = half(la, along)                       # how far the first part reaches along the length
        far_corner = (cx + (la - 1) * along[0] + (strip - 1) * across[0], cy + (la - 1) * along[1] + (strip - 1) * across[1])
        todo.append((far_corner, (-across[0], -across[1]), strip, back, la - near))
        todo.append(((cx + strip * across[0], cy + strip * across[1]), along, la, across, lc - strip))
        todo.append(((cx, cy), across, strip, along, near))
    return out


def hilbert_rect(Tm: int, Tn: int) -> List[int]:
    """x runs along the tile columns, y along the tile rows."""
    return [y * Tn + x for (x, y) in hilbert_rect_cells(Tn, Tm)]


def xcd_window(n: int, X: int, balanced: bool) -> List[int]:
    """Image of the local ids 0..n-1 of one window under the paper's swizzle.

    literal : p -> (p mod X) * ceil(n / X) + p div X       (exactly as printed)
    balanced: when X does not divide n the printed form leaves [0, n); here chiplet x
              owns floor(n/X) ids plus one more if x < n mod X, contiguous, in order.
              It coincides with the literal form whenever X divides n.
    """
    if X < 1:
        raise ValueError("num_xcds must be >= 1")
    out = []
    if not balanced:
        per = ceil_div(n, X)
        for p in range(n):
            out.append((p % X) * per + p // X)
        return out
    # balanced: enumerate which ids each chiplet owns, then hand them out in turn
    q, r = divmod(n, X)
    first = []
    nxt = 0
    for x in range(X):
        first.append(nxt)
        nxt += q + (1 if x < r else 0)
    for p in range(n):
        out.append(first[p % X] + p // X)
    return out


def xcd(T: int, X: int, W: int = 0, balanced: bool = False) -> List[int]:
    """The paper's remap applied to consecutive windows of W slots (W = 0 means one
    window over all T slots, which is what its 4 x 5 figure shows; W = number of
    resident blocks is its persistent-kernel listing)."""
    if W < 0:
        raise ValueError("wave must be >= 0")
    if W == 0:
        W = T
    out = []
    for base in range(0, T, W):
        n = min(W, T - base)
        for v in xcd_window(n, X, balanced):
            out.append(base + v)
    if not is_bijection(out, T):
        raise NotBijective(f"XCD remap (T={T}, X={X}, W={W}) leaves [0,{T})")
    return out


# ----------------------------------------------------------------------------------
# die-aware split: two halves of the tile space, each ordered on its own
# ----------------------------------------------------------------------------------
def _inner(Tm: int, Tn: int, scheme: int, G: int, serpentine: bool = False) -> List[int]:
    if scheme == ROW_MAJOR:
        return row_major(Tm, Tn)
    if scheme == COL_MAJOR:
        return col_major(Tm, Tn)
    if scheme == GROUP_M:
        return group_m(Tm, Tn, G, serpentine)
    if scheme == GROUP_N:
        return group_n(Tm, Tn, G, serpentine)
    if scheme == MORTON:
        return morton(Tm, Tn)
    if scheme == HILBERT:
        return hilbert(Tm, Tn)
    raise ValueError("inner scheme must be one of the plain orders")


def die_split_halves(Tm: int, Tn: int, axis: int, inner: int, G: int, serpentine: bool = False) -> Tuple[List[int], List[int]]:
    """The two queues.  axis 0 halves the tile rows (half 0 = rows [0, ceil(Tm/2))),
    axis 1 halves the tile columns.  Each half is a grid of its own, ordered by the
    inner scheme; its local ids are mapped back to ids of the whole grid."""
    if axis not in (0, 1):
        raise ValueError("split_axis must be 0 or 1")
    halves = []
    if axis == 0:
        cut = ceil_div(Tm, 2)
        for (r0, r1) in ((0, cut), (cut, Tm)):
            rows = r1 - r0
            q = []
            if rows > 0:
                for local in _inner(rows, Tn, inner, G, serpentine):
                    lm, ln = divmod(local, Tn)
                    q.append((r0 + lm) * Tn + ln)
            halves.append(q)
    else:
        cut = ceil_div(Tn, 2)
        for (c0, c1) in ((0, cut), (cut, Tn)):
            cols = c1 - c0
            q = []
            if cols > 0:
                for local in _inner(Tm, cols, inner, G, serpentine):
                    lm, ln = divmod(local, cols)
                    q.append(lm * Tn + (c0 + ln))
            halves.append(q)
    return halves[0], halves[1]


def die_split(Tm: int, Tn: int, axis: int = 0, inner: int = ROW_MAJOR, G: int = 1,
              interleave: bool = False, serpentine: bool = False) -> List[int]:
    h0, h1 = die_split_halves(Tm, Tn, axis, inner, G, serpentine)
    if not interleave:
        return h0 + h1
    out = []
    for i in range(len(h0)):          # len(h0) >= len(h1) by construction
        out.append(h0[i])
        if i < len(h1):
            out.append(h1[i])
    return out


def custom(T: int, table: Sequence[int]) -> List[int]:
    out = [int(v) for v in table]
    if not is_bijection(out, T):
        raise NotBijective("custom table is not a permutation of the tile ids")
    return out


# ----------------------------------------------------------------------------------
# the call the library's sp_tile_map mirrors
# ----------------------------------------------------------------------------------
@dataclass
class Params:
    group: int = 1
    num_xcds: int = 1
    wave: int = 0
    xcd_balanced: int = 0
    split_axis: int = 0
    inner_scheme: int = ROW_MAJOR
    inner_group: int = 1
    interleave: int = 0
    custom_perm: Optional[Sequence[int]] = field(default=None)
    flags: int = 0          # bit 2 (value 4): serpentine bands; bit 1 (value 2) only affects placement, not the map


def tile_map(M: int, N: int, tile_m: int, tile_n: int, scheme: int, p: Optional[Params] = None) -> List[int]:
    p = p or Params()
    Tm, Tn = grid(M, N, tile_m, tile_n)
    T = Tm * Tn
    if scheme == ROW_MAJOR:
        out = row_major(Tm, Tn)
    elif scheme == COL_MAJOR:
        out = col_major(Tm, Tn)
    elif scheme == GROUP_M:
        out = group_m(Tm, Tn, p.group, bool(p.flags & 4))
    elif scheme == GROUP_N:
        out = group_n(Tm, Tn, p.group, bool(p.flags & 4))
    elif scheme == MORTON:
        out = morton(Tm, Tn)
    elif scheme == HILBERT:
        out = hilbert(Tm, Tn)
    elif scheme == XCD:
        out = xcd(T, p.num_xcds, p.wave, bool(p.xcd_balanced))
    elif scheme == DIE_SPLIT:
        out = die_split(Tm, Tn, p.split_axis, p.inner_scheme, p.inner_group, bool(p.interleave), bool(p.flags & 4))
    elif scheme == HILBERT_RECT:
        out = hilbert_rect(Tm, Tn)
    elif scheme == CUSTOM:
        if p.custom_perm is None:
            raise ValueError("custom scheme needs a table")
        out = custom(T, p.custom_perm)
    else:
        raise ValueError("unknown scheme")
    if not is_bijection(out, T):
        raise NotBijective("remap is not a bijection")
    return out
