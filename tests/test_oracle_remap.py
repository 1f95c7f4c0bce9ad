"""Pins for the remap oracle: hand-written permutations, the paper's worked example,
independent second derivations, reductions between schemes, and brute-force invariants.
A plausible slip anywhere in the oracle (swapped loop order, wrong band edge, transposed
axes, off-by-one in a window) fails at least one of these."""

import itertools
import os

import pytest
from hypothesis import given, settings, strategies as st

from oracle import remap as R


def _read_ints(path):
    vals = []
    with open(path) as f:
        for line in f:
            if line.startswith("#"):
                continue
            vals += [int(v) for v in line.split()]
    return vals


# ---------------------------------------------------------------- paper's worked example
def test_paper_gemm_example_4x5(golden_dir):
    want = _read_ints(os.path.join(golden_dir, "xcd_gemm_4x5.txt"))
    got = R.xcd(20, 4)
    assert got == want
    # Caption of the GEMM swizzling figure: blocks are dealt round-robin to the XCDs
    # (slot s lands on XCD s mod 4); after the swizzle each XCD holds one row of C.
    Tn = 5
    for x in range(4):
        rows = {got[s] // Tn for s in range(20) if s % 4 == x}
        assert rows == {x}


def test_paper_listing_mi300x(golden_dir):
    want = _read_ints(os.path.join(golden_dir, "xcd_mi300x_304.txt"))
    got = R.xcd(304, 8)
    assert got[:16] == want
    assert R.is_bijection(got, 304)


def test_paper_formula_not_bijective_when_x_does_not_divide():
    # ceil(10/4) = 3: p = 3 -> 3*3 + 0 = 9, p = 7 -> 3*3 + 1 = 10 which is outside [0, 10)
    with pytest.raises(R.NotBijective):
        R.xcd(10, 4)
    with pytest.raises(R.NotBijective):
        R.xcd(148, 8)
    assert R.xcd_window(10, 4, False)[7] == 10


def test_xcd_more_examples():
    assert R.xcd(74, 2)[:4] == [0, 37, 1, 38]
    assert R.xcd(148, 2)[:4] == [0, 74, 1, 75]
    assert R.xcd(10, 4, balanced=True) == [0, 3, 6, 8, 1, 4, 7, 9, 2, 5]
    assert R.xcd(7, 3, balanced=True) == [0, 3, 5, 1, 4, 6, 2]
    assert R.xcd(5, 8, balanced=True) == [0, 1, 2, 3, 4]
    # windows of 8 on 16 tiles, 2 chiplets; on a 4 x 4 grid this is a 2-row supertile order
    assert R.xcd(16, 2, W=8) == [0, 4, 1, 5, 2, 6, 3, 7, 8, 12, 9, 13, 10, 14, 11, 15]
    assert R.xcd(16, 2, W=8) == R.group_m(4, 4, 2)


@given(n=st.integers(1, 400), X=st.integers(1, 64))
@settings(max_examples=200, deadline=None)
def test_xcd_contiguity_property(n, X):
    """Listing comment: contiguous new ids all sit on one XCD before the next XCD starts."""
    img = R.xcd_window(n, X, True)
    assert sorted(img) == list(range(n))
    for x in range(min(X, n)):
        mine = [img[p] for p in range(n) if p % X == x]
        assert mine == list(range(mine[0], mine[0] + len(mine)))
    if n % X == 0:
        assert R.xcd_window(n, X, False) == img


# ---------------------------------------------------------------- grouped orders
def test_group_hand_examples():
    assert R.group_m(4, 4, 2) == [0, 4, 1, 5, 2, 6, 3, 7, 8, 12, 9, 13, 10, 14, 11, 15]
    assert R.group_m(5, 3, 2) == [0, 3, 1, 4, 2, 5, 6, 9, 7, 10, 8, 11, 12, 13, 14]
    assert R.group_n(4, 4, 2) == [0, 1, 4, 5, 8, 9, 12, 13, 2, 3, 6, 7, 10, 11, 14, 15]
    assert R.group_n(3, 5, 2) == [0, 1, 5, 6, 10, 11, 2, 3, 7, 8, 12, 13, 4, 9, 14]
    assert R.group_m(3, 4, 3) == [0, 4, 8, 1, 5, 9, 2, 6, 10, 3, 7, 11]
    assert R.col_major(3, 4) == [0, 4, 8, 1, 5, 9, 2, 6, 10, 3, 7, 11]
    assert R.row_major(2, 3) == [0, 1, 2, 3, 4, 5]


def test_serpentine_bands_by_hand():
    # 4 x 3 grid, bands of 2 rows: the second band walks its columns right to left
    assert R.group_m(4, 3, 2, serpentine=True) == [0, 3, 1, 4, 2, 5, 8, 11, 7, 10, 6, 9]
    # 3 x 4 grid, bands of 2 columns: the second band walks its rows bottom to top
    assert R.group_n(3, 4, 2, serpentine=True) == [0, 1, 4, 5, 8, 9, 10, 11, 6, 7, 2, 3]
    for Tm, Tn, G in [(5, 7, 2), (8, 8, 3), (1, 9, 4)]:
        plain, serp = R.group_m(Tm, Tn, G), R.group_m(Tm, Tn, G, True)
        assert R.is_bijection(serp, Tm * Tn)
        band = G * Tn
        for b in range(0, Tm * Tn, band):
            chunk_p, chunk_s = plain[b:b + band], serp[b:b + band]
            g = len(chunk_p) // Tn
            if (b // band) % 2 == 0:
                assert chunk_s == chunk_p
            else:   # same band, columns in reverse order, rows inside a column unchanged
                cols = [chunk_p[i * g:(i + 1) * g] for i in range(Tn)]
                assert chunk_s == [t for col in reversed(cols) for t in col]
        # the first tile column of a band is the last one of the band before
        for b in range(band, Tm * Tn, band):
            assert serp[b] % Tn == serp[b - 1] % Tn


@given(Tm=st.integers(1, 60), Tn=st.integers(1, 60), G=st.integers(1, 80))
@settings(max_examples=150, deadline=None)
def test_group_reductions(Tm, Tn, G):
    T = Tm * Tn
    gm, gn = R.group_m(Tm, Tn, G), R.group_n(Tm, Tn, G)
    assert R.is_bijection(gm, T) and R.is_bijection(gn, T)
    assert R.group_m(Tm, Tn, 1) == R.row_major(Tm, Tn)
    assert R.group_n(Tm, Tn, 1) == R.col_major(Tm, Tn)
    if G >= Tm:
        assert gm == R.col_major(Tm, Tn)
    if G >= Tn:
        assert gn == R.row_major(Tm, Tn)
    # group_n on (Tm, Tn) is group_m on the transposed grid, ids transposed back
    gmt = R.group_m(Tn, Tm, G)
    assert gn == [(t % Tm) * Tn + (t // Tm) for t in gmt]
    # band structure: within the first full band all G rows of a column are consecutive
    if G <= Tm:
        for tn in range(Tn):
            chunk = gm[tn * G:(tn + 1) * G]
            assert chunk == [tm * Tn + tn for tm in range(G)]


# ---------------------------------------------------------------- curves
def _d2xy(order, d):
    """Independent derivation: the iterative bit-pair decode of the Hilbert index."""
    x = y = 0
    t = d
    s = 1
    while s < (1 << order):
        rx = 1 & (t // 2)
        ry = 1 & (t ^ rx)
        if ry == 0:
            if rx == 1:
                x, y = s - 1 - x, s - 1 - y
            x, y = y, x
        x += s * rx
        y += s * ry
        t //= 4
        s *= 2
    return x, y


def test_hilbert_h2_golden(golden_dir):
    flat = _read_ints(os.path.join(golden_dir, "hilbert_h2.txt"))
    want = list(zip(flat[0::2], flat[1::2]))
    assert R.hilbert_cells(2) == want


@pytest.mark.parametrize("k", range(0, 7))
def test_hilbert_two_derivations_and_geometry(k):
    cells = R.hilbert_cells(k)
    n = 1 << k
    assert len(cells) == n * n and len(set(cells)) == n * n
    assert cells[0] == (0, 0) and cells[-1] == (n - 1, 0)
    for (a, b) in zip(cells, cells[1:]):
        assert abs(a[0] - b[0]) + abs(a[1] - b[1]) == 1
    # the iterative decode visits the same cells, up to the x<->y orientation it fixes per order
    other = [_d2xy(k, d) for d in range(n * n)]
    assert other == cells or [(y, x) for (x, y) in other] == cells


def test_curve_hand_examples():
    assert R.hilbert(4, 4) == [0, 1, 5, 4, 8, 12, 13, 9, 10, 14, 15, 11, 7, 6, 2, 3]
    assert R.morton(4, 4) == [0, 1, 4, 5, 2, 3, 6, 7, 8, 9, 12, 13, 10, 11, 14, 15]
    assert R.hilbert(4, 2) == [0, 1, 3, 2, 4, 6, 7, 5]
    assert R.hilbert(2, 4) == [0, 4, 5, 1, 2, 3, 7, 6]
    assert R.hilbert(3, 3) == [0, 1, 4, 3, 6, 7, 8, 5, 2]
    assert R.morton(3, 3) == [0, 1, 3, 4, 2, 5, 6, 7, 8]
    assert R.hilbert(32, 16)[:24] == [0, 16, 17, 1, 2, 3, 19, 18, 34, 35, 51, 50, 49, 33, 32, 48, 64, 65, 81, 80,
                                      96, 112, 113, 97]


@pytest.mark.parametrize("Tm,Tn", [(32, 32), (32, 16), (16, 32), (64, 64), (128, 64)])
def test_hilbert_unit_steps_on_square_and_2to1_grids(Tm, Tn):
    p = R.hilbert(Tm, Tn)
    assert R.is_bijection(p, Tm * Tn)
    for a, b in zip(p, p[1:]):
        assert abs(a // Tn - b // Tn) + abs(a % Tn - b % Tn) == 1


@pytest.mark.parametrize("fn", [R.hilbert, R.morton])
@pytest.mark.parametrize("Tm,Tn", [(8, 8), (7, 5), (5, 12), (16, 4), (3, 3), (1, 9), (9, 1)])
def test_curves_keep_aligned_squares_contiguous(fn, Tm, Tn):
    p = fn(Tm, Tn)
    assert R.is_bijection(p, Tm * Tn)
    slot = {t: s for s, t in enumerate(p)}
    j = 1
    while (1 << j) <= min(Tm, Tn):
        w = 1 << j
        for m0 in range(0, Tm - w + 1, w):
            for n0 in range(0, Tn - w + 1, w):
                slots = sorted(slot[(m0 + a) * Tn + (n0 + b)] for a in range(w) for b in range(w))
                assert slots == list(range(slots[0], slots[0] + w * w))
        j += 1


def test_morton_is_bit_interleave_on_squares():
    p = R.morton(8, 8)
    for s, t in enumerate(p):
        tm, tn = divmod(t, 8)
        z = 0
        for b in range(3):
            z |= ((tn >> b) & 1) << (2 * b)
            z |= ((tm >> b) & 1) << (2 * b + 1)
        assert z == s


# ---------------------------------------------------------------- die split
def test_die_split_hand_examples():
    assert R.die_split(4, 4, 0, R.ROW_MAJOR) == list(range(16))
    assert R.die_split(4, 4, 0, R.ROW_MAJOR, interleave=True) == [0, 8, 1, 9, 2, 10, 3, 11, 4, 12, 5, 13, 6, 14, 7, 15]
    assert R.die_split(4, 4, 1, R.ROW_MAJOR) == [0, 1, 4, 5, 8, 9, 12, 13, 2, 3, 6, 7, 10, 11, 14, 15]
    assert R.die_split(5, 2, 0, R.ROW_MAJOR) == list(range(10))
    assert R.die_split(5, 2, 0, R.ROW_MAJOR, interleave=True) == [0, 6, 1, 7, 2, 8, 3, 9, 4, 5]
    assert R.die_split(4, 4, 0, R.GROUP_M, 2) == [0, 4, 1, 5, 2, 6, 3, 7, 8, 12, 9, 13, 10, 14, 11, 15]
    h0, h1 = R.die_split_halves(5, 2, 0, R.ROW_MAJOR, 1)
    assert (len(h0), len(h1)) == (6, 4)


@given(Tm=st.integers(1, 40), Tn=st.integers(1, 40), axis=st.integers(0, 1),
       inner=st.sampled_from([R.ROW_MAJOR, R.COL_MAJOR, R.GROUP_M, R.GROUP_N, R.MORTON, R.HILBERT]),
       G=st.integers(1, 9), inter=st.booleans())
@settings(max_examples=150, deadline=None)
def test_die_split_properties(Tm, Tn, axis, inner, G, inter):
    p = R.die_split(Tm, Tn, axis, inner, G, inter)
    T = Tm * Tn
    assert R.is_bijection(p, T)
    h0, h1 = R.die_split_halves(Tm, Tn, axis, inner, G)
    assert len(h0) >= len(h1)
    cut = R.ceil_div(Tm if axis == 0 else Tn, 2)

    def half(t):
        return int((t // Tn if axis == 0 else t % Tn) >= cut)

    assert all(half(t) == 0 for t in h0) and all(half(t) == 1 for t in h1)
    if not inter:
        assert p[:len(h0)] == h0
    else:
        # with equal halves the alternating merge is the paper's formula with two chiplets
        if len(h0) == len(h1):
            base = h0 + h1
            x2 = R.xcd(T, 2)
            assert p == [base[x2[s]] for s in range(T)]


# ---------------------------------------------------------------- everything, brute force
def test_all_schemes_bijective_on_every_small_grid():
    for Tm, Tn in itertools.product(range(1, 13), repeat=2):
        T = Tm * Tn
        for perm in (R.row_major(Tm, Tn), R.col_major(Tm, Tn), R.morton(Tm, Tn), R.hilbert(Tm, Tn)):
            assert R.is_bijection(perm, T)
        for G in (1, 2, 3, 5, 12, 13):
            assert R.is_bijection(R.group_m(Tm, Tn, G), T)
            assert R.is_bijection(R.group_n(Tm, Tn, G), T)
        for X in (1, 2, 3, 8):
            assert R.is_bijection(R.xcd(T, X, 0, True), T)
            assert R.is_bijection(R.xcd(T, X, 7, True), T)


def test_tile_map_front_door():
    P = R.Params
    assert R.tile_map(512, 512, 128, 128, R.GROUP_M, P(group=2)) == R.group_m(4, 4, 2)
    assert R.tile_map(500, 300, 128, 128, R.ROW_MAJOR) == list(range(12))        # ragged: 4 x 3 tiles
    assert R.tile_map(512, 640, 128, 128, R.XCD, P(num_xcds=4)) == R.xcd(20, 4)
    with pytest.raises(R.NotBijective):
        R.tile_map(512, 512, 128, 128, R.CUSTOM, P(custom_perm=[0] * 16))
    with pytest.raises(R.NotBijective):
        R.tile_map(256, 640, 128, 128, R.XCD, P(num_xcds=4))                     # n = 10, X = 4
    assert R.tile_map(256, 256, 128, 128, R.CUSTOM, P(custom_perm=[3, 1, 2, 0])) == [3, 1, 2, 0]


# ------------------------------------------------- printed formulas of other kernels as negative vectors
def test_bit_swap_pattern_breaks_when_grid_changes():
    """The appendix's bitwise pattern (swap adjacent bits) is a permutation only on
    power-of-four-sized ranges; the paper reports such patterns failing bijectivity."""
    def swap(p):
        return ((p >> 1) & 0x55555555) | ((p & 0x55555555) << 1)
    for n in (16, 64, 1024):
        assert R.is_bijection([swap(p) for p in range(n)], n)
    for n in (6, 20, 100):
        assert not R.is_bijection([swap(p) for p in range(n)], n)


def test_exactly_when_the_printed_formula_is_a_bijection():
    """Counting argument: chiplet x receives ceil(n/X) ids if x < n mod X, else floor(n/X), but the printed
    form starts every chiplet at x * ceil(n/X); the ranges tile [0, n) only if at most one (the last)
    chiplet is short: n mod X in {0, X-1}, or X > n (then it is the identity)."""
    for n in range(1, 161):
        for X in range(1, 25):
            bij = R.is_bijection(R.xcd_window(n, X, False), n)
            assert bij == (X > n or n % X in (0, X - 1)), (n, X)


# ------------------------------------------------- generalised Hilbert curve over a rectangle (not in the paper)
def test_hilbert_rect_hand_derived_examples():
    # 4 wide, 2 high: long case, two 2 x 2 blocks each walked down, along, up
    assert R.hilbert_rect_cells(4, 2) == [(0, 0), (0, 1), (1, 1), (1, 0), (2, 0), (2, 1), (3, 1), (3, 0)]
    assert R.hilbert_rect(2, 4) == [0, 4, 5, 1, 2, 6, 7, 3]
    # 2 wide, 3 high: major axis along y; one cell, then a column of three, then back up the first column
    assert R.hilbert_rect_cells(2, 3) == [(0, 0), (1, 0), (1, 1), (1, 2), (0, 2), (0, 1)]
    assert R.hilbert_rect(3, 2) == [0, 1, 3, 5, 4, 2]
    assert R.hilbert_rect(1, 5) == [0, 1, 2, 3, 4] and R.hilbert_rect(5, 1) == [0, 1, 2, 3, 4]


def test_hilbert_rect_on_power_of_two_squares_is_a_hilbert_curve():
    for k in range(1, 6):
        n = 1 << k
        cells = R.hilbert_rect_cells(n, n)
        h = R.hilbert_cells(k)                               # the independent construction pinned above
        assert cells == h or cells == [(y, x) for (x, y) in h]


def test_hilbert_rect_visits_every_cell_once_in_unit_steps():
    for W in range(1, 26):
        for H in range(1, 26):
            cells = R.hilbert_rect_cells(W, H)
            assert len(cells) == W * H and len(set(cells)) == W * H
            assert all(0 <= x < W and 0 <= y < H for (x, y) in cells)
            assert cells[0] == (0, 0)
            steps = [abs(a[0] - b[0]) + abs(a[1] - b[1]) for a, b in zip(cells, cells[1:])]
            diagonal = [s for s in steps if s != 1]
            assert all(s == 2 for s in diagonal) and len(diagonal) <= 1      # at most one diagonal step, never a jump
            if W % 2 == 0 and H % 2 == 0:
                assert not diagonal
