"""Host remap (closed forms in the library) against the enumerating oracle: bit-exact."""

import ctypes

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import paper_2508_20258_b200 as sp
from oracle import remap as R


def _lib_map(Tm, Tn, scheme, **kw):
    return sp.tile_map(Tm * 128, Tn * 64, 128, 64, scheme, sp.make_params(**kw)).tolist()


@given(Tm=st.integers(1, 150), Tn=st.integers(1, 150), G=st.integers(1, 200))
@settings(max_examples=120, deadline=None)
def test_plain_and_grouped_orders(Tm, Tn, G):
    assert _lib_map(Tm, Tn, sp.ROW_MAJOR) == R.row_major(Tm, Tn)
    assert _lib_map(Tm, Tn, sp.COL_MAJOR) == R.col_major(Tm, Tn)
    assert _lib_map(Tm, Tn, sp.GROUP_M, group=G) == R.group_m(Tm, Tn, G)
    assert _lib_map(Tm, Tn, sp.GROUP_N, group=G) == R.group_n(Tm, Tn, G)
    assert _lib_map(Tm, Tn, sp.GROUP_M, group=G, flags=4) == R.group_m(Tm, Tn, G, True)
    assert _lib_map(Tm, Tn, sp.GROUP_N, group=G, flags=4) == R.group_n(Tm, Tn, G, True)


@given(Tm=st.integers(1, 70), Tn=st.integers(1, 70))
@settings(max_examples=60, deadline=None)
def test_curves(Tm, Tn):
    assert _lib_map(Tm, Tn, sp.MORTON) == R.morton(Tm, Tn)
    assert _lib_map(Tm, Tn, sp.HILBERT) == R.hilbert(Tm, Tn)


@pytest.mark.parametrize("Tm,Tn", [(1, 1), (32, 32), (32, 16), (64, 8), (64, 64), (128, 8), (5, 100)])
def test_curves_on_config_grids(Tm, Tn):
    assert _lib_map(Tm, Tn, sp.MORTON) == R.morton(Tm, Tn)
    assert _lib_map(Tm, Tn, sp.HILBERT) == R.hilbert(Tm, Tn)


@given(T=st.integers(1, 3000), X=st.integers(1, 200), W=st.integers(0, 400), bal=st.booleans())
@settings(max_examples=200, deadline=None)
def test_xcd(T, X, W, bal):
    try:
        want = R.xcd(T, X, W, bal)
    except R.NotBijective:
        want = None
    out = np.full(T, -7, dtype=np.int32)
    p = sp.make_params(num_xcds=X, wave=W, xcd_balanced=int(bal))
    rc = sp.lib().sp_tile_map(128, T * 128, 128, 128, sp.XCD, ctypes.byref(p), out.ctypes.data)
    if want is None:
        assert rc == sp.ERR_NOT_BIJECTIVE
        assert (out == -7).all()          # untouched on rejection
    else:
        assert rc == sp.OK and out.tolist() == want


@given(Tm=st.integers(1, 40), Tn=st.integers(1, 40), axis=st.integers(0, 1),
       inner=st.sampled_from([R.ROW_MAJOR, R.COL_MAJOR, R.GROUP_M, R.GROUP_N, R.MORTON, R.HILBERT]),
       G=st.integers(1, 9), inter=st.booleans())
@settings(max_examples=200, deadline=None)
def test_die_split(Tm, Tn, axis, inner, G, inter):
    got = _lib_map(Tm, Tn, sp.DIE_SPLIT, split_axis=axis, inner_scheme=inner, inner_group=G, interleave=int(inter))
    assert got == R.die_split(Tm, Tn, axis, inner, G, inter)
    got = _lib_map(Tm, Tn, sp.DIE_SPLIT, split_axis=axis, inner_scheme=inner, inner_group=G, interleave=int(inter), flags=4)
    assert got == R.die_split(Tm, Tn, axis, inner, G, inter, True)


def test_front_door_matches_oracle_on_the_five_workload_grids():
    cases = [(512, 512, 128, 128), (4096, 4096, 128, 256), (8192, 8192, 256, 256), (16384, 2048, 256, 256),
             (16384, 2048, 128, 256), (16384, 16384, 256, 256), (1000, 520, 128, 128)]
    for (M, N, tm, tn) in cases:
        for scheme, kw in [(sp.ROW_MAJOR, {}), (sp.COL_MAJOR, {}), (sp.GROUP_M, dict(group=8)),
                           (sp.GROUP_N, dict(group=4)), (sp.MORTON, {}), (sp.HILBERT, {}),
                           (sp.XCD, dict(num_xcds=2, wave=74, xcd_balanced=1)),
                           (sp.DIE_SPLIT, dict(split_axis=0, inner_scheme=sp.HILBERT)),
                           (sp.DIE_SPLIT, dict(split_axis=1, inner_scheme=sp.GROUP_M, inner_group=8, interleave=1))]:
            got = sp.tile_map(M, N, tm, tn, scheme, sp.make_params(**kw)).tolist()
            want = R.tile_map(M, N, tm, tn, scheme, R.Params(**kw))
            assert got == want, (M, N, tm, tn, scheme, kw)


def test_custom_tables():
    good = [3, 1, 2, 0]
    assert sp.tile_map(256, 256, 128, 128, sp.CUSTOM, sp.make_params(custom_perm=good)).tolist() == good
    for bad in ([0, 0, 1, 2], [0, 1, 2, 4], [0, 1, 2, -1]):
        with pytest.raises(sp.SpError) as e:
            sp.tile_map(256, 256, 128, 128, sp.CUSTOM, sp.make_params(custom_perm=bad))
        assert e.value.status == sp.ERR_NOT_BIJECTIVE


def test_argument_errors():
    L = sp.lib()
    out = np.zeros(16, dtype=np.int32)
    ok = sp.make_params(group=2)
    assert L.sp_tile_map(0, 512, 128, 128, sp.ROW_MAJOR, None, out.ctypes.data) == sp.ERR_INVALID_ARG
    assert L.sp_tile_map(512, 512, 128, 0, sp.ROW_MAJOR, None, out.ctypes.data) == sp.ERR_INVALID_ARG
    assert L.sp_tile_map(512, 512, 128, 128, 99, None, out.ctypes.data) == sp.ERR_INVALID_ARG
    assert L.sp_tile_map(512, 512, 128, 128, sp.GROUP_M, None, out.ctypes.data) == sp.ERR_INVALID_ARG
    assert L.sp_tile_map(512, 512, 128, 128, sp.GROUP_M, ctypes.byref(ok), None) == sp.ERR_INVALID_ARG
    for kw in (dict(group=0), ):
        p = sp.make_params(**kw)
        assert L.sp_tile_map(512, 512, 128, 128, sp.GROUP_M, ctypes.byref(p), out.ctypes.data) == sp.ERR_INVALID_ARG
    p = sp.make_params(num_xcds=0)
    assert L.sp_tile_map(512, 512, 128, 128, sp.XCD, ctypes.byref(p), out.ctypes.data) == sp.ERR_INVALID_ARG
    p = sp.make_params(num_xcds=2, wave=-1)
    assert L.sp_tile_map(512, 512, 128, 128, sp.XCD, ctypes.byref(p), out.ctypes.data) == sp.ERR_INVALID_ARG
    p = sp.make_params(split_axis=2)
    assert L.sp_tile_map(512, 512, 128, 128, sp.DIE_SPLIT, ctypes.byref(p), out.ctypes.data) == sp.ERR_INVALID_ARG
    p = sp.make_params(inner_scheme=sp.XCD)
    assert L.sp_tile_map(512, 512, 128, 128, sp.DIE_SPLIT, ctypes.byref(p), out.ctypes.data) == sp.ERR_INVALID_ARG
    p = sp.make_params(group=2)
    p.struct_size = 12
    assert L.sp_tile_map(512, 512, 128, 128, sp.GROUP_M, ctypes.byref(p), out.ctypes.data) == sp.ERR_INVALID_ARG
    assert "struct_size" in sp.last_error()
    # more than 2^24 tiles
    assert L.sp_tile_map(1 << 20, 1 << 20, 128, 128, sp.ROW_MAJOR, None, out.ctypes.data) == sp.ERR_INVALID_ARG
    # curve on a grid too elongated for its enclosing square
    assert L.sp_tile_map(128 * 5000, 128, 128, 128, sp.HILBERT, None, out.ctypes.data) == sp.ERR_UNSUPPORTED
    assert sp.tile_count(512, 640, 128, 128) == 20 and sp.tile_count(1, 1, 128, 128) == 1
    assert sp.tile_count(0, 5, 1, 1) == -1


def test_paper_example_through_the_library():
    got = sp.tile_map(4 * 128, 5 * 128, 128, 128, sp.XCD, sp.make_params(num_xcds=4)).tolist()
    assert got == [0, 5, 10, 15, 1, 6, 11, 16, 2, 7, 12, 17, 3, 8, 13, 18, 4, 9, 14, 19]
    with pytest.raises(sp.SpError) as e:      # 148 blocks over 8 chiplets: printed form leaves the range
        sp.tile_map(128, 148 * 128, 128, 128, sp.XCD, sp.make_params(num_xcds=8))
    assert e.value.status == sp.ERR_NOT_BIJECTIVE


def test_die_pinned_rank_assignment_covers_every_rank_under_any_placement():
    """If the GPU is shared, more units than measured may land on one L2 half; the surplus must take exactly
    the ranks left free on the other half (host self-test of the function the kernel uses)."""
    L = sp.lib()
    for n0, n1 in [(37, 37), (74, 74), (1, 1), (3, 5), (0, 4)]:
        for arrivals0 in range(0, n0 + n1 + 1):
            assert L.sp_selftest_pinned_tickets(n0, n1, arrivals0) == sp.OK, (n0, n1, arrivals0)
    assert L.sp_selftest_pinned_tickets(2, 2, 5) == sp.ERR_INVALID_ARG


def test_largest_accepted_grids():
    """The documented limits: 2^24 tiles, curve orders up to 4096 tiles per side.  At the limit the maps are still
    bijections (checked with numpy; the enumerating oracle would take minutes), one tile beyond is refused."""
    T = 1 << 24
    for scheme, kw in [(sp.ROW_MAJOR, {}), (sp.GROUP_M, dict(group=5)), (sp.GROUP_N, dict(group=7)),
                       (sp.XCD, dict(num_xcds=8, wave=148, xcd_balanced=1)),
                       (sp.DIE_SPLIT, dict(split_axis=1, inner_scheme=sp.GROUP_M, inner_group=3, interleave=1))]:
        perm = np.asarray(sp.tile_map(4096, 4096, 1, 1, scheme, sp.make_params(**kw)))
        assert perm.shape == (T,)
        seen = np.zeros(T, dtype=bool)
        seen[perm] = True
        assert seen.all(), scheme
    h = np.asarray(sp.tile_map(4096, 4096, 1, 1, sp.HILBERT))
    tm, tn = np.divmod(h, 4096)
    assert (np.abs(np.diff(tm)) + np.abs(np.diff(tn)) == 1).all()          # a Hilbert walk moves one cell at a time
    assert h[0] == 0 and np.array_equal(np.sort(h), np.arange(T))
    with pytest.raises(sp.SpError) as e:
        sp.tile_map(4097, 4096, 1, 1, sp.ROW_MAJOR)
    assert e.value.status == sp.ERR_INVALID_ARG
    with pytest.raises(sp.SpError) as e:
        sp.tile_map(4097, 8, 1, 1, sp.HILBERT)
    assert e.value.status == sp.ERR_UNSUPPORTED
    assert sp.tile_count(1 << 40, 1 << 40, 1 << 30, 1 << 30) == 1 << 20


def test_the_papers_other_printed_remaps_meet_the_gate_as_caller_tables():
    """The appendix prints a remap for each of its other kernels (with eight chiplets).  Restated here as functions of
    the linear block id and handed to the library as SP_CUSTOM tables: the gate must accept exactly those that are
    permutations, which is what the paper's loop needs from it (a broken remap is a failed attempt, not a launch)."""
    X = 8

    def chunked(p, n):            # layer-norm / softmax figures: chiplet from (p div X) mod X, position p mod X
        return ((p // X) % X) * (-(-n // X)) + p % X

    def floor_form(p, n):         # the hardware-aware transpose figure: the GEMM formula with floor for ceil
        return p // X + (p % X) * (n // X)

    def strided(p, n):            # the transpose figure: chiplet from (p div X) mod X, then p div X
        return ((p // X) % X) * (n // X) + p // X

    def collapsed(p, n, rows):    # the stencil figure: a whole chunk of `rows` ids lands on one id
        return (p // (X * rows)) * X + (p // rows) % X

    def gate(table, T):
        seen = np.zeros(T, dtype=bool)
        ok = all(0 <= t < T for t in table)
        if ok:
            seen[np.asarray(table)] = True
        want = ok and bool(seen.all())
        try:
            got = list(sp.tile_map(T, 1, 1, 1, sp.CUSTOM, sp.make_params(custom_perm=list(table))))
            assert got == list(table)
            accepted = True
        except sp.SpError as e:
            assert e.status == sp.ERR_NOT_BIJECTIVE
            accepted = False
        assert accepted == want
        return accepted

    assert gate([chunked(p, 64) for p in range(64)], 64)                  # 64 blocks: the identity
    assert not gate([chunked(p, 128) for p in range(128)], 128)           # beyond 64 blocks ids repeat (p and p + 64)
    assert not gate([chunked(p, 40) for p in range(40)], 40)
    for n in (64, 128, 1024):
        assert gate([floor_form(p, n) for p in range(n)], n)              # X divides n: a transposition of the id space
    for n in (20, 100, 148):
        assert not gate([floor_form(p, n) for p in range(n)], n)          # it does not: ids collide
    for n in (64, 256):
        assert not gate([strided(p, n) for p in range(n)], n)             # both terms depend on p div X only: X ids share a target
    assert not gate([collapsed(p, 64, 4) for p in range(64)], 64)         # four ids per target
    assert gate([collapsed(p, 64, 1) for p in range(64)], 64)             # one row per chunk: the identity


def test_recommendation_is_valid_and_matches_what_the_sweeps_found():
    found = {  # (M, N, K) -> (tile, scheme, group): the fastest (or within noise of it) in sustained sweeps of every tile and order on B200
        (4096, 4096, 4096): ((256, 512), sp.ROW_MAJOR, 1),
        (8192, 8192, 8192): ((256, 512), sp.GROUP_N, 8),
        (16384, 2048, 8192): ((256, 256), sp.ROW_MAJOR, 1),
        (16384, 16384, 4096): ((256, 512), sp.GROUP_N, 8),
        (2048, 2048, 2048): ((256, 256), sp.ROW_MAJOR, 1),
    }
    for (M, N, K), (tile, scheme, group) in found.items():
        s, p = sp.recommend(M, N, K)
        assert (p.tile_m, p.tile_n) == tile and s == scheme and p.group == group, (M, N, K)
    s, p = sp.recommend(1024, 1024, 8192)                 # few tiles, long k: the k-split is suggested
    assert p.flags == sp.FLAG_STREAM_K and p.tile_n <= 256
    # band orders come with serpentine bands, alternating K and evict_first C stores; orders that need no bands with no flag
    bands = sp.FLAG_SERPENTINE | sp.FLAG_K_ALTERNATE | sp.FLAG_HINT_C_EVICT_FIRST
    assert sp.recommend(8192, 8192, 8192)[1].flags == bands and sp.recommend(16384, 16384, 4096)[1].flags == bands
    assert sp.recommend(512, 512, 512)[1].flags == 0 and sp.recommend(4096, 4096, 4096)[1].flags == 0
    # a narrow grid whose operands exceed L2: row-major, K alternating, evict_first C stores
    assert sp.recommend(16384, 2048, 8192)[1].flags == sp.FLAG_K_ALTERNATE | sp.FLAG_HINT_C_EVICT_FIRST
    rng = np.random.default_rng(0)
    for _ in range(200):                                  # always a supported tile and a bijective order
        M, N, K = (int(rng.integers(1, 40000)), int(rng.integers(1, 5000)) * 8, int(rng.integers(1, 3000)) * 8)
        s, p = sp.recommend(M, N, K, out_dtype=int(rng.integers(2)), b_layout=int(rng.integers(2)))
        assert (p.tile_m, p.tile_n) in [(128, 128), (128, 256), (256, 128), (256, 256), (256, 512)]
        perm = np.asarray(sp.tile_map(M, N, p.tile_m, p.tile_n, s, p))
        assert np.array_equal(np.sort(perm), np.arange(len(perm)))
    with pytest.raises(sp.SpError):
        sp.recommend(0, 8, 8)
    with pytest.raises(sp.SpError):
        sp.recommend(8, 8, 8, out_dtype=3)


def test_hilbert_rect_index_descent_matches_the_recursive_construction():
    """The library finds cell s by descending into the part of the rectangle that holds it; the oracle generates the
    whole curve recursively.  Every grid up to 40 x 40, the five workload grids, and some long thin ones."""
    grids = [(a, b) for a in range(1, 41) for b in range(1, 41)]
    grids += [(4, 4), (32, 16), (32, 32), (64, 8), (64, 64), (32, 64), (1, 300), (300, 1), (3, 1000), (1000, 3), (127, 255)]
    for Tm, Tn in grids:
        got = list(sp.tile_map(Tm, Tn, 1, 1, sp.HILBERT_RECT))
        assert got == R.hilbert_rect(Tm, Tn), (Tm, Tn)
    with pytest.raises(sp.SpError) as e:                  # not available inside DIE_SPLIT
        sp.tile_map(8, 8, 1, 1, sp.DIE_SPLIT, sp.make_params(inner_scheme=sp.HILBERT_RECT))
    assert e.value.status == sp.ERR_INVALID_ARG
