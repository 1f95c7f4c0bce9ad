"""The L2 reuse model: exact small cases by hand, limits, and the orderings it must predict."""

from oracle import l2model as L
from oracle import remap as R


def test_single_tile_only_compulsory_misses():
    r = L.simulate([0], 1, 1, 256, 128, 128, units=1, capacity=1 << 30)
    assert r["hit_bytes"] == 0 and r["read_bytes"] == 4 * (128 * 64 * 2 * 2)


def test_two_tiles_in_one_row_share_a_by_hand():
    # 1 x 2 grid, one k-block, both tiles concurrent: A chunk read twice (one hit), two distinct B chunks
    r = L.simulate([0, 1], 1, 2, 64, 128, 128, units=2, capacity=1 << 30)
    chunk = 128 * 64 * 2
    assert r["read_bytes"] == 4 * chunk and r["hit_bytes"] == chunk
    # sequential on one unit with a cache too small to keep anything: no hit
    r = L.simulate([0, 1], 1, 2, 64, 128, 128, units=1, capacity=chunk)
    assert r["hit_bytes"] == 0


def test_infinite_cache_gives_compulsory_traffic_and_capacity_is_monotone():
    Tm = Tn = 8
    perm = R.row_major(Tm, Tn)
    kw = dict(Tm=Tm, Tn=Tn, K=512, tile_m=128, tile_n=128, units=8)
    big = L.simulate(perm, capacity=1 << 40, **kw)
    assert big["dram_read_bytes"] == (Tm * 128 * 512 + 512 * Tn * 128) * 2      # A and B once each
    last = None
    for cap in (1 << 16, 1 << 19, 1 << 21, 1 << 23, 1 << 26):
        r = L.simulate(perm, capacity=cap, **kw)
        assert last is None or r["hit_rate"] >= last - 1e-12
        last = r["hit_rate"]


def test_model_orders_schemes_like_the_measurements():
    """8192^3 with 256x256 tiles, 74 units, 126 MiB: grouped supertiles beat row-major; and for the
    tall-skinny problem (B small) row-major is already the best order."""
    cap = 126 << 20
    kw = dict(Tm=32, Tn=32, K=8192, tile_m=256, tile_n=256, units=74, capacity=cap)
    row = L.simulate(R.row_major(32, 32), **kw)["hit_rate"]
    g8 = L.simulate(R.group_m(32, 32, 8), **kw)["hit_rate"]
    hil = L.simulate(R.hilbert(32, 32), **kw)["hit_rate"]
    assert g8 > row + 0.05 and hil > row + 0.05
    kw4 = dict(Tm=64, Tn=8, K=8192, tile_m=256, tile_n=256, units=74, capacity=cap)
    row4 = L.simulate(R.row_major(64, 8), **kw4)["hit_rate"]
    g64 = L.simulate(R.group_m(64, 8, 64), **kw4)["hit_rate"]
    assert row4 > g64 + 0.1


def test_split_cache_rewards_pinning_halves():
    """Two caches of half the size: when every unit of a half only ever touches one half of A, the
    halves stop duplicating each other's A panels."""
    cap = 126 << 20
    Tm = Tn = 64
    perm = R.die_split(Tm, Tn, 0, R.GROUP_M, 8)
    h0 = len(R.die_split_halves(Tm, Tn, 0, R.GROUP_M, 8)[0])
    kw = dict(Tm=Tm, Tn=Tn, K=4096, tile_m=256, tile_n=256, units=74, capacity=cap, halves=2)
    unpinned = L.simulate(R.group_m(Tm, Tn, 8), **kw)
    pinned = L.simulate(perm, half_of_unit=lambda u: u % 2,
                        slots_of_unit=lambda u: range((u % 2) * h0 + u // 2, h0 if u % 2 == 0 else Tm * Tn, 37), **kw)
    assert pinned["read_bytes"] == unpinned["read_bytes"]
    assert pinned["dram_read_bytes"] < unpinned["dram_read_bytes"]
