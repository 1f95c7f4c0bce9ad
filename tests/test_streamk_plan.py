"""The k-split of the tail wave (SP_FLAG_STREAM_K): host plan of the library against the enumerative
oracle, and both against the properties the kernel relies on.  No GPU needed."""

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import streamk as O

CASES = [
    # (T, units, kblocks)
    (256, 74, 64),      # 4096^3 with 256x256 pair tiles: 3 full waves + 34 tiles, each cut in two
    (1024, 74, 128),    # 8192^3: 13 full waves + 62: more than half a wave, nothing is split
    (512, 148, 64),     # 4096^3 with 128x256 tiles: 68 left, cut in two
    (16, 148, 8),       # smaller than a wave: pieces of 4 k-blocks (two per tile) although nine units per tile are free
    (16, 148, 64),      # ... eight pieces per tile (nine units per tile are free, eight is the cap)
    (16, 148, 2),       # ... too few k-blocks to split
    (3, 74, 64), (75, 74, 5), (75, 74, 64), (147, 74, 3), (149, 148, 16), (100, 7, 13), (101, 7, 13), (5, 4, 256),
    (9, 4, 1),
    (148, 74, 64), (74, 74, 10),   # units divide T: nothing to split
]


@pytest.mark.parametrize("T,units,kb", CASES)
def test_plan_matches_enumeration(T, units, kb):
    first, segs = sp.streamk_plan(T, units, kb)
    ofirst, osegs = O.plan(T, units, kb)
    assert first == ofirst
    assert segs == osegs


@pytest.mark.parametrize("T,units,kb", CASES)
def test_plan_properties(T, units, kb):
    first, segs = sp.streamk_plan(T, units, kb)
    R = T % units
    f = min(units // R, kb // 4, 8) if R else 0
    if f < 2:
        assert first == T and all(s == [] for s in segs)
        return
    assert first == T - R and first % units == 0     # the whole tiles before the tail form full waves
    assert sum(1 for ss in segs if ss) == R * f      # f units per remainder tile
    assert all(len(ss) <= 1 for ss in segs)          # one piece each: nobody waits while still holding other work
    cover = np.zeros((T - first, kb), dtype=np.int32)
    finisher = {}
    for u, ss in enumerate(segs):
        kinds = [k for (_, _, _, k) in ss]
        assert kinds.count(sp.WORK_CONTRIB) <= 1 and kinds.count(sp.WORK_OWNER) <= 1
        if sp.WORK_CONTRIB in kinds:
            assert kinds[0] == sp.WORK_CONTRIB       # walked first: it never waits
        if sp.WORK_OWNER in kinds:
            assert kinds[-1] == sp.WORK_OWNER        # walked last: the partials it needs are long done
        slots = [s for (s, _, _, _) in ss]
        assert slots == sorted(slots, reverse=True)
        for (s, k0, k1, kind) in ss:
            assert first <= s < T and 0 <= k0 < k1 <= kb
            cover[s - first, k0:k1] += 1
            if kind == sp.WORK_FULL:
                assert (k0, k1) == (0, kb)
            if kind == sp.WORK_CONTRIB:
                assert k1 < kb
            if kind == sp.WORK_OWNER:
                assert k0 > 0 and k1 == kb
            if kind != sp.WORK_CONTRIB:
                assert s not in finisher
                finisher[s] = u
    assert (cover == 1).all()                         # every k-block of every tail tile exactly once
    assert sorted(finisher) == list(range(first, T))  # every tail tile is stored by exactly one unit
    # contributors of a tile are the units directly below its finisher, contiguous, in k order
    for u, ss in enumerate(segs):
        for (s, k0, k1, kind) in ss:
            if kind == sp.WORK_CONTRIB:
                assert u < finisher[s]
    work = [sum(k1 - k0 for (_, k0, k1, _) in ss) for ss in segs]
    busy = [w for w in work if w]
    assert max(busy) - min(busy) <= 1                 # equal shares to within one k-block
    assert min(busy) >= 4                             # no piece shorter than 4 k-blocks
    # pieces with the same index start at the same k-block in every tile: they walk k in step
    starts = sorted({k0 for ss in segs for (_, k0, _, _) in ss})
    assert len(starts) == f


def test_plan_worked_example():
    # 9 tiles of 10 k-blocks on 8 units: one full wave, then the last tile cut into min(8 // 1, 10 // 4) = 2 pieces
    first, segs = sp.streamk_plan(9, 8, 10)
    assert first == 8
    assert segs[0] == [(8, 0, 5, 1)]
    assert segs[1] == [(8, 5, 10, 2)]
    assert all(s == [] for s in segs[2:])
    # 14 tiles of 12 k-blocks on 12 units: remainder 2, f = min(6, 3) = 3 pieces of 4 k-blocks, units 0..5
    first, segs = sp.streamk_plan(14, 12, 12)
    assert first == 12
    assert segs[:6] == [[(12, 0, 4, 1)], [(12, 4, 8, 1)], [(12, 8, 12, 2)], [(13, 0, 4, 1)], [(13, 4, 8, 1)], [(13, 8, 12, 2)]]


def test_plan_rejects_bad_arguments():
    for bad in [(0, 4, 4), (5, 0, 4), (5, 4, 0)]:
        with pytest.raises(sp.SpError) as e:
            sp.streamk_plan(*bad)
        assert e.value.status == sp.ERR_INVALID_ARG
