"""Seeded random combinations of shape, tile, order, parameters and flags through the C ABI against the CPU oracle.

Inputs are small integers, so every fp32 partial sum is exact in any accumulation order and the fp32 output must
equal the oracle's bit for bit whatever the tile order, the direction K is walked in, or the way the last wave is
split.  The fixed cases elsewhere pick their combinations by hand; these are drawn, so that pairings nobody thought of
get run too (ragged edges with every tile, bands wider than the grid, pinned halves of odd grids, hints with every
scheduler).
"""

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import gemm as G
from oracle import remap as R
from paper_2508_20258_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

TILES = [(128, 128), (128, 256), (256, 128), (256, 256), (256, 512)]
HINTS = [0, sp.FLAG_HINT_C_EVICT_FIRST, sp.FLAG_HINT_A_EVICT_FIRST, sp.FLAG_HINT_B_EVICT_FIRST,
         sp.FLAG_HINT_A_EVICT_LAST | sp.FLAG_HINT_B_EVICT_FIRST, sp.FLAG_HINT_B_EVICT_LAST | sp.FLAG_HINT_C_EVICT_FIRST]


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def draw_case(rng):
    tm, tn = TILES[rng.integers(len(TILES))]
    # up to a few waves of tiles; ragged in M (any size) and N (multiple of 8: 16-byte rows); K a multiple of 8
    Tm, Tn = int(rng.integers(1, 13)), int(rng.integers(1, 13))
    M = (Tm - 1) * tm + int(rng.integers(1, tm + 1))
    N = (Tn - 1) * tn + 8 * int(rng.integers(1, tn // 8 + 1))
    K = 8 * int(rng.integers(1, 97)) if rng.random() < 0.8 else 64 * int(rng.integers(16, 80))
    b_nk = int(rng.integers(2))
    kind = int(rng.integers(9))
    kw = {}
    if kind == 0:
        scheme = sp.ROW_MAJOR
    elif kind == 1:
        scheme = sp.COL_MAJOR
    elif kind in (2, 3):
        scheme = sp.GROUP_M if kind == 2 else sp.GROUP_N
        kw = dict(group=int(rng.integers(1, 20)), flags=sp.FLAG_SERPENTINE * int(rng.integers(2)))
    elif kind == 4:
        scheme = [sp.MORTON, sp.HILBERT, sp.HILBERT_RECT][rng.integers(3)]
    elif kind == 5:
        scheme = sp.XCD
        kw = dict(num_xcds=int(rng.integers(1, 10)), wave=int(rng.integers(0, 3)) * 37, xcd_balanced=1)
    elif kind in (6, 7):
        scheme = sp.DIE_SPLIT
        inner = [sp.ROW_MAJOR, sp.COL_MAJOR, sp.GROUP_M, sp.GROUP_N, sp.MORTON, sp.HILBERT][rng.integers(6)]
        pinned = kind == 7
        kw = dict(split_axis=int(rng.integers(2)), inner_scheme=inner, inner_group=int(rng.integers(1, 10)),
                  interleave=0 if pinned else int(rng.integers(2)),
                  flags=sp.FLAG_SERPENTINE * int(rng.integers(2)) | (sp.FLAG_DIE_PINNED if pinned else 0))
        if pinned and rng.random() < 0.4:
            kw["flags"] |= sp.FLAG_STEAL
    else:
        scheme = sp.CUSTOM
        kw = dict(custom_perm=rng.permutation(Tm * Tn).astype(np.int32))
    flags = kw.get("flags", 0)
    if rng.random() < 0.5:
        flags |= sp.FLAG_K_ALTERNATE
    flags |= HINTS[rng.integers(len(HINTS))]
    if not (flags & sp.FLAG_DIE_PINNED):
        mode = rng.random()
        if mode < 0.2 and tn <= 256:
            flags |= sp.FLAG_STREAM_K
        elif mode < 0.4:
            flags |= sp.FLAG_CLC
        elif mode < 0.5:
            flags |= sp.FLAG_OVERLAP
    kw["flags"] = flags
    return M, N, K, (tm, tn), b_nk, scheme, kw


@pytest.mark.parametrize("seed", range(12))
def test_random_combinations_are_bit_exact(seed):
    rng = np.random.default_rng(4200 + seed)
    ran = 0
    for _ in range(10):
        M, N, K, (tm, tn), b_nk, scheme, kw = draw_case(rng)
        A, B = synth.make_int_inputs(M, N, K, seed=int(rng.integers(1 << 30)))
        ref, _ = G.gemm_full(A, B)
        dA, dB = dev_bf16(A), dev_bf16(np.ascontiguousarray(B.T) if b_nk else B)
        dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        p = sp.make_params(tile_m=tm, tile_n=tn, out_dtype=1, b_layout=b_nk, **kw)
        what = (M, N, K, tm, tn, b_nk, scheme, {k: v for k, v in kw.items() if k != "custom_perm"})
        try:
            sp.gemm(dA, dB, dC, scheme, p)
        except sp.SpError as err:
            # the only refusal a drawn case may meet: pinning on a device whose probe found no two L2 halves
            assert err.status == sp.ERR_UNSUPPORTED and (kw["flags"] & sp.FLAG_DIE_PINNED), (what, str(err))
            continue
        assert sp.get_status() == 0, what
        got = dC.cpu().numpy().astype(np.float64)
        assert np.array_equal(got, ref), (what, int((got != ref).sum()))
        ran += 1
    assert ran >= 5


@pytest.mark.parametrize("seed", range(3))
def test_random_orders_on_the_device_equal_the_oracle(seed):
    """The device decode of every drawn (grid, order, parameters) is the oracle's permutation, entry by entry."""
    rng = np.random.default_rng(900 + seed)
    for _ in range(25):
        M, N, K, (tm, tn), b_nk, scheme, kw = draw_case(rng)
        kw = {k: v for k, v in kw.items()}
        kw["flags"] = kw.get("flags", 0) & sp.FLAG_SERPENTINE          # the order itself: the other flags do not enter it
        if scheme == sp.CUSTOM:
            want = [int(v) for v in kw["custom_perm"]]
            okw = None
        else:
            okw = {k: v for k, v in kw.items()}
            want = R.tile_map(M, N, tm, tn, scheme, R.Params(**okw))
        got = sp.tile_map_device(M, N, tm, tn, scheme, sp.make_params(**kw)).cpu().numpy().tolist()
        assert got == want, (M, N, tm, tn, scheme, okw)
        assert sorted(got) == list(range(len(got)))
