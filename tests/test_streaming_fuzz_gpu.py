"""Seeded random shapes and orders for the three memory-bound kernels (tile transpose, 2-D stencil, row softmax)
through the C ABI against their oracles.  The hand-picked cases elsewhere fix the interesting sizes; these draw sizes and
order parameters, so that the tile grids (64 x 64, 64 x 128 and 32 x 512 tiles) get ragged edges, single rows and
columns of tiles, and bands wider than the grid in combinations nobody listed.
"""

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import softmax as SM
from oracle import stencil as S
from oracle import transpose as T

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def draw_order(rng, Tm, Tn):
    kind = int(rng.integers(8))
    if kind == 0:
        return sp.ROW_MAJOR, {}
    if kind == 1:
        return sp.COL_MAJOR, {}
    if kind in (2, 3):
        return (sp.GROUP_M if kind == 2 else sp.GROUP_N), dict(group=int(rng.integers(1, 12)), flags=sp.FLAG_SERPENTINE * int(rng.integers(2)))
    if kind == 4:
        return [sp.MORTON, sp.HILBERT, sp.HILBERT_RECT][rng.integers(3)], {}
    if kind == 5:
        return sp.XCD, dict(num_xcds=int(rng.integers(1, 10)), wave=int(rng.integers(0, 2)) * 148, xcd_balanced=1)
    if kind == 6:
        inner = [sp.ROW_MAJOR, sp.GROUP_M, sp.GROUP_N, sp.HILBERT][rng.integers(4)]
        return sp.DIE_SPLIT, dict(split_axis=int(rng.integers(2)), inner_scheme=inner, inner_group=int(rng.integers(1, 6)),
                                  interleave=int(rng.integers(2)))
    return sp.CUSTOM, dict(custom_perm=rng.permutation(Tm * Tn).astype(np.int32))


def describe(kw):
    return {k: v for k, v in kw.items() if k != "custom_perm"}


@pytest.mark.parametrize("seed", range(4))
def test_transpose_random_shapes_and_orders(seed):
    rng = np.random.default_rng(7100 + seed)
    for _ in range(12):
        M, N = 8 * int(rng.integers(1, 200)), 8 * int(rng.integers(1, 200))        # 16-byte rows on both sides
        x = rng.integers(0, 65536, size=(M, N)).astype(np.uint16)
        scheme, kw = draw_order(rng, -(-M // 64), -(-N // 64))
        dx = torch.from_numpy(x.view(np.int16)).cuda()
        out = torch.full((N, M), -1, dtype=torch.int16, device="cuda")
        sp.transpose(dx, out, scheme, sp.make_params(**kw))
        assert sp.get_status() == 0
        assert np.array_equal(out.cpu().numpy().view(np.uint16), T.transpose(x)), (M, N, scheme, describe(kw))


@pytest.mark.parametrize("seed", range(4))
def test_stencil_random_shapes_and_orders(seed):
    rng = np.random.default_rng(7200 + seed)
    for _ in range(12):
        M, N = int(rng.integers(1, 700)), 4 * int(rng.integers(1, 300))            # 16-byte rows
        x = rng.integers(-8, 9, size=(M, N)).astype(np.float32)
        c0, c1 = [(0.5, 0.125), (-0.25, 0.5), (1.0, -0.125)][rng.integers(3)]   # dyadic weights: exact in fp32 in any order
        scheme, kw = draw_order(rng, -(-M // 64), -(-N // 128))
        dx = torch.from_numpy(x).cuda()
        out = torch.full_like(dx, float("nan"))
        sp.stencil2d(dx, out, c0, c1, scheme, sp.make_params(**kw))
        assert sp.get_status() == 0
        assert np.array_equal(out.cpu().numpy().astype(np.float64), S.stencil2d(x, c0, c1)), (M, N, scheme, describe(kw))


@pytest.mark.parametrize("seed", range(4))
def test_softmax_random_shapes_modes_and_orders(seed):
    rng = np.random.default_rng(7300 + seed)
    for _ in range(12):
        M = int(rng.integers(1, 400))
        N = 4 * int(rng.integers(1, 1400)) if rng.random() < 0.8 else 4 * int(rng.integers(4000, 10000))   # 16-byte rows
        x = (rng.standard_normal((M, N)) * float(rng.uniform(0.5, 6.0))).astype(np.float32)
        x[int(rng.integers(M)), int(rng.integers(N))] += 50.0
        mode = [sp.SOFTMAX_SINGLE_PASS, sp.SOFTMAX_TWO_PHASE, sp.SOFTMAX_TWO_PHASE_REVERSED][rng.integers(3)]
        if mode == sp.SOFTMAX_SINGLE_PASS:                          # blocks of whole rows: a grid of one column
            rows = min(96, max(8, 12288 // N // 8 * 8)) if N <= 1792 else max(1, 12288 // N)   # the header's rule
            grid = (-(-M // rows), 1)
        else:
            grid = (-(-M // sp.SOFTMAX_TILE[0]), -(-N // sp.SOFTMAX_TILE[1]))
        scheme, kw = draw_order(rng, *grid)
        dx = torch.from_numpy(x).cuda()
        out = torch.full_like(dx, float("nan"))
        sp.softmax(dx, out, mode, scheme, sp.make_params(**kw))
        assert sp.get_status() == 0
        got, ref = out.cpu().numpy(), SM.softmax(x)
        what = (M, N, mode, scheme, describe(kw))
        assert not np.isnan(got).any(), what
        assert (np.abs(got.astype(np.float64) - ref) <= 2e-5 * ref + 2e-38).all(), what
        assert np.abs(got.astype(np.float64).sum(axis=1) - 1.0).max() <= 1e-5, what
