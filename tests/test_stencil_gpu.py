"""sp_stencil2d through the C ABI against the oracle: exact on dyadic inputs, within a derived fp32 bound on random
ones, identical bits under every tile order, ragged and degenerate grids, rejections."""

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import stencil as S

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

ORDERS = [(sp.ROW_MAJOR, {}), (sp.COL_MAJOR, {}), (sp.GROUP_M, dict(group=3)), (sp.GROUP_N, dict(group=2)), (sp.MORTON, {}),
          (sp.HILBERT, {}), (sp.HILBERT_RECT, {}), (sp.XCD, dict(num_xcds=8, xcd_balanced=1)),
          (sp.DIE_SPLIT, dict(split_axis=0, inner_scheme=sp.GROUP_M, inner_group=2, interleave=1))]


def run(x, c0, c1, scheme=sp.ROW_MAJOR, **kw):
    dx = torch.from_numpy(x).cuda()
    out = torch.full_like(dx, float("nan"))
    sp.stencil2d(dx, out, c0, c1, scheme, sp.make_params(**kw))
    assert sp.get_status() == 0
    return out.cpu().numpy()


# sizes span several 64 x 128 tiles, ragged edges in both directions, a single tile, fewer than three rows / columns
@pytest.mark.parametrize("M,N", [(64, 128), (200, 388), (513, 1028), (1, 4), (2, 260), (300, 4), (67, 132), (1000, 8)])
def test_small_integers_with_dyadic_weights_are_exact(M, N):
    rng = np.random.default_rng(M * 131 + N)
    x = rng.integers(-8, 9, size=(M, N)).astype(np.float32)
    ref = S.stencil2d(x, 0.5, 0.125)                 # multiples of 1/8 below 2^7: exact in fp32 in any order
    for scheme, kw in ORDERS[:4]:
        got = run(x, 0.5, 0.125, scheme, **kw)
        assert np.array_equal(got.astype(np.float64), ref), (scheme, kw)


def test_random_grid_within_the_fp32_bound_and_same_bits_under_every_order():
    M, N = 1100, 1540
    rng = np.random.default_rng(3)
    x = rng.standard_normal((M, N)).astype(np.float32)
    c0, c1 = np.float32(-0.6), np.float32(0.2)
    ref = S.stencil2d(x, float(c0), float(c1))
    mag = S.magnitude(x, float(c0), float(c1))
    first = None
    for scheme, kw in ORDERS:
        got = run(x, float(c0), float(c1), scheme, **kw)
        if first is None:
            first = got
            # three additions, one product, one fused multiply-add: at most 5 roundings of 2^-24 each, relative to the
            # sum of the magnitudes of the terms
            assert (np.abs(got.astype(np.float64) - ref) <= 5.01 * 2.0 ** -24 * mag + 1e-30).all()
            assert not np.isnan(got).any()
        else:
            assert np.array_equal(got.view(np.uint32), first.view(np.uint32)), (scheme, kw)


def test_rim_is_carried_over_and_impulses_land_on_the_star_across_tile_borders():
    M, N = 192, 384                                   # 3 x 3 tiles
    x = np.zeros((M, N), dtype=np.float32)
    pts = [(63, 127), (64, 128), (64, 127), (63, 128), (1, 1), (M - 2, N - 2), (100, 255), (100, 256), (127, 5), (128, 5)]
    for k, (i, j) in enumerate(pts):
        x[i, j] = float(2 ** (k % 5))
    x[0, :] = 3.0
    x[:, 0] = 5.0
    x[M - 1, :] = 7.0
    x[:, N - 1] = 9.0
    got = run(x, 0.25, 0.5, sp.HILBERT)
    assert np.array_equal(got.astype(np.float64), S.stencil2d(x, 0.25, 0.5))
    assert np.array_equal(got[0], x[0]) and np.array_equal(got[:, N - 1], x[:, N - 1])


def test_full_size_grid_sampled_rows_and_columns():
    M = N = 8192                                      # the size bench.py --stencil times by default is 16384^2; same launch shape
    g = torch.Generator(device="cuda").manual_seed(11)
    dx = torch.randn((M, N), device="cuda", generator=g, dtype=torch.float32)
    out = torch.full_like(dx, float("nan"))
    sp.stencil2d(dx, out, 0.5, 0.125, sp.GROUP_M, sp.make_params(group=4))
    assert sp.get_status() == 0
    x = dx.cpu().numpy()
    got = out.cpu().numpy()
    assert not np.isnan(got).any()
    rows = sorted({0, 1, 63, 64, 65, 4095, 4096, M - 2, M - 1} | set(np.random.default_rng(5).integers(0, M, 40).tolist()))
    for i in rows:                                    # whole rows: they cross every tile column
        lo, hi = max(i - 1, 0), min(i + 2, M)
        ref = S.stencil2d(x[lo:hi], 0.5, 0.125)[i - lo] if 0 < i < M - 1 else x[i].astype(np.float64)
        mag = S.magnitude(x[lo:hi], 0.5, 0.125)[i - lo]
        assert (np.abs(got[i].astype(np.float64) - ref) <= 5.01 * 2.0 ** -24 * mag + 1e-30).all(), i
    cols = [0, 1, 127, 128, 129, 4095, 4096, N - 2, N - 1]
    for j in cols:                                    # whole columns: they cross every tile row
        lo, hi = max(j - 1, 0), min(j + 2, N)
        ref = S.stencil2d(x[:, lo:hi], 0.5, 0.125)[:, j - lo] if 0 < j < N - 1 else x[:, j].astype(np.float64)
        mag = S.magnitude(x[:, lo:hi], 0.5, 0.125)[:, j - lo]
        assert (np.abs(got[:, j].astype(np.float64) - ref) <= 5.01 * 2.0 ** -24 * mag + 1e-30).all(), j


def test_stencil_rejections():
    x = torch.zeros((64, 128), dtype=torch.float32, device="cuda")
    out = torch.zeros_like(x)
    L = sp.lib()
    assert L.sp_stencil2d(x.data_ptr(), out.data_ptr(), 64, 126, 1.0, 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_ALIGNMENT
    assert L.sp_stencil2d(x.data_ptr() + 4, out.data_ptr(), 64, 128, 1.0, 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_ALIGNMENT
    assert L.sp_stencil2d(x.data_ptr(), x.data_ptr(), 64, 128, 1.0, 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    assert L.sp_stencil2d(None, out.data_ptr(), 64, 128, 1.0, 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    assert L.sp_stencil2d(x.data_ptr(), out.data_ptr(), 0, 128, 1.0, 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    assert L.sp_stencil2d(x.data_ptr(), out.data_ptr(), 64, 128, float("nan"), 0.0, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    bad = sp.make_params(num_xcds=4, xcd_balanced=0)
    xw = torch.zeros((64 * 10, 128), dtype=torch.float32, device="cuda")   # 10 tiles: the printed formula with X = 4 hits 10
    import ctypes
    assert L.sp_stencil2d(xw.data_ptr(), torch.zeros_like(xw).data_ptr(), 640, 128, 1.0, 0.0, sp.XCD, ctypes.byref(bad),
                          None) == sp.ERR_NOT_BIJECTIVE
    assert sp.get_status() == 0


def test_grid_larger_than_4_gib_is_addressed_correctly():
    M, N = 36864, 32768                                # 4.8 GB per fp32 grid: byte offsets beyond 2^32
    g = torch.Generator(device="cuda").manual_seed(5)
    dx = torch.randint(-8, 9, (M, N), device="cuda", generator=g, dtype=torch.int32).float()
    out = torch.full_like(dx, float("nan"))
    sp.stencil2d(dx, out, 0.5, 0.125, sp.HILBERT)
    assert sp.get_status() == 0
    for i in [0, 1, 63, 64, 16383, 16384, 32767, 32768, 32769, M - 65, M - 2, M - 1]:
        lo, hi = max(i - 1, 0), min(i + 2, M)
        x = dx[lo:hi].cpu().numpy()
        ref = S.stencil2d(x, 0.5, 0.125)[i - lo] if 0 < i < M - 1 else x[i - lo].astype(np.float64)
        assert np.array_equal(out[i].cpu().numpy().astype(np.float64), ref), i      # dyadic weights, small integers: exact
    assert not bool(torch.isnan(out[:, N - 1]).any()) and not bool(torch.isnan(out[::1013]).any())
