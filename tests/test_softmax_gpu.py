"""sp_softmax through the C ABI against the oracle (the definition in float64), in all three modes, under several tile
orders, on ragged and degenerate shapes.

Tolerance, from the arithmetic (fp32; t = x - max <= 0): the difference is rounded once and its product with log2(e) once
(together |t| * 2^-23 absolute in the exponent, i.e. relative in the exponential), the hardware's 2^x is good to 2 ulp
(2^-22), the sums are taken by lanes and then by a shuffle tree (a few times 2^-24 on top of the terms' own error, all
terms being non-negative), then one reciprocal and one product.  For |t| <= 87 (beyond, exp underflows fp32) that is at
most about 1.5e-5 relative; the gate is 2e-5 * ref + 2e-38 (the hardware flushes denormal results to zero)."""

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import softmax as SM

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

MODES = [sp.SOFTMAX_SINGLE_PASS, sp.SOFTMAX_TWO_PHASE, sp.SOFTMAX_TWO_PHASE_REVERSED]
ORDERS = [(sp.ROW_MAJOR, {}), (sp.COL_MAJOR, {}), (sp.GROUP_M, dict(group=3)), (sp.GROUP_N, dict(group=2)),
          (sp.HILBERT, {}), (sp.HILBERT_RECT, {}), (sp.XCD, dict(num_xcds=8, xcd_balanced=1)),
          (sp.DIE_SPLIT, dict(split_axis=0, inner_scheme=sp.GROUP_M, inner_group=2, interleave=1))]


def run(x, mode, scheme=sp.ROW_MAJOR, **kw):
    dx = torch.from_numpy(x).cuda()
    out = torch.full_like(dx, float("nan"))
    sp.softmax(dx, out, mode, scheme, sp.make_params(**kw))
    assert sp.get_status() == 0
    return out.cpu().numpy()


def close(got, ref):
    return bool((np.abs(got.astype(np.float64) - ref) <= 2e-5 * ref + 2e-38).all()) and not np.isnan(got).any()


# sizes span several 32 x 512 tiles with ragged edges both ways, one tile, one row, one 16-byte unit per row, rows of
# 16384 (one row per single-pass block) and 2048 (six)
@pytest.mark.parametrize("M,N", [(32, 512), (100, 1300), (257, 4100), (1, 4), (3, 16384), (70, 2048), (9, 8), (33, 520),
                                 (1003, 64), (77, 128), (50, 32), (333, 96), (201, 20)])   # the last five: 8 or 16 lanes per row, ragged last block
@pytest.mark.parametrize("mode", MODES)
def test_matches_the_definition(M, N, mode):
    rng = np.random.default_rng(M * 7 + N)
    x = (rng.standard_normal((M, N)) * 3.0).astype(np.float32)
    x[M // 2, N // 3] += 40.0                                   # one row with a dominant entry far from the rest
    ref = SM.softmax(x)
    got = run(x, mode)
    assert close(got, ref)
    assert np.abs(got.astype(np.float64).sum(axis=1) - 1.0).max() <= 1e-5


@pytest.mark.parametrize("mode", MODES)
def test_every_order_gives_the_same_bits(mode):
    M, N = 200, 2600
    rng = np.random.default_rng(5)
    x = rng.standard_normal((M, N)).astype(np.float32) * 2
    ref = SM.softmax(x)
    first = None
    for scheme, kw in ORDERS:
        got = run(x, mode, scheme, **kw)
        if first is None:
            first = got
            assert close(got, ref)
        else:
            assert np.array_equal(got.view(np.uint32), first.view(np.uint32)), (scheme, kw)   # an order moves work, not sums


def test_closed_forms_uniform_rows_and_logarithms():
    for mode in MODES:
        x = np.full((40, 1024), -3.25, dtype=np.float32)
        assert np.array_equal(run(x, mode), np.full((40, 1024), 1.0 / 1024, dtype=np.float32))   # exp(0) = 1 exactly, 1024 = 2^10
        # entries ln(1..4) repeated: out = k / sum; the logarithms are rounded to fp32 first, the oracle sees the same values
        row = np.log(np.tile(np.arange(1, 5, dtype=np.float64), 130)).astype(np.float32)
        x = np.tile(row, (5, 1))
        assert close(run(x, mode), SM.softmax(x))
        # a shift per row changes nothing beyond rounding: compare with the oracle of the shifted input
        xs = (x + np.arange(5, dtype=np.float32)[:, None] * 11.0).astype(np.float32)
        assert close(run(xs, mode), SM.softmax(xs))


def test_large_spread_and_tiny_outputs():
    rng = np.random.default_rng(9)
    x = (rng.standard_normal((64, 3000)) * 25.0).astype(np.float32)      # differences beyond 87: exp underflows to zero
    ref = SM.softmax(x)
    for mode in MODES:
        got = run(x, mode)
        assert close(got, ref) and (got >= 0).all()


def test_rejections_launch_nothing():
    x = torch.zeros((8, 16), dtype=torch.float32, device="cuda")
    out = torch.full_like(x, 7.0)
    L = sp.lib()
    import ctypes
    p = sp.make_params()
    assert L.sp_softmax(x.data_ptr(), x.data_ptr(), 8, 16, 0, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_INVALID_ARG
    assert L.sp_softmax(x.data_ptr(), out.data_ptr(), 8, 16, 3, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_INVALID_ARG
    assert L.sp_softmax(x.data_ptr(), out.data_ptr(), 8, 18, 0, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_ALIGNMENT
    assert L.sp_softmax(x.data_ptr() + 4, out.data_ptr(), 8, 12, 0, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_ALIGNMENT
    assert L.sp_softmax(x.data_ptr(), out.data_ptr(), 1, 131076, 0, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_UNSUPPORTED
    assert L.sp_softmax(None, out.data_ptr(), 8, 16, 0, sp.ROW_MAJOR, ctypes.byref(p), None) == sp.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())


def test_rows_longer_than_a_buffer_take_the_two_phase_form():
    M, N = 5, 40000
    rng = np.random.default_rng(2)
    x = rng.standard_normal((M, N)).astype(np.float32) * 4
    ref = SM.softmax(x)
    for mode in MODES[1:]:
        assert close(run(x, mode, sp.GROUP_N, group=7), ref)


# rows spread over a cluster of 2, 4 or 8 CTAs: the shortest and longest row of each cluster size, shares with a ragged last
# CTA, more rows than resident clusters, fewer rows than that, one row
@pytest.mark.parametrize("M,N", [(5, 16388), (300, 32768), (7, 32772), (3, 50000), (200, 65536), (2, 65540), (9, 100000),
                                 (150, 131072), (1, 131072), (40, 16400), (11, 98308)])
def test_single_pass_with_a_cluster_per_row(M, N):
    rng = np.random.default_rng(M * 13 + N)
    x = (rng.standard_normal((M, N)) * 3.0).astype(np.float32)
    x[M // 2, (2 * N) // 3] += 35.0                     # a dominant entry in one CTA's share: every share needs its maximum
    ref = SM.softmax(x)
    for scheme, kw in [(sp.ROW_MAJOR, {}), (sp.GROUP_M, dict(group=3)), (sp.HILBERT, {})]:
        got = run(x, sp.SOFTMAX_SINGLE_PASS, scheme, **kw)
        assert close(got, ref), (M, N, scheme)
        assert np.abs(got.astype(np.float64).sum(axis=1) - 1.0).max() <= 1e-5


def test_single_pass_refuses_rows_beyond_eight_buffers():
    x = torch.zeros((2, 131076), dtype=torch.float32, device="cuda")
    out = torch.empty_like(x)
    with pytest.raises(sp.SpError) as e:
        sp.softmax(x, out, sp.SOFTMAX_SINGLE_PASS, sp.ROW_MAJOR, sp.make_params())
    assert e.value.status == sp.ERR_UNSUPPORTED


def test_single_pass_at_every_row_length_of_the_long_row_kernels():
    """Rows of 1796 to 16384 elements in steps of 4: every pairing of rows per block, warps per row and units per lane the
    long-row dispatch can choose, each with a last block that is short of rows."""
    rng = np.random.default_rng(77)
    base = (rng.standard_normal((17, 16384)) * 3.0).astype(np.float32)
    worst = 0.0
    for N in range(1796, 16385, 4):
        rows = max(1, 12288 // N)
        M = 2 * rows + 1 if N % 64 == 0 else rows + 1
        x = np.ascontiguousarray(base[:M, 16384 - N:])
        x[M - 1, N - 1] += 30.0
        got = run(x, sp.SOFTMAX_SINGLE_PASS)
        ref = SM.softmax(x)
        assert close(got, ref), N
        worst = max(worst, float(np.abs(got.astype(np.float64).sum(axis=1) - 1.0).max()))
    assert worst <= 1e-5
