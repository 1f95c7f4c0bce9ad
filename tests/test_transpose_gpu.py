"""Parity of sp_transpose (through the C ABI) against the oracle: bit-exact, every element."""

import ctypes

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import remap as R
from oracle import transpose as T

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def run(x, scheme=sp.ROW_MAJOR, **kw):
    dx = torch.from_numpy(x.view(np.int16)).cuda()
    out = torch.full((x.shape[1], x.shape[0]), -1, dtype=torch.int16, device="cuda")
    sp.transpose(dx, out, scheme, sp.make_params(**kw) if kw else None)
    assert sp.get_status() == 0
    return out.cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("M,N", [(8, 8), (64, 64), (64, 128), (200, 72), (1000, 520), (4096, 4096), (8200, 1032)])
def test_transpose_is_bit_exact_under_every_order(M, N):
    rng = np.random.default_rng(M * 31 + N)
    x = rng.integers(0, 65536, size=(M, N)).astype(np.uint16)
    want = T.transpose(x)
    Tm, Tn = -(-M // 64), -(-N // 64)
    table = np.random.default_rng(5).permutation(Tm * Tn).astype(np.int32)
    for scheme, kw in [(sp.ROW_MAJOR, {}), (sp.COL_MAJOR, {}), (sp.GROUP_M, dict(group=8)), (sp.HILBERT, {}), (sp.HILBERT_RECT, {}),
                       (sp.XCD, dict(num_xcds=8, xcd_balanced=1)), (sp.CUSTOM, dict(custom_perm=table)),
                       (sp.DIE_SPLIT, dict(split_axis=1, inner_scheme=sp.GROUP_N, inner_group=4, interleave=1))]:
        assert np.array_equal(run(x, scheme, **kw), want), (scheme, kw)


def test_position_revealing_pattern_and_involution():
    M, N = 384, 640
    x = (np.arange(M, dtype=np.uint32)[:, None] * 131 + np.arange(N, dtype=np.uint32)[None, :] * 7).astype(np.uint16)
    y = run(x, sp.MORTON)
    assert np.array_equal(y, T.transpose(x))
    assert np.array_equal(run(y, sp.GROUP_N, group=3), x)


def test_transpose_rejections():
    L = sp.lib()
    a = torch.zeros(64 * 64, dtype=torch.int16, device="cuda")
    b = torch.zeros(64 * 64, dtype=torch.int16, device="cuda")
    assert L.sp_transpose(a.data_ptr(), b.data_ptr(), 60, 64, sp.ROW_MAJOR, None, None) == sp.ERR_ALIGNMENT
    assert L.sp_transpose(a.data_ptr(), a.data_ptr(), 64, 64, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    assert L.sp_transpose(a.data_ptr() + 2, b.data_ptr(), 64, 64, sp.ROW_MAJOR, None, None) == sp.ERR_ALIGNMENT
    assert L.sp_transpose(None, b.data_ptr(), 64, 64, sp.ROW_MAJOR, None, None) == sp.ERR_INVALID_ARG
    p = sp.make_params(num_xcds=8)          # 5 x 2 tiles, 8 chiplets: printed formula leaves the range
    assert L.sp_transpose(a.data_ptr(), b.data_ptr(), 320, 128, sp.XCD, ctypes.byref(p), None) == sp.ERR_NOT_BIJECTIVE


def test_matrix_larger_than_4_gib_is_addressed_correctly():
    M, N = 40960, 61440                                # 5 GB of 16-bit elements: byte offsets beyond 2^32
    g = torch.Generator(device="cuda").manual_seed(9)
    x = torch.randint(-32768, 32768, (M, N), device="cuda", generator=g, dtype=torch.int16)
    out = torch.zeros((N, M), dtype=torch.int16, device="cuda")
    sp.transpose(x, out, sp.DIE_SPLIT, sp.make_params(split_axis=0, inner_scheme=sp.HILBERT, interleave=1))
    assert sp.get_status() == 0
    for j in [0, 1, 63, 64, 30719, 30720, N - 65, N - 1]:            # rows of the output = columns of the input
        assert torch.equal(out[j], x[:, j]), j
    for i in [0, 4095, 20480, M - 1]:
        assert torch.equal(out[:, i], x[i]), i
