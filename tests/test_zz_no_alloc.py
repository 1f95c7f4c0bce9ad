"""sp_gemm_noalloc, the entry point for callers that cannot allocate device memory (their pool
owns the whole GPU, or an allocation's hidden synchronisation is not acceptable): called through
the C ABI, twice in a row, its output must equal sp_gemm's bit for bit -- both run the same kernel,
only the home of the tile table and the status word differs.  The file name sorts last on purpose."""

import ctypes

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from paper_2508_20258_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def test_noalloc_matches_gemm_on_two_calls_in_a_row():
    L = sp.lib()
    M, N, K = 1160, 1544, 520                      # 5 x 7 tiles of 256 x 256: a ragged, non-square grid
    A, B = synth.make_inputs(M, N, K, "normal", 1.0, seed=21)
    dA, dB = _dev(A), _dev(B)
    stream = torch.cuda.current_stream().cuda_stream
    table = np.random.default_rng(3).permutation(5 * 7).astype(np.int32)
    # first a curve order (table built on the device), then a caller table (table copied): the second
    # call finds the first call's table in the shared array and must replace it
    calls = [(sp.HILBERT, sp.make_params(tile_m=256, tile_n=256)),
             (sp.CUSTOM, sp.make_params(tile_m=256, tile_n=256, custom_perm=table)),
             (sp.GROUP_M, sp.make_params(tile_m=256, tile_n=256, group=2))]
    for scheme, p in calls:
        want = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        got = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        sp.gemm(dA, dB, want, scheme, p)
        assert sp.get_status() == 0
        word = ctypes.c_int32(-1)
        rc = L.sp_gemm_noalloc(dA.data_ptr(), dB.data_ptr(), got.data_ptr(), M, N, K, scheme, ctypes.byref(p), stream,
                               ctypes.byref(word))
        assert rc == sp.OK, sp.last_error()
        assert word.value == 0
        torch.cuda.synchronize()
        assert not torch.isnan(got.float()).any()
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    # asynchronous form (no status pointer), through the Python wrapper
    got2 = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    sp.gemm_noalloc(dA, dB, got2, scheme, p)
    torch.cuda.synchronize()
    assert torch.equal(got2.view(torch.int16), want.view(torch.int16))


def test_noalloc_rejects_more_tiles_than_its_array_holds():
    L = sp.lib()
    a = torch.zeros(16, dtype=torch.bfloat16, device="cuda")      # never read: rejected on the host
    p = sp.make_params(tile_m=128, tile_n=128)
    M = N = 128 * 257                                               # 66049 tiles > 65536
    rc = L.sp_gemm_noalloc(a.data_ptr(), a.data_ptr(), a.data_ptr(), M, N, 64, sp.ROW_MAJOR, ctypes.byref(p), None, None)
    assert rc == sp.ERR_UNSUPPORTED
    assert "65536" in sp.last_error()
