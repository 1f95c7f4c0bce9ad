"""sp_gemm_noalloc, the entry point for callers that cannot allocate device memory (their pool
owns the whole GPU, or an allocation's hidden synchronisation is not acceptable): called through
the C ABI, several times in a row, its output must equal sp_gemm's bit for bit -- both run the same
kernel, only the home of the tile table and the status word differs -- and must match the CPU oracle
within the GEMM tolerance; and it must leave the amount of free device memory untouched on orders
for which sp_gemm would allocate a table.  The file name sorts last on purpose."""

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
    from oracle import gemm as G
    L = sp.lib()
    M, N, K = 1160, 1544, 520                      # 5 x 7 tiles of 256 x 256: a ragged, non-square grid
    A, B = synth.make_inputs(M, N, K, "normal", 1.0, seed=21)
    dA, dB = _dev(A), _dev(B)
    ref, S = G.gemm_full(A, B)
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
        r = G.compare(G.bf16_bits_to_f64(got.view(torch.int16).cpu().numpy().view(np.uint16)), ref, S)
        assert r["max_err"] <= 1e-2, r               # the benchmark spec's tolerance: floored relative error vs the fp64 oracle
    # asynchronous form (no status pointer), through the Python wrapper
    got2 = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    sp.gemm_noalloc(dA, dB, got2, scheme, p)
    torch.cuda.synchronize()
    assert torch.equal(got2.view(torch.int16), want.view(torch.int16))


def test_noalloc_leaves_free_device_memory_untouched():
    """Orders on grids this process has not used before: sp_gemm would cudaMalloc a tile table for each."""
    L = sp.lib()
    M, N, K = 1928, 1672, 136                      # 16 x 14 tiles of 128 x 128 (also 8 x 7 of 256 x 256): nowhere else in the suite
    A, B = synth.make_inputs(M, N, K, "uniform", 1.0, seed=22)
    dA, dB = _dev(A), _dev(B)
    want = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    got = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    word = ctypes.c_int32(-1)
    # Everything that may load code or reserve memory on first use happens before the measurement: the kernels of the
    # three tile shapes (arithmetic order: no table), the table builder (into a caller buffer), this entry point's own
    # first call on the device, and the comparison's temporaries in torch's pool.
    for tm, tn in ((256, 256), (128, 256), (128, 128)):
        sp.gemm(dA, dB, want, sp.ROW_MAJOR, sp.make_params(tile_m=tm, tile_n=tn))
    sp.tile_map_device(640, 384, 128, 128, sp.HILBERT, sp.make_params())
    p0 = sp.make_params(tile_m=128, tile_n=128)
    assert L.sp_gemm_noalloc(dA.data_ptr(), dB.data_ptr(), got.data_ptr(), M, N, K, sp.ROW_MAJOR, ctypes.byref(p0), stream,
                             ctypes.byref(word)) == sp.OK, sp.last_error()
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for scheme, kw in [(sp.HILBERT, dict(tile_m=128, tile_n=128)), (sp.MORTON, dict(tile_m=256, tile_n=256)),
                       (sp.HILBERT_RECT, dict(tile_m=128, tile_n=256)),
                       (sp.DIE_SPLIT, dict(tile_m=128, tile_n=128, inner_scheme=sp.HILBERT)),
                       (sp.HILBERT, dict(tile_m=128, tile_n=128))]:       # the last one finds its table already in the array
        p = sp.make_params(**kw)
        rc = L.sp_gemm_noalloc(dA.data_ptr(), dB.data_ptr(), got.data_ptr(), M, N, K, scheme, ctypes.byref(p), stream,
                               ctypes.byref(word))
        assert rc == sp.OK, sp.last_error()
        assert word.value == 0
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))   # the order never changes the bits of C
        assert torch.cuda.mem_get_info()[0] == free0


def test_noalloc_rejects_flags_that_need_allocated_memory():
    L = sp.lib()
    a = torch.zeros(256 * 64, dtype=torch.bfloat16, device="cuda")
    for flag in (sp.FLAG_DIE_PINNED, sp.FLAG_STREAM_K, sp.FLAG_CLC, sp.FLAG_OVERLAP):
        p = sp.make_params(tile_m=128, tile_n=128, inner_scheme=sp.GROUP_M, inner_group=2, flags=flag)
        rc = L.sp_gemm_noalloc(a.data_ptr(), a.data_ptr(), a.data_ptr(), 128, 128, 64, sp.DIE_SPLIT, ctypes.byref(p), None, None)
        assert rc == sp.ERR_INVALID_ARG, flag
        assert "SP_FLAG_SERPENTINE" in sp.last_error()


def test_noalloc_rejects_more_tiles_than_its_array_holds():
    L = sp.lib()
    a = torch.zeros(16, dtype=torch.bfloat16, device="cuda")      # never read: rejected on the host
    p = sp.make_params(tile_m=128, tile_n=128)
    M = N = 128 * 257                                               # 66049 tiles > 65536
    rc = L.sp_gemm_noalloc(a.data_ptr(), a.data_ptr(), a.data_ptr(), M, N, 64, sp.ROW_MAJOR, ctypes.byref(p), None, None)
    assert rc == sp.ERR_UNSUPPORTED
    assert "65536" in sp.last_error()
