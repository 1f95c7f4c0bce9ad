"""SP_FLAG_OVERLAP: launches declared independent of their predecessor start while it is still running.  The results
must be those of ordinary launches, and whatever follows on the stream must still see both kernels complete."""

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import gemm as G
from paper_2508_20258_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
OV = sp.FLAG_OVERLAP


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def test_chain_of_independent_gemms_matches_the_oracle():
    shapes = [(1024, 1280, 768, (256, 256)), (640, 896, 1000, (128, 128)), (2304, 2560, 512, (256, 512)),
              (512, 512, 512, (128, 256)), (1160, 600, 520, (256, 128))]
    problems = []
    for i, (M, N, K, tile) in enumerate(shapes):
        A, B = synth.make_int_inputs(M, N, K, seed=40 + i)
        problems.append((dev_bf16(A), dev_bf16(B), torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda"),
                         tile, G.gemm_full(A, B)[0]))
    orders = [(sp.HILBERT, {}), (sp.GROUP_M, dict(group=2)), (sp.ROW_MAJOR, {}), (sp.MORTON, {}), (sp.GROUP_N, dict(group=3))]
    for rep in range(3):                                  # the first round builds tile tables, later rounds overlap fully
        for (dA, dB, dC, tile, _), (scheme, kw) in zip(problems, orders):
            if rep:
                dC.fill_(float("nan"))
        for (dA, dB, dC, tile, _), (scheme, kw) in zip(problems, orders):
            sp.gemm(dA, dB, dC, scheme, sp.make_params(tile_m=tile[0], tile_n=tile[1], out_dtype=1, flags=OV, **kw))
        assert sp.get_status() == 0
        for (_, _, dC, _, ref) in problems:
            assert np.array_equal(dC.cpu().numpy().astype(np.float64), ref)


def test_a_copy_behind_a_short_overlapped_launch_still_sees_the_long_predecessor_complete():
    w, A, B = synth.make_workload("cfg2")
    dA, dB = dev_bf16(A), dev_bf16(B)
    big = torch.empty((w.M, w.N), dtype=torch.bfloat16, device="cuda")
    p = sp.make_params(tile_m=256, tile_n=256)
    sp.gemm(dA, dB, big, sp.ROW_MAJOR, p)
    want = big.cpu()
    a2, b2 = synth.make_int_inputs(128, 128, 64, seed=3)
    dA2, dB2 = dev_bf16(a2), dev_bf16(b2)
    small = torch.empty((128, 128), dtype=torch.bfloat16, device="cuda")
    host = torch.empty((w.M, w.N), dtype=torch.bfloat16).pin_memory()
    for _ in range(5):
        big.zero_()
        torch.cuda.synchronize()
        sp.gemm(dA, dB, big, sp.ROW_MAJOR, p)                                        # about 0.1 ms
        sp.gemm(dA2, dB2, small, sp.ROW_MAJOR, sp.make_params(tile_m=128, tile_n=128, flags=OV))   # microseconds, overlapped
        host.copy_(big, non_blocking=True)                                            # ordered behind both
        torch.cuda.synchronize()
        assert torch.equal(host.view(torch.int16), want.view(torch.int16))
    assert sp.get_status() == 0


def test_overlap_rejections():
    A, B = synth.make_int_inputs(512, 512, 512, seed=1)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.zeros((512, 512), dtype=torch.bfloat16, device="cuda")
    for bad in (OV | sp.FLAG_STREAM_K, OV | sp.FLAG_DIE_PINNED):
        with pytest.raises(sp.SpError) as e:
            sp.gemm(dA, dB, dC, sp.DIE_SPLIT, sp.make_params(tile_m=128, tile_n=128, inner_scheme=sp.ROW_MAJOR, flags=bad))
        assert e.value.status == sp.ERR_INVALID_ARG
    with pytest.raises(sp.SpError) as e:
        sp.gemm_trace(dA, dB, dC, sp.ROW_MAJOR, sp.make_params(tile_m=128, tile_n=128, flags=OV))
    assert e.value.status == sp.ERR_INVALID_ARG
    with pytest.raises(sp.SpError) as e:
        sp.gemm_noalloc(dA, dB, dC, sp.ROW_MAJOR, sp.make_params(tile_m=128, tile_n=128, flags=OV))
    assert e.value.status == sp.ERR_INVALID_ARG
    with pytest.raises(sp.SpError) as e:
        sp.gemm_host(A.view(np.int16), B.view(np.int16), np.zeros((512, 512), dtype=np.int16), sp.ROW_MAJOR,
                     sp.make_params(tile_m=128, tile_n=128, flags=OV))
    assert e.value.status == sp.ERR_INVALID_ARG
    assert sp.get_status() == 0 and float(dC.float().abs().sum()) == 0.0


def test_dependent_gemms_back_to_back_see_each_others_results():
    """Ordinary launches are programmatic too (their set-up overlaps the predecessor's tail), so the wait that orders them
    is checked where it matters: a chain in which every GEMM reads, as its A operand, what the GEMM before it wrote.
    The GEMMs are large enough for the GPU, not the host, to set the pace, and every other one walks its tiles in reverse,
    so that its first tiles need what its predecessor writes last (with SP_FLAG_OVERLAP set against its contract, this
    very chain comes out wrong every time; with ordinary launches it must be exact)."""
    M = N = K = 4096
    rng = np.random.default_rng(3)
    a0 = rng.integers(-3, 4, size=(M, K)).astype(np.float32)
    A0 = synth.f32_to_bf16_bits(a0)
    want = a0.astype(np.float64)
    dPs = []
    for seed in range(6):                                # right factors: signed permutation matrices, products stay small integers
        r = np.random.default_rng(seed)
        j, sg = r.permutation(N), r.choice([-1.0, 1.0], size=K).astype(np.float32)
        P = np.zeros((K, N), dtype=np.float32)
        P[np.arange(K), j] = sg
        dPs.append(dev_bf16(synth.f32_to_bf16_bits(P)))
        nxt = np.zeros_like(want)
        nxt[:, j] = want * sg
        want = nxt
    for tile, kw in [((256, 256), {}), ((256, 512), {}), ((128, 256), {}), ((256, 256), dict(flags=sp.FLAG_CLC)),
                     ((256, 256), dict(flags=sp.FLAG_STREAM_K))]:
        T = sp.tile_count(M, N, tile[0], tile[1])
        fwd = sp.make_params(tile_m=tile[0], tile_n=tile[1], **kw)
        rev = sp.make_params(tile_m=tile[0], tile_n=tile[1], custom_perm=np.arange(T - 1, -1, -1, dtype=np.int32), **kw)
        bufs = [dev_bf16(A0), torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")]
        sp.gemm(bufs[0], dPs[0], bufs[1], sp.CUSTOM, rev)                 # uploads the table once, outside the chain
        torch.cuda.synchronize()
        bufs[1].zero_()
        src = 0
        for i, dP in enumerate(dPs):                     # no synchronisation anywhere in the chain
            if i % 2 == 0:
                sp.gemm(bufs[src], dP, bufs[1 - src], sp.ROW_MAJOR, fwd)
            else:
                sp.gemm(bufs[src], dP, bufs[1 - src], sp.CUSTOM, rev)
            src = 1 - src
        assert sp.get_status() == 0
        got = G.bf16_bits_to_f64(bufs[src].view(torch.int16).cpu().numpy().view(np.uint16))
        assert np.array_equal(got, want), (tile, kw)


def test_other_kernels_behind_a_gemm_wait_for_all_of_it():
    """A GEMM tells the hardware at its start that a programmatic successor may be scheduled; a kernel launched the
    ordinary way behind it (here the transpose, walking its tiles from the end) must still see all of C."""
    M = N = K = 4096
    A, B = synth.make_int_inputs(M, N, K, seed=12)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    dT = torch.zeros((N, M), dtype=torch.bfloat16, device="cuda")
    p = sp.make_params(tile_m=256, tile_n=512)
    sp.gemm(dA, dB, dC, sp.ROW_MAJOR, p)
    torch.cuda.synchronize()
    want = dC.t().contiguous()
    Tt = sp.tile_count(M, N, 64, 64)
    rev = sp.make_params(custom_perm=np.arange(Tt - 1, -1, -1, dtype=np.int32))
    sp.transpose(dC.view(torch.int16), dT.view(torch.int16), sp.CUSTOM, rev)          # uploads the table
    for _ in range(5):
        dC.zero_()
        dT.zero_()
        torch.cuda.synchronize()
        sp.gemm(dA, dB, dC, sp.ROW_MAJOR, p)
        sp.transpose(dC.view(torch.int16), dT.view(torch.int16), sp.CUSTOM, rev)      # starts with the tiles C gets last
        torch.cuda.synchronize()
        assert torch.equal(dT.view(torch.int16), want.view(torch.int16))
    assert sp.get_status() == 0


def test_gemm_behind_a_library_kernel_reads_its_complete_output():
    """The producer of A is another library's GEMM (which may itself release its programmatic successors early): our
    launch, walking its tiles from the end, must still read all of it."""
    M = N = K = 4096
    rng = np.random.default_rng(8)
    x = torch.from_numpy(rng.integers(-2, 3, size=(M, K)).astype(np.float32)).cuda().bfloat16()
    j = torch.from_numpy(rng.permutation(K)).cuda()
    P = torch.zeros((K, K), dtype=torch.bfloat16, device="cuda")
    P[torch.arange(K, device="cuda"), j] = 1.0                      # permutation matrix: x @ P is exact
    E = torch.zeros((K, N), dtype=torch.bfloat16, device="cuda")
    E[torch.arange(K, device="cuda"), torch.arange(K, device="cuda").flip(0)] = -1.0
    mid = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    want = -(x.float()[:, torch.argsort(j)]).flip(1)                 # (x P) E, both factors signed permutations
    T = sp.tile_count(M, N, 256, 256)
    rev = sp.make_params(tile_m=256, tile_n=256, custom_perm=np.arange(T - 1, -1, -1, dtype=np.int32))
    sp.gemm(mid, E, out, sp.CUSTOM, rev)
    torch.cuda.synchronize()
    for _ in range(5):
        mid.zero_()
        out.zero_()
        torch.cuda.synchronize()
        torch.matmul(x, P, out=mid)
        sp.gemm(mid, E, out, sp.CUSTOM, rev)
        torch.cuda.synchronize()
        assert torch.equal(out.float(), want)
    assert sp.get_status() == 0
