"""SP_FLAG_STREAM_K on the GPU, through the C ABI: the k-split of the last, partly empty wave must give the GEMM
the oracle defines (exactly on integer inputs, within the usual tolerance on random ones), the same bits run to
run, and the documented rejections."""

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import gemm as G
from paper_2508_20258_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
SK = sp.FLAG_STREAM_K


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def launch(A, B, scheme, tile, out, b_is_nk=False, **kw):
    M, K = A.shape
    N = B.shape[1]
    dA, dB = dev_bf16(A), dev_bf16(np.ascontiguousarray(B.T) if b_is_nk else B)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32 if out == "fp32" else torch.bfloat16, device="cuda")
    p = sp.make_params(tile_m=tile[0], tile_n=tile[1], out_dtype=int(out == "fp32"), b_layout=int(b_is_nk), **kw)
    sp.gemm(dA, dB, dC, scheme, p)
    assert sp.get_status() == 0
    return dC


def pieces_of(M, N, K, tile):
    """(first_slot, number of units with a piece) of the plan the library uses for this launch."""
    T = sp.tile_count(M, N, *tile)
    units = sp.gemm_units(tile[0], tile[1], 1 << 24)
    first, segs = sp.streamk_plan(T, units, -(-K // 64))
    return T, first, sum(1 for s in segs if s)


# shapes chosen so that the remainder wave is split 2, 3, 4 and 9 ways on a 148-SM device, with ragged edges and a
# ragged last k-block; (tile, M, N, K)
SPLIT_SHAPES = [
    ((256, 256), 2304, 2560, 1024),    # 90 tiles on 74 units: 16 left, 4 pieces each
    ((256, 256), 4096, 4096, 512),     # 256 tiles: 34 left, 2 pieces
    ((256, 128), 2300, 1096, 840),     # ragged in M, N and K: 81 tiles, 7 left, 3 pieces
    ((128, 256), 128 * 13, 256 * 12, 64 * 12),   # 156 tiles on 148 units: 8 left, 3 pieces of 4 k-blocks
    ((128, 128), 512, 512, 2304),      # smaller than a wave: 16 tiles, 8 pieces each (the cap)
    ((128, 128), 1024, 1280, 768),     # 80 tiles on 148 units: no split (f = 1)
]


@pytest.mark.parametrize("tile,M,N,K", SPLIT_SHAPES)
@pytest.mark.parametrize("b_is_nk", [False, True])
def test_split_tail_is_exact_on_integer_inputs(tile, M, N, K, b_is_nk):
    A, B = synth.make_int_inputs(M, N, K, seed=21)
    ref, _ = G.gemm_full(A, B)                      # small integers: every partial sum is exact in fp32
    for scheme, kw in [(sp.ROW_MAJOR, {}), (sp.HILBERT, {}), (sp.GROUP_M, dict(group=4))]:
        dC = launch(A, B, scheme, tile, "fp32", b_is_nk, flags=SK, **kw)
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), ref), (scheme, kw)
    dC = launch(A, B, sp.GROUP_N, tile, "bf16", b_is_nk, flags=SK, group=3)
    got = G.bf16_bits_to_f64(dC.view(torch.int16).cpu().numpy().view(np.uint16))
    want = G.bf16_bits_to_f64(synth.f32_to_bf16_bits(ref.astype(np.float32)))
    assert np.array_equal(got, want)


def test_the_shapes_above_do_split():
    expect = {0: 64, 1: 68, 3: 24, 4: 128, 5: 0}    # units holding a piece (256x128 case depends on raggedness: skipped)
    for i, n in expect.items():
        tile, M, N, K = SPLIT_SHAPES[i]
        if sp.gemm_units(tile[0], tile[1], 1 << 24) != (74 if tile[0] == 256 else 148):
            pytest.skip("unit count differs from a full B200")
        T, first, busy = pieces_of(M, N, K, tile)
        assert busy == n, (SPLIT_SHAPES[i], T, first, busy)


def test_split_tail_on_random_inputs_matches_the_oracle_and_repeats_bit_for_bit():
    M, N, K, tile = 2304, 2560, 2048, (256, 256)
    A, B = synth.make_inputs(M, N, K, dist="normal", seed=33)
    ref, S = G.gemm_full(A, B)
    outs = []
    for _ in range(3):
        dC = launch(A, B, sp.GROUP_M, tile, "bf16", flags=SK, group=4)
        outs.append(dC.view(torch.int16).cpu().numpy().view(np.uint16).copy())
    r = G.compare(G.bf16_bits_to_f64(outs[0]), ref, S)
    assert r["max_err"] <= 1e-2 and r["fro_rel"] <= 3e-3, r
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
    # fp32 output: the split sum differs from the unsplit one only by rounding order
    c_split = launch(A, B, sp.GROUP_M, tile, "fp32", flags=SK, group=4).cpu().numpy().astype(np.float64)
    c_plain = launch(A, B, sp.GROUP_M, tile, "fp32", group=4).cpu().numpy().astype(np.float64)
    r32, p32 = G.compare(c_split, ref, S), G.compare(c_plain, ref, S)
    assert r32["fro_rel"] <= 1e-5 and p32["fro_rel"] <= 1e-5, (r32, p32)   # fp32 output: only accumulation rounding remains
    assert r32["max_err"] <= 2.0 * p32["max_err"] + 1e-6, (r32, p32)       # ... and the split adds none to speak of
    # only tiles of the split remainder may differ at all
    T, first, _ = pieces_of(M, N, K, tile)
    perm = sp.tile_map(M, N, tile[0], tile[1], sp.GROUP_M, sp.make_params(group=4))
    Tn = -(-N // tile[1])
    whole = np.ones((M, N), dtype=bool)
    for s in range(first, T):
        tm, tn = divmod(int(perm[s]), Tn)
        whole[tm * tile[0]:(tm + 1) * tile[0], tn * tile[1]:(tn + 1) * tile[1]] = False
    assert first < T and np.array_equal(c_split[whole], c_plain[whole])


def test_trace_of_a_split_launch_has_one_record_per_tile():
    M, N, K, tile = 2304, 2560, 1024, (256, 256)
    A, B = synth.make_int_inputs(M, N, K, seed=5)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    p = sp.make_params(tile_m=tile[0], tile_n=tile[1], flags=SK)
    tr = sp.gemm_trace(dA, dB, dC, sp.HILBERT, p)
    perm = sp.tile_map(M, N, tile[0], tile[1], sp.HILBERT, p)
    assert np.array_equal(tr["slot"], np.arange(len(perm)))
    assert np.array_equal(tr["tile"], perm)
    assert (tr["t_end"] >= tr["t_begin"]).all()
    T, first, _ = pieces_of(M, N, K, tile)
    units = sp.gemm_units(tile[0], tile[1], 1 << 24)
    _, segs = sp.streamk_plan(T, units, K // 64)
    for u, ss in enumerate(segs):
        for (slot, k0, k1, kind) in ss:
            if kind != sp.WORK_CONTRIB:
                assert tr["unit"][slot] == u          # the storing piece wrote the record


def test_split_rejections_launch_nothing():
    A, B = synth.make_int_inputs(512, 512, 512, seed=1)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.zeros((512, 512), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sp.SpError) as e:
        sp.gemm(dA, dB, dC, sp.ROW_MAJOR, sp.make_params(tile_m=256, tile_n=512, flags=SK))
    assert e.value.status == sp.ERR_UNSUPPORTED
    with pytest.raises(sp.SpError) as e:
        sp.gemm(dA, dB, dC, sp.DIE_SPLIT, sp.make_params(tile_m=128, tile_n=128, inner_scheme=sp.ROW_MAJOR,
                                                         flags=SK | sp.FLAG_DIE_PINNED))
    assert e.value.status in (sp.ERR_INVALID_ARG, sp.ERR_UNSUPPORTED)
    with pytest.raises(sp.SpError) as e:
        sp.gemm_noalloc(dA, dB, dC, sp.ROW_MAJOR, sp.make_params(tile_m=128, tile_n=128, flags=SK))
    assert e.value.status == sp.ERR_INVALID_ARG
    assert sp.get_status() == 0 and float(dC.float().abs().sum()) == 0.0


def test_split_through_the_host_entry_point():
    M, N, K = 2304, 2560, 1024
    A, B = synth.make_int_inputs(M, N, K, seed=8)
    ref, _ = G.gemm_full(A, B)
    hC = np.zeros((M, N), dtype=np.float32)
    sp.gemm_host(A.view(np.int16), B.view(np.int16), hC, sp.GROUP_M,
                 sp.make_params(tile_m=256, tile_n=256, out_dtype=1, group=2, flags=SK))
    assert np.array_equal(hC.astype(np.float64), ref)


def test_split_launches_of_different_shapes_back_to_back_and_on_two_streams():
    """The workspace and its flags are reused from launch to launch on a stream (a launch counter tells the flags of one
    launch from the next) and are separate per stream: different split shapes queued back to back on two streams at once."""
    shapes = [(2304, 2560, 1024, (256, 256)), (512, 512, 2304, (128, 128)), (4096, 4096, 512, (256, 256)),
              (128 * 13, 256 * 12, 64 * 12, (128, 256)), (2300, 1096, 840, (256, 128))]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    work = []
    for i, (M, N, K, tile) in enumerate(shapes):
        A, B = synth.make_int_inputs(M, N, K, seed=90 + i)
        work.append((dev_bf16(A), dev_bf16(B), G.gemm_full(A, B)[0], tile,
                     [torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") for _ in range(4)]))
    torch.cuda.synchronize()
    for rep in range(2):
        for k, st in enumerate(streams):
            for (dA, dB, _, tile, outs) in work:
                sp.gemm(dA, dB, outs[2 * rep + k], sp.GROUP_M, sp.make_params(tile_m=tile[0], tile_n=tile[1], out_dtype=1, group=2, flags=SK), st)
    torch.cuda.synchronize()
    assert sp.get_status() == 0
    for (_, _, ref, _, outs) in work:
        for o in outs:
            assert np.array_equal(o.cpu().numpy().astype(np.float64), ref)
