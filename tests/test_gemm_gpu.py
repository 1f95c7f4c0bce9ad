"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element.

Bars: remaps bit-exact; GEMM max floored relative error <= 1e-2 for bf16 inputs with fp32
accumulation (the stated tolerance); integer-valued inputs and stamp matrices bit-exact,
because every fp32 partial sum is then exact in any accumulation order.
"""

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import gemm as G
from oracle import remap as R
from paper_2508_20258_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 1e-2

torch = pytest.importorskip("torch")


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def run_gemm(A, B, scheme=sp.ROW_MAJOR, tile=(256, 256), out="bf16", b_is_nk=False, **kw):
    """A, B: uint16 bit patterns on the host (B as K x N).  Returns C as float64 on the host."""
    M, K = A.shape
    N = B.shape[1]
    Bd = np.ascontiguousarray(B.T) if b_is_nk else B
    dA, dB = dev_bf16(A), dev_bf16(Bd)
    dC = torch.full((M, N), float("nan"), dtype=torch.float32 if out == "fp32" else torch.bfloat16, device="cuda")
    p = sp.make_params(tile_m=tile[0], tile_n=tile[1], out_dtype=int(out == "fp32"), b_layout=int(b_is_nk), **kw)
    sp.gemm(dA, dB, dC, scheme, p)
    assert sp.get_status() == 0
    if out == "fp32":
        return dC.cpu().numpy().astype(np.float64), dC
    return G.bf16_bits_to_f64(dC.view(torch.int16).cpu().numpy().view(np.uint16)), dC


# ------------------------------------------------------------------ remap: device code == oracle
@pytest.mark.parametrize("M,N,tm,tn", [(512, 512, 128, 128), (4096, 4096, 128, 256), (8192, 8192, 256, 256),
                                        (16384, 2048, 256, 256), (16384, 16384, 256, 256), (1000, 520, 128, 128),
                                        (128 * 37, 128 * 5, 128, 128), (128, 128 * 300, 128, 128)])
def test_device_remap_matches_oracle(M, N, tm, tn):
    cases = [(sp.ROW_MAJOR, {}), (sp.COL_MAJOR, {}), (sp.GROUP_M, dict(group=8)), (sp.GROUP_M, dict(group=3)),
             (sp.GROUP_N, dict(group=4)), (sp.MORTON, {}), (sp.HILBERT, {}), (sp.HILBERT_RECT, {}),
             (sp.XCD, dict(num_xcds=2, wave=74, xcd_balanced=1)), (sp.XCD, dict(num_xcds=8, xcd_balanced=1)),
             (sp.DIE_SPLIT, dict(split_axis=0, inner_scheme=sp.HILBERT)),
             (sp.DIE_SPLIT, dict(split_axis=1, inner_scheme=sp.GROUP_M, inner_group=8, interleave=1)),
             (sp.DIE_SPLIT, dict(split_axis=1, inner_scheme=sp.MORTON, interleave=1)),
             (sp.GROUP_M, dict(group=8, flags=4)), (sp.GROUP_N, dict(group=3, flags=4)),
             (sp.DIE_SPLIT, dict(split_axis=0, inner_scheme=sp.GROUP_M, inner_group=8, flags=4))]
    for scheme, kw in cases:
        want = R.tile_map(M, N, tm, tn, scheme, R.Params(**kw))
        got = sp.tile_map_device(M, N, tm, tn, scheme, sp.make_params(**kw)).cpu().numpy().tolist()
        assert got == want, (scheme, kw)
    table = np.random.default_rng(0).permutation(sp.tile_count(M, N, tm, tn)).astype(np.int32)
    got = sp.tile_map_device(M, N, tm, tn, sp.CUSTOM, sp.make_params(custom_perm=table)).cpu().numpy()
    assert np.array_equal(got, table)


# ------------------------------------------------------------------ exact cases
SHAPES = [(128, 128), (128, 256), (256, 128), (256, 256), (256, 512)]


@pytest.mark.parametrize("tile", SHAPES)
@pytest.mark.parametrize("b_is_nk", [False, True])
@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (300, 328, 200), (1000, 520, 264), (768, 1024, 8192)])
def test_integer_inputs_are_bit_exact(tile, b_is_nk, M, N, K):
    A, B = synth.make_int_inputs(M, N, K, seed=M + K)
    ref, _ = G.gemm_full(A, B)
    got, _ = run_gemm(A, B, sp.GROUP_M, tile, "fp32", b_is_nk, group=2)
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("tile", SHAPES)
@pytest.mark.parametrize("b_is_nk", [False, True])
@pytest.mark.parametrize("kk", [0, 17, 63, 100])
def test_stamp_matrices_pin_addressing(tile, b_is_nk, kk):
    """One non-zero k: C[i,j] = 2^(i mod 8) * 2^-(j mod 16) names its own position, so a
    misplaced row, column, k-slice or a transposed operand cannot pass."""
    M, N, K = 520, 776, 128
    Af = np.zeros((M, K), np.float32)
    Bf = np.zeros((K, N), np.float32)
    Af[:, kk] = 2.0 ** (np.arange(M) % 8) * (1 + (np.arange(M) // 8) % 2)
    Bf[kk, :] = 2.0 ** -(np.arange(N) % 16) * (1 + 2 * ((np.arange(N) // 16) % 2))
    A, B = synth.f32_to_bf16_bits(Af), synth.f32_to_bf16_bits(Bf)
    ref, _ = G.gemm_full(A, B)
    got, _ = run_gemm(A, B, sp.COL_MAJOR, tile, "fp32", b_is_nk)
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("tile", [(128, 256), (256, 256)])
def test_bf16_output_is_rne_of_the_fp32_result(tile):
    A, B = synth.make_inputs(512, 768, 1024, "normal", 1.0, 9)
    f32, _ = run_gemm(A, B, sp.ROW_MAJOR, tile, "fp32")
    b16, _ = run_gemm(A, B, sp.ROW_MAJOR, tile, "bf16")
    want = G.bf16_bits_to_f64(synth.f32_to_bf16_bits(f32.astype(np.float32)))
    assert np.array_equal(b16, want)


# ------------------------------------------------------------------ small workloads, every element
@pytest.mark.parametrize("scheme,kw", [(sp.ROW_MAJOR, {}), (sp.GROUP_M, dict(group=2))])
def test_cfg1_full(scheme, kw):
    w, A, B = synth.make_workload("cfg1")
    ref, S = G.gemm_full(A, B)
    got, _ = run_gemm(A, B, scheme, (w.tile_m, w.tile_n), w.out_dtype, **kw)
    r = G.compare(got, ref, S)
    assert r["max_err"] <= TOL, r
    assert r["fro_rel"] <= 1e-5, r          # fp32 output: only accumulation rounding remains


@pytest.mark.parametrize("M,N,K,tile,out", [(640, 896, 1000, (128, 128), "bf16"), (1160, 600, 520, (128, 256), "fp32"),
                                             (1160, 1096, 776, (256, 256), "bf16"), (904, 648, 1288, (256, 128), "bf16"), (1160, 1608, 776, (256, 512), "bf16"),
                                             (520, 2056, 328, (256, 512), "fp32")])
@pytest.mark.parametrize("b_is_nk", [False, True])
def test_ragged_sizes_full(M, N, K, tile, out, b_is_nk):
    """Several tiles, ragged M / N tails, K not a multiple of the 64-wide k-block."""
    A, B = synth.make_inputs(M, N, K, "normal", 1.0, seed=M)
    ref, S = G.gemm_full(A, B)
    for scheme, kw in [(sp.HILBERT, {}), (sp.HILBERT_RECT, {}), (sp.XCD, dict(num_xcds=2, xcd_balanced=1))]:
        got, _ = run_gemm(A, B, scheme, tile, out, b_is_nk, **kw)
        r = G.compare(got, ref, S)
        assert r["max_err"] <= TOL, (scheme, r)


def test_tiny_and_degenerate_sizes():
    for (M, N, K) in [(1, 8, 8), (8, 8, 8), (129, 264, 72), (256, 8, 64)]:
        A, B = synth.make_int_inputs(M, N, K, seed=3)
        ref, _ = G.gemm_full(A, B)
        for tile in SHAPES:
            got, _ = run_gemm(A, B, sp.ROW_MAJOR, tile, "fp32")
            assert np.array_equal(got, ref), (M, N, K, tile)


def test_cfg2_full():
    w, A, B = synth.make_workload("cfg2")
    ref, S = G.gemm_full(A, B)
    first = None
    for scheme, kw in [(sp.ROW_MAJOR, {}), (sp.GROUP_M, dict(group=4)), (sp.GROUP_M, dict(group=8)),
                       (sp.GROUP_M, dict(group=16)), (sp.HILBERT, {})]:
        got, dC = run_gemm(A, B, scheme, (w.tile_m, w.tile_n), w.out_dtype, **kw)
        r = G.compare(got, ref, S)
        assert r["max_err"] <= TOL, (scheme, kw, r)
        assert r["fro_rel"] <= 3e-3, r
        bits = dC.view(torch.int16).cpu().numpy()
        if first is None:
            first = bits
        else:
            assert np.array_equal(bits, first)      # a swizzle only reorders tiles: same bits


# ------------------------------------------------------------------ schedule evidence
@pytest.mark.parametrize("tile", [(128, 256), (256, 256)])
def test_trace_runs_every_tile_once_under_the_remap(tile):
    M, N, K = 4096, 4096, 256
    A, B = synth.make_int_inputs(M, N, K, seed=5)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    for scheme, kw in [(sp.ROW_MAJOR, {}), (sp.HILBERT, {}), (sp.GROUP_M, dict(group=4)),
                       (sp.DIE_SPLIT, dict(split_axis=0, inner_scheme=sp.GROUP_N, inner_group=2, interleave=1))]:
        p = sp.make_params(tile_m=tile[0], tile_n=tile[1], **kw)
        tr = sp.gemm_trace(dA, dB, dC, scheme, p)
        assert sp.get_status() == 0
        want = R.tile_map(M, N, tile[0], tile[1], scheme, R.Params(**kw))
        T = len(want)
        assert tr["slot"].tolist() == list(range(T))
        assert tr["tile"].tolist() == want
        assert sorted(tr["tile"].tolist()) == list(range(T))
        units = sp.gemm_units(tile[0], tile[1], T)
        assert tr["unit"].tolist() == [s % units for s in range(T)]
        assert (tr["t_end"] > tr["t_begin"]).all()
        # a unit runs its slots in increasing order
        for u in range(min(units, 4)):
            mine = tr[tr["unit"] == u]
            assert (np.diff(mine["t_begin"].astype(np.int64)) > 0).all()
            assert len(set(mine["smid"].tolist())) == 1


def test_output_bits_do_not_depend_on_the_scheme():
    A, B = synth.make_inputs(2048, 2304, 1024, "normal", 1.0, 12)
    ref = None
    table = np.random.default_rng(1).permutation(8 * 9).astype(np.int32)
    for scheme, kw in [(sp.ROW_MAJOR, {}), (sp.COL_MAJOR, {}), (sp.GROUP_N, dict(group=3)), (sp.MORTON, {}), (sp.HILBERT_RECT, {}),
                       (sp.XCD, dict(num_xcds=4, wave=16, xcd_balanced=1)), (sp.CUSTOM, dict(custom_perm=table)),
                       (sp.DIE_SPLIT, dict(split_axis=1, inner_scheme=sp.HILBERT))]:
        _, dC = run_gemm(A, B, scheme, (256, 256), "bf16", **kw)
        bits = dC.view(torch.int16).cpu().numpy()
        if ref is None:
            ref = bits
        assert np.array_equal(bits, ref), scheme


def test_runtime_rejections_launch_nothing():
    A = torch.zeros((256, 256), dtype=torch.bfloat16, device="cuda")
    C = torch.full((256, 256), 7.0, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sp.SpError) as e:
        sp.gemm(A, A, C, sp.XCD, sp.make_params(tile_m=128, tile_n=128, num_xcds=3))   # 4 tiles, X = 3
    assert e.value.status == sp.ERR_NOT_BIJECTIVE
    with pytest.raises(sp.SpError) as e:
        sp.gemm(A, A, C, sp.CUSTOM, sp.make_params(tile_m=128, tile_n=128, custom_perm=[0, 1, 1, 3]))
    assert e.value.status == sp.ERR_NOT_BIJECTIVE
    torch.cuda.synchronize()
    assert (C == 7.0).all()
    assert sp.get_status() == 0


def test_die_pinned_schedule_keeps_each_half_on_one_l2_half():
    """SP_FLAG_DIE_PINNED: units run only the slots of the tile-space half that matches the L2 half
    (die) their SM was measured on; every tile still runs exactly once and C has the same bits."""
    die, conf, _ = sp.probe_topology()
    if conf < 0.8 or (die < 0).any():
        pytest.skip("no two-way L2 structure measured on this device")
    M = N = 8192
    K = 256
    A, B = synth.make_int_inputs(M, N, K, seed=8)
    dA, dB = dev_bf16(A), dev_bf16(B)
    ref = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    sp.gemm(dA, dB, ref, sp.ROW_MAJOR, sp.make_params(tile_m=256, tile_n=256))
    for tile in [(256, 256), (128, 256)]:
        for axis in (0, 1):
            kw = dict(split_axis=axis, inner_scheme=sp.GROUP_M, inner_group=4)
            p = sp.make_params(tile_m=tile[0], tile_n=tile[1], flags=2, **kw)
            dC = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
            tr = sp.gemm_trace(dA, dB, dC, sp.DIE_SPLIT, p)
            assert sp.get_status() == 0
            assert torch.equal(dC.view(torch.int16), ref.view(torch.int16))
            want = R.tile_map(M, N, tile[0], tile[1], sp.DIE_SPLIT, R.Params(**kw))
            assert tr["tile"].tolist() == want                       # record s still describes slot s
            h0 = len(R.die_split_halves(-(-M // tile[0]), -(-N // tile[1]), axis, sp.GROUP_M, 4)[0])
            on_die = die[tr["smid"]]
            # each half runs on one L2 half; where the GPU's halves have unequal SM counts (72 / 76) the surplus
            # units of the larger side help out on the other half of the tile space
            d0 = int(np.bincount(on_die[:h0], minlength=2).argmax())
            d1 = int(np.bincount(on_die[h0:], minlength=2).argmax())
            assert d0 != d1
            assert (on_die[:h0] == d0).mean() >= 0.9 and (on_die[h0:] == d1).mean() >= 0.9
            if (die == 0).sum() == (die == 1).sum():
                assert (on_die[:h0] == d0).all() and (on_die[h0:] == d1).all()
    with pytest.raises(sp.SpError) as e:                              # pinning is defined for the split order only
        sp.gemm(dA, dB, ref, sp.GROUP_M, sp.make_params(tile_m=256, tile_n=256, group=4, flags=2))
    assert e.value.status == sp.ERR_INVALID_ARG


def test_topology_probe_finds_two_equal_l2_halves_and_pairs_stay_together():
    die, conf, lat = sp.probe_topology()
    assert len(die) == torch.cuda.get_device_properties(0).multi_processor_count
    assert lat.shape == (len(die), sp.binding.PROBE_LINES) and (lat > 0).all()
    if conf < 0.8:
        pytest.skip("no two-way L2 structure measured on this device")
    # the two halves need not be equal: parts differ in which SMs are fused off (74/74 and 72/76 have been seen)
    n0, n1 = int((die == 0).sum()), int((die == 1).sum())
    assert set(die.tolist()) == {0, 1} and n0 % 2 == 0 and n1 % 2 == 0 and abs(n0 - n1) <= len(die) // 8
    assert (die[0::2] == die[1::2]).all()          # the two SMs of a CTA pair share a half
    near = np.median(lat[die == 0][:, :], axis=0)  # per line: latency seen from half 0 ...
    far = np.median(lat[die == 1][:, :], axis=0)   # ... and from half 1: one of them is the home half
    assert (np.maximum(near, far) > 1.5 * np.minimum(near, far)).mean() > 0.9


def test_bounded_wait_expires_with_a_status_and_leaves_the_context_usable():
    """Failure detection without a fault: a wait on a barrier nobody arrives on gives up after its
    limit, records (role << 8 | wait) and the kernel ends normally."""
    code, waited = sp.selftest_timeout(20000)                 # 20 ms
    assert code == (3 << 8) | 0x7f
    assert 20000 <= waited < 200000
    assert sp.get_status() == 0                               # the word was cleared
    A, B = synth.make_int_inputs(256, 256, 64, seed=1)        # and the device still computes
    ref, _ = G.gemm_full(A, B)
    got, _ = run_gemm(A, B, sp.ROW_MAJOR, (256, 256), "fp32")
    assert np.array_equal(got, ref)


def test_device_remap_matches_oracle_on_random_grids():
    """Seeded random grids and parameters: the scheduler's device code against the enumerating oracle."""
    rng = np.random.default_rng(2024)
    for _ in range(40):
        Tm, Tn = int(rng.integers(1, 90)), int(rng.integers(1, 90))
        G, X, W = int(rng.integers(1, 20)), int(rng.integers(1, 12)), int(rng.integers(0, 200))
        inner = int(rng.choice([sp.ROW_MAJOR, sp.COL_MAJOR, sp.GROUP_M, sp.GROUP_N, sp.MORTON, sp.HILBERT]))
        axis, inter, serp = int(rng.integers(2)), int(rng.integers(2)), int(rng.integers(2)) * 4
        for scheme, kw in [(sp.GROUP_M, dict(group=G, flags=serp)), (sp.GROUP_N, dict(group=G, flags=serp)),
                           (sp.MORTON, {}), (sp.HILBERT, {}), (sp.HILBERT_RECT, {}), (sp.XCD, dict(num_xcds=X, wave=W, xcd_balanced=1)),
                           (sp.DIE_SPLIT, dict(split_axis=axis, inner_scheme=inner, inner_group=G, interleave=inter, flags=serp))]:
            want = R.tile_map(Tm * 64, Tn * 64, 64, 64, scheme, R.Params(**kw))
            got = sp.tile_map_device(Tm * 64, Tn * 64, 64, 64, scheme, sp.make_params(**kw)).cpu().numpy().tolist()
            assert got == want, (Tm, Tn, scheme, kw)


def test_l2_capacity_probe_sees_the_knee():
    MB = 1 << 20
    rates = sp.probe_l2_capacity([16 * MB, 256 * MB], -1)
    assert rates.shape == (2,) and (rates > 0).all()
    assert rates[0] > 1.3 * rates[1]          # 16 MiB is served from L2, 256 MiB is not
    with pytest.raises(sp.SpError):
        sp.probe_l2_capacity([100], -1)       # not a multiple of 16, below the minimum


def test_gemm_host_pipelined_row_blocks_match_gemm():
    """sp_gemm_host splits tall problems into row blocks to overlap copies with compute: same bits as sp_gemm."""
    M, N, K = 6400, 1024, 520                          # 4 row blocks of 2048 (the last one 256 rows), ragged K
    A, B = synth.make_inputs(M, N, K, "normal", 1.0, seed=31)
    for scheme, kw in [(sp.GROUP_M, dict(group=4)), (sp.HILBERT, {})]:
        p = sp.make_params(tile_m=256, tile_n=256, **kw)
        want = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        sp.gemm(dev_bf16(A), dev_bf16(B), want, scheme, p)
        hA = torch.from_numpy(A.view(np.int16)).pin_memory()
        hB = torch.from_numpy(B.view(np.int16)).pin_memory()
        hC = torch.full((M, N), -1, dtype=torch.int16).pin_memory()
        sp.gemm_host(hA, hB, hC, scheme, p)
        assert np.array_equal(hC.numpy(), want.view(torch.int16).cpu().numpy())
    hC2 = np.full((M, N), -1, dtype=np.int16)          # pageable host memory works too
    sp.gemm_host(A.view(np.int16), B.view(np.int16), hC2, scheme, p)
    assert np.array_equal(hC2, hC.numpy())


def test_small_host_gemm_and_shutdown_then_reuse():
    A, B = synth.make_int_inputs(512, 640, 256, seed=17)
    ref, _ = G.gemm_full(A, B)
    hC = np.zeros((512, 640), dtype=np.float32)
    p = sp.make_params(tile_m=128, tile_n=128, out_dtype=1)
    sp.gemm_host(A.view(np.int16), B.view(np.int16), hC, sp.HILBERT, p)      # below the row-block threshold: one launch
    assert np.array_equal(hC.astype(np.float64), ref)
    torch.cuda.synchronize()
    sp.shutdown()                                                             # caches, staging, streams released
    got, _ = run_gemm(A, B, sp.HILBERT, (128, 128), "fp32")                   # and rebuilt on demand
    assert np.array_equal(got, ref)
    hC[:] = 0
    sp.gemm_host(A.view(np.int16), B.view(np.int16), hC, sp.DIE_SPLIT, sp.make_params(tile_m=128, tile_n=128, out_dtype=1,
                                                                                   inner_scheme=sp.MORTON))
    assert np.array_equal(hC.astype(np.float64), ref)


def test_gemm_launches_replay_from_a_cuda_graph():
    # warm caches first (tile table, status word), then capture three launches on a side stream and replay them
    A, B = synth.make_int_inputs(768, 1024, 512, seed=23)
    ref, _ = G.gemm_full(A, B)
    dA, dB = dev_bf16(A), dev_bf16(B)
    outs = [torch.zeros((768, 1024), dtype=torch.float32, device="cuda") for _ in range(3)]
    cases = [(sp.HILBERT, sp.make_params(tile_m=128, tile_n=128, out_dtype=1)),
             (sp.GROUP_M, sp.make_params(tile_m=256, tile_n=256, out_dtype=1, group=2)),
             (sp.ROW_MAJOR, sp.make_params(tile_m=256, tile_n=512, out_dtype=1))]
    for (scheme, p), o in zip(cases, outs):
        sp.gemm(dA, dB, o, scheme, p)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for (scheme, p), o in zip(cases, outs):
                sp.gemm(dA, dB, o, scheme, p, side)
    for rep in range(3):
        for o in outs:
            o.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        for o in outs:
            assert np.array_equal(o.cpu().numpy().astype(np.float64), ref)
    assert sp.get_status() == 0


def test_host_threads_on_separate_streams():
    """Four host threads, each with its own stream and problem, call the library at the same time (plain, table-based,
    die-pinned when available, k-split and cluster-launch-control launches mixed): every result is exact."""
    import threading
    jobs = []
    flags = [0, sp.FLAG_STREAM_K, sp.FLAG_CLC, 0]
    schemes = [(sp.HILBERT, {}), (sp.GROUP_M, dict(group=4)), (sp.ROW_MAJOR, {}), (sp.DIE_SPLIT, dict(inner_scheme=sp.GROUP_M, inner_group=2))]
    shapes = [(1024, 1280, 512), (2304, 2560, 1024), (1160, 600, 520), (2048, 2304, 256)]
    for i in range(4):
        M, N, K = shapes[i]
        A, B = synth.make_int_inputs(M, N, K, seed=60 + i)
        jobs.append(dict(dA=dev_bf16(A), dB=dev_bf16(B), ref=G.gemm_full(A, B)[0],
                         out=[torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") for _ in range(6)],
                         stream=torch.cuda.Stream(), scheme=schemes[i][0],
                         p=sp.make_params(tile_m=256 if i % 2 else 128, tile_n=256, out_dtype=1, flags=flags[i], **schemes[i][1])))
    torch.cuda.synchronize()
    errors = []

    def work(j):
        try:
            for o in j["out"]:
                sp.gemm(j["dA"], j["dB"], o, j["scheme"], j["p"], j["stream"])
        except Exception as e:      # noqa: BLE001
            errors.append(e)
    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    torch.cuda.synchronize()
    assert sp.get_status() == 0
    for j in jobs:
        for o in j["out"]:
            assert np.array_equal(o.cpu().numpy().astype(np.float64), j["ref"])


def test_very_long_k():
    """Eight tiles at most, 1024 k-blocks: the ring, the phase bits and the accumulation run far longer than in any workload."""
    M, N, K = 256, 512, 65536
    A, B = synth.make_int_inputs(M, N, K, seed=9)
    ref, _ = G.gemm_full(A, B)
    for tile in [(256, 512), (256, 256), (128, 128)]:
        got, _ = run_gemm(A, B, sp.ROW_MAJOR, tile, "fp32")
        assert np.array_equal(got, ref), tile
    got, _ = run_gemm(A, B, sp.ROW_MAJOR, (128, 128), "fp32", flags=sp.FLAG_STREAM_K)     # 8 tiles on 148 units: 8 pieces each
    assert np.array_equal(got, ref)


def test_die_pinned_launches_on_two_streams_at_once():
    """Each die-pinned launch takes its ranks from its own set of counters; two such launches sharing the GPU land on
    whatever SMs are free, and the overflow rule must still hand out every (half, rank) pair of each launch exactly once."""
    M, N, K = 4096, 4608, 512
    A, B = synth.make_int_inputs(M, N, K, seed=31)
    ref, _ = G.gemm_full(A, B)
    dA, dB = dev_bf16(A), dev_bf16(B)
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [[torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda") for _ in range(6)] for _ in streams]
    p = sp.make_params(tile_m=256, tile_n=256, out_dtype=1, split_axis=0, inner_scheme=sp.GROUP_M, inner_group=4, flags=sp.FLAG_DIE_PINNED)
    try:
        sp.gemm(dA, dB, outs[0][0], sp.DIE_SPLIT, p)
    except sp.SpError as e:
        if e.status == sp.ERR_UNSUPPORTED:
            pytest.skip("no two-way L2 structure measured on this device")
        raise
    torch.cuda.synchronize()
    for i in range(6):
        for k, st in enumerate(streams):
            sp.gemm(dA, dB, outs[k][i], sp.DIE_SPLIT, p, st)
    torch.cuda.synchronize()
    assert sp.get_status() == 0
    for k in range(2):
        for o in outs[k]:
            assert np.array_equal(o.cpu().numpy().astype(np.float64), ref)


def test_host_entry_point_from_two_threads():
    import threading
    jobs = []
    for i, (M, N, K) in enumerate([(4608, 1024, 512), (1024, 768, 256)]):
        A, B = synth.make_int_inputs(M, N, K, seed=70 + i)
        jobs.append((A, B, G.gemm_full(A, B)[0], [np.zeros((M, N), dtype=np.float32) for _ in range(3)]))
    errors = []

    def work(j):
        A, B, _, outs = j
        try:
            for o in outs:
                sp.gemm_host(A.view(np.int16), B.view(np.int16), o, sp.GROUP_M, sp.make_params(tile_m=128, tile_n=256, out_dtype=1, group=2),
                             torch.cuda.Stream())
        except Exception as e:      # noqa: BLE001
            errors.append(e)
    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for (_, _, ref, outs) in jobs:
        for o in outs:
            assert np.array_equal(o.astype(np.float64), ref)


def test_table_built_on_one_stream_is_complete_for_the_next_stream():
    """First use of a table order on stream X, and at once the same order on stream Y: the second call finds the
    table in the cache and launches without waiting for X, so the table must have been complete before it was
    published.  Fresh grid shapes (used nowhere else in this suite), so the build really happens here; X is kept busy
    beforehand so that an unfinished build would still be queued when Y's kernel reads the table."""
    sx, sy = torch.cuda.Stream(), torch.cuda.Stream()
    big = torch.empty(1 << 28, dtype=torch.uint8, device="cuda")
    for (M, N, K, tile, scheme, kw) in [(128 * 19, 128 * 23, 264, (128, 128), sp.HILBERT, {}),
                                        (256 * 9, 256 * 11, 200, (256, 256), sp.HILBERT_RECT, {}),
                                        (128 * 21, 256 * 7, 136, (128, 256), sp.DIE_SPLIT, dict(inner_scheme=sp.MORTON))]:
        A, B = synth.make_inputs(M, N, K, "normal", 1.0, seed=31)
        dA, dB = dev_bf16(A), dev_bf16(B)
        want = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        sp.gemm(dA, dB, want, sp.ROW_MAJOR, sp.make_params(tile_m=tile[0], tile_n=tile[1]))
        cx = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        cy = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        p = sp.make_params(tile_m=tile[0], tile_n=tile[1], **kw)
        with torch.cuda.stream(sx):
            for _ in range(8):
                big.fill_(1)                                 # about a millisecond of queued work ahead of the build
        sp.gemm(dA, dB, cx, scheme, p, sx)
        sp.gemm(dA, dB, cy, scheme, p, sy)
        torch.cuda.synchronize()
        assert sp.get_status() == 0
        assert torch.equal(cx.view(torch.int16), want.view(torch.int16))
        assert torch.equal(cy.view(torch.int16), want.view(torch.int16))


@pytest.mark.parametrize("tile", [(128, 128), (128, 256), (256, 256), (256, 512)])
def test_k_alternate_walks_every_k_block_once(tile):
    """SP_FLAG_K_ALTERNATE: odd rounds of a unit take their k-blocks in descending order.  Small integers make every
    partial sum exact, so C must equal the oracle bit for bit whatever the order of the k-blocks -- a k-block loaded
    twice, skipped, or taken from the wrong end of a ragged K shows up as a wrong integer.  Grids with several rounds
    per unit (more tiles than SMs), ragged M, N and K."""
    M, N, K = tile[0] * 13 + 40, tile[1] * 15 + 72, 64 * 9 + 24
    A, B = synth.make_int_inputs(M, N, K, seed=41)
    ref, _ = G.gemm_full(A, B)
    for scheme, kw in [(sp.GROUP_N, dict(group=8)), (sp.HILBERT, {}), (sp.ROW_MAJOR, {})]:
        got, _ = run_gemm(A, B, scheme, tile, out="fp32", flags=sp.FLAG_K_ALTERNATE, **kw)
        assert np.array_equal(got, ref), (scheme, tile)
    got, _ = run_gemm(A, B, sp.GROUP_M, tile, out="fp32", b_is_nk=True, group=4, flags=sp.FLAG_K_ALTERNATE)
    assert np.array_equal(got, ref)


def test_k_alternate_within_tolerance_and_with_the_other_schedulers():
    M, N, K = 256 * 11, 512 * 9 + 128, 1096
    A, B = synth.make_inputs(M, N, K, "normal", 1.0, seed=42)
    ref, S = G.gemm_full(A, B)
    cases = [((256, 512), sp.GROUP_N, dict(group=8, flags=sp.FLAG_K_ALTERNATE)),
             ((256, 256), sp.GROUP_M, dict(group=8, flags=sp.FLAG_K_ALTERNATE | sp.FLAG_STREAM_K)),
             ((256, 256), sp.ROW_MAJOR, dict(flags=sp.FLAG_K_ALTERNATE | sp.FLAG_CLC)),
             ((256, 512), sp.DIE_SPLIT, dict(inner_scheme=sp.GROUP_M, inner_group=4, flags=sp.FLAG_K_ALTERNATE | sp.FLAG_DIE_PINNED))]
    for tile, scheme, kw in cases:
        try:
            got, _ = run_gemm(A, B, scheme, tile, **kw)
        except sp.SpError as err:                     # die-pinned orders need the two-way L2 structure and enough tiles
            assert err.status == sp.ERR_UNSUPPORTED and (kw["flags"] & sp.FLAG_DIE_PINNED)
            continue
        r = G.compare(got, ref, S)
        assert r["max_err"] <= TOL, (tile, scheme, r)


def test_stealing_between_the_die_queues():
    """SP_FLAG_STEAL: each half's slots are handed out by ticket to the units of its L2 half; a unit whose own queue
    is empty takes tickets of the other half.  Every tile must still run exactly once, under the same map, with the
    same bits; on a lopsided grid (half 0 holds two tile rows, half 1 one) units of half 1's die must end up running
    slots of half 0, which the fixed die-pinned assignment never lets them do; and on an even grid nothing needs to
    be stolen in bulk."""
    die, conf, _ = sp.probe_topology()
    if conf < 0.8 or (die < 0).any():
        pytest.skip("no two-way L2 structure measured on this device")
    K = 512
    kw = dict(split_axis=0, inner_scheme=sp.GROUP_N, inner_group=8)
    for (M, N, tile, lopsided) in [(3 * 256, 60 * 256, (256, 256), True), (8 * 256, 40 * 256, (256, 256), False),
                                   (2 * 128 + 40, 80 * 256 + 8, (128, 256), True), (6 * 256, 20 * 512, (256, 512), False)]:
        A, B = synth.make_int_inputs(M, N, K, seed=M + N)
        dA, dB = dev_bf16(A), dev_bf16(B)
        ref = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        sp.gemm(dA, dB, ref, sp.ROW_MAJOR, sp.make_params(tile_m=tile[0], tile_n=tile[1]))
        want = R.tile_map(M, N, tile[0], tile[1], sp.DIE_SPLIT, R.Params(**kw))
        Tm, Tn = -(-M // tile[0]), -(-N // tile[1])
        h0 = len(R.die_split_halves(Tm, Tn, 0, sp.GROUP_N, 8)[0])
        crossed = {}
        for flags in (sp.FLAG_DIE_PINNED, sp.FLAG_DIE_PINNED | sp.FLAG_STEAL):
            p = sp.make_params(tile_m=tile[0], tile_n=tile[1], flags=flags, **kw)
            dC = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
            tr = sp.gemm_trace(dA, dB, dC, sp.DIE_SPLIT, p)
            assert sp.get_status() == 0
            assert torch.equal(dC.view(torch.int16), ref.view(torch.int16))
            assert tr["slot"].tolist() == list(range(Tm * Tn)) and tr["tile"].tolist() == want   # every slot once, same map
            on_die = die[tr["smid"]]
            d0 = int(np.bincount(on_die[:h0], minlength=2).argmax())          # the die that serves half 0
            crossed[flags] = int((on_die[:h0] != d0).sum()) + int((on_die[h0:] == d0).sum())
            # plain launches (not traced) of the same mode, twice: the ticket counters must come back to zero
            for _ in range(2):
                dC.fill_(float("nan"))
                sp.gemm(dA, dB, dC, sp.DIE_SPLIT, p)
                assert sp.get_status() == 0
                assert torch.equal(dC.view(torch.int16), ref.view(torch.int16))
        if lopsided:
            # half 0 has twice the tiles: with tickets the other die's units come over for a good share of them
            assert crossed[sp.FLAG_DIE_PINNED | sp.FLAG_STEAL] >= h0 // 8, crossed
            assert crossed[sp.FLAG_DIE_PINNED | sp.FLAG_STEAL] > crossed[sp.FLAG_DIE_PINNED]
    with pytest.raises(sp.SpError) as e:                                      # a mode of the pinned split only
        sp.gemm(dA, dB, ref, sp.GROUP_M, sp.make_params(tile_m=256, tile_n=256, group=4, flags=sp.FLAG_STEAL))
    assert e.value.status == sp.ERR_INVALID_ARG


def test_flag_combinations_refused_and_accepted():
    """Every clash between flags is refused before anything is launched (C keeps its contents); the combinations that are
    allowed give the oracle's result, exactly (small integers)."""
    M, N, K = 2048, 2560, 192
    A, B = synth.make_int_inputs(M, N, K, seed=77)
    ref, _ = G.gemm_full(A, B)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.full((M, N), 7.0, dtype=torch.float32, device="cuda")
    split = dict(inner_scheme=sp.GROUP_M, inner_group=4)

    def call(scheme, tile=(256, 256), **kw):
        sp.gemm(dA, dB, dC, scheme, sp.make_params(tile_m=tile[0], tile_n=tile[1], out_dtype=1, **kw))

    refused = [(sp.GROUP_M, dict(group=4, flags=sp.FLAG_STEAL)),                                   # a mode of the pinned split
               (sp.GROUP_M, dict(group=4, flags=sp.FLAG_DIE_PINNED)),                              # pinning needs the split order
               (sp.DIE_SPLIT, dict(interleave=1, flags=sp.FLAG_DIE_PINNED, **split)),
               (sp.ROW_MAJOR, dict(flags=sp.FLAG_HINT_A_EVICT_FIRST | sp.FLAG_HINT_A_EVICT_LAST)),
               (sp.ROW_MAJOR, dict(flags=sp.FLAG_HINT_B_EVICT_FIRST | sp.FLAG_HINT_B_EVICT_LAST)),
               (sp.DIE_SPLIT, dict(flags=sp.FLAG_DIE_PINNED | sp.FLAG_CLC, **split)),
               (sp.DIE_SPLIT, dict(flags=sp.FLAG_DIE_PINNED | sp.FLAG_STREAM_K, **split)),
               (sp.DIE_SPLIT, dict(flags=sp.FLAG_DIE_PINNED | sp.FLAG_OVERLAP, **split)),
               (sp.ROW_MAJOR, dict(flags=sp.FLAG_CLC | sp.FLAG_STREAM_K)),
               (sp.ROW_MAJOR, dict(flags=sp.FLAG_OVERLAP | sp.FLAG_STREAM_K))]
    for scheme, kw in refused:
        with pytest.raises(sp.SpError) as e:
            call(scheme, **kw)
        assert e.value.status == sp.ERR_INVALID_ARG, (scheme, kw)
    with pytest.raises(sp.SpError) as e:
        call(sp.ROW_MAJOR, tile=(256, 512), flags=sp.FLAG_STREAM_K)
    assert e.value.status == sp.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert bool((dC == 7.0).all())                                                                  # nothing ran

    mem = sp.FLAG_K_ALTERNATE | sp.FLAG_HINT_C_EVICT_FIRST | sp.FLAG_HINT_A_EVICT_LAST | sp.FLAG_HINT_B_EVICT_FIRST
    accepted = [(sp.GROUP_N, (256, 512), dict(group=2, flags=mem | sp.FLAG_SERPENTINE)),
                (sp.GROUP_M, (256, 256), dict(group=2, flags=mem | sp.FLAG_STREAM_K)),
                (sp.HILBERT, (128, 256), dict(flags=mem | sp.FLAG_CLC)),
                (sp.ROW_MAJOR, (128, 128), dict(flags=mem | sp.FLAG_OVERLAP)),
                (sp.DIE_SPLIT, (128, 256), dict(flags=mem | sp.FLAG_SERPENTINE | sp.FLAG_DIE_PINNED | sp.FLAG_STEAL, **split)),
                (sp.DIE_SPLIT, (256, 128), dict(flags=mem | sp.FLAG_DIE_PINNED, **split))]
    for scheme, tile, kw in accepted:
        dC.fill_(float("nan"))
        try:
            call(scheme, tile=tile, **kw)
        except sp.SpError as err:                      # die-pinned modes need the two-way L2 structure
            assert err.status == sp.ERR_UNSUPPORTED and (kw["flags"] & sp.FLAG_DIE_PINNED)
            continue
        assert sp.get_status() == 0
        assert np.array_equal(dC.cpu().numpy().astype(np.float64), ref), (scheme, tile, kw)
