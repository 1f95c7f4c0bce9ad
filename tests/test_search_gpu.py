"""The enumerative search loop: broken remaps are recorded as failures, valid ones are checked
against the ground truth and ranked, the best is a validated candidate."""

import pytest

import paper_2508_20258_b200 as sp
from paper_2508_20258_b200 import search

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def test_search_loop_validates_ranks_and_keeps_history():
    M, N, K = 4096, 5120, 512                     # 16 x 20 tiles of 256 x 256
    g = torch.Generator(device="cuda").manual_seed(1)
    A = torch.randn((M, K), device="cuda", generator=g).bfloat16()
    B = torch.randn((K, N), device="cuda", generator=g).bfloat16()
    C = torch.empty((M, N), device="cuda", dtype=torch.bfloat16)
    cands = [("row_major", sp.ROW_MAJOR, {}), ("group_m:4", sp.GROUP_M, dict(group=4)), ("hilbert", sp.HILBERT, {}),
             ("xcd:4:74:literal", sp.XCD, dict(num_xcds=4, wave=74, xcd_balanced=0)),       # 74 = 19+19+18+18: reaches 74
             ("xcd:2:74", sp.XCD, dict(num_xcds=2, wave=74, xcd_balanced=1)),
             ("custom:dup", sp.CUSTOM, dict(custom_perm=[0] * 320))]
    r = search.search(A, B, C, (256, 256), cands, launches=5)
    by = {h.name: h for h in r.history}
    assert [h.name for h in r.history] == [c[0] for c in cands]
    assert by["xcd:4:74:literal"].status == "broken" and by["custom:dup"].status == "broken"
    ok = [h for h in r.history if h.status == "ok"]
    assert {h.name for h in ok} == {"row_major", "group_m:4", "hilbert", "xcd:2:74"}
    assert all(h.ms > 0 and h.tflops > 0 for h in ok) and by["row_major"].speedup == 1.0
    assert r.best is not None and r.best.status == "ok" and r.best.ms == min(h.ms for h in ok)
    assert len(search.default_candidates(74)) > 20


def test_recommended_configuration_runs_and_beats_the_smallest_tile():
    import numpy as np
    from oracle import gemm as G
    from paper_2508_20258_b200 import synth
    M, N, K = 4096, 6144, 2048
    A, B = synth.make_int_inputs(M, N, K, seed=4)
    dA = torch.from_numpy(A.view(np.int16)).cuda().view(torch.bfloat16)
    dB = torch.from_numpy(B.view(np.int16)).cuda().view(torch.bfloat16)
    dC = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    scheme, p = sp.recommend(M, N, K)
    sp.gemm(dA, dB, dC, scheme, p)
    assert sp.get_status() == 0
    rows = [0, 255, 256, 2047, M - 1]
    ref, _ = G.gemm_rows(A, B, rows)
    want = G.bf16_bits_to_f64(synth.f32_to_bf16_bits(ref.astype(np.float32)))
    assert np.array_equal(G.bf16_bits_to_f64(dC[rows].view(torch.int16).cpu().numpy().view(np.uint16)), want)

    def timed(s_, p_):
        for _ in range(5):
            sp.gemm(dA, dB, dC, s_, p_)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(50):
            sp.gemm(dA, dB, dC, s_, p_)
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1)
    small = timed(sp.ROW_MAJOR, sp.make_params(tile_m=128, tile_n=128))
    assert timed(scheme, p) < small / 1.2
