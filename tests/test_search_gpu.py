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
