"""SP_FLAG_CLC: slots handed out by cluster launch control.  Same GEMM, same bits; every tile exactly once; the
clusters that run start on the slot of their own index and take over slots of clusters that never started."""

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import gemm as G
from paper_2508_20258_b200 import synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
CLC = sp.FLAG_CLC


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("tile", [(128, 128), (128, 256), (256, 128), (256, 256), (256, 512)])
@pytest.mark.parametrize("M,N,K", [(512, 512, 512), (2304, 2560, 1024), (2000, 1096, 840), (128 * 37, 128 * 5, 192)])
def test_integer_inputs_are_exact_under_dynamic_scheduling(tile, M, N, K):
    A, B = synth.make_int_inputs(M, N, K, seed=13)
    ref, _ = G.gemm_full(A, B)
    dA, dB = dev_bf16(A), dev_bf16(B)
    for scheme, kw in [(sp.ROW_MAJOR, {}), (sp.HILBERT, {}), (sp.GROUP_N, dict(group=3))]:
        for b_nk in (0, 1):
            dBx = dev_bf16(np.ascontiguousarray(B.T)) if b_nk else dB
            dC = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
            sp.gemm(dA, dBx, dC, scheme, sp.make_params(tile_m=tile[0], tile_n=tile[1], out_dtype=1, b_layout=b_nk, flags=CLC, **kw))
            assert sp.get_status() == 0
            assert np.array_equal(dC.cpu().numpy().astype(np.float64), ref), (scheme, kw, b_nk)


def test_same_bits_as_the_static_schedule_on_random_inputs():
    w, A, B = synth.make_workload("cfg2")
    dA, dB = dev_bf16(A), dev_bf16(B)
    outs = []
    for flags in (0, CLC, CLC | sp.FLAG_OVERLAP):
        dC = torch.full((w.M, w.N), float("nan"), dtype=torch.bfloat16, device="cuda")
        for _ in range(3):
            sp.gemm(dA, dB, dC, sp.GROUP_M, sp.make_params(tile_m=256, tile_n=512, group=4, flags=flags))
        assert sp.get_status() == 0
        outs.append(dC.view(torch.int16).cpu().numpy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])


@pytest.mark.parametrize("tile", [(256, 256), (128, 256), (256, 512)])
def test_trace_every_slot_once_and_clusters_start_on_their_own_slot(tile):
    M, N, K = 4096, 4096, 1024
    A, B = synth.make_int_inputs(M, N, K, seed=2)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    p = sp.make_params(tile_m=tile[0], tile_n=tile[1], group=4, flags=CLC)
    tr = sp.gemm_trace(dA, dB, dC, sp.GROUP_M, p)
    perm = sp.tile_map(M, N, tile[0], tile[1], sp.GROUP_M, p)
    T = len(perm)
    assert np.array_equal(tr["slot"], np.arange(T))          # record s was written, by whoever ran slot s
    assert np.array_equal(tr["tile"], perm)
    ran = np.unique(tr["unit"])                               # indices of the clusters that actually started
    resident = sp.gemm_units(tile[0], tile[1], 1 << 24)
    assert len(ran) <= resident < T                           # the rest were cancelled before they started
    for u in ran:
        mine = tr[tr["unit"] == u]
        first = mine[np.argmin(mine["t_begin"])]
        assert first["slot"] == u                             # a cluster's first slot is its own index
    assert sorted(np.bincount(tr["unit"])[ran].tolist())[0] >= 1
    assert len(np.unique(tr["smid"])) <= resident


def test_clc_rejections_and_host_entry_point():
    A, B = synth.make_int_inputs(2304, 2560, 512, seed=1)
    ref, _ = G.gemm_full(A, B)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.zeros((2304, 2560), dtype=torch.bfloat16, device="cuda")
    for bad in (CLC | sp.FLAG_STREAM_K, CLC | sp.FLAG_DIE_PINNED):
        with pytest.raises(sp.SpError) as e:
            sp.gemm(dA, dB, dC, sp.DIE_SPLIT, sp.make_params(tile_m=128, tile_n=128, inner_scheme=sp.ROW_MAJOR, flags=bad))
        assert e.value.status == sp.ERR_INVALID_ARG
    with pytest.raises(sp.SpError) as e:
        sp.gemm_noalloc(dA, dB, dC, sp.ROW_MAJOR, sp.make_params(tile_m=128, tile_n=128, flags=CLC))
    assert e.value.status == sp.ERR_INVALID_ARG
    assert sp.get_status() == 0 and float(dC.float().abs().sum()) == 0.0
    hC = np.zeros((2304, 2560), dtype=np.float32)
    sp.gemm_host(A.view(np.int16), B.view(np.int16), hC, sp.MORTON, sp.make_params(tile_m=256, tile_n=256, out_dtype=1, flags=CLC))
    assert np.array_equal(hC.astype(np.float64), ref)
