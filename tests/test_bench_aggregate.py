"""The multi-rank bookkeeping of the benchmark (max of times, sum of work) under gloo, world size 2."""

import os
import socket
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2508_20258_b200 import benchutil
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    agg = benchutil.aggregate(10.0 + 5.0 * rank, 100.0 * (rank + 1), world)
    out[rank] = (agg["ms"], agg["units"])
    dist.destroy_process_group()


def test_aggregate_two_ranks():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
        assert out[0] == out[1] == (15.0, 300.0)


def test_aggregate_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2508_20258_b200 import benchutil
    assert benchutil.aggregate(3.0, 7.0, 1) == {"ms": 3.0, "units": 7.0}
    p = benchutil.measured_peaks(ROOT)
    assert p["bf16_tflops"] > 0 and p["source"] in ("measured", "fallback")


def test_scheme_specs_parse():
    sys.path.insert(0, ROOT)
    import bench
    import paper_2508_20258_b200 as sp
    assert bench.parse_scheme("group_m:8") == (sp.GROUP_M, dict(group=8))
    assert bench.parse_scheme("xcd:2:74") == (sp.XCD, dict(num_xcds=2, wave=74, xcd_balanced=1))
    assert bench.parse_scheme("die_split:n:group_m:8:i") == (
        sp.DIE_SPLIT, dict(split_axis=1, inner_scheme=sp.GROUP_M, inner_group=8, interleave=1))
    assert bench.parse_scheme("die_split:m:group_m:8:p")[1]["flags"] == 2
    for name, specs in bench.SWEEPS.items():
        for s in specs:
            bench.parse_scheme(s)


def test_scheme_specs_parse_to_library_parameters():
    import bench
    import paper_2508_20258_b200 as sp
    assert bench.parse_scheme("row_major") == (sp.ROW_MAJOR, {})
    assert bench.parse_scheme("hilbert_rect") == (sp.HILBERT_RECT, {})
    assert bench.parse_scheme("group_n:8:s") == (sp.GROUP_N, dict(group=8, flags=sp.FLAG_SERPENTINE))
    assert bench.parse_scheme("xcd:8:148") == (sp.XCD, dict(num_xcds=8, wave=148, xcd_balanced=1))
    s, kw = bench.parse_scheme("die_split:n:group_m:4:i:p")
    assert s == sp.DIE_SPLIT and kw == dict(split_axis=1, inner_scheme=sp.GROUP_M, inner_group=4, interleave=1, flags=sp.FLAG_DIE_PINNED)
    for suffix, flag in (("+k", sp.FLAG_STREAM_K), ("+o", sp.FLAG_OVERLAP), ("+c", sp.FLAG_CLC)):
        s, kw = bench.parse_scheme("group_m:8" + suffix)
        assert s == sp.GROUP_M and kw == dict(group=8, flags=flag)
    # every spec of every sweep list is understood and, on its workload's grid, a bijection (or refused as documented)
    from paper_2508_20258_b200 import synth
    for name, specs in bench.SWEEPS.items():
        w = synth.WORKLOADS[name]
        for spec in specs:
            s, kw = bench.parse_scheme(spec)
            perm = sp.tile_map(w.M, w.N, w.tile_m, w.tile_n, s, sp.make_params(**kw))
            assert sorted(perm) == list(range(len(perm))), (name, spec)
