"""The reader of the profiler's CSV, on a small hand-written file in the profiler's format (tests/golden/ncu_small.csv:
a table builder launch and three GEMM launches with units as the profiler prints them: Mbyte / byte, us / ms, hz / Ghz,
thousands separators, '==PROF==' lines around the table): unit conversion, launch list, per-order table, the paper's
ranking (L2 hit rate first, time second), the traffic table, and the answer when there is no table at all."""

import json
import os

import pytest

from paper_2508_20258_b200 import ncuparse as NP


@pytest.fixture()
def csv_path(golden_dir):
    return os.path.join(golden_dir, "ncu_small.csv")


def test_launches_and_unit_conversion(csv_path):
    ls = NP.launches(csv_path)
    assert [l["id"] for l in ls] == [0, 1, 2, 3]
    assert NP.short_kernel_name(ls[1]["kernel"]) == "sp::gemm_kernel<2, 512, 0, 0, 0>"
    m1, m2 = ls[1]["metrics"], ls[2]["metrics"]
    assert m1["dram__bytes_read.sum"] == 1097.5e6 and m2["dram__bytes_read.sum"] == 655e6      # "1,097.5" Mbyte; plain bytes
    assert m2["gpu__time_duration.sum"] == pytest.approx(659.0) and m1["gpu__time_duration.sum"] == 678.0   # ms -> us
    assert m1["sm__cycles_elapsed.avg.per_second"] == pytest.approx(1.44) and m2["sm__cycles_elapsed.avg.per_second"] == 1.48


def test_launch_list_shares(csv_path):
    rows = NP.launch_list(csv_path)
    assert [r["kernel"] for r in rows] == ["sp::gemm_kernel<2, 512, 0, 0, 0>", "sp::build_perm_kernel"]
    assert rows[0]["launches"] == 3 and rows[0]["total_us"] == pytest.approx(678.0 + 659.0 + 667.0)
    assert sum(r["share"] for r in rows) == pytest.approx(1.0) and rows[1]["share"] == pytest.approx(3.2 / 2007.2)


def test_per_order_table_ranking_and_markdown(csv_path):
    order = ["row_major", "die_split:m:group_m:8:p:s+a+hc", "group_n:8"]
    rows = NP.per_launch_table(csv_path, order)            # the table builder's launch is not a GEMM launch
    assert [r["scheme"] for r in rows] == order
    assert rows[0]["dram_bytes"] == 1227.5e6 and rows[1]["l2_hit_pct"] == 78.9 and rows[2]["time_us"] == 667.0
    ranked = NP.rank_by_l2(rows)
    # 78.9 and 78.94 tie at one decimal: time decides (659 < 667); row-major is last
    assert [r["scheme"] for r in ranked] == [order[1], order[2], order[0]]
    md = NP.markdown(rows, {"row_major": {"tflops": 1356.0, "speedup_vs_first": 1.0}})
    assert "| row_major | 67.6 | +0.0 (+0 %)" in md and "+11.3 (+17 %)" in md and "| 1356 | 1.000 |" in md
    with pytest.raises(ValueError):
        NP.per_launch_table(csv_path, order[:2])          # three launches cannot be two orders


def test_traffic_table_round_trip(csv_path, tmp_path):
    path = str(tmp_path / "traffic.json")
    rows = NP.per_launch_table(csv_path, ["a", "b", "c"])
    assert NP.update_traffic(rows, "cfg3", "256x512", "2026-01-01", "ncu ...", path) == 3
    assert NP.update_traffic(rows[:1], "cfg3", "256x512", "2026-01-02", "ncu again", path) == 1     # replaces, does not append
    table = json.load(open(path))["captures"]
    assert len(table) == 3 and {c["scheme"] for c in table} == {"a", "b", "c"}
    a = next(c for c in table if c["scheme"] == "a")
    assert a["captured"] == "2026-01-02" and a["dram_bytes"] == 1227.5e6 and a["command"] == "ncu again"


def test_a_log_without_a_table_is_reported_as_unavailable(tmp_path):
    p = tmp_path / "closed.csv"
    p.write_text("==ERROR== profiling is closed on this pool\n")
    with pytest.raises(NP.NcuUnavailable) as e:
        NP.launches(str(p))
    assert "closed on this pool" in str(e.value)


def test_committed_traffic_table_covers_what_the_benchmark_times_by_default():
    import bench
    table = {(c["workload"], c["tile"], c["scheme"]) for c in NP.load_traffic()["captures"]}
    for w in ("cfg3", "cfg5"):
        tile = bench.DEFAULT_TILE[w]
        assert (w, tile, bench.DEFAULT_SCHEME_BY_TILE[(w, tile)]) in table
        assert (w, tile, bench.FALLBACK_SCHEME_BY_TILE[(w, tile)]) in table
