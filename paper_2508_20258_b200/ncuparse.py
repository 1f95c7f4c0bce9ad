"""Reads the CSV that `ncu --csv --log-file FILE` writes and turns it into the tables this package reports.

Three uses, all from one parser:

* `launches(path)` / `launch_list(path)` -- every captured launch with its metrics; per kernel the number of launches,
  the total time and the share of the total (the launch list of a benchmark command).
* `per_launch_table(path, order)` -- one row per launch of the GEMM kernel, labelled by the tile order that launch ran
  under (the order list is what `bench.py --profile-sweep` prints): L2 hit rate, DRAM bytes, duration.  This is what
  the search loop ranks by and what the per-scheme tables are made of.
* `update_traffic(...)` -- stores DRAM bytes per launch for (workload, tile, order) in `ncu_traffic.json` beside this
  file, with the capture's command and date; `bench.py` reports them as `roofline.traffic`.

Command line:

    python -m paper_2508_20258_b200.ncuparse --launch-list launches.csv
    python -m paper_2508_20258_b200.ncuparse --sweep l2sweep.csv --order plain.log [--markdown [--sustained sweep.jsonl]]
    python -m paper_2508_20258_b200.ncuparse --sweep l2sweep.csv --order plain.log --traffic \
        --workload cfg3 --tile 256x512 --date 2026-11-25 --command "ncu ... python bench.py --profile-sweep ..."

Nothing here runs a profiler or touches a GPU; it only reads text.
"""

from __future__ import annotations

import argparse
import csv
import json
import os
import sys
from collections import OrderedDict
from typing import Dict, List, Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
TRAFFIC_PATH = os.path.join(HERE, "ncu_traffic.json")

_TIME_TO_US = {"ns": 1e-3, "nsecond": 1e-3, "us": 1.0, "usecond": 1.0, "ms": 1e3, "msecond": 1e3, "s": 1e6, "second": 1e6}
_BYTES = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12}
_TO_GHZ = {"hz": 1e-9, "khz": 1e-6, "mhz": 1e-3, "ghz": 1.0}


class NcuUnavailable(RuntimeError):
    """The profiler answered that it may not be used here (or produced no table)."""


def _number(text: str) -> float:
    return float(text.replace(",", ""))


def launches(path: str) -> List[Dict]:
    """Captured launches in capture order: {"id", "kernel", "metrics": {name: value}, "units": {name: unit}}.
    Durations are converted to microseconds and byte counts to bytes, frequencies to GHz; other values are kept as printed."""
    with open(path, newline="") as fh:
        lines = [l for l in fh if l.startswith('"')]
    if not lines:
        with open(path) as fh:
            head = fh.read(2000)
        raise NcuUnavailable(f"no metric table in {path}: {head.strip()[:300]!r}")
    rows = list(csv.reader(lines))
    hdr = rows[0]
    need = ["ID", "Kernel Name", "Metric Name", "Metric Unit", "Metric Value"]
    if any(c not in hdr for c in need):
        raise NcuUnavailable(f"unexpected header in {path}: {hdr}")
    iid, ik, im, iu, iv = (hdr.index(c) for c in need)
    out: "OrderedDict[str, Dict]" = OrderedDict()
    for r in rows[1:]:
        if len(r) <= iv:
            continue
        rec = out.setdefault(r[iid], {"id": int(r[iid]), "kernel": r[ik], "metrics": {}, "units": {}})
        name, unit = r[im], r[iu]
        try:
            val = _number(r[iv])
        except ValueError:
            continue
        if unit in _TIME_TO_US:
            val, unit = val * _TIME_TO_US[unit], "us"
        elif unit in _BYTES:
            val, unit = val * _BYTES[unit], "byte"
        elif unit.lower() in _TO_GHZ:
            val, unit = val * _TO_GHZ[unit.lower()], "Ghz"
        rec["metrics"][name] = val
        rec["units"][name] = unit
    return list(out.values())


def short_kernel_name(name: str) -> str:
    """'void sp::gemm_kernel<2, 512, 0, 0>(CUtensorMap_st, ...)' -> 'sp::gemm_kernel<2, 512, 0, 0>'."""
    n = name.split("(")[0].strip()
    return n[5:] if n.startswith("void ") else n


def launch_list(path: str) -> List[Dict]:
    """Per kernel: launches, total microseconds (gpu__time_duration.sum) and share of the total, largest first."""
    agg: "OrderedDict[str, List[float]]" = OrderedDict()
    for l in launches(path):
        t = l["metrics"].get("gpu__time_duration.sum")
        if t is None:
            continue
        a = agg.setdefault(short_kernel_name(l["kernel"]), [0, 0.0])
        a[0] += 1
        a[1] += t
    total = sum(a[1] for a in agg.values()) or 1.0
    rows = [{"kernel": k, "launches": int(n), "total_us": us, "share": us / total} for k, (n, us) in agg.items()]
    return sorted(rows, key=lambda r: -r["total_us"])


def read_order(path: str) -> Dict:
    """The JSON line `bench.py --profile-sweep` prints: {"profile_sweep": W, "tile": "MxN", "launch_order": [...]}."""
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if line.startswith("{") and "launch_order" in line:
                return json.loads(line)
    raise ValueError(f"no launch_order line in {path}")


def per_launch_table(path: str, order: Sequence[str], kernel_substr: str = "gemm_kernel") -> List[Dict]:
    """One row per launch of the kernel, labelled with order[i] for the i-th such launch.  A capture holds either one
    launch per order or a whole number of repeats of the list (the last repeat wins)."""
    ls = [l for l in launches(path) if kernel_substr in l["kernel"]]
    if not ls or len(ls) % len(order) != 0:
        raise ValueError(f"{len(ls)} launches of {kernel_substr} for {len(order)} orders in {path}")
    ls = ls[-len(order):]
    rows = []
    for spec, l in zip(order, ls):
        m = l["metrics"]
        rd, wr = m.get("dram__bytes_read.sum"), m.get("dram__bytes_write.sum")
        rows.append({
            "scheme": spec, "kernel": short_kernel_name(l["kernel"]),
            "l2_hit_pct": m.get("lts__t_sector_hit_rate.pct"),
            "l2_read_hit_pct": m.get("lts__t_sector_op_read_hit_rate.pct"),
            "dram_read_bytes": rd, "dram_write_bytes": wr,
            "dram_bytes": (rd + wr) if rd is not None and wr is not None else None,
            "time_us": m.get("gpu__time_duration.sum"),
            "sm_ghz": m.get("sm__cycles_elapsed.avg.per_second"),
            "tensor_active_pct": m.get("sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active"),
            "l2_sectors": m.get("lts__t_sectors.sum"),
            "l2_to_sm_bytes": m.get("l1tex__m_xbar2l1tex_read_bytes.sum"),
        })
    return rows


def rank_by_l2(rows: Sequence[Dict]) -> List[Dict]:
    """The paper's ranking: L2 hit rate first (higher is better), time second (lower is better)."""
    usable = [r for r in rows if r.get("l2_hit_pct") is not None]
    return sorted(usable, key=lambda r: (-round(r["l2_hit_pct"], 1), r.get("time_us") or float("inf")))


def read_sustained(path: str) -> Dict[str, Dict]:
    """The JSON lines of `bench.py --sweep-sustained`: scheme -> {"tflops", "speedup_vs_first"}."""
    out: Dict[str, Dict] = {}
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if line.startswith("{") and "sweep_sustained" in line:
                j = json.loads(line)
                out[j["scheme"]] = {"tflops": j["tflops"], "speedup_vs_first": j["speedup_vs_first"]}
    return out


def markdown(rows: Sequence[Dict], sustained: Optional[Dict[str, Dict]] = None) -> str:
    base = next((r for r in rows if r["scheme"] == "row_major"), rows[0] if rows else None)
    out = ["| scheme | L2 hit % | dL2 vs first/row-major | read hit % | DRAM rd MB | DRAM wr MB | ncu us | SM GHz | tensor % |"
           + (" sustained TF | x first |" if sustained else ""),
           "|---|---|---|---|---|---|---|---|---|" + ("---|---|" if sustained else "")]

    def f(v, spec="{:.1f}"):
        return "-" if v is None else spec.format(v)
    for r in rows:
        d = None
        if base and r.get("l2_hit_pct") is not None and base.get("l2_hit_pct"):
            d = f"{r['l2_hit_pct'] - base['l2_hit_pct']:+.1f} ({100 * (r['l2_hit_pct'] / base['l2_hit_pct'] - 1):+.0f} %)"
        out.append(f"| {r['scheme']} | {f(r['l2_hit_pct'])} | {d or '-'} | {f(r['l2_read_hit_pct'])} | "
                   f"{f(r['dram_read_bytes'] and r['dram_read_bytes'] / 1e6, '{:.0f}')} | "
                   f"{f(r['dram_write_bytes'] and r['dram_write_bytes'] / 1e6, '{:.0f}')} | {f(r['time_us'], '{:.0f}')} | "
                   f"{f(r['sm_ghz'], '{:.2f}')} | {f(r['tensor_active_pct'])} |"
                   + ((f" {f(sustained.get(r['scheme'], {}).get('tflops'), '{:.0f}')} |"
                       f" {f(sustained.get(r['scheme'], {}).get('speedup_vs_first'), '{:.3f}')} |") if sustained else ""))
    return "\n".join(out)


def load_traffic(path: str = TRAFFIC_PATH) -> Dict:
    if not os.path.exists(path):
        return {"captures": []}
    with open(path) as fh:
        return json.load(fh)


def update_traffic(rows: Sequence[Dict], workload: str, tile: str, date: str, command: str, path: str = TRAFFIC_PATH) -> int:
    """Adds or replaces the entries (workload, tile, scheme) for every row that has DRAM counters."""
    table = load_traffic(path)
    keep = {(c["workload"], c["tile"], c["scheme"]): c for c in table["captures"]}
    n = 0
    for r in rows:
        if r.get("dram_bytes") is None:
            continue
        keep[(workload, tile, r["scheme"])] = {
            "workload": workload, "tile": tile, "scheme": r["scheme"], "dram_read_bytes": r["dram_read_bytes"],
            "dram_write_bytes": r["dram_write_bytes"], "dram_bytes": r["dram_bytes"], "l2_hit_pct": r.get("l2_hit_pct"),
            "time_us": r.get("time_us"), "captured": date, "command": command}
        n += 1
    table["captures"] = sorted(keep.values(), key=lambda c: (c["workload"], c["tile"], c["scheme"]))
    with open(path, "w") as fh:
        json.dump(table, fh, indent=1)
        fh.write("\n")
    return n


def main(argv: Optional[Sequence[str]] = None) -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--launch-list", metavar="CSV")
    ap.add_argument("--sweep", metavar="CSV")
    ap.add_argument("--order", metavar="LOG", help="output of the same command run without the profiler (holds the launch order)")
    ap.add_argument("--sustained", metavar="JSONL", help="output of bench.py --sweep-sustained: adds its columns to the table")
    ap.add_argument("--kernel", default="gemm_kernel")
    ap.add_argument("--markdown", action="store_true")
    ap.add_argument("--traffic", action="store_true", help="store DRAM bytes per (workload, tile, order) in ncu_traffic.json")
    ap.add_argument("--workload")
    ap.add_argument("--tile")
    ap.add_argument("--date")
    ap.add_argument("--command")
    a = ap.parse_args(argv)
    if a.launch_list:
        rows = launch_list(a.launch_list)
        print("| kernel | launches | total ms | share |\n|---|---|---|---|")
        for r in rows:
            print(f"| `{r['kernel']}` | {r['launches']} | {r['total_us'] / 1e3:.3f} | {100 * r['share']:.2f} % |")
        return 0
    if a.sweep:
        if not a.order:
            ap.error("--sweep needs --order")
        o = read_order(a.order)
        rows = per_launch_table(a.sweep, o["launch_order"], a.kernel)
        if a.traffic:
            if not (a.date and a.command):
                ap.error("--traffic needs --date and --command")
            n = update_traffic(rows, a.workload or o["profile_sweep"], a.tile or o["tile"], a.date, a.command)
            print(f"{n} entries written to {TRAFFIC_PATH}")
        if a.markdown or not a.traffic:
            print(markdown(rows, read_sustained(a.sustained) if a.sustained else None) if a.markdown else json.dumps(rows, indent=1))
        return 0
    ap.error("nothing to do")
    return 2


if __name__ == "__main__":
    sys.exit(main())
