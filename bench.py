#!/usr/bin/env python
"""Benchmark of the swizzled tiled GEMM on B200.

A step is one pass of the whole hot path (remap -> TMA producer -> tcgen05 mainloop ->
epilogue, one kernel launch) over one synthetic GEMM.  The default workload is the
8192^3 bf16 GEMM with 256x256 CTA-pair tiles, the configuration the throughput target is
quoted on.  One JSON line is printed by rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                  [--workload cfg1..cfg5] [--scheme SPEC] [--tile MxN] [--kernel-only] [--sweep]

With N > 1 (under torchrun) every rank runs an independent replica of the same GEMM on
its own GPU: the path has no exchange step, so no collective touches the data.
"""

from __future__ import annotations

import argparse
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2508_20258_b200 import benchutil, synth  # noqa: E402

L2_BYTES = 126 * 2 ** 20



def captured_traffic(workload: str, tile: str, spec: str):
    """DRAM bytes per launch of the GEMM kernel for (workload, tile, order), from the table of profiler captures kept
    beside the package (written by `python -m paper_2508_20258_b200.ncuparse --traffic`); None when that combination
    was never captured."""
    path = os.path.join(ROOT, "paper_2508_20258_b200", "ncu_traffic.json")
    with open(path) as fh:
        for rec in json.load(fh)["captures"]:
            if (rec["workload"], rec["tile"], rec["scheme"]) == (workload, tile, spec):
                return rec
    return None


def parse_scheme(spec: str):
    """'group_m:8' -> (scheme id, keyword dict for make_params)."""
    import paper_2508_20258_b200 as sp
    if spec.endswith("+k"):    # any order + stream-K split of the tail wave
        scheme, kw = parse_scheme(spec[:-2])
        kw["flags"] = kw.get("flags", 0) | sp.FLAG_STREAM_K
        return scheme, kw
    if spec.endswith("+c"):    # any order, slots handed out by cluster launch control instead of a fixed stride
        scheme, kw = parse_scheme(spec[:-2])
        kw["flags"] = kw.get("flags", 0) | sp.FLAG_CLC
        return scheme, kw
    for suffix, bit in (("+hc", 128), ("+ha", 256), ("+hb", 512), ("+ka", 1024), ("+kb", 2048)):
        if spec.endswith(suffix):    # L2 eviction hints: C / A / B evict_first, A / B evict_last
            scheme, kw = parse_scheme(spec[:-len(suffix)])
            kw["flags"] = kw.get("flags", 0) | bit
            return scheme, kw
    if spec.endswith("+a"):    # any order, every other tile of a unit walks K from the far end
        scheme, kw = parse_scheme(spec[:-2])
        kw["flags"] = kw.get("flags", 0) | sp.FLAG_K_ALTERNATE
        return scheme, kw
    if spec.endswith("+o"):    # any order, launches declared independent of their predecessor (they overlap its tail)
        scheme, kw = parse_scheme(spec[:-2])
        kw["flags"] = kw.get("flags", 0) | sp.FLAG_OVERLAP
        return scheme, kw
    a = spec.split(":")
    name = a[0]
    if name == "row_major":
        return sp.ROW_MAJOR, {}
    if name == "col_major":
        return sp.COL_MAJOR, {}
    if name == "group_m":      # group_m:G[:s]   (s = serpentine bands)
        return sp.GROUP_M, dict(group=int(a[1]), **({"flags": 4} if "s" in a[2:] else {}))
    if name == "group_n":
        return sp.GROUP_N, dict(group=int(a[1]), **({"flags": 4} if "s" in a[2:] else {}))
    if name == "morton":
        return sp.MORTON, {}
    if name == "hilbert":
        return sp.HILBERT, {}
    if name == "hilbert_rect":
        return sp.HILBERT_RECT, {}
    if name == "xcd":      # xcd:X[:W]  (balanced form)
        return sp.XCD, dict(num_xcds=int(a[1]), wave=int(a[2]) if len(a) > 2 else 0, xcd_balanced=1)
    if name == "die_split":  # die_split:{m|n}:inner[:G][:i][:p][:s]
        inner = {"row_major": sp.ROW_MAJOR, "col_major": sp.COL_MAJOR, "group_m": sp.GROUP_M, "group_n": sp.GROUP_N,
                 "morton": sp.MORTON, "hilbert": sp.HILBERT}[a[2]]
        rest = a[3:]
        inter = int("i" in rest)
        g = [int(v) for v in rest if v.isdigit()]
        kw = dict(split_axis=int(a[1] == "n"), inner_scheme=inner, inner_group=g[0] if g else 1, interleave=inter)
        # p: units pinned to their L2 half; s: serpentine; t: per-half ticket queues with stealing (with p)
        flags = (2 if "p" in rest else 0) | (4 if "s" in rest else 0) | (4096 if "t" in rest else 0)
        if flags:
            kw["flags"] = flags
        return sp.DIE_SPLIT, kw
    raise ValueError(f"unknown scheme spec {spec!r}")


SWEEPS = {
    "cfg1": ["row_major", "group_m:2"],
    "cfg2": ["row_major", "group_m:4", "group_m:8", "group_m:16", "hilbert"],
    "cfg3": ["row_major", "col_major", "group_m:2", "group_m:4", "group_m:8", "group_m:16", "group_n:2", "group_n:4",
             "group_n:8", "group_n:16", "morton", "hilbert", "xcd:2:74", "xcd:2", "die_split:m:group_m:8",
             "die_split:n:group_m:8", "die_split:m:hilbert", "die_split:n:hilbert", "die_split:m:group_m:8:i",
             "die_split:m:group_m:8:p", "die_split:n:group_m:8:p", "die_split:m:group_m:4:p", "die_split:n:group_n:4:p",
             "die_split:m:hilbert:p", "die_split:m:group_n:8:p", "die_split:n:group_n:8:p", "die_split:m:group_m:16:p",
             "group_m:8:s", "group_m:8+a", "group_m:8:s+a", "group_n:8:s+a", "group_m:16:s+a", "group_m:8:s+a+hc",
             "die_split:m:group_m:8:p:s+a", "die_split:m:group_m:8:p:s+a+hc", "die_split:n:group_n:4:p:s+a+hc",
             "die_split:m:group_m:8:p:t:s+a+hc"],
    "cfg4": [f"group_m:{g}" for g in (1, 2, 4, 8, 16, 32, 64)] + [f"group_n:{g}" for g in (1, 2, 4, 8)] + ["row_major+a+hc"],
    "cfg5": [f"group_m:{g}" for g in (1, 2, 4, 8, 16, 32)] + [f"group_n:{g}" for g in (2, 4, 8, 16, 32)] +
            ["hilbert", "die_split:m:group_m:8", "die_split:m:hilbert", "die_split:m:group_m:8:i",
             "die_split:m:group_m:8:p", "die_split:m:group_m:16:p", "die_split:n:group_n:16:p", "die_split:m:hilbert:p",
             "die_split:n:group_m:16:p", "die_split:m:group_n:16:p", "group_m:16:s+a", "group_m:16:s+a+hc", "group_n:8:s+a+hc",
             "die_split:m:group_m:8:p:s+a+hc", "die_split:m:group_m:16:p:s+a+hc"],
}
DEFAULT_SCHEME = {"cfg1": "group_m:2", "cfg2": "group_m:8", "cfg3": "die_split:m:group_m:8:p:s+a+hc", "cfg4": "row_major+a+hc",
                  "cfg5": "die_split:m:group_m:16:p:s+a+hc"}
FALLBACK_SCHEME = {"cfg3": "group_m:8:s+a+hc", "cfg5": "group_m:16:s+a+hc"}   # if the topology probe finds no two-way L2 structure
FALLBACK_SCHEME_BY_TILE = {("cfg3", "256x512"): "group_m:16:s+a+hc", ("cfg5", "256x512"): "group_m:16:s+a+hc"}
# 8192^3 is timed with two 256x256 2-CTA MMA tiles per scheduler tile (they share the A panel: a quarter less operand
# traffic from L2); the plain 256x256 scheduler tile is timed beside it and reported in the same line.
DEFAULT_TILE = {"cfg3": "256x512", "cfg2": "256x512",   # 4096^3: A and B fit in L2, the order hardly matters, the wider tile does
                "cfg5": "256x512",
                "cfg1": "256x128"}   # 512^3: 8 CTA pairs, a quarter fewer operand bytes per SM than 16 CTAs of 128x128 (7.34 against 7.67 us)
DEFAULT_SCHEME_BY_TILE = {("cfg3", "256x512"): "die_split:m:group_m:8:p:s+a+hc", ("cfg5", "256x512"): "die_split:m:group_m:8:p:s+a+hc",
                          ("cfg2", "256x512"): "row_major"}


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def _rows_for_seconds(G, A, B, M, seconds):
    """How many rows of C the oracle computes in about `seconds` (two probes separate the fixed
    cost of widening the B panel from the per-row cost)."""
    t0 = time.perf_counter()
    G.gemm_rows(A, B, np.arange(4))
    t4 = time.perf_counter() - t0
    t0 = time.perf_counter()
    G.gemm_rows(A, B, np.arange(36))
    t36 = time.perf_counter() - t0
    per_row = max((t36 - t4) / 32.0, 1e-6)
    fixed = max(t4 - 4 * per_row, 0.0)
    return int(max(1, min(M, (seconds - fixed) / per_row)))


# ---------------------------------------------------------------------------------- reference arm
def run_reference(args) -> int:
    """Times the CPU oracle, as it stands, on a bounded sample of the same workload."""
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    from oracle import gemm as G
    w = synth.WORKLOADS[args.workload]
    _, A, B = synth.make_workload(args.workload)
    cores = G.threads()
    rows = min(_rows_for_seconds(G, A, B, w.M, 150.0 / (args.steps + args.warmup)), max(1, w.M // 16))
    band = np.arange(rows)
    for _ in range(args.warmup):
        G.gemm_rows(A, B, band)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        G.gemm_rows(A, B, band)
    dt = time.perf_counter() - t0
    tflops = 2.0 * rows * w.N * w.K * args.steps / dt / 1e12
    sample = f"{rows} contiguous rows of C ({rows}x{w.N}x{w.K}) per step, of the {w.M}-row product"
    line = {
        "impl": "reference", "metric": "bf16 GEMM TFLOP/s", "value": tflops, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: M={w.M} N={w.N} K={w.K} bf16 inputs, fp64 CPU oracle", "sample": sample},
        "cpu_baseline": {"value": tflops, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def sustained_leg(fn, flops, stream, gpu_index, seconds=4.0):
    """`fn` launched back to back for at least `seconds` (how the pool's sustained peak was taken): mean TFLOP/s over
    the whole stretch, the SM clock sampled through it, and time x clock = SM cycles per launch, which separates what
    the kernel needs from what the power limiter grants."""
    import math
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        fn()
    e0.record(stream)
    for _ in range(10):
        fn()
    e1.record(stream)
    e1.synchronize()
    one = e0.elapsed_time(e1) / 10
    n = int(math.ceil(seconds * 1e3 / one * 1.06))           # launches get slower as the clock settles: aim a little high
    sampler = benchutil.ClockSampler(gpu_index, period_s=0.02).start()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0.record(stream)
    for _ in range(n):
        fn()
    e1.record(stream)
    e1.synchronize()
    t1 = time.perf_counter()
    sampler.stop()
    ms = e0.elapsed_time(e1)
    c = sampler.summary(t0, t1)
    inside = [x[1] for x in sampler.samples if t0 <= x[0] <= t1]
    watts = c.get("power_w")       # board power, median over the stretch: at the power limit time is energy / power
    return {"launches": n, "seconds": ms / 1e3, "ms_per_launch": ms / n, "tflops": flops * n / ms / 1e9,
            "clocks": c, "sm_mhz_min": min(inside) if inside else None, "sm_mhz_max": max(inside) if inside else None,
            "sm_cycles_per_launch": None if not c.get("sm_mhz") else ms / n * 1e3 * c["sm_mhz"],
            "joules_per_launch": None if not watts else watts * ms / n / 1e3,
            "pj_per_flop": None if not watts else watts * ms / n / 1e3 / flops * 1e12}


def workloads_block(sp, names, peaks, stream):
    """The other named workloads, each timed briefly in the same process: the fastest known (tile, order) for it beside
    row-major on the same tile (alternating blocks of a quarter of a second, mean of two; best of four for the launch-bound 512^3), `torch.matmul`
    in the same alternation as context where the output is bf16, and the workload's nominal tile when that is another one.  For the launch-bound 512^3 also what a call costs on the host and how long one launch takes from call to
    completion."""
    import torch
    out = {}
    for name in names:
        w, A, B = synth.make_workload(name)
        out_f32 = int(w.out_dtype == "fp32")
        dA = torch.from_numpy(A.view(np.int16)).cuda().view(torch.bfloat16)
        dB = torch.from_numpy(B.view(np.int16)).cuda().view(torch.bfloat16)
        dC = torch.empty((w.M, w.N), dtype=torch.float32 if out_f32 else torch.bfloat16, device="cuda")
        flops = 2.0 * w.M * w.N * w.K
        tile = DEFAULT_TILE.get(name) or f"{w.tile_m}x{w.tile_n}"
        spec = DEFAULT_SCHEME_BY_TILE.get((name, tile)) or DEFAULT_SCHEME[name]

        def arm(tile_s, spec_s):
            tm, tn = (int(v) for v in tile_s.split("x"))
            scheme, kw = parse_scheme(spec_s)
            return scheme, sp.make_params(tile_m=tm, tile_n=tn, out_dtype=out_f32, **kw)

        def usable(tile_s, spec_s):
            try:
                sp.gemm(dA, dB, dC, *arm(tile_s, spec_s), stream)
                return True
            except sp.SpError as err:
                if err.status != sp.ERR_UNSUPPORTED:
                    raise
                return False
        if not usable(tile, spec):
            spec = FALLBACK_SCHEME_BY_TILE.get((name, tile)) or FALLBACK_SCHEME.get(name, "row_major")
        arms = [("best", tile, spec), ("row_major", tile, "row_major")]
        nominal_tile = f"{w.tile_m}x{w.tile_n}"
        if nominal_tile != tile:
            nspec = DEFAULT_SCHEME[name] if usable(nominal_tile, DEFAULT_SCHEME[name]) else FALLBACK_SCHEME.get(name, "row_major")
            arms.append(("nominal_tile", nominal_tile, nspec))
        for _, t_, s_ in arms:
            for _ in range(3):
                sp.gemm(dA, dB, dC, *arm(t_, s_), stream)
        est = time_steps(sp, dA, dB, dC, *arm(tile, spec), 5, stream) / 5
        # blocks of about 0.25 s: long enough for the power limiter to act, which is where a tile order's saved DRAM
        # traffic turns into clock and time (in a burst of a few milliseconds every order runs at the full clock)
        n = int(max(10, min(20000, 250.0 / est)))
        ms = {k: [] for k, _, _ in arms}
        lib_ms = []                # torch.matmul on the same tensors in the same alternation (bf16 output only): context
        if not out_f32:
            for _ in range(3):
                torch.matmul(dA, dB, out=dC)
        # one untimed block first: the first timed block must not run in the boost the later ones never see
        time_steps(sp, dA, dB, dC, *arm(tile, spec), n, stream)
        launch_bound = flops < 1e9      # 512^3: host and launch jitter is one-sided, so more rounds and the best of them
        for _ in range(4 if launch_bound else 2):
            for k, t_, s_ in arms:
                ms[k].append(time_steps(sp, dA, dB, dC, *arm(t_, s_), n, stream) / n)
            if not out_f32:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(n):
                    torch.matmul(dA, dB, out=dC)
                e1.record(stream)
                e1.synchronize()
                lib_ms.append(e0.elapsed_time(e1) / n)
        med = {k: (min(v) if launch_bound else sum(v) / len(v)) for k, v in ms.items()}
        rec = {"shape": [w.M, w.N, w.K], "out": w.out_dtype, "tile": tile, "scheme": spec, "launches_per_block": n,
               "ms": med["best"], "tflops": flops / med["best"] / 1e9,
               "frac_of_sustained_peak": flops / med["best"] / 1e9 / peaks["bf16_tflops_sustained"],
               "row_major_tflops": flops / med["row_major"] / 1e9, "speedup_over_row_major": med["row_major"] / med["best"]}
        if "nominal_tile" in med:
            rec["nominal_tile"] = {"tile": nominal_tile, "scheme": arms[2][2], "tflops": flops / med["nominal_tile"] / 1e9}
        if lib_ms:
            lib = sum(lib_ms) / len(lib_ms)
            rec["cublas_context"] = {"tflops": flops / lib / 1e9, "ours_over_it": lib / med["best"],
                                     "note": "torch.matmul in the same alternating blocks; context only, not a target"}
        if flops < 1e9:      # launch-bound: what a call costs
            scheme, p = arm(tile, spec)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(200):     # few enough for the launch queue never to fill: pure host cost of the call
                sp.gemm(dA, dB, dC, scheme, p, stream)
            rec["host_us_per_call"] = (time.perf_counter() - t0) / 200 * 1e6
            torch.cuda.synchronize()
            lat = []
            for _ in range(20):
                t0 = time.perf_counter()
                sp.gemm(dA, dB, dC, scheme, p, stream)
                torch.cuda.synchronize()
                lat.append((time.perf_counter() - t0) * 1e6)
            rec["call_to_completion_us"] = min(lat)
            rec["device_us_per_launch_back_to_back"] = med["best"] * 1e3
            # the same launches replayed from a CUDA graph (200 per graph): what a launch-bound loop should use
            side, graph, per_graph = torch.cuda.Stream(), torch.cuda.CUDAGraph(), 200
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph, stream=side):
                    for _ in range(per_graph):
                        sp.gemm(dA, dB, dC, scheme, p, side)
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(50):
                graph.replay()
            e1.record()
            e1.synchronize()
            rec["device_us_per_launch_from_a_cuda_graph"] = e0.elapsed_time(e1) / (50 * per_graph) * 1e3
            del graph
        assert sp.get_status() == 0
        out[name] = rec
        del dA, dB, dC
    return out


# ---------------------------------------------------------------------------------- our arm
def time_steps(sp, dA, dB, dC, scheme, p, steps, stream):
    import torch
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        sp.gemm(dA, dB, dC, scheme, p, stream)
    e1.record(stream)
    e1.synchronize()
    return e0.elapsed_time(e1)


def run_ours(args) -> int:
    import torch
    import paper_2508_20258_b200 as sp

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    sp.lib()  # fail loudly if the extension is missing

    b_nk = int(args.b_layout == "nk")
    if args.shape:                             # free shape for ablations: N(0,1) inputs, seed 5, 256x256 tiles, bf16 out
        Ms, Ns, Ks = (int(v) for v in args.shape.split("x"))
        w = synth.Workload(args.shape, Ms, Ns, Ks, "normal", 1.0, 5, 256, 256, "bf16")
        A, B = synth.make_inputs(Ms, Ns, Ks, w.dist, w.std, w.seed, bool(b_nk))
        SWEEPS[w.name] = ["row_major", "group_m:4", "group_m:8", "group_m:16", "hilbert", "die_split:m:group_m:8:p"]
        DEFAULT_SCHEME[w.name] = "group_m:8"
        args.workload = w.name
        if not (args.tile or args.scheme or args.sweep or args.sweep_sustained or args.profile_sweep or args.alternate):
            rs, rp = sp.recommend(Ms, Ns, Ks, 0, b_nk)      # nothing asked for: the library's own suggestion for the shape
            args.tile = f"{rp.tile_m}x{rp.tile_n}"
            args.scheme = ({sp.ROW_MAJOR: "row_major", sp.COL_MAJOR: "col_major", sp.GROUP_M: f"group_m:{rp.group}",
                            sp.GROUP_N: f"group_n:{rp.group}"}[rs] + (":s" if rp.flags & sp.FLAG_SERPENTINE else "")
                           + ("+a" if rp.flags & sp.FLAG_K_ALTERNATE else "") + ("+hc" if rp.flags & sp.FLAG_HINT_C_EVICT_FIRST else "")
                           + ("+k" if rp.flags & sp.FLAG_STREAM_K else ""))
    else:
        w = synth.WORKLOADS[args.workload]
        _, A, B = synth.make_workload(args.workload, b_is_nk=bool(b_nk))
    if not args.tile and args.workload in DEFAULT_TILE and not (args.sweep or args.sweep_sustained or args.profile_sweep or args.alternate):
        args.tile = DEFAULT_TILE[args.workload]
    tile_m, tile_n = (int(v) for v in args.tile.split("x")) if args.tile else (w.tile_m, w.tile_n)
    out_f32 = int(w.out_dtype == "fp32")
    dA = torch.from_numpy(A.view(np.int16)).cuda().view(torch.bfloat16)
    dB = torch.from_numpy(B.view(np.int16)).cuda().view(torch.bfloat16)
    dC = torch.empty((w.M, w.N), dtype=torch.float32 if out_f32 else torch.bfloat16, device="cuda")
    stream = torch.cuda.current_stream()
    flops = 2.0 * w.M * w.N * w.K
    resident = A.nbytes + B.nbytes + dC.numel() * dC.element_size()

    def params_for(spec):
        scheme, kw = parse_scheme(spec)
        return scheme, sp.make_params(tile_m=tile_m, tile_n=tile_n, out_dtype=out_f32, b_layout=b_nk, **kw)

    def supported(spec):                       # the die-pinned orders need at least as many tiles as units
        s_, p_ = params_for(spec)
        try:
            sp.gemm(dA, dB, dC, s_, p_, stream)
            return True
        except sp.SpError as err:
            if err.status == sp.ERR_UNSUPPORTED:
                return False
            raise

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    if args.sweep_sustained:
        return run_sweep_sustained(args, sp, w, dA, dB, dC, params_for, flops, stream)
    if args.alternate:
        return run_alternate(args, sp, w, dA, dB, dC, params_for, flops, stream)
    if args.sweep:
        return run_sweep(args, sp, w, dA, dB, dC, params_for, flops, stream)
    if args.profile_sweep:                     # one launch per scheme, in SWEEPS order: the command ncu wraps
        specs = [x for x in (args.scheme.split(",") if args.scheme else SWEEPS[args.workload]) if supported(x)]
        for spec in specs:
            s_, p_ = params_for(spec)
            sp.gemm(dA, dB, dC, s_, p_, stream)
        assert sp.get_status() == 0
        print(json.dumps({"profile_sweep": w.name, "tile": f"{tile_m}x{tile_n}", "launch_order": specs}), flush=True)
        return 0

    spec = args.scheme or DEFAULT_SCHEME_BY_TILE.get((args.workload, f"{tile_m}x{tile_n}")) or DEFAULT_SCHEME[args.workload]
    scheme, p = params_for(spec)
    try:
        sp.gemm(dA, dB, dC, scheme, p, stream)
    except sp.SpError as err:
        if args.scheme or err.status != sp.ERR_UNSUPPORTED or args.workload not in FALLBACK_SCHEME:
            raise
        spec = FALLBACK_SCHEME_BY_TILE.get((args.workload, f"{tile_m}x{tile_n}")) or FALLBACK_SCHEME[args.workload]
        scheme, p = params_for(spec)
    tile_s = f"{tile_m}x{tile_n}"
    traffic = None
    if not (args.kernel_only or args.no_traffic):
        traffic = captured_traffic(w.name, tile_s, spec)
        if traffic is None:
            raise SystemExit(f"no profiler capture of DRAM traffic for ({w.name}, {tile_s}, {spec}): capture it (ncu over "
                             f"`bench.py --profile-sweep`, then `python -m paper_2508_20258_b200.ncuparse --sweep ... --traffic`) "
                             f"or pass --no-traffic to report roofline.traffic as null")
    sampler = None if args.kernel_only else benchutil.ClockSampler(local_rank, period_s=0.002).start()   # before the warm-up: no idle gap later
    for _ in range(max(args.warmup, 3)):
        sp.gemm(dA, dB, dC, scheme, p, stream)
    torch.cuda.synchronize()
    if args.kernel_only:                       # the command profilers wrap: nothing but the kernel
        ms = time_steps(sp, dA, dB, dC, scheme, p, args.steps, stream)
        sp.get_status()
        print(json.dumps({"kernel_only": True, "workload": w.name, "scheme": spec, "tile": f"{tile_m}x{tile_n}",
                          "ms_per_step": ms / args.steps, "tflops": flops * args.steps / ms / 1e9}), flush=True)
        return 0

    barrier()
    t_host0 = time.perf_counter()
    ms_total = time_steps(sp, dA, dB, dC, scheme, p, args.steps, stream)
    torch.cuda.synchronize()
    t_host1 = time.perf_counter()
    barrier()
    sampler.stop()
    assert sp.get_status() == 0
    agg = benchutil.aggregate(ms_total, flops * args.steps, world)
    value = agg["units"] / agg["ms"] / 1e9                      # TFLOP/s, whole job
    clocks = sampler.summary(t_host0, t_host1)

    # burst protocol: one launch timed on its own, best of 10 (how the pool's peak itself was measured); the
    # launch before it keeps the host's launch latency out of the bracket, the sleep lets the clocks recover
    def one_launch():
        sp.gemm(dA, dB, dC, scheme, p, stream)
        ms = time_steps(sp, dA, dB, dC, scheme, p, 1, stream)
        time.sleep(0.05)
        return ms
    burst_ms = min(one_launch() for _ in range(10))
    row_scheme, row_p = params_for("row_major")
    for _ in range(3):
        sp.gemm(dA, dB, dC, row_scheme, row_p, stream)
    row_ms = time_steps(sp, dA, dB, dC, row_scheme, row_p, args.steps, stream) / args.steps

    # The same launches declared independent of their predecessor (SP_FLAG_OVERLAP): CTAs of launch i+1 take over SMs as
    # those of launch i finish, so the partly empty last wave is filled.  Reported beside the headline, not as it: the
    # headline keeps every launch ordered after the previous one.
    overlapped = None
    if "+" not in spec and not (p.flags & sp.FLAG_DIE_PINNED):
        ov_scheme, ov_p = params_for(spec + "+o")
        for _ in range(3):
            sp.gemm(dA, dB, dC, ov_scheme, ov_p, stream)
        pl, ov = [], []
        for _ in range(3):                      # alternating, so both see the same thermal state
            pl.append(time_steps(sp, dA, dB, dC, scheme, p, args.steps, stream) / args.steps)
            ov.append(time_steps(sp, dA, dB, dC, ov_scheme, ov_p, args.steps, stream) / args.steps)
        ov_ms, pl_ms = sorted(ov)[1], sorted(pl)[1]
        overlapped = {"ms_per_step": ov_ms, "tflops": flops / ov_ms / 1e9, "ordered_launches_alternating_tflops": flops / pl_ms / 1e9,
                      "speedup": pl_ms / ov_ms,
                      "note": "SP_FLAG_OVERLAP: successive launches not ordered against each other; same work per launch"}

    # the workload's nominal scheduler tile, when the timed one differs from it
    nominal = None
    if (tile_m, tile_n) != (w.tile_m, w.tile_n):
        nspec = DEFAULT_SCHEME[args.workload]
        ns, kw = parse_scheme(nspec)
        npar = sp.make_params(tile_m=w.tile_m, tile_n=w.tile_n, out_dtype=out_f32, b_layout=b_nk, **kw)
        try:
            sp.gemm(dA, dB, dC, ns, npar, stream)
        except sp.SpError:
            nspec = FALLBACK_SCHEME.get(args.workload, "row_major")
            ns, kw = parse_scheme(nspec)
            npar = sp.make_params(tile_m=w.tile_m, tile_n=w.tile_n, out_dtype=out_f32, b_layout=b_nk, **kw)
        for _ in range(3):
            sp.gemm(dA, dB, dC, ns, npar, stream)
        n_ms = time_steps(sp, dA, dB, dC, ns, npar, args.steps, stream) / args.steps
        nrs, nrkw = parse_scheme("row_major")
        nrp = sp.make_params(tile_m=w.tile_m, tile_n=w.tile_n, out_dtype=out_f32, b_layout=b_nk)
        nr_ms = time_steps(sp, dA, dB, dC, nrs, nrp, args.steps, stream) / args.steps
        nominal = {"tile": f"{w.tile_m}x{w.tile_n}", "scheme": nspec, "ms_per_step": n_ms, "tflops": flops / n_ms / 1e9,
                   "row_major_tflops": flops / nr_ms / 1e9, "speedup_over_row_major": nr_ms / n_ms}

    # context only: cuBLAS (torch.matmul) on the same tensors, same back-to-back protocol, same thermal state
    cublas = None
    if dC.dtype == torch.bfloat16 and not b_nk:
        ref = torch.empty_like(dC)
        for _ in range(3):
            torch.matmul(dA, dB, out=ref)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            torch.matmul(dA, dB, out=ref)
        e1.record(stream)
        e1.synchronize()
        cublas = {"tflops": flops * args.steps / e0.elapsed_time(e1) / 1e9, "note": "torch.matmul, context only, not a target"}
        ours_again = time_steps(sp, dA, dB, dC, scheme, p, args.steps, stream) / args.steps
        cublas["ours_right_after_tflops"] = flops / ours_again / 1e9

        # single launches of both, alternating, in the burst protocol (on this GPU, now: the pool's burst peak was taken on
        # another day, possibly on another GPU of the pool)
        def one(fn):
            fn()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            fn()
            a1.record(stream)
            a1.synchronize()
            time.sleep(0.05)
            return a0.elapsed_time(a1)
        time.sleep(0.5)
        b_ours, b_lib = [], []
        for _ in range(8):
            b_lib.append(one(lambda: torch.matmul(dA, dB, out=ref)))
            b_ours.append(one(lambda: sp.gemm(dA, dB, dC, scheme, p, stream)))
        cublas["burst_tflops"] = flops / min(b_lib) / 1e9
        cublas["ours_burst_alternating_tflops"] = flops / min(b_ours) / 1e9
        del ref

    # the same launches back to back for four seconds, against the pool's sustained peak, with the clocks
    sustained = None
    if not args.no_sustained:
        sustained = sustained_leg(lambda: sp.gemm(dA, dB, dC, scheme, p, stream), flops, stream, local_rank, args.sustained_seconds)
        sustained["peak"] = benchutil.measured_peaks(ROOT)["bf16_tflops_sustained"]
        sustained["frac"] = sustained["tflops"] / sustained["peak"]
        sustained["protocol"] = f"launches back to back for >= {args.sustained_seconds:g} s, mean over the whole stretch; clock sampled every 20 ms"
        if cublas is not None:
            time.sleep(1.0)
            ref = torch.empty_like(dC)
            lib = sustained_leg(lambda: torch.matmul(dA, dB, out=ref), flops, stream, local_rank, args.sustained_seconds)
            cublas["sustained"] = {k: lib[k] for k in ("tflops", "seconds", "sm_cycles_per_launch", "joules_per_launch", "pj_per_flop")}
            cublas["sustained"]["sm_mhz"] = lib["clocks"]["sm_mhz"]
            cublas["sustained"]["power_w"] = lib["clocks"].get("power_w")
            sustained["over_cublas_same_run"] = sustained["tflops"] / lib["tflops"]
            del ref
    assert sp.get_status() == 0

    workloads = None
    if rank == 0 and not args.no_workloads and not args.shape:
        workloads = workloads_block(sp, [n_ for n_ in ("cfg1", "cfg2", "cfg4", "cfg5") if n_ != args.workload],
                                    benchutil.measured_peaks(ROOT), stream)

    # end to end through the C ABI with host buffers (pinned): H2D of A and B, kernel, D2H of C, every step
    e2e = None
    if not args.no_e2e:
        hA = torch.from_numpy(A.view(np.int16)).pin_memory()
        hB = torch.from_numpy(B.view(np.int16)).pin_memory()
        hC = torch.empty((w.M, w.N), dtype=torch.float32 if out_f32 else torch.int16).pin_memory()
        e2e_steps = max(1, min(args.steps, 5))
        sp.gemm_host(hA, hB, hC, scheme, p, stream)
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            sp.gemm_host(hA, hB, hC, scheme, p, stream)        # synchronises before returning
        e2e_ms = (time.perf_counter() - t0) * 1e3
        barrier()
        eagg = benchutil.aggregate(e2e_ms, flops * e2e_steps, world)
        e2e = {"value": eagg["units"] / eagg["ms"] / 1e9, "unit": "TFLOP/s", "h2d_bytes_per_step": int(A.nbytes + B.nbytes),
               "d2h_bytes_per_step": int(hC.numel() * hC.element_size()), "steps": e2e_steps,
               "ms_per_step": eagg["ms"] / e2e_steps, "api": "sp_gemm_host (pinned host buffers)"}
        # the floor the copies alone set on this machine: the same bytes over PCIe with nothing else going on, each direction
        # on its own and both at once (what the pipelined call does); floor = the slower direction
        dAB = torch.empty(A.nbytes + B.nbytes, dtype=torch.uint8, device="cuda")
        hAB = torch.empty(A.nbytes + B.nbytes, dtype=torch.uint8).pin_memory()
        hCb = hC.view(torch.uint8).reshape(-1)
        dCb = dC.view(torch.uint8).reshape(-1)
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

        def copies(h2d, d2h):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            if h2d:
                with torch.cuda.stream(s_in):
                    dAB.copy_(hAB, non_blocking=True)
            if d2h:
                with torch.cuda.stream(s_out):
                    hCb.copy_(dCb, non_blocking=True)
            torch.cuda.synchronize()
            return (time.perf_counter() - t0) * 1e3
        copies(True, True)
        h2d_ms = min(copies(True, False) for _ in range(3))
        d2h_ms = min(copies(False, True) for _ in range(3))
        both_ms = min(copies(True, True) for _ in range(3))
        e2e["pcie_floor"] = {"h2d_GBps": dAB.numel() / h2d_ms / 1e6, "d2h_GBps": dCb.numel() / d2h_ms / 1e6, "h2d_ms": h2d_ms,
                             "d2h_ms": d2h_ms, "both_directions_at_once_ms": both_ms, "floor_ms": max(h2d_ms, d2h_ms),
                             "e2e_over_floor": e2e["ms_per_step"] / max(h2d_ms, d2h_ms),
                             "e2e_over_both_directions_at_once": e2e["ms_per_step"] / both_ms,
                             "note": "pinned host memory, one copy per direction, best of 3; rank 0's box"}
        del dAB, hAB
        del hA, hB, hC

    peaks = benchutil.measured_peaks(ROOT)
    launch_ms = ms_total / args.steps
    achieved = flops / launch_ms / 1e9
    # Which measured peak the timed region is compared with follows from its length: the pool's burst figure was taken on
    # single launches, its sustained figure on launches back to back for 4 s (the chip then sits at its power limit and
    # the clock has settled).  A timed region of under a second has not settled: it is a burst and is divided by the burst
    # peak.  The `sustained` record below repeats the measurement the other way.
    is_burst = ms_total < 1000.0
    peak = peaks["bf16_tflops"] if is_burst else peaks["bf16_tflops_sustained"]
    out_bytes = 4 if out_f32 else 2
    algorithmic_bytes = 2.0 * (w.M * w.K + w.K * w.N) + out_bytes * w.M * w.N
    roofline = {
        "bound": "tensor", "kernel": f"gemm_kernel<CG={tile_m // 128},BN={tile_n}>" + (" (two 256x256 2-CTA MMA tiles sharing A)" if tile_n == 512 else ""),
        "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
        "peak_kind": (f"cuBLAS bf16 {'burst (best single launch)' if is_burst else 'sustained (4 s back to back)'}, {peaks['source']}; "
                      f"the timed region lasted {ms_total:.1f} ms"
                      + ("; that is long enough for the power limiter to have begun to act (it does within 100 ms) and too short for"
                         " the clock to have settled: no kernel holds the burst figure that long, see `sustained` for the like-for-like"
                         if 50.0 < ms_total < 1000.0 else "")),
        "traffic": None if traffic is None else traffic["dram_bytes"],
        "traffic_source": None if traffic is None else {"captured": traffic["captured"], "command": traffic["command"],
                                                        "dram_read_bytes": traffic["dram_read_bytes"],
                                                        "dram_write_bytes": traffic["dram_write_bytes"]},
        "algorithmic_bytes": algorithmic_bytes,
        "traffic_over_algorithmic": None if traffic is None else traffic["dram_bytes"] / algorithmic_bytes,
        "algorithmic_flops_per_launch": flops,
        "sm_cycles_per_launch": None if not clocks.get("sm_mhz") else launch_ms * 1e3 * clocks["sm_mhz"],
        "burst": {"achieved": flops / burst_ms / 1e9, "peak": peaks["bf16_tflops"],
                  "frac": flops / burst_ms / 1e9 / peaks["bf16_tflops"], "protocol": "best of 10 single launches, each queued behind one untimed launch"},
        "sustained": sustained,
        "frac_of_nominal_2250": achieved / 2250.0,
    }

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import gemm as G
        rows = _rows_for_seconds(G, A, B, w.M, 15.0)
        t0 = time.perf_counter()
        G.gemm_rows(A, B, np.arange(rows))
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": 2.0 * rows * w.N * w.K / dt / 1e12, "unit": "TFLOP/s", "cores": G.threads(),
                        "kind": "oracle", "seconds": dt,
                        "sample": f"first {rows} rows of C ({rows}x{w.N}x{w.K}) of the {w.M}-row product"}
        # the other half of the oracle: the enumerated remap of this workload's tile grid under the timed order
        from oracle import remap as OR
        kw_o = parse_scheme(spec)[1]
        op = OR.Params(**{k: v for k, v in kw_o.items() if k in OR.Params.__dataclass_fields__})
        t0 = time.perf_counter()
        OR.tile_map(w.M, w.N, tile_m, tile_n, scheme, op)
        cpu_baseline["remap_oracle_ms"] = (time.perf_counter() - t0) * 1e3
        if w.M * w.N * w.K <= 2 ** 28:                      # small enough to also time on one core (512^3)
            t0 = time.perf_counter()
            G.gemm_rows(A, B, np.arange(w.M), nthreads=1)
            cpu_baseline["single_thread_tflops"] = 2.0 * w.M * w.N * w.K / (time.perf_counter() - t0) / 1e12
            G.gemm_rows(A, B, np.arange(1), nthreads=cpu_baseline["cores"])    # the thread count is sticky: put it back

    if rank == 0:
        line = {
            "metric": "bf16 GEMM TFLOP/s", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": agg["ms"] / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{w.name}: C=A.B M={w.M} N={w.N} K={w.K}, bf16 in ({w.dist}, seed {w.seed}), fp32 "
                                   f"accumulate, {w.out_dtype} out", "tile": f"{tile_m}x{tile_n}", "scheme": spec,
                       "units": sp.gemm_units(tile_m, tile_n, sp.tile_count(w.M, w.N, tile_m, tile_n)),
                       "l2": f"no flush: {resident / 1e6:.0f} MB resident per step vs {L2_BYTES / 1e6:.0f} MB L2",
                       "parallelism": "replicas only" if world > 1 else "1 GPU"},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": args.steps,
            "clocks": clocks,
            "workloads": workloads,
            "nominal_tile": nominal, "cublas_context": cublas, "overlapped_launches": overlapped,
            "row_major": {"ms_per_step": row_ms, "tflops": flops / row_ms / 1e9, "speedup_of_scheme": row_ms / launch_ms},
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def run_sweep_sustained(args, sp, w, dA, dB, dC, params_for, flops, stream) -> int:
    """Every scheme timed on its own in back-to-back launches (about 0.3 s each, two passes): the power-capped
    steady state, where traffic saved by a tile order shows up as clock and therefore as time."""
    import torch
    specs = []
    for spec in (args.scheme.split(",") if args.scheme else SWEEPS[args.workload]):
        try:
            sp.gemm(dA, dB, dC, *params_for(spec), stream)
            specs.append(spec)
        except sp.SpError as err:
            if err.status != sp.ERR_UNSUPPORTED:
                raise
    done = {}
    if args.resume and os.path.exists(args.resume):     # an interrupted sweep picks up where it stopped
        for l in open(args.resume):
            try:
                j = json.loads(l)
                if j.get("sweep_sustained") == w.name and j.get("key") == args.resume_key:
                    done[j["scheme"]] = j
            except ValueError:
                pass
        specs = [s_ for s_ in specs if s_ not in done]
    acc = {spec: [] for spec in specs}
    if specs:            # half a second of load first: the first scheme must not be timed in the boost the others never see
        s, p = params_for(specs[0])
        one = time_steps(sp, dA, dB, dC, s, p, 10, stream) / 10
        time_steps(sp, dA, dB, dC, s, p, int(max(20, min(5000, 500.0 / one))), stream)
    for _ in range(2):
        for spec in specs:
            s, p = params_for(spec)
            for _ in range(3):
                sp.gemm(dA, dB, dC, s, p, stream)
            torch.cuda.synchronize()
            one = time_steps(sp, dA, dB, dC, s, p, 10, stream) / 10
            n = int(max(20, min(2000, 300.0 / one)))
            acc[spec].append(time_steps(sp, dA, dB, dC, s, p, n, stream) / n)
    assert sp.get_status() == 0
    base = None
    for j in done.values():
        print(json.dumps(j), flush=True)
        base = base or j["ms"]
    for spec in specs:
        ms = sum(acc[spec]) / len(acc[spec])
        if base is None:
            base = ms
        line = {"sweep_sustained": w.name, "scheme": spec, "ms": ms, "tflops": flops / ms / 1e9,
                "speedup_vs_first": base / ms, "passes_ms": acc[spec], "key": args.resume_key}
        print(json.dumps(line), flush=True)
        if args.resume:
            with open(args.resume, "a") as fh:
                fh.write(json.dumps(line) + "\n")
    return 0


def run_alternate(args, sp, w, dA, dB, dC, params_for, flops, stream) -> int:
    """The given schemes (and, with the pseudo-scheme 'cublas', torch.matmul on the same tensors) in alternating blocks of
    --steps launches, --rounds rounds, median per arm: every arm sees the same thermal state.  JSON lines to stdout."""
    import torch
    arms = []
    ref = None
    for spec in args.alternate.split(","):
        if spec == "cublas":
            if args.b_layout != "kn" or dC.dtype != torch.bfloat16:
                raise SystemExit("the cublas arm needs B stored K x N and bf16 output")
            ref = torch.empty_like(dC)
            arms.append((spec, lambda: torch.matmul(dA, dB, out=ref)))
        else:
            s, p = params_for(spec)
            arms.append((spec, lambda s=s, p=p: sp.gemm(dA, dB, dC, s, p, stream)))
    n = max(args.steps, 1)
    for _, fn in arms:
        for _ in range(n):
            fn()
    torch.cuda.synchronize()
    times = {spec: [] for spec, _ in arms}
    mhz = {spec: [] for spec, _ in arms}
    sampler = benchutil.ClockSampler(0).start()
    for _ in range(args.rounds):
        for spec, fn in arms:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.perf_counter()
            e0.record(stream)
            for _ in range(n):
                fn()
            e1.record(stream)
            e1.synchronize()
            t1 = time.perf_counter()
            times[spec].append(e0.elapsed_time(e1) / n)
            # the host runs ahead of the GPU: only the second half of the block is sure to have the GPU busy with this arm
            c = sampler.summary(0.5 * (t0 + t1), t1)
            if c["sm_mhz"] is not None and c["samples"] >= 3 and "+-" not in c["window"]:
                mhz[spec].append(c["sm_mhz"])
    sampler.stop()
    assert sp.get_status() == 0
    base = None
    for spec, _ in arms:
        ms = float(np.median(times[spec]))
        base = base or ms
        clk = float(np.median(mhz[spec])) if mhz[spec] else None
        print(json.dumps({"alternate": w.name, "arm": spec, "ms": ms, "tflops": flops / ms / 1e9, "first_arm_over_this": base / ms,
                          "block_launches": n, "rounds": args.rounds, "sm_mhz": clk,
                          "sm_cycles_per_launch": None if clk is None else ms * 1e-3 * clk * 1e6}), flush=True)
    return 0


def run_sweep(args, sp, w, dA, dB, dC, params_for, flops, stream) -> int:
    """Every scheme of the workload, interleaved (ABAB) to share thermal state; JSON lines to stdout."""
    import torch
    specs = SWEEPS[args.workload]
    for spec in specs:
        s, p = params_for(spec)
        for _ in range(3):
            sp.gemm(dA, dB, dC, s, p, stream)
    torch.cuda.synchronize()
    best = {spec: 1e30 for spec in specs}
    total = {spec: 0.0 for spec in specs}
    rounds = max(args.steps, 1)
    for _ in range(rounds):
        for spec in specs:
            s, p = params_for(spec)
            ms = time_steps(sp, dA, dB, dC, s, p, 1, stream)
            best[spec] = min(best[spec], ms)
            total[spec] += ms
    assert sp.get_status() == 0
    ref = torch.empty_like(dC)
    tb = 1e30
    if dC.dtype == torch.bfloat16:
        for _ in range(3):
            torch.matmul(dA, dB, out=ref)
        for _ in range(rounds):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); torch.matmul(dA, dB, out=ref); e1.record(); e1.synchronize()
            tb = min(tb, e0.elapsed_time(e1))
    for spec in specs:
        print(json.dumps({"sweep": w.name, "scheme": spec, "best_ms": best[spec], "mean_ms": total[spec] / rounds,
                          "best_tflops": flops / best[spec] / 1e9, "mean_tflops": flops * rounds / total[spec] / 1e9}),
              flush=True)
    if tb < 1e30:
        print(json.dumps({"sweep": w.name, "scheme": "torch.matmul (cuBLAS, context only)", "best_ms": tb,
                          "best_tflops": flops / tb / 1e9}), flush=True)
    return 0


TRANSPOSE_SWEEP = ["row_major", "col_major", "group_m:2", "group_m:4", "group_m:8", "group_m:16", "group_m:32", "group_n:4",
                   "group_n:8", "group_n:16", "morton", "hilbert", "xcd:2", "xcd:8", "die_split:m:group_m:8",
                   "die_split:m:group_m:8:i"]


def run_transpose(args) -> int:
    """Second workload (the paper's largest win): 16-bit transpose under each tile order.  HBM bound:
    algorithmic bytes = 2 * M * N * 2 (every element read once, written once).  JSON lines to stdout."""
    import torch
    import paper_2508_20258_b200 as sp
    M, N = (int(v) for v in args.transpose.split("x"))
    torch.cuda.set_device(0)
    rng = np.random.Generator(np.random.PCG64(7))
    x = torch.from_numpy(rng.integers(-32768, 32768, size=(M, N), dtype=np.int16)).cuda()
    out = torch.empty((N, M), dtype=torch.int16, device="cuda")
    stream = torch.cuda.current_stream()
    peaks = benchutil.measured_peaks(ROOT)
    nbytes = 2.0 * M * N * 2
    specs = args.scheme.split(",") if args.scheme else TRANSPOSE_SWEEP

    def timed(spec, n):
        scheme, kw = parse_scheme(spec)
        p = sp.make_params(**kw)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            sp.transpose(x, out, scheme, p, stream)
        e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1) / n

    if args.profile_sweep:
        for spec in specs:
            timed(spec, 1)
        assert sp.get_status() == 0
        print(json.dumps({"profile_sweep": "transpose", "shape": [M, N], "launch_order": specs}), flush=True)
        return 0
    for spec in specs:
        timed(spec, 3)
        one = timed(spec, 5)
        n = int(max(10, min(1000, 200.0 / one)))
        ms = min(timed(spec, n) for _ in range(2))
        gbs = nbytes / ms / 1e6
        print(json.dumps({"transpose": [M, N], "scheme": spec, "ms": ms, "GB/s": gbs,
                          "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                       "frac": gbs / peaks["hbm_gbs"], "peak_kind": f"copy bandwidth, {peaks['source']}"}}),
              flush=True)
    assert sp.get_status() == 0
    xt = torch.empty_like(out)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        xt.copy_(x.t())
    e0.record(stream)
    for _ in range(20):
        xt.copy_(x.t())
    e1.record(stream)
    e1.synchronize()
    ms = e0.elapsed_time(e1) / 20
    print(json.dumps({"transpose": [M, N], "scheme": "torch copy_ of a transposed view (context only)", "ms": ms,
                      "GB/s": nbytes / ms / 1e6}), flush=True)
    return 0


STENCIL_SWEEP = ["row_major", "col_major", "group_m:2", "group_m:4", "group_m:8", "group_n:2", "group_n:4", "group_n:8",
                 "morton", "hilbert", "xcd:2", "xcd:8", "die_split:m:row_major", "die_split:m:row_major:i",
                 "die_split:m:group_m:4"]


def run_stencil(args) -> int:
    """Third workload (the paper's Stencil 2D): one five-point sweep over an fp32 grid under each tile order.  HBM
    bound: algorithmic bytes = 2 * M * N * 4 (every point read once, written once; halos come from L2)."""
    import torch
    import paper_2508_20258_b200 as sp
    M, N = (int(v) for v in args.stencil.split("x"))
    torch.cuda.set_device(0)
    g = torch.Generator(device="cuda").manual_seed(11)
    x = torch.randn((M, N), device="cuda", generator=g, dtype=torch.float32)
    out = torch.empty_like(x)
    stream = torch.cuda.current_stream()
    peaks = benchutil.measured_peaks(ROOT)
    nbytes = 2.0 * M * N * 4
    specs = args.scheme.split(",") if args.scheme else STENCIL_SWEEP

    def timed(spec, n):
        scheme, kw = parse_scheme(spec)
        p = sp.make_params(**kw)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            sp.stencil2d(x, out, 0.5, 0.125, scheme, p, stream)
        e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1) / n

    if args.profile_sweep:
        for spec in specs:
            timed(spec, 1)
        assert sp.get_status() == 0
        print(json.dumps({"profile_sweep": "stencil2d", "shape": [M, N], "launch_order": specs}), flush=True)
        return 0
    for spec in specs:
        timed(spec, 3)
        one = timed(spec, 5)
        n = int(max(10, min(1000, 200.0 / one)))
        ms = min(timed(spec, n) for _ in range(2))
        gbs = nbytes / ms / 1e6
        print(json.dumps({"stencil2d": [M, N], "scheme": spec, "ms": ms, "GB/s": gbs,
                          "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                       "frac": gbs / peaks["hbm_gbs"], "peak_kind": f"copy bandwidth, {peaks['source']}"}}),
              flush=True)
    assert sp.get_status() == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        out.copy_(x)
    e0.record(stream)
    for _ in range(20):
        out.copy_(x)
    e1.record(stream)
    e1.synchronize()
    ms = e0.elapsed_time(e1) / 20
    print(json.dumps({"stencil2d": [M, N], "scheme": "torch copy_ of the grid (context only)", "ms": ms,
                      "GB/s": nbytes / ms / 1e6}), flush=True)
    return 0


SOFTMAX_SWEEP = ["single:row_major", "single:group_m:8", "two:row_major", "two:col_major", "two:group_m:8", "two:hilbert",
                 "rev:row_major", "rev:col_major", "rev:group_m:8", "rev:group_n:4", "rev:hilbert", "rev:hilbert_rect"]


def run_softmax(args) -> int:
    """Fourth workload (the paper's softmax case study): row softmax of an fp32 matrix, single pass and in the two-phase
    tiled form under each tile order, the second phase in the same or in reverse slot order.  HBM bound: algorithmic
    bytes = 2 * M * N * 4 (every element read once, written once).  Specs are `mode:order` with mode single / two / rev."""
    import torch
    import paper_2508_20258_b200 as sp
    M, N = (int(v) for v in args.softmax.split("x"))
    torch.cuda.set_device(0)
    g = torch.Generator(device="cuda").manual_seed(13)
    x = torch.randn((M, N), device="cuda", generator=g, dtype=torch.float32) * 3.0
    out = torch.empty_like(x)
    stream = torch.cuda.current_stream()
    peaks = benchutil.measured_peaks(ROOT)
    nbytes = 2.0 * M * N * 4
    specs = args.scheme.split(",") if args.scheme else SOFTMAX_SWEEP
    modes = {"single": sp.SOFTMAX_SINGLE_PASS, "two": sp.SOFTMAX_TWO_PHASE, "rev": sp.SOFTMAX_TWO_PHASE_REVERSED}

    def timed(spec, n):
        mode, order = spec.split(":", 1)
        scheme, kw = parse_scheme(order)
        p = sp.make_params(**kw)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            sp.softmax(x, out, modes[mode], scheme, p, stream)
        e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1) / n

    if args.profile_sweep:
        for spec in specs:
            timed(spec, 1)
        assert sp.get_status() == 0
        print(json.dumps({"profile_sweep": "softmax", "shape": [M, N], "launch_order": specs}), flush=True)
        return 0
    for spec in specs:
        timed(spec, 3)
        one = timed(spec, 5)
        n = int(max(10, min(1000, 200.0 / one)))
        ms = min(timed(spec, n) for _ in range(2))
        gbs = nbytes / ms / 1e6
        print(json.dumps({"softmax": [M, N], "scheme": spec, "ms": ms, "GB/s": gbs,
                          "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                       "frac": gbs / peaks["hbm_gbs"], "peak_kind": f"copy bandwidth, {peaks['source']}"}}),
              flush=True)
    assert sp.get_status() == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name, fn in (("torch.softmax (context only)", lambda: torch.softmax(x, dim=1, out=out)),
                     ("torch copy_ of the matrix (context only)", lambda: out.copy_(x))):
        for _ in range(3):
            fn()
        e0.record(stream)
        for _ in range(20):
            fn()
        e1.record(stream)
        e1.synchronize()
        ms = e0.elapsed_time(e1) / 20
        print(json.dumps({"softmax": [M, N], "scheme": name, "ms": ms, "GB/s": nbytes / ms / 1e6}), flush=True)
    return 0


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20,
                    help="timed launches (20 of the 8192^3 GEMM last 14 ms: a burst, compared with the burst peak; the sustained record times four seconds)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--shape", default=None, metavar="MxNxK", help="free GEMM shape instead of a named workload (ablations)")
    ap.add_argument("--scheme", default=None)
    ap.add_argument("--tile", default=None, help="MxN override, e.g. 128x256")
    ap.add_argument("--kernel-only", action="store_true", help="time the kernel only (the command profilers wrap)")
    ap.add_argument("--sweep", action="store_true", help="time every scheme of the workload")
    ap.add_argument("--sweep-sustained", action="store_true", help="time every scheme in its own back-to-back loop")
    ap.add_argument("--profile-sweep", action="store_true", help="launch each scheme once (for ncu counters)")
    ap.add_argument("--alternate", default=None, metavar="SPEC,SPEC[,cublas]",
                    help="time the given schemes in alternating blocks of --steps launches (--rounds rounds, median)")
    ap.add_argument("--rounds", type=int, default=6)
    ap.add_argument("--resume", default=None, metavar="FILE.jsonl",
                    help="--sweep-sustained: append each scheme's line to FILE and skip schemes already in it")
    ap.add_argument("--b-layout", default="kn", choices=["kn", "nk"], help="B stored K x N (default) or N x K")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the four-second back-to-back leg")
    ap.add_argument("--sustained-seconds", type=float, default=4.0)
    ap.add_argument("--no-workloads", action="store_true", help="skip the brief timings of the other named workloads")
    ap.add_argument("--no-traffic", action="store_true", help="report roofline.traffic as null when no capture exists")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--transpose", default=None, metavar="MxN", help="time sp_transpose on an M x N 16-bit matrix instead")
    ap.add_argument("--stencil", default=None, metavar="MxN", help="time sp_stencil2d on an M x N fp32 grid instead")
    ap.add_argument("--softmax", default=None, metavar="MxN", help="time sp_softmax on an M x N fp32 matrix instead")
    args = ap.parse_args()
    args.resume_key = f"{args.workload}|{args.shape}|{args.tile}|{args.b_layout}"
    if args.transpose:
        return run_transpose(args)
    if args.stencil:
        return run_stencil(args)
    if args.softmax:
        return run_softmax(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
