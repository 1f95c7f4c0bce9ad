"""Helpers for the benchmark: clock sampling, cross-rank aggregation, roofline records.

No arithmetic of the method lives here.
"""

from __future__ import annotations

import json
import os
import statistics
import subprocess
import threading
import time
from typing import Dict, List, Optional


class ClockSampler:
    """Samples SM clock, throttle reasons and board power of one GPU in a background thread.

    Uses NVML when the Python binding is importable, else polls ``nvidia-smi``.  It only
    reads; it never changes a setting of the GPU.
    """

    BAD = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}
    NOTED = {"sw_power_cap": 0x4}

    def __init__(self, index: int = 0, period_s: float = 0.01):
        self.index = index
        self.period_s = period_s
        self.samples: List[tuple] = []      # (t, sm_mhz, reasons_bitmask, watts or None)
        self.max_mhz: Optional[float] = None
        self._stop = threading.Event()
        self._thread: Optional[threading.Thread] = None
        self._nvml = None

    def _init_nvml(self) -> bool:
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._handle, pynvml.NVML_CLOCK_SM))
            # the first call of each query takes milliseconds (later ones microseconds): make them here, not inside the
            # region that is about to be sampled
            for _ in range(2):
                pynvml.nvmlDeviceGetClockInfo(self._handle, pynvml.NVML_CLOCK_SM)
                pynvml.nvmlDeviceGetCurrentClocksEventReasons(self._handle)
                try:
                    pynvml.nvmlDeviceGetPowerUsage(self._handle)
                except Exception:
                    pass
            return True
        except Exception:
            self._nvml = None
            return False

    def _loop_nvml(self) -> None:
        n = self._nvml
        watts, reasons, i = None, 0, 0
        while not self._stop.is_set():
            try:
                # every query costs a good part of a sampling period (more on some hosts): the clock is read every time,
                # the reasons every second time (a sample carries the last mask read, and the union over a window is
                # what is reported), the power every sixteenth
                mhz = float(n.nvmlDeviceGetClockInfo(self._handle, n.NVML_CLOCK_SM))
                if i % 2 == 0:
                    reasons = int(n.nvmlDeviceGetCurrentClocksEventReasons(self._handle))
                if i % 16 == 1:
                    try:
                        watts = n.nvmlDeviceGetPowerUsage(self._handle) / 1000.0
                    except Exception:
                        watts = None
                i += 1
                self.samples.append((time.perf_counter(), mhz, reasons, watts))
            except Exception:
                pass
            self._stop.wait(self.period_s)

    def _loop_smi(self) -> None:
        q = "clocks.sm,clocks.max.sm,clocks_event_reasons.active,power.draw"
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.index}", f"--query-gpu={q}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
                a = [v.strip() for v in out.strip().split(",")]
                self.max_mhz = float(a[1])
                try:
                    watts = float(a[3])
                except (IndexError, ValueError):
                    watts = None
                self.samples.append((time.perf_counter(), float(a[0]), int(a[2], 16), watts))
            except Exception:
                pass
            self._stop.wait(max(self.period_s, 0.05))

    def start(self) -> "ClockSampler":
        # the sampling thread re-acquires the interpreter lock after every query; with the default 5 ms switch interval a
        # busy main thread would hold it off for most of a short timed region
        import sys
        if sys.getswitchinterval() > 0.0005:
            sys.setswitchinterval(0.0005)
        target = self._loop_nvml if self._init_nvml() else self._loop_smi
        self._thread = threading.Thread(target=target, daemon=True)
        self._thread.start()
        return self

    def stop(self) -> None:
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=10)

    def summary(self, t0: float, t1: float) -> Dict:
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed region"
        for pad in (0.05, 0.2):      # a region of a few milliseconds may hold fewer than three samples: say how far the window was widened
            if len(inside) >= 3:
                break
            inside = [s for s in self.samples if t0 - pad <= s[0] <= t1 + pad]
            window = f"timed region +-{int(pad * 1000)} ms (too short for 3 samples)"
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "window": window}
        mask = 0
        for s in inside:
            mask |= s[2]
        reasons = [k for k, b in {**self.BAD, **self.NOTED}.items() if mask & b]
        watts = [s[3] for s in inside if s[3] is not None]
        return {"sm_mhz": statistics.median(s[1] for s in inside), "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(inside), "window": window, "power_w": statistics.median(watts) if watts else None}


def aggregate(ms_local: float, units_local: float, world_size: int) -> Dict[str, float]:
    """Whole-job figure from per-rank timings: time = max over ranks, units = sum over ranks.

    With world_size > 1 this runs two all-reduces on the default process group (any backend).
    """
    if world_size <= 1:
        return {"ms": ms_local, "units": units_local}
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    u = torch.tensor([units_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return {"ms": float(t.item()), "units": float(u.item())}


def measured_peaks(root: str) -> Dict:
    """Measured peaks for this machine, else the stated fallback."""
    path = os.path.join(root, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": float(d["bf16_tflops"]), "bf16_tflops_sustained": float(d["bf16_tflops_sustained"]),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    except Exception:
        return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}
