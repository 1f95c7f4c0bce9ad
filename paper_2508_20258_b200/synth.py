"""Seeded synthetic GEMM inputs, shared by the tests, the benchmark and the oracle's callers.

This module holds no arithmetic of the method: it only draws matrices and rounds them
to bf16 once, so that the CPU oracle and the GPU library are fed the very same bit
patterns.  The paper gives no GEMM shape, dtype or data ("medium problem sizes" only),
so these workloads stand in for it.

Recipe (fixed): ``rng = numpy.random.Generator(numpy.random.PCG64(seed))``; A is drawn
first, then B, from the same generator; the fp64 draw is narrowed to fp32 and then to
bf16 with round-to-nearest-even; matrices are returned as uint16 bit patterns.
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import Tuple

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    M: int
    N: int
    K: int
    dist: str          # "uniform" -> U[-1, 1);  "normal" -> N(0, std^2)
    std: float
    seed: int
    tile_m: int
    tile_n: int
    out_dtype: str     # "bf16" | "fp32"


WORKLOADS = {
    "cfg1": Workload("cfg1", 512, 512, 512, "uniform", 1.0, 0, 128, 128, "fp32"),
    "cfg2": Workload("cfg2", 4096, 4096, 4096, "uniform", 1.0, 1, 128, 256, "bf16"),
    "cfg3": Workload("cfg3", 8192, 8192, 8192, "normal", 1.0, 2, 256, 256, "bf16"),
    "cfg4": Workload("cfg4", 16384, 2048, 8192, "uniform", 1.0, 3, 256, 256, "bf16"),
    "cfg5": Workload("cfg5", 16384, 16384, 4096, "normal", 0.5, 4, 256, 256, "bf16"),
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _draw(rng: np.random.Generator, shape: Tuple[int, int], dist: str, std: float) -> np.ndarray:
    if dist == "uniform":
        x = rng.uniform(-1.0, 1.0, size=shape)
    elif dist == "normal":
        x = rng.normal(0.0, std, size=shape)
    else:
        raise ValueError(dist)
    return f32_to_bf16_bits(x.astype(np.float32))


def make_inputs(M: int, N: int, K: int, dist: str = "uniform", std: float = 1.0, seed: int = 0,
                b_is_nk: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """A [M, K] and B [K, N] (or B [N, K] when ``b_is_nk``) as uint16 bf16 bit patterns."""
    rng = np.random.Generator(np.random.PCG64(seed))
    A = _draw(rng, (M, K), dist, std)
    B = _draw(rng, (K, N), dist, std)
    if b_is_nk:
        B = np.ascontiguousarray(B.T)
    return A, B


def make_workload(name: str, b_is_nk: bool = False) -> Tuple[Workload, np.ndarray, np.ndarray]:
    w = WORKLOADS[name]
    A, B = make_inputs(w.M, w.N, w.K, w.dist, w.std, w.seed, b_is_nk)
    return w, A, B


def make_int_inputs(M: int, N: int, K: int, seed: int, lo: int = -2, hi: int = 2) -> Tuple[np.ndarray, np.ndarray]:
    """Small-integer matrices (exactly representable; every fp32 partial sum is exact)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    A = rng.integers(lo, hi + 1, size=(M, K)).astype(np.float32)
    B = rng.integers(lo, hi + 1, size=(K, N)).astype(np.float32)
    return f32_to_bf16_bits(A), f32_to_bf16_bits(B)
