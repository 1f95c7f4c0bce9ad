"""GEMM oracle driver: compiles ``gemm_oracle.c`` with gcc and calls it through ctypes.

TEST INFRASTRUCTURE.  The arithmetic lives in ``gemm_oracle.c`` (plain i-k-j loops,
fp64 accumulation of exactly-widened bf16 inputs).  This file only builds the shared
object, marshals numpy arrays, and states the comparison metric used by the parity
tests.
"""

from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
from typing import Dict, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gemm_oracle.c")
_LIB = None


def _cpu_tag() -> str:
    """The object is built with -march=native, so it is keyed by the host's ISA flags."""
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    with open(_SRC, "rb") as f:
        src = f.read()
    return hashlib.sha1(flags.encode() + src).hexdigest()[:12]


def lib_path() -> str:
    return os.path.join(_HERE, f"liboracle_{_cpu_tag()}.so")


def build(force: bool = False) -> str:
    """Compile the C oracle (idempotent).  Returns the path of the shared object."""
    out = lib_path()
    if force or not os.path.exists(out):
        tmp = out + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-march=native", "-fopenmp", "-fno-fast-math", "-std=c99", "-shared", "-fPIC",
               _SRC, "-o", tmp, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, out)
    return out


def _lib():
    global _LIB
    if _LIB is None:
        L = ctypes.CDLL(build())
        L.sp_oracle_gemm_rows.restype = ctypes.c_int
        L.sp_oracle_gemm_rows.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int,
            ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_int]
        L.sp_oracle_threads.restype = ctypes.c_int
        _LIB = L
    return _LIB


def threads() -> int:
    """Number of host threads the C oracle uses by default."""
    return int(_lib().sp_oracle_threads())


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def gemm_rows(A: np.ndarray, B: np.ndarray, rows: Sequence[int], c0: int = 0, c1: Optional[int] = None,
              b_is_nk: bool = False, nthreads: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """Rows ``rows`` and columns [c0, c1) of C = A.B in fp64, plus S = |A|.|B|.

    A: uint16 [M, K] bf16 bits.  B: uint16 [K, N] (default) or [N, K] when ``b_is_nk``.
    """
    A = np.ascontiguousarray(A, dtype=np.uint16)
    B = np.ascontiguousarray(B, dtype=np.uint16)
    M, K = A.shape
    if b_is_nk:
        N, K2 = B.shape
    else:
        K2, N = B.shape
    if K2 != K:
        raise ValueError("inner dimensions differ")
    if c1 is None:
        c1 = N
    rows_a = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    W = c1 - c0
    ref = np.empty((len(rows_a), W), dtype=np.float64)
    S = np.empty((len(rows_a), W), dtype=np.float64)
    rc = _lib().sp_oracle_gemm_rows(A.ctypes.data, B.ctypes.data, M, N, K, int(b_is_nk), rows_a.ctypes.data,
                                    len(rows_a), c0, c1, ref.ctypes.data, S.ctypes.data, nthreads)
    if rc != 0:
        raise ValueError("oracle rejected the arguments")
    return ref, S


def gemm_full(A: np.ndarray, B: np.ndarray, b_is_nk: bool = False, nthreads: int = 0):
    return gemm_rows(A, B, np.arange(A.shape[0]), 0, None, b_is_nk, nthreads)


def gemm_block(A: np.ndarray, B: np.ndarray, r0: int, r1: int, c0: int, c1: int, b_is_nk: bool = False,
               nthreads: int = 0):
    return gemm_rows(A, B, np.arange(r0, r1), c0, c1, b_is_nk, nthreads)


PHI = 2.0 ** -10


def compare(got: np.ndarray, ref: np.ndarray, S: np.ndarray, phi: float = PHI, K: int = 0, bf16_out: bool = True) -> Dict[str, float]:
    """Element-wise error of a GPU result against the oracle.

    err_ij = |got - ref| / max(|ref|, phi * S).  With zero-mean inputs a few outputs
    cancel to |ref| far below the rounding noise of ANY fp32 accumulation (which scales
    with S, not with ref), so the relative error is floored at phi * S; a dropped term
    or k-block is still orders of magnitude above 1e-2 * phi * S.
    Returns the gated figure (``max_err``) and diagnostics.  With ``K`` given, also counts (never gates) the elements
    outside the strict tier |got - ref| <= 2^-8 |ref| + 2 K 2^-24 S for bf16 output (half an ulp of the rounding to
    bf16 plus a worst-case fp32 accumulation) or <= 2 K 2^-24 S for fp32 output: ``strict_violations``.
    """
    got = np.asarray(got, dtype=np.float64)
    diff = np.abs(got - ref)
    floor = phi * S
    den = np.maximum(np.abs(ref), floor)
    den = np.where(den == 0.0, 1.0, den)          # all-zero row/column: diff must be 0
    err = diff / den
    unfloored = np.abs(ref) >= floor
    fro = float(np.sqrt((diff ** 2).sum()) / max(np.sqrt((ref ** 2).sum()), 1e-300))
    strict = None
    if K > 0:
        bound = 2.0 * K * 2.0 ** -24 * S + (2.0 ** -8 * np.abs(ref) if bf16_out else 0.0)
        strict = int((diff > bound).sum())
    return {
        "strict_violations": strict,
        "max_err": float(err.max()) if err.size else 0.0,
        "max_err_unfloored": float(err[unfloored].max()) if unfloored.any() else 0.0,
        "n_floored": int((~unfloored).sum()),
        "fro_rel": fro,
        "max_abs": float(diff.max()) if diff.size else 0.0,
        "n": int(err.size),
    }
