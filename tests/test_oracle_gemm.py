"""Pins for the GEMM oracle: closed-form special cases, exact rational arithmetic on tiny
inputs, a library routine on medium sizes, and layout/subset consistency.  A dropped
term, a transposed operand, a wrong stride or a swapped B layout fails one of them."""

from fractions import Fraction

import numpy as np
import pytest

from oracle import gemm as G
from paper_2508_20258_b200 import synth


def _bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _f64(bits):
    return G.bf16_bits_to_f64(bits)


def test_widening_is_exact_and_rne():
    # 1 + 2^-8 is halfway between two bf16 values (1 and 1 + 2^-7): ties go to even (1.0)
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -0.5, 3.140625], dtype=np.float32)
    b = _bits(x)
    assert _f64(b).tolist() == [1.0, 1.0, 1.0 + 2.0 ** -6, -0.5, 3.140625]
    assert b[0] == 0x3F80


def test_identity_left_and_right():
    rng = np.random.default_rng(5)
    X = _bits(rng.uniform(-1, 1, (48, 48)))
    eye = _bits(np.eye(48))
    ref, S = G.gemm_full(eye, X)
    assert np.array_equal(ref, _f64(X))
    assert np.array_equal(S, np.abs(_f64(X)))
    ref, _ = G.gemm_full(X, eye)
    assert np.array_equal(ref, _f64(X))


def test_all_ones_gives_column_sums():
    rng = np.random.default_rng(6)
    B = _bits(rng.integers(-8, 9, (40, 24)))
    ones = _bits(np.ones((7, 40)))
    ref, _ = G.gemm_full(ones, B)
    assert np.array_equal(ref, np.tile(_f64(B).sum(axis=0), (7, 1)))


def test_stamp_matrices_reveal_position():
    """A[i,0] = 2^(i mod 8), B[0,j] = 2^-(j mod 16), zero elsewhere: C[i,j] is a power of
    two that names (i, j); a transposed operand or wrong stride cannot reproduce it."""
    M, N, K = 24, 40, 16
    A = np.zeros((M, K)); B = np.zeros((K, N))
    A[:, 0] = 2.0 ** (np.arange(M) % 8)
    B[0, :] = 2.0 ** -(np.arange(N) % 16)
    ref, _ = G.gemm_full(_bits(A), _bits(B))
    want = np.outer(A[:, 0], B[0, :])
    assert np.array_equal(ref, want)


def test_against_exact_rationals():
    rng = np.random.default_rng(7)
    A = _bits(rng.normal(0, 1, (5, 8)))
    B = _bits(rng.normal(0, 1, (8, 6)))
    ref, S = G.gemm_full(A, B)
    Af, Bf = _f64(A), _f64(B)
    for i in range(5):
        for j in range(6):
            exact = sum(Fraction(Af[i, k]) * Fraction(Bf[k, j]) for k in range(8))
            absx = sum(abs(Fraction(Af[i, k]) * Fraction(Bf[k, j])) for k in range(8))
            assert abs(Fraction(ref[i, j]) - exact) <= Fraction(1, 2 ** 45) * absx
            assert abs(Fraction(S[i, j]) - absx) <= Fraction(1, 2 ** 45) * absx


@pytest.mark.parametrize("M,N,K,seed", [(64, 96, 128, 0), (257, 129, 511, 1), (512, 512, 512, 2)])
def test_against_numpy_float64_matmul(M, N, K, seed):
    A, B = synth.make_inputs(M, N, K, "normal", 1.0, seed)
    ref, S = G.gemm_full(A, B)
    lib = _f64(A) @ _f64(B)
    libS = np.abs(_f64(A)) @ np.abs(_f64(B))
    assert np.max(np.abs(ref - lib) / S) <= 1e-12
    assert np.max(np.abs(S - libS) / S) <= 1e-12


def test_b_layouts_agree_and_subsets_agree():
    A, B = synth.make_inputs(96, 80, 64, "uniform", 1.0, 3)
    ref, S = G.gemm_full(A, B)
    ref2, S2 = G.gemm_full(A, np.ascontiguousarray(B.T), b_is_nk=True)
    assert np.array_equal(ref, ref2) and np.array_equal(S, S2)
    rows = [5, 0, 95, 17]
    sub, subS = G.gemm_rows(A, B, rows, 16, 48)
    assert np.array_equal(sub, ref[rows, 16:48]) and np.array_equal(subS, S[rows, 16:48])
    blk, _ = G.gemm_block(A, B, 32, 64, 8, 24)
    assert np.array_equal(blk, ref[32:64, 8:24])
    # thread count does not change any value (each row is summed by one thread, k ascending)
    one, _ = G.gemm_full(A, B, nthreads=1)
    assert np.array_equal(one, ref)


def test_compare_metric_flags_a_dropped_term_and_passes_rounding():
    A, B = synth.make_inputs(128, 128, 512, "normal", 1.0, 4)
    ref, S = G.gemm_full(A, B)
    # honest result: fp32-rounded reference, then rounded to bf16
    honest = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(ref.astype(np.float32))).astype(np.float64)
    assert G.compare(honest, ref, S)["max_err"] <= 2.0 ** -8 + 1e-6
    # drop the last k term everywhere
    Af, Bf = _f64(A), _f64(B)
    broken = ref - np.outer(Af[:, -1], Bf[-1, :])
    assert G.compare(broken, ref, S)["max_err"] > 1e-2


def test_input_recipe_is_deterministic_and_a_is_drawn_first():
    A1, B1 = synth.make_inputs(8, 6, 4, "uniform", 1.0, 0)
    A2, B2 = synth.make_inputs(8, 6, 4, "uniform", 1.0, 0)
    assert np.array_equal(A1, A2) and np.array_equal(B1, B2)
    rng = np.random.Generator(np.random.PCG64(0))
    a = rng.uniform(-1.0, 1.0, size=(8, 4)).astype(np.float32)
    assert np.array_equal(A1, synth.f32_to_bf16_bits(a))
    vals = synth.bf16_bits_to_f32(A1)
    assert vals.min() >= -1.0 and vals.max() <= 1.0
    w = synth.WORKLOADS["cfg5"]
    assert (w.M, w.N, w.K, w.std, w.seed) == (16384, 16384, 4096, 0.5, 4)


def test_strict_tier_is_a_diagnostic_that_honest_rounding_passes_and_a_dropped_term_fails():
    rng = np.random.default_rng(11)
    M, N, K = 24, 40, 512
    a = rng.standard_normal((M, K)).astype(np.float32)
    b = rng.standard_normal((K, N)).astype(np.float32)
    A = (a.view(np.uint32) >> 16).astype(np.uint16)              # truncation to bf16 bits: any bf16 values will do
    B = (b.view(np.uint32) >> 16).astype(np.uint16)
    ref, S = G.gemm_full(A, B)
    honest = G.bf16_bits_to_f64(((ref.astype(np.float32).view(np.uint32) + 0x8000) >> 16).astype(np.uint16))
    r = G.compare(honest, ref, S, K=K)
    assert r["strict_violations"] == 0 and r["max_err"] <= 1e-2
    broken = honest.copy()
    broken[3, 5] -= G.bf16_bits_to_f64(A[3:4, 7:8])[0, 0] * G.bf16_bits_to_f64(B[7:8, 5:6])[0, 0] + 0.5
    assert G.compare(broken, ref, S, K=K)["strict_violations"] >= 1
    assert G.compare(ref, ref, S, K=K, bf16_out=False)["strict_violations"] == 0
    assert G.compare(ref, ref, S)["strict_violations"] is None
