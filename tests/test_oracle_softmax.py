"""Pins of the softmax oracle: a hand case, closed forms, invariants, a library routine, and the chunked two-phase form
against the definition.  Each would fail for a missing maximum shift (overflow), a sum over the wrong axis, a dropped
chunk, or partial sums combined without their exp(m_c - M) weights."""

import numpy as np
import pytest
from scipy import special

from oracle import softmax as SM


def test_hand_case_with_logarithms():
    # exp(ln a) = a: rows [ln 1, ln 2, ln 3] and [ln 4, ln 4, ln 8] give [1/6, 2/6, 3/6] and [1/4, 1/4, 1/2]
    x = np.log(np.array([[1.0, 2.0, 3.0], [4.0, 4.0, 8.0]]))
    want = np.array([[1 / 6, 2 / 6, 3 / 6], [0.25, 0.25, 0.5]])
    assert np.allclose(SM.softmax(x), want, rtol=0, atol=1e-15)
    assert np.allclose(SM.softmax_chunked(x, 2), want, rtol=0, atol=1e-15)


def test_uniform_rows_and_single_columns():
    assert np.allclose(SM.softmax(np.full((3, 7), -2.5)), 1 / 7, rtol=0, atol=1e-16)
    assert np.array_equal(SM.softmax(np.array([[3.0], [-1e300]])), np.ones((2, 1)))


def test_rows_sum_to_one_and_shift_invariance_and_no_overflow():
    rng = np.random.default_rng(0)
    x = rng.normal(0, 30, size=(17, 301))
    y = SM.softmax(x)
    assert np.allclose(y.sum(axis=1), 1.0, rtol=0, atol=1e-14)
    assert (y >= 0).all() and (y <= 1).all()
    shift = rng.normal(0, 100, size=(17, 1))
    assert np.allclose(SM.softmax(x + shift), y, rtol=1e-10, atol=1e-300)   # a constant per row changes nothing
    big = SM.softmax(np.array([[1000.0, 1001.0, 999.0]]))                     # exp(1000) overflows float64: the shift must be there
    assert np.isfinite(big).all() and np.allclose(big, SM.softmax(np.array([[0.0, 1.0, -1.0]])), rtol=1e-12)
    assert np.argmax(y, axis=1).tolist() == np.argmax(x, axis=1).tolist()    # monotone: the largest entry stays the largest


def test_equals_the_library_routine():
    rng = np.random.default_rng(1)
    for shape in [(1, 1), (5, 2), (33, 1000), (4, 4097)]:
        x = rng.normal(0, 4, size=shape)
        assert np.allclose(SM.softmax(x), special.softmax(x, axis=1), rtol=1e-13, atol=1e-300)


def test_one_dominant_entry_takes_almost_everything():
    x = np.zeros((1, 1000))
    x[0, 123] = 50.0
    y = SM.softmax(x)
    assert y[0, 123] == pytest.approx(1.0 - 999 * np.exp(-50.0), rel=1e-12)
    assert np.allclose(np.delete(y[0], 123), np.exp(-50.0), rtol=1e-12)


@pytest.mark.parametrize("chunk", [1, 2, 7, 512, 4096])
def test_chunked_two_phase_form_is_the_definition(chunk):
    rng = np.random.default_rng(chunk)
    x = rng.normal(0, 10, size=(9, 1300))            # 1300 is not a multiple of any of the chunk widths but 1 and 2
    x[3, 700:] += 60.0                               # chunks whose maxima differ by far more than the spread inside them
    assert np.allclose(SM.softmax_chunked(x, chunk), SM.softmax(x), rtol=1e-12, atol=1e-300)
