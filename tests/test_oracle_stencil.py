"""Pins of the stencil oracle: closed forms, the textbook discrete Laplacian, a library correlation, and the
point-by-point definition.  Each would fail for a dropped neighbour, a wrong sign, swapped coefficients, a
transposed axis or a rim handled as interior."""

import numpy as np
import pytest
from scipy import ndimage

from oracle import stencil as S


def test_slices_equal_the_point_by_point_definition():
    rng = np.random.default_rng(0)
    for (M, N) in [(3, 3), (4, 7), (9, 5), (16, 12)]:
        x = rng.standard_normal((M, N))
        assert np.array_equal(S.stencil2d(x, 0.3, -0.7), S.stencil2d_points(x, 0.3, -0.7))


def test_impulse_response_is_the_star():
    x = np.zeros((7, 9))
    x[3, 4] = 2.0
    out = S.stencil2d(x, 0.5, 0.125)
    want = np.zeros((7, 9))
    want[3, 4] = 1.0
    want[2, 4] = want[4, 4] = want[3, 3] = want[3, 5] = 0.25
    assert np.array_equal(out, want)
    # asymmetric probe: distinct values on the four neighbours must each be weighted by c_neighbor only
    y = np.zeros((5, 5))
    y[1, 2], y[3, 2], y[2, 1], y[2, 3], y[2, 2] = 1.0, 10.0, 100.0, 1000.0, 7.0
    assert S.stencil2d(y, 2.0, 3.0)[2, 2] == 2.0 * 7.0 + 3.0 * 1111.0


def test_constant_and_linear_fields_are_fixed_points_when_weights_sum_to_one():
    M, N = 11, 13
    i, j = np.meshgrid(np.arange(M), np.arange(N), indexing="ij")
    for field in (np.full((M, N), 4.25), 3.0 * i - 2.0 * j + 5.0):
        out = S.stencil2d(field, 0.5, 0.125)            # 0.5 + 4 * 0.125 = 1
        assert np.array_equal(out, field)


def test_quadratic_field_gives_the_discrete_laplacian():
    M, N = 10, 8
    i, j = np.meshgrid(np.arange(M, dtype=np.float64), np.arange(N, dtype=np.float64), indexing="ij")
    f = i * i + 3.0 * j * j
    # neighbours sum to 4 f + (2 + 6): the 5-point Laplacian of i^2 + 3 j^2 is 2 + 6
    out = S.stencil2d(f, -4.0, 1.0)
    assert np.array_equal(out[1:-1, 1:-1], np.full((M - 2, N - 2), 8.0))
    assert np.array_equal(out[0], f[0]) and np.array_equal(out[:, -1], f[:, -1])      # rim carried over


def test_interior_matches_a_library_correlation():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((33, 47))
    k = np.array([[0.0, 0.2, 0.0], [0.2, -0.6, 0.2], [0.0, 0.2, 0.0]])
    lib = ndimage.correlate(x, k, mode="constant")
    out = S.stencil2d(x, -0.6, 0.2)
    assert np.allclose(out[1:-1, 1:-1], lib[1:-1, 1:-1], rtol=0, atol=1e-14)
    assert np.array_equal(out[0], x[0]) and np.array_equal(out[-1], x[-1])
    assert np.array_equal(out[:, 0], x[:, 0]) and np.array_equal(out[:, -1], x[:, -1])


def test_axes_are_not_interchangeable():
    # a field varying along i only: the stencil of its transpose is the transpose of its stencil, and the values
    # come from the two i neighbours plus twice the point itself (its j neighbours equal it)
    x = np.tile(np.array([0.0, 1.0, 4.0, 9.0, 16.0])[:, None], (1, 6))
    out = S.stencil2d(x, 0.0, 1.0)
    assert np.array_equal(out[1:-1, 1:-1], np.tile(np.array([6.0, 18.0, 38.0])[:, None], (1, 4)))
    assert np.array_equal(S.stencil2d(x.T, 0.0, 1.0), out.T)


@pytest.mark.parametrize("shape", [(1, 1), (1, 9), (2, 5), (6, 2)])
def test_grids_without_interior_are_copied(shape):
    x = np.arange(shape[0] * shape[1], dtype=np.float64).reshape(shape)
    assert np.array_equal(S.stencil2d(x, 9.0, 9.0), x)
    assert np.array_equal(S.stencil2d_points(x, 9.0, 9.0), x)


def test_magnitude_hand_case():
    """The error scale of the GPU tolerance, on a 3 x 3 grid worked by hand: the one interior point gets
    |c0||x11| + |c1|(|x01| + |x21| + |x10| + |x12|) = 0.5 * 5 + 0.25 * (2 + 8 + 4 + 6) = 7.5 (signs of the inputs
    and of the weights dropped), the rim its own absolute value."""
    x = np.array([[1.0, -2.0, 3.0], [-4.0, 5.0, -6.0], [7.0, -8.0, 9.0]])
    m = S.magnitude(x, -0.5, 0.25)
    want = np.abs(x)
    want[1, 1] = 7.5
    assert np.array_equal(m, want)
    # the plain stencil of the same grid cancels instead: -0.5 * 5 + 0.25 * (-2 - 8 - 4 - 6) = -7.5
    assert S.stencil2d(x, -0.5, 0.25)[1, 1] == -7.5
    # and with weights of one sign on a grid of one sign, magnitude and stencil coincide
    y = np.abs(x)
    assert np.array_equal(S.magnitude(y, 0.5, 0.25), S.stencil2d(y, 0.5, 0.25))
