"""CPU oracle (test infrastructure, never on the product path) for the 2-D stencil workload.

The paper lists "Stencil 2D" among its science kernels (evaluation section; its swizzle is shown in
the appendix figure for the stencil kernel) and checks it against a CPU implementation, but does not
print the stencil itself.  Reading taken here: the 5-point star, one sweep, values on the rim of the
grid carried over unchanged,

    out[i, j] = c_center * in[i, j] + c_neighbor * (in[i-1, j] + in[i+1, j] + in[i, j-1] + in[i, j+1])
                                                              for 0 < i < M-1 and 0 < j < N-1,
    out[i, j] = in[i, j]                                      on the rim.

Written twice: by slices (used at test sizes) and point by point (tiny grids; pins the slices).
All arithmetic in float64.
"""

from __future__ import annotations

import numpy as np


def stencil2d(x: np.ndarray, c_center: float, c_neighbor: float) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    out = x.copy()
    if x.shape[0] >= 3 and x.shape[1] >= 3:
        out[1:-1, 1:-1] = c_center * x[1:-1, 1:-1] + c_neighbor * (x[:-2, 1:-1] + x[2:, 1:-1] + x[1:-1, :-2] + x[1:-1, 2:])
    return out


def stencil2d_points(x: np.ndarray, c_center: float, c_neighbor: float) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    M, N = x.shape
    out = np.empty_like(x)
    for i in range(M):
        for j in range(N):
            if i == 0 or j == 0 or i == M - 1 or j == N - 1:
                out[i, j] = x[i, j]
            else:
                out[i, j] = c_center * x[i, j] + c_neighbor * (x[i - 1, j] + x[i + 1, j] + x[i, j - 1] + x[i, j + 1])
    return out


def magnitude(x: np.ndarray, c_center: float, c_neighbor: float) -> np.ndarray:
    """Sum of the absolute values of the terms of each output: the scale rounding errors are measured against."""
    return stencil2d(np.abs(np.asarray(x, dtype=np.float64)), abs(c_center), abs(c_neighbor))
