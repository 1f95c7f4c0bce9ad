"""Transpose oracle (TEST INFRASTRUCTURE): out[j][i] = in[i][j], written out as the definition.

The tile order of the paper's transpose kernel only changes which block moves which tile;
the result is the plain transpose, bit for bit.
"""

from __future__ import annotations

import numpy as np


def transpose_loops(x: np.ndarray) -> np.ndarray:
    """The definition, element by element (small inputs)."""
    M, N = x.shape
    out = np.empty((N, M), dtype=x.dtype)
    for i in range(M):
        for j in range(N):
            out[j, i] = x[i, j]
    return out


def transpose(x: np.ndarray) -> np.ndarray:
    """The same result through the library's strided copy (any size)."""
    return np.ascontiguousarray(x.T)
