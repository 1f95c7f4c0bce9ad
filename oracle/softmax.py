"""CPU oracle (test infrastructure, never on the product path) for the row softmax workload.

The paper's softmax case study re-orders the blocks of a softmax kernel in which every row is reduced in two phases
(first the maximum, then the exponentials and their sum), the row being cut into BLOCK_SIZE chunks handled by
different blocks.  The result has a plain definition, which is what this file writes out, in float64:

    out[i, j] = exp(x[i, j] - max_j x[i, :]) / sum_j exp(x[i, j] - max_j x[i, :])

Second, the chunked two-phase evaluation as the paper describes it -- per chunk a partial maximum m_c and a partial sum
s_c = sum exp(x - m_c); per row M = max_c m_c, S = sum_c s_c exp(m_c - M); out = exp(x - M) / S -- in plain loops; its only
role is to show (in the pins) that the chunked form is the definition re-associated, so that a kernel built that way can
be held to the definition.  Entries must be finite.
"""

from __future__ import annotations

import numpy as np


def softmax(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    if x.ndim != 2:
        raise ValueError("softmax works on the rows of a matrix")
    out = np.empty_like(x)
    for i in range(x.shape[0]):
        row = x[i]
        if row.size == 0:
            continue
        m = row.max()
        e = np.exp(row - m)
        out[i] = e / e.sum()
    return out


def softmax_chunked(x: np.ndarray, chunk: int) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    if chunk < 1:
        raise ValueError("chunk must be >= 1")
    M, N = x.shape
    out = np.empty_like(x)
    for i in range(M):
        parts = []
        for c0 in range(0, N, chunk):               # phase 1: one (maximum, sum) pair per chunk
            seg = x[i, c0:c0 + chunk]
            m = seg.max()
            parts.append((m, np.exp(seg - m).sum()))
        big = max(m for m, _ in parts)               # phase 2: combine, then normalise
        total = sum(s * np.exp(m - big) for m, s in parts)
        out[i] = np.exp(x[i] - big) / total
    return out
