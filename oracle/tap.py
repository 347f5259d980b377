"""Matrix steps of Temporal-Aware Parallel Clustering (section "Temporal-Aware Parallel Clustering for
Calibration", Algorithm 1) for ONE subsample.  Test infrastructure.

For a subsample of n calibration samples x_k (flattened features) with timestamps t_k:
    A_spatial[k,h]  = x_k . x_h / (|x_k| |x_h|)
    A_temporal[k,h] = exp(-|t_k - t_h|)
    A_final         = alpha A_spatial + (1 - alpha) A_temporal
    L               = D_r^e A_final D_c^e,   D_r = diag(row sums), D_c = diag(column sums)
The paper prints the exponent e = +1/2; the usual normalised adjacency has e = -1/2.  Both are available
(default: as printed).  Readings: the pairs are those inside the subsample (square n x n matrices, as in
Algorithm 1); a zero feature vector has similarity 0 with everything.  Eigenvectors, k-means and the aggregation
over subsamples are not part of this module.
"""
from __future__ import annotations

import numpy as np


def affinity(x, t, alpha: float) -> np.ndarray:
    """A_final [n,n], float64.  x [n,d], t [n]."""
    x = np.asarray(x, dtype=np.float64).reshape(len(x), -1)
    t = np.asarray(t, dtype=np.float64)
    norm = np.sqrt((x * x).sum(axis=1))
    safe = np.where(norm > 0, norm, 1.0)
    xn = x / safe[:, None]
    xn[norm == 0] = 0.0
    spatial = xn @ xn.T
    temporal = np.exp(-np.abs(t[:, None] - t[None, :]))
    return alpha * spatial + (1.0 - alpha) * temporal


def laplacian(A, exponent: float = 0.5) -> np.ndarray:
    """L = D_r^e A D_c^e with the row-sum and column-sum degrees of A."""
    A = np.asarray(A, dtype=np.float64)
    dr = A.sum(axis=1)
    dc = A.sum(axis=0)
    return (dr ** exponent)[:, None] * A * (dc ** exponent)[None, :]
