"""Matrix steps of Temporal-Aware Parallel Clustering (section "Temporal-Aware Parallel Clustering for
Calibration", Algorithm 1) for ONE subsample.  Test infrastructure.

For a subsample of n calibration samples x_k (flattened features) with timestamps t_k:
    A_spatial[k,h]  = x_k . x_h / (|x_k| |x_h|)
    A_temporal[k,h] = exp(-|t_k - t_h|)
    A_final         = alpha A_spatial + (1 - alpha) A_temporal
    L               = D_r^e A_final D_c^e,   D_r = diag(row sums), D_c = diag(column sums)
The paper prints the exponent e = +1/2; the usual normalised adjacency has e = -1/2.  Both are available
(default: as printed).  Readings: the pairs are those inside the subsample (square n x n matrices, as in
Algorithm 1); a zero feature vector has similarity 0 with everything.

The spectral step of Algorithm 1 follows: the top k eigenvectors of L (largest eigenvalues; L is symmetric
positive semi-definite whenever the degrees are positive, being a congruence of a sum of two Gram / kernel
matrices), k-means on the rows of the n x k eigenvector matrix, and the aggregation over the m subsamples.
The paper fixes none of the details of k-means or of the aggregation; the readings taken here:
  * rows are used as they are (no row normalisation);
  * k-means = Lloyd's iterations from a deterministic farthest-point start (first centre = row 0, each further
    centre = the row farthest from the centres chosen so far, ties to the lowest index), nearest centre by squared
    Euclidean distance with ties to the lowest centre, an emptied cluster keeps its centre, a fixed iteration count
    with early exit when no label changes;
  * aggregation: every cluster of a subsample is summarised by the mean of its members' unit-length features and
    the mean of their timestamps; the clusters of subsample i > 1 are matched one-to-one to those of subsample 1
    greedily by the same similarity measure as A_final (largest remaining entry first, ties to the lowest pair);
    matched summaries are averaged with the cluster sizes as weights; every sample of the whole dataset is then
    assigned to the aggregated cluster it is most similar to (ties to the lowest cluster).  This is linear in the
    dataset size per subsample, as the complexity the paper states for TAP.
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


def top_eigenvectors(L, k: int):
    """The k largest eigenvalues of the symmetric matrix L (descending) and their orthonormal eigenvectors [n,k]."""
    L = np.asarray(L, dtype=np.float64)
    w, V = np.linalg.eigh(0.5 * (L + L.T))
    order = np.argsort(-w, kind="stable")[:k]
    return w[order], V[:, order]


def kmeans(Y, k: int, iters: int = 50):
    """Lloyd's k-means on the rows of Y [n,p] from the farthest-point start described in the module header.
    Returns (labels int64 [n], centres float64 [k,p])."""
    Y = np.asarray(Y, dtype=np.float64)
    n = Y.shape[0]
    if not 1 <= k <= n:
        raise ValueError("need 1 <= k <= n")
    chosen = [0]
    dmin = ((Y - Y[0]) ** 2).sum(axis=1)
    for _ in range(1, k):
        nxt = int(np.argmax(dmin))          # first maximum = lowest index
        chosen.append(nxt)
        dmin = np.minimum(dmin, ((Y - Y[nxt]) ** 2).sum(axis=1))
    C = Y[chosen].copy()
    labels = np.full(n, -1, dtype=np.int64)
    for _ in range(iters):
        d2 = ((Y[:, None, :] - C[None, :, :]) ** 2).sum(axis=2)
        new = np.argmin(d2, axis=1)         # first minimum = lowest centre
        if np.array_equal(new, labels):
            break
        labels = new
        for c in range(k):
            members = Y[labels == c]
            if len(members):
                C[c] = members.mean(axis=0)
    return labels, C


def spectral_labels(x, t, alpha: float, k: int, exponent: float = 0.5, iters: int = 50):
    """One subsample of Algorithm 1: affinity -> L -> top-k eigenvectors -> k-means on the rows.
    Returns (labels [n], eigenvalues [k], eigenvectors [n,k])."""
    L = laplacian(affinity(x, t, alpha), exponent)
    w, V = top_eigenvectors(L, k)
    labels, _ = kmeans(V, k, iters)
    return labels, w, V


def _unit_rows(x):
    x = np.asarray(x, dtype=np.float64).reshape(len(x), -1)
    norm = np.sqrt((x * x).sum(axis=1))
    out = x / np.where(norm > 0, norm, 1.0)[:, None]
    out[norm == 0] = 0.0
    return out


def cluster_summaries(x, t, labels, k: int):
    """Per cluster: mean of the members' unit-length features [k,d], mean timestamp [k], size [k]."""
    xn = _unit_rows(x)
    t = np.asarray(t, dtype=np.float64)
    labels = np.asarray(labels)
    F = np.zeros((k, xn.shape[1]))
    tau = np.zeros(k)
    size = np.zeros(k, dtype=np.int64)
    for c in range(k):
        sel = labels == c
        size[c] = int(sel.sum())
        if size[c]:
            F[c] = xn[sel].mean(axis=0)
            tau[c] = t[sel].mean()
    return F, tau, size


def _similarity(Fa, ta, Fb, tb, alpha: float):
    return alpha * (_unit_rows(Fa) @ _unit_rows(Fb).T) + (1.0 - alpha) * np.exp(-np.abs(ta[:, None] - tb[None, :]))


def match_clusters(S):
    """Greedy one-to-one matching on a k x k similarity matrix: repeatedly the largest remaining entry (ties to the
    lowest row, then column).  Returns perm with perm[b] = row matched to column b."""
    S = np.array(S, dtype=np.float64)
    k = S.shape[0]
    perm = np.full(k, -1, dtype=np.int64)
    for _ in range(k):
        a, b = np.unravel_index(int(np.argmax(S)), S.shape)
        perm[b] = a
        S[a, :] = -np.inf
        S[:, b] = -np.inf
    return perm


def aggregate(subsamples, x_all, t_all, alpha: float, k: int):
    """Aggregation over the m subsamples (last step of Algorithm 1), as read in the module header.

    subsamples: list of (x_i [n,d], t_i [n], labels_i [n]).  x_all [N,d], t_all [N]: the whole dataset.
    Returns (labels of all N samples, aggregated feature summaries [k,d], aggregated timestamps [k])."""
    F0, tau0, size0 = cluster_summaries(*subsamples[0], k)
    accF = F0 * size0[:, None]
    accT = tau0 * size0
    accN = size0.astype(np.float64)
    for x_i, t_i, lab_i in subsamples[1:]:
        Fi, taui, sizei = cluster_summaries(x_i, t_i, lab_i, k)
        perm = match_clusters(_similarity(F0, tau0, Fi, taui, alpha))
        for b in range(k):
            a = perm[b]
            accF[a] += Fi[b] * sizei[b]
            accT[a] += taui[b] * sizei[b]
            accN[a] += sizei[b]
    safe = np.where(accN > 0, accN, 1.0)
    F = accF / safe[:, None]
    tau = accT / safe
    S = _similarity(np.asarray(x_all, dtype=np.float64).reshape(len(x_all), -1), np.asarray(t_all, dtype=np.float64), F, tau, alpha)
    return np.argmax(S, axis=1), F, tau
