"""Pins for oracle.tap: the similarity matrices and the degree normalisation of Algorithm 1."""
import numpy as np

from oracle import tap


def test_affinity_definition_by_loops_and_special_cases():
    rng = np.random.default_rng(31)
    n, d = 7, 12
    x = rng.standard_normal((n, d))
    x[3] = 2.5 * x[1]                  # parallel vectors: cosine 1
    x[5] = 0                           # zero vector: similarity 0
    t = np.array([0, 1, 1, 5, 9, 2, 0], dtype=np.float64)
    alpha = 0.7
    A = tap.affinity(x, t, alpha)
    for k in range(n):
        for h in range(n):
            nk, nh = np.linalg.norm(x[k]), np.linalg.norm(x[h])
            cos = float(x[k] @ x[h]) / (nk * nh) if nk > 0 and nh > 0 else 0.0
            want = alpha * cos + (1 - alpha) * np.exp(-abs(t[k] - t[h]))
            assert abs(A[k, h] - want) < 1e-12
    np.testing.assert_allclose(A, A.T, atol=1e-15)
    assert abs(A[1, 3] - (alpha + (1 - alpha) * np.exp(-4.0))) < 1e-12      # parallel features, |dt| = 4
    assert abs(A[0, 6] - (alpha * (x[0] @ x[6]) / np.linalg.norm(x[0]) / np.linalg.norm(x[6]) + (1 - alpha))) < 1e-12
    np.testing.assert_allclose(tap.affinity(x, t, 0.0), np.exp(-np.abs(t[:, None] - t[None, :])), atol=1e-15)
    np.testing.assert_allclose(np.diag(tap.affinity(x[:5], t[:5], 1.0)), np.ones(5), atol=1e-12)
    # scale invariance of the spatial part
    np.testing.assert_allclose(tap.affinity(3.0 * x, t, alpha), A, atol=1e-12)


def test_laplacian_degrees_and_textbook_eigenvector():
    rng = np.random.default_rng(32)
    A = np.abs(rng.standard_normal((6, 6)))
    A = A + A.T
    d = A.sum(axis=1)
    L = tap.laplacian(A, 0.5)                  # as printed
    for k in range(6):
        for h in range(6):
            assert abs(L[k, h] - np.sqrt(d[k]) * A[k, h] * np.sqrt(d[h])) < 1e-12
    # the usual normalised adjacency D^-1/2 A D^-1/2 has eigenvalue 1 with eigenvector D^1/2 1
    Ln = tap.laplacian(A, -0.5)
    v = np.sqrt(d)
    np.testing.assert_allclose(Ln @ v, v, rtol=1e-12)
    assert np.max(np.abs(np.linalg.eigvalsh(Ln))) < 1 + 1e-12
    # rectangular input: row and column degrees differ
    R = np.abs(rng.standard_normal((4, 3)))
    Lr = tap.laplacian(R, 0.5)
    assert abs(Lr[2, 1] - np.sqrt(R[2].sum()) * R[2, 1] * np.sqrt(R[:, 1].sum())) < 1e-12
