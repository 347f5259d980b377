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


def _blobs(rng, sizes, d, t_centres, spread=0.05):
    """Well separated groups: a private random direction and a private timestamp per group."""
    xs, ts, ys = [], [], []
    dirs = np.linalg.qr(rng.standard_normal((d, len(sizes))))[0].T      # orthonormal directions
    for g, (sz, tc) in enumerate(zip(sizes, t_centres)):
        xs.append(dirs[g] * (1.0 + rng.random((sz, 1))) + spread * rng.standard_normal((sz, d)))
        ts.append(tc + 0.01 * rng.standard_normal(sz))
        ys += [g] * sz
    return np.concatenate(xs), np.concatenate(ts), np.array(ys)


def _same_partition(a, b):
    pairs = set(zip(a.tolist(), b.tolist()))
    return len(pairs) == len(set(a.tolist())) == len(set(b.tolist()))


def test_top_eigenvectors_against_definition_and_block_structure():
    rng = np.random.default_rng(40)
    B = rng.standard_normal((9, 9))
    L = B @ B.T
    w, V = tap.top_eigenvectors(L, 3)
    assert np.all(np.diff(w) <= 0)
    np.testing.assert_allclose(L @ V, V * w, atol=1e-9)                   # eigen-pairs
    np.testing.assert_allclose(V.T @ V, np.eye(3), atol=1e-12)            # orthonormal
    assert abs(w[0] - np.linalg.norm(L, 2)) < 1e-9                        # largest eigenvalue of a PSD matrix = its 2-norm
    # block-diagonal matrix of all-ones blocks: the top eigenvectors are the block indicators
    Lb = np.zeros((7, 7))
    Lb[:3, :3] = 1.0
    Lb[3:, 3:] = 1.0
    wb, Vb = tap.top_eigenvectors(Lb, 2)
    np.testing.assert_allclose(wb, [4.0, 3.0], atol=1e-12)
    np.testing.assert_allclose(np.abs(Vb[:, 0]), np.r_[np.zeros(3), np.full(4, 0.5)], atol=1e-12)
    np.testing.assert_allclose(np.abs(Vb[:, 1]), np.r_[np.full(3, 3 ** -0.5), np.zeros(4)], atol=1e-12)


def test_kmeans_known_clusters_start_rule_and_fixed_point():
    rng = np.random.default_rng(41)
    centres = np.array([[0.0, 0.0], [10.0, 0.0], [0.0, 10.0]])
    truth = np.array([0, 1, 2, 0, 1, 2, 0, 0, 1, 2, 2, 1])
    Y = centres[truth] + 0.1 * rng.standard_normal((12, 2))
    labels, C = tap.kmeans(Y, 3)
    assert _same_partition(labels, truth)
    for c in range(3):                                                    # a fixed point: centres are member means
        np.testing.assert_allclose(C[c], Y[labels == c].mean(axis=0), atol=1e-12)
    d2 = ((Y[:, None] - C[None]) ** 2).sum(-1)
    np.testing.assert_array_equal(labels, d2.argmin(1))                   # and every point sits with its nearest centre
    assert labels[0] == 0                                                 # start rule: row 0 seeds centre 0
    # 1-D textbook case, k = 2: points {0, 1, 9, 10} -> {0,1} and {9,10}, centres 0.5 and 9.5
    l1, C1 = tap.kmeans(np.array([[0.0], [1.0], [9.0], [10.0]]), 2)
    assert l1.tolist() == [0, 0, 1, 1] and np.allclose(C1[:, 0], [0.5, 9.5])
    # k = n: every point its own cluster; k = 1: one cluster at the mean
    ln, _ = tap.kmeans(Y, 12)
    assert sorted(ln.tolist()) == list(range(12))
    l0, C0 = tap.kmeans(Y, 1)
    assert set(l0.tolist()) == {0} and np.allclose(C0[0], Y.mean(0))


def test_spectral_labels_recover_planted_groups():
    rng = np.random.default_rng(42)
    x, t, y = _blobs(rng, [9, 7, 8], d=16, t_centres=[0.0, 5.0, 10.0])
    shuffle = rng.permutation(len(y))
    x, t, y = x[shuffle], t[shuffle], y[shuffle]
    for exponent in (0.5, -0.5):
        labels, w, V = tap.spectral_labels(x, t, alpha=0.5, k=3, exponent=exponent)
        assert _same_partition(labels, y)
        L = tap.laplacian(tap.affinity(x, t, 0.5), exponent)
        np.testing.assert_allclose(L @ V, V * w, atol=1e-8 * abs(w[0]))
    # a clear spectral gap after the 3rd eigenvalue is what makes the groups recoverable
    L = tap.laplacian(tap.affinity(x, t, 0.5), -0.5)
    ev = np.sort(np.linalg.eigvalsh(L))[::-1]
    assert ev[2] > 0.8 and ev[3] < 0.3


def test_match_clusters_is_the_greedy_rule():
    S = np.array([[0.9, 0.8, 0.1], [0.95, 0.2, 0.3], [0.1, 0.7, 0.6]])
    # largest 0.95 at (1,0); then among rows {0,2} x cols {1,2}: 0.8 at (0,1); then (2,2)
    assert tap.match_clusters(S).tolist() == [1, 0, 2]
    assert tap.match_clusters(np.eye(4)[[2, 0, 3, 1]]).tolist() == [1, 3, 0, 2]


def test_aggregate_relabels_subsamples_consistently_and_covers_the_dataset():
    rng = np.random.default_rng(43)
    x, t, y = _blobs(rng, [40, 30, 50], d=24, t_centres=[0.0, 4.0, 8.0])
    N, k, alpha = len(y), 3, 0.6
    subs = []
    for i in range(3):
        idx = rng.choice(N, size=30, replace=False)
        labels, _, _ = tap.spectral_labels(x[idx], t[idx], alpha, k, exponent=-0.5)
        assert _same_partition(labels, y[idx])
        labels = (labels + i) % k                                         # arbitrary per-subsample cluster numbering
        subs.append((x[idx], t[idx], labels))
    final, F, tau = tap.aggregate(subs, x, t, alpha, k)
    assert final.shape == (N,) and _same_partition(final, y)              # whole dataset split into the planted groups
    # numbering follows subsample 1
    x0, t0, l0 = subs[0]
    F0, tau0, n0 = tap.cluster_summaries(x0, t0, l0, k)
    for c in range(k):
        assert abs(tau[c] - tau0[c]) < 0.05
    # a single subsample aggregates to its own summaries
    f1, F1, tau1 = tap.aggregate(subs[:1], x, t, alpha, k)
    np.testing.assert_allclose(F1, F0, atol=1e-12)
    np.testing.assert_allclose(tau1, tau0, atol=1e-12)
    # summaries by loops
    xn = x0 / np.linalg.norm(x0, axis=1, keepdims=True)
    for c in range(k):
        np.testing.assert_allclose(F0[c], xn[l0 == c].mean(0), atol=1e-12)
        assert n0[c] == (l0 == c).sum()
