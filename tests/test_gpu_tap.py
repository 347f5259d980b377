"""GPU parity of the spectral step of Temporal-Aware Parallel Clustering (Algorithm 1): eigenvectors, k-means and the
aggregation over subsamples, against oracle.tap.  Several answers are valid (an eigenvector's sign, rotations inside a
repeated eigenvalue, cluster numbering), so what is unique is compared (eigenvalues, the spanned subspace, the
partition) and the rest is checked for validity (eigen-residual, orthonormality)."""
import numpy as np
import pytest
import torch

from oracle import tap

from gpu_util import dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q():
    import paper_2503_02508_b200 as q
    return q


@pytest.fixture(scope="module")
def ctx(q):
    c = q.qdit_create(0, None)
    yield c
    q.qdit_destroy(c)


def _blobs(rng, sizes, d, t_centres, spread=0.05):
    """Well separated groups: a private random direction and a private timestamp per group."""
    xs, ts, ys = [], [], []
    dirs = np.linalg.qr(rng.standard_normal((d, len(sizes))))[0].T
    for g, (sz, tc) in enumerate(zip(sizes, t_centres)):
        xs.append(dirs[g] * (1.0 + rng.random((sz, 1))) + spread * rng.standard_normal((sz, d)))
        ts.append(tc + 0.01 * rng.standard_normal(sz))
        ys += [g] * sz
    return np.concatenate(xs).astype(np.float32), np.concatenate(ts).astype(np.float32), np.array(ys)


def _same_partition(a, b):
    pairs = set(zip(np.asarray(a).tolist(), np.asarray(b).tolist()))
    return len(pairs) == len(set(np.asarray(a).tolist())) == len(set(np.asarray(b).tolist()))


@pytest.mark.parametrize("sizes,d,n,m,exponent", [([50, 40, 30, 40], 32, 64, 3, -0.5), ([300, 200, 250, 150, 220, 180, 160, 240], 64, 256, 2, 0.5)])
def test_cluster_and_aggregate_match_the_oracle(q, ctx, sizes, d, n, m, exponent):
    rng = np.random.default_rng(601 + n)
    k, alpha = len(sizes), 0.6
    x_all, t_all, y_all = _blobs(rng, sizes, d, [3.0 * g for g in range(k)])
    N = len(y_all)
    idx = np.stack([rng.choice(N, size=n, replace=False) for _ in range(m)])
    for i in range(m):                      # every subsample sees every group
        assert len(set(y_all[idx[i]].tolist())) == k
    xs, ts = x_all[idx], t_all[idx]         # [m, n, d], [m, n]
    ws = torch.empty(q.qdit_tap_cluster_workspace(m, n, d, k), dtype=torch.float32, device="cuda")
    evals = torch.empty((m, k), dtype=torch.float32, device="cuda")
    evecs = torch.empty((m, n, k), dtype=torch.float32, device="cuda")
    labels = torch.empty((m, n), dtype=torch.int32, device="cuda")
    q.qdit_tap_cluster(ctx, dev(xs), dev(ts), m, n, d, alpha, exponent, k, 30, 50, ws, evals, evecs, labels)
    q.qdit_sync(ctx)
    ev, V, lab = evals.cpu().numpy().astype(np.float64), evecs.cpu().numpy().astype(np.float64), labels.cpu().numpy()
    subs = []
    for i in range(m):
        L = tap.laplacian(tap.affinity(xs[i], ts[i], alpha), exponent)
        w_o, V_o = tap.top_eigenvectors(L, k)
        assert np.all(np.diff(ev[i]) <= 1e-6 * w_o[0])
        np.testing.assert_allclose(ev[i], w_o, rtol=2e-4)                                   # eigenvalues
        np.testing.assert_allclose(V[i].T @ V[i], np.eye(k), atol=2e-4)                      # orthonormal columns
        assert np.abs(L @ V[i] - V[i] * ev[i]).max() <= 2e-3 * w_o[0]                        # eigen-residual
        sv = np.linalg.svd(V_o.T @ V[i], compute_uv=False)
        assert sv.min() > 1 - 1e-4                                                           # the same subspace (principal angles)
        lab_o, _ = tap.kmeans(V_o, k)
        assert _same_partition(lab[i], lab_o) and _same_partition(lab[i], y_all[idx[i]])     # the planted groups
        assert lab[i].min() == 0 and lab[i].max() == k - 1 and lab[i][0] == 0                # numbering: row 0 seeds centre 0
        subs.append((xs[i], ts[i], lab[i]))
    wa = torch.empty(q.qdit_tap_aggregate_workspace(m, n, d, k, N), dtype=torch.float32, device="cuda")
    lab_all = torch.empty(N, dtype=torch.int32, device="cuda")
    cent = torch.empty((k, d), dtype=torch.float32, device="cuda")
    tau = torch.empty(k, dtype=torch.float32, device="cuda")
    q.qdit_tap_aggregate(ctx, dev(xs), dev(ts), labels, m, n, d, k, alpha, dev(x_all), dev(t_all), N, wa, lab_all, cent, tau)
    q.qdit_sync(ctx)
    want_lab, want_F, want_tau = tap.aggregate(subs, x_all, t_all, alpha, k)
    np.testing.assert_array_equal(lab_all.cpu().numpy(), want_lab)
    np.testing.assert_allclose(cent.cpu().numpy(), want_F, atol=2e-6)
    np.testing.assert_allclose(tau.cpu().numpy(), want_tau, atol=2e-5)
    assert _same_partition(want_lab, y_all)                                                  # the whole dataset, planted groups


def test_cluster_argument_errors(q, ctx):
    f = q.lib.qdit_tap_cluster
    a = torch.zeros(64 * 64, dtype=torch.float32, device="cuda").data_ptr()
    assert f(ctx, a, a, 1, 60, 32, 0.5, 0.5, 4, 10, 10, a, a, a, a) == q.QDIT_ERR_SHAPE      # n not a multiple of 16
    assert f(ctx, a, a, 1, 16, 32, 0.5, 0.5, 12, 10, 10, a, a, a, a) == q.QDIT_ERR_SHAPE     # block of k + 8 vectors exceeds n
    assert f(ctx, a, None, 1, 64, 32, 0.5, 0.5, 4, 10, 10, a, a, a, a) == q.QDIT_ERR_INVALID_ARG
    assert q.qdit_tap_cluster_workspace(0, 64, 32, 4) == 0
