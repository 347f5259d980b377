"""Pins for oracle.linear: brute-force integer products, structure, zero-point algebra, error bound."""
import numpy as np
import pytest

from oracle import linear, quant
from oracle.quant import QParams


def brute(qa, qw):
    M, K = qa.shape
    N = qw.shape[0]
    out = [[0] * N for _ in range(M)]
    for m in range(M):
        for n in range(N):
            acc = 0
            for k in range(K):
                acc += int(qa[m, k]) * int(qw[n, k])
            out[m][n] = acc
    return np.array(out, dtype=np.int64)


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (3, 5, 7), (17, 9, 32), (32, 31, 29)])
def test_gemm_matches_triple_loop(M, N, K):
    rng = np.random.default_rng(M * 100 + N * 10 + K)
    qa = rng.integers(-128, 128, (M, K))
    qw = rng.integers(-127, 128, (N, K))
    np.testing.assert_array_equal(linear.gemm_i8(qa, qw), brute(qa, qw))


def test_gemm_is_not_transposed_and_not_symmetric():
    # rectangular operands with distinct rows: A @ W^T, indexed [m, n]
    qa = np.array([[1, 2, 3], [4, 5, 6]])
    qw = np.array([[1, 0, 0], [0, 1, 0], [0, 0, 1], [1, 1, 1]])
    np.testing.assert_array_equal(linear.gemm_i8(qa, qw), [[1, 2, 3, 6], [4, 5, 6, 15]])


def test_gemm_structure_cases():
    K = 4608
    ones = np.ones((4, K), dtype=np.int32)
    assert (linear.gemm_i8(ones, ones[:3]) == K).all()
    A = np.random.default_rng(0).integers(-128, 128, (6, 24))
    np.testing.assert_array_equal(linear.gemm_i8(A, np.eye(24, dtype=np.int32)), A)
    # extremes stay exact and inside int32
    lo = np.full((2, K), -128)
    hi = np.full((2, K), 127)
    u8 = np.full((2, K), 255)
    assert (linear.gemm_i8(lo, lo) == 128 * 128 * K).all()
    assert (linear.gemm_i8(lo, hi) == -128 * 127 * K).all()
    assert (linear.gemm_i8(u8, hi) == 255 * 127 * K).all()
    assert 255 * 128 * K < 2 ** 31
    # linearity in W
    rng = np.random.default_rng(1)
    A = rng.integers(-128, 128, (5, 64))
    W1, W2 = rng.integers(-60, 60, (7, 64)), rng.integers(-60, 60, (7, 64))
    np.testing.assert_array_equal(linear.gemm_i8(A, W1 + W2), linear.gemm_i8(A, W1) + linear.gemm_i8(A, W2))


def test_zero_point_algebra():
    rng = np.random.default_rng(5)
    M, N, K = 6, 7, 48
    qa = rng.integers(0, 256, (M, K))
    qw = rng.integers(-127, 128, (N, K))
    a_qp = QParams(0.031, 113, 0, 255)
    s_w = rng.uniform(1e-3, 1e-2, N).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    got = linear.w8a8_linear(qa, a_qp, qw, s_w, qw.sum(axis=1), bias)
    # definition: sum_k deq(qa) * deq(qw) + bias
    want = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            sp = np.float64(np.float32(a_qp.scale) * s_w[n])
            want[m, n] = sp * sum((int(qa[m, k]) - 113) * int(qw[n, k]) for k in range(K)) + float(bias[n])
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    # a zero-point shift of the codes with the same real values leaves the output unchanged
    a_qp0 = QParams(0.031, 0, -128, 127)
    got0 = linear.w8a8_linear(qa - 113, a_qp0, qw, s_w, qw.sum(axis=1), bias)
    np.testing.assert_allclose(got, got0, rtol=1e-12, atol=1e-12)


def test_quantized_linear_within_analytic_error_bound():
    # |y_q - y_fp| <= sum_k (|x_k| s_w/2 + |w_k| s_a/2 + s_a s_w/4) for values inside the clip range
    rng = np.random.default_rng(11)
    M, N, K = 16, 12, 96
    x = rng.standard_normal((M, K)).astype(np.float32)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    b = (rng.standard_normal(N) * 0.02).astype(np.float32)
    qw, s_w, cs = quant.quantize_weight_per_channel(W)
    for a_qp in (quant.qparams_symmetric(float(np.abs(x).max())), quant.qparams_minmax(x)):
        y = linear.w8a8_linear(quant.quantize(x, a_qp), a_qp, qw, s_w, cs, b)
        ref = x.astype(np.float64) @ W.astype(np.float64).T + b
        s_a = a_qp.scale
        bound = (np.abs(x).astype(np.float64) @ np.ones((K, 1))) * (s_w[None, :] / 2) \
            + (np.abs(W).astype(np.float64).sum(axis=1))[None, :] * s_a / 2 + K * s_a * s_w[None, :] / 4
        assert (np.abs(y - ref) <= bound * (1 + 1e-4)).all()
        # and it is a real approximation, not garbage: typical error is far below the bound
        assert np.abs(y - ref).mean() < 0.2 * bound.mean()
