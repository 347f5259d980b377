"""Quantized linear layer: exact integer product and its de-quantisation.  Test infrastructure.

An 8-bit weight / 8-bit activation layer ("W8A8", Table 1) computes, for codes
qa = Q(x) (Eq. 1, tensor-wise s_a, z_a) and qw[n,:] = Q(W[n,:]) (channel-wise
s_w[n], z = 0):

    acc[m,n] = sum_k qa[m,k] * qw[n,k]                       (exact integers)
    y[m,n]   = s_a*s_w[n] * (acc[m,n] - z_a * sum_k qw[n,k]) + bias[n]

which is sum_k deq(qa)[m,k] * deq(qw)[n,k] + bias[n] written with the integer
sum pulled out.  The product s_a*s_w[n] is formed in float32 (both scales are
float32 data); everything else is float64.
"""
from __future__ import annotations

import numpy as np

from .quant import F32, QParams


def gemm_i8(qa: np.ndarray, qw: np.ndarray) -> np.ndarray:
    """acc[M,N] = qa[M,K] @ qw[N,K]^T as exact int64.

    Uses the float64 matrix product as a library step: every partial sum is an
    integer below 2^53 (|code| <= 255, K < 2^37), so the result is exact.
    """
    a = np.asarray(qa, dtype=np.float64)
    w = np.asarray(qw, dtype=np.float64)
    acc = a @ w.T
    return np.rint(acc).astype(np.int64)


def dequant_affine(acc: np.ndarray, a_qp: QParams, w_scale: np.ndarray, w_colsum: np.ndarray,
                   bias: np.ndarray | None) -> np.ndarray:
    """y = (s_a*s_w[n]) * (acc - z_a*colsum[n]) + bias[n], float64 [M,N]."""
    sprod = (F32(a_qp.scale) * np.asarray(w_scale, dtype=F32)).astype(np.float64)
    t = acc.astype(np.float64) - np.float64(a_qp.zero_point) * np.asarray(w_colsum, dtype=np.float64)[None, :]
    y = t * sprod[None, :]
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :]
    return y


def w8a8_linear_per_token(qa: np.ndarray, a_scales: np.ndarray, qw: np.ndarray, w_scale: np.ndarray,
                          bias: np.ndarray | None) -> np.ndarray:
    """Quantized linear whose activations carry one scale per row (symmetric, z = 0):
    y[m,n] = (s_a[m] * s_w[n]) * acc[m,n] + bias[n], the scale product formed in float32; float64 [M,N]."""
    acc = gemm_i8(qa, qw).astype(np.float64)
    sprod = (np.asarray(a_scales, dtype=F32)[:, None] * np.asarray(w_scale, dtype=F32)[None, :]).astype(np.float64)
    y = acc * sprod
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :]
    return y


def w8a8_linear(qa: np.ndarray, a_qp: QParams, qw: np.ndarray, w_scale: np.ndarray, w_colsum: np.ndarray,
                bias: np.ndarray | None) -> np.ndarray:
    """Full quantized linear on already-quantized activations; float64 [M,N]."""
    return dequant_affine(gemm_i8(qa, qw), a_qp, w_scale, w_colsum, bias)
