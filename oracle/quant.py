"""Uniform quantizer of the paper's Background section (Eq. 1-3).  Test infrastructure.

Q(X|b) = clip(round(X / s) + z, 0, 2^b - 1)                                  (Eq. 1)
l = min X, u = max X                                                        (Eq. 2)
s = (u - l) / (2^b - 1),  z = clip(round(-l / s), 0, 2^b - 1)                (Eq. 3)

Readings taken where the paper is silent or garbled:
  * Eq. 3 prints z on both sides; the inner "+z" is dropped.
  * round() is round-half-to-even.
  * X / s is evaluated as one float32 product X * (1/s) with 1/s rounded to
    float32 once; the rounding decision is taken in float32.
  * Besides the unsigned range of Eq. 1 a symmetric signed range [-127, 127]
    with z = 0 is supported (s = max|X| / 127); weights use it per output channel
    and activations per tensor (granularities as stated in the section
    "Comparison on Performance").
  * A degenerate range (u == l, or max|X| == 0) takes s = 1.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

F32 = np.float32


@dataclass(frozen=True)
class QParams:
    scale: float       # s, representable in float32
    zero_point: int    # z
    qmin: int
    qmax: int

    @property
    def inv_scale(self) -> np.float32:
        return F32(1.0) / F32(self.scale)


def qparams_minmax(X: np.ndarray, bits: int = 8) -> QParams:
    """Eq. 2-3: asymmetric parameters from the range of X; codes in [0, 2^b - 1]."""
    levels = (1 << bits) - 1
    l = F32(np.min(X))
    u = F32(np.max(X))
    s = F32(u - l) / F32(levels)
    if not s > 0:
        s = F32(1.0)
    z = int(np.clip(np.rint(np.float64(-l) / np.float64(s)), 0, levels))
    return QParams(float(s), z, 0, levels)


def qparams_symmetric(absmax: float, bits: int = 8) -> QParams:
    """Signed symmetric parameters: s = absmax / (2^(b-1) - 1), z = 0."""
    top = (1 << (bits - 1)) - 1
    s = F32(absmax) / F32(top)
    if not s > 0:
        s = F32(1.0)
    return QParams(float(s), 0, -top, top)


def quantize(X: np.ndarray, qp: QParams) -> np.ndarray:
    """Eq. 1.  X is rounded to float32 first; returns int32 codes in [qmin, qmax]."""
    x32 = np.asarray(X).astype(F32)
    r = np.rint(x32 * qp.inv_scale)          # float32 product, half-to-even
    r = r.astype(np.float64) + qp.zero_point
    return np.clip(r, qp.qmin, qp.qmax).astype(np.int32)


def quantize_per_token(X: np.ndarray):
    """Dynamic per-token (per-row) symmetric quantizer: Eq. 1 with s[m] = max_k |X[m,k]| / 127, z = 0, range
    [-127, 127] (s = 1 for an all-zero row).  Returns (codes int32 [M,K], scales float32 [M])."""
    x32 = np.asarray(X).astype(F32)
    s = (np.max(np.abs(x32), axis=1) / F32(127)).astype(F32)
    s[~(s > 0)] = F32(1.0)
    inv = (F32(1.0) / s).astype(F32)
    r = np.rint(x32 * inv[:, None])
    return np.clip(r, -127, 127).astype(np.int32), s


def dequantize(q: np.ndarray, qp: QParams) -> np.ndarray:
    """Inverse map of Eq. 1 inside the clip range: s * (q - z), float64."""
    return np.float64(F32(qp.scale)) * (np.asarray(q, dtype=np.float64) - qp.zero_point)


def quantize_weight_per_channel(W: np.ndarray, bits: int = 8):
    """Channel-wise symmetric weights: one scale per output row of W[N, K].

    Returns (q int32 [N,K], scale float32 [N], colsum int64 [N]) where
    colsum[n] = sum_k q[n,k] (needed to undo an activation zero-point).
    """
    W = np.asarray(W, dtype=F32)
    top = (1 << (bits - 1)) - 1
    absmax = np.max(np.abs(W), axis=1)
    s = (absmax / F32(top)).astype(F32)
    s[~(s > 0)] = F32(1.0)
    inv = (F32(1.0) / s).astype(F32)
    q = np.clip(np.rint(W * inv[:, None]), -top, top).astype(np.int32)
    return q, s, q.sum(axis=1, dtype=np.int64)


def pack_int4(q: np.ndarray) -> np.ndarray:
    """Storage form of 4-bit weight codes (the W4A8 setting of Table 2): two signed codes per byte.

    q: integer codes in [-8, 7], shape [N, K] with K even.  Byte j of a row holds code 2j in its low nibble and
    code 2j + 1 in its high nibble, each as a 4-bit two's-complement number.  Returns uint8 [N, K/2].
    (The byte layout is this build's choice: the paper fixes the code width only.)
    """
    q = np.asarray(q)
    if q.ndim != 2 or q.shape[1] % 2:
        raise ValueError("codes must be [N, K] with K even")
    if q.min(initial=0) < -8 or q.max(initial=0) > 7:
        raise ValueError("codes outside the 4-bit range [-8, 7]")
    n = (q.astype(np.int64) & 0xF).astype(np.uint8)
    return (n[:, 0::2] | (n[:, 1::2] << 4)).astype(np.uint8)


def unpack_int4(p: np.ndarray) -> np.ndarray:
    """Inverse of pack_int4: uint8 [N, K/2] -> int32 codes [N, K] (nibbles sign-extended)."""
    p = np.asarray(p, dtype=np.uint8)
    lo = (p & 0xF).astype(np.int32)
    hi = (p >> 4).astype(np.int32)
    lo = np.where(lo >= 8, lo - 16, lo)
    hi = np.where(hi >= 8, hi - 16, hi)
    out = np.empty((p.shape[0], 2 * p.shape[1]), dtype=np.int32)
    out[:, 0::2] = lo
    out[:, 1::2] = hi
    return out
