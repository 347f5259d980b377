"""GPU parity: bf16 attention (and its fused output quantizer) vs the oracle."""
import numpy as np
import pytest
import torch

import synth
from oracle import dit, quant

from gpu_util import bf16_to_f64, code_mismatch_report, dev, host_codes

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


def _run(q, ctx, qkv_dev, B, T, H, dh, out_dtype, qp=None):
    D = H * dh
    M = B * T
    if out_dtype == q.QDIT_F32:
        out = torch.empty((M, D), dtype=torch.float32, device="cuda")
    elif out_dtype == q.QDIT_BF16:
        out = torch.empty((M, D), dtype=torch.bfloat16, device="cuda")
    else:
        out = torch.empty((M, D), dtype=torch.uint8, device="cuda")
    base = qkv_dev.data_ptr()
    q.qdit_attention(ctx, base, base + 2 * D, base + 4 * D, 3 * D, B, H, T, dh, 1.0 / np.sqrt(dh), out, out_dtype, qp)
    q.qdit_sync(ctx)
    return out


# Tolerance: the probabilities enter the P.V product as bf16 (relative step 2^-8, error <= 2^-9 each) and
# V is exact, so |o - o_ref| <= 2^-9 * max|v| in the worst case; everything else is f32.
def _tol(v):
    return 2.0 ** -9 * np.abs(v).max() * 1.1


@pytest.mark.parametrize("B,T,H,dh", [(2, 256, 6, 64), (2, 256, 16, 72), (1, 64, 2, 72), (1, 1024, 3, 72), (3, 128, 2, 64)])
def test_attention_matches_oracle(q, ctx, B, T, H, dh):
    D = H * dh
    x = synth.normal(51, f"qkv{T}.{H}.{dh}", (B * T, 3 * D), 1.0)
    x[:, :D] *= 2.0                                 # sharper softmax than pure noise
    xd = dev(x).to(torch.bfloat16)
    xh = bf16_to_f64(xd).reshape(B, T, 3, H, dh)
    ref = dit.attention(xh[:, :, 0], xh[:, :, 1], xh[:, :, 2]).reshape(B * T, D)
    got = _run(q, ctx, xd, B, T, H, dh, q.QDIT_F32).cpu().numpy().astype(np.float64)
    err = np.abs(got - ref).max()
    assert err <= _tol(xh[:, :, 2]), err
    assert np.sqrt(np.mean((got - ref) ** 2)) < 0.15 * _tol(xh[:, :, 2])     # typical error far below the bound
    gb = bf16_to_f64(_run(q, ctx, xd, B, T, H, dh, q.QDIT_BF16))
    np.testing.assert_array_equal(gb, dit.round_bf16(got))


@pytest.mark.parametrize("T", [128, 256])            # one key block (online kernel) / two (whole row in tensor memory)
def test_attention_special_cases(q, ctx, T):
    B, H, dh = 1, 2, 72
    D = H * dh
    x = synth.normal(52, "qkv0", (B * T, 3 * D), 1.0)
    x[:, :D] = 0                                     # zero queries -> mean of V
    xd = dev(x).to(torch.bfloat16)
    v = bf16_to_f64(xd)[:, 2 * D:]
    got = _run(q, ctx, xd, B, T, H, dh, q.QDIT_F32).cpu().numpy()
    np.testing.assert_allclose(got, np.broadcast_to(v.mean(axis=0, keepdims=True), got.shape), atol=_tol(v))
    # one dominant key per query -> that key's V row (softmax saturates)
    x = np.zeros((B * T, 3 * D), dtype=np.float32)
    perm = synth.stream(52, "perm").permutation(T)
    onehot = np.zeros((T, dh), dtype=np.float32)
    onehot[np.arange(T), np.arange(T) % dh] = 1.0
    codes = synth.normal(52, "codes", (T, dh), 1.0)
    codes /= np.linalg.norm(codes, axis=1, keepdims=True)
    for h in range(H):
        x[:, D + h * dh:D + (h + 1) * dh] = codes * 30.0           # keys
        x[:, h * dh:(h + 1) * dh] = codes[perm] * 30.0             # query t looks for key perm[t]
    x[:, 2 * D:] = synth.normal(52, "v", (T, D))
    xd = dev(x).to(torch.bfloat16)
    v = bf16_to_f64(xd)[:, 2 * D:]
    got = _run(q, ctx, xd, B, T, H, dh, q.QDIT_F32).cpu().numpy()
    np.testing.assert_allclose(got, v[perm], atol=_tol(v))


def test_attention_fused_quantizer(q, ctx):
    B, T, H, dh = 2, 256, 16, 72
    D = H * dh
    x = synth.normal(53, "qkvq", (B * T, 3 * D), 1.0)
    xd = dev(x).to(torch.bfloat16)
    xh = bf16_to_f64(xd).reshape(B, T, 3, H, dh)
    ref = dit.attention(xh[:, :, 0], xh[:, :, 1], xh[:, :, 2]).reshape(B * T, D)
    qp = quant.qparams_symmetric(float(np.abs(ref).max()) * 0.9)
    got = host_codes(_run(q, ctx, xd, B, T, H, dh, q.QDIT_I8, q.qparams(qp.scale)))
    gf = _run(q, ctx, xd, B, T, H, dh, q.QDIT_F32).cpu().numpy()
    # the codes are the quantizer (Eq. 1) applied to the kernel's own f32 output ...
    np.testing.assert_array_equal(got, quant.quantize(gf, qp))
    # ... and differ from the oracle's codes by at most one step, only where the oracle's value is
    # within the attention tolerance of a rounding boundary
    pre = ref.astype(np.float32).astype(np.float64) * float(qp.inv_scale)
    n_bad, ok = code_mismatch_report(got, quant.quantize(ref, qp), pre, _tol(xh[:, :, 2]) / qp.scale)
    assert ok, n_bad
    assert n_bad < 0.2 * got.size


def test_attention_start_stagger_changes_no_value(q, ctx):
    """The start delay of an SM's second CTA (a scheduling option) must not change a single output byte: 12 samples x
    16 heads x 2 query blocks = 384 CTAs, so the delayed group (CTAs 148..295) exists."""
    B, T, H, dh = 12, 256, 16, 72
    D = H * dh
    xd = dev(synth.normal(54, "qkvs", (B * T, 3 * D), 1.0)).to(torch.bfloat16)
    qp = q.qparams(0.01)
    assert q.qdit_get_option(ctx, q.QDIT_OPT_ATTN_STAGGER_NS) == 2000
    a = host_codes(_run(q, ctx, xd, B, T, H, dh, q.QDIT_I8, qp))
    try:
        for ns in (0, 20000):
            q.qdit_set_option(ctx, q.QDIT_OPT_ATTN_STAGGER_NS, ns)
            np.testing.assert_array_equal(host_codes(_run(q, ctx, xd, B, T, H, dh, q.QDIT_I8, qp)), a)
        assert q.lib.qdit_set_option(ctx, q.QDIT_OPT_ATTN_STAGGER_NS, 20001) == q.QDIT_ERR_INVALID_ARG
        assert q.lib.qdit_set_option(ctx, q.QDIT_OPT_ATTN_STAGGER_NS, -1) == q.QDIT_ERR_INVALID_ARG
    finally:
        q.qdit_set_option(ctx, q.QDIT_OPT_ATTN_STAGGER_NS, 2000)


def test_attention_rejects_bad_arguments(q, ctx):
    t = torch.zeros((64, 3 * 64), dtype=torch.bfloat16, device="cuda")
    o = torch.zeros((64, 64), dtype=torch.float32, device="cuda")
    f = q.lib.qdit_attention
    p = t.data_ptr()
    assert f(ctx, p, p + 128, p + 256, 192, 1, 1, 64, 48, 0.1, o.data_ptr(), q.QDIT_F32, None, None) == q.QDIT_ERR_SHAPE
    assert f(ctx, p, p + 128, p + 256, 192, 1, 1, 50, 64, 0.1, o.data_ptr(), q.QDIT_F32, None, None) == q.QDIT_ERR_SHAPE
    assert f(ctx, p, None, p + 256, 192, 1, 1, 64, 64, 0.1, o.data_ptr(), q.QDIT_F32, None, None) == q.QDIT_ERR_INVALID_ARG
    assert f(ctx, p, p + 128, p + 256, 192, 1, 1, 64, 64, 0.1, o.data_ptr(), q.QDIT_I8, None, None) == q.QDIT_ERR_INVALID_ARG
    q.qdit_sync(ctx)
