"""GPU parity: activation quantizer (Eq. 1), weight quantizer, LayerNorm + adaLN modulate, vs the oracle."""
import numpy as np
import pytest
import torch

import synth
from oracle import dit, quant
from oracle.quant import QParams

from gpu_util import bf16_to_f64, code_mismatch_report, dev, host_codes, max_rel_err

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


@pytest.mark.parametrize("M,K", [(1, 8), (3, 24), (257, 1152), (64, 4608), (1000, 384)])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("qp", [QParams(0.0371, 0, -127, 127), QParams(0.0521, 117, 0, 255)])
def test_quantize_act_static_bit_exact(q, ctx, M, K, dtype, qp):
    x = synth.outlier_activations(5, f"x{M}x{K}", M, K)
    x[0, :8] = np.array([0.5, 1.5, 2.5, -0.5, -1.5, 1e9, -1e9, 0.0], dtype=np.float32) * np.float32(qp.scale)
    if dtype == "bf16":
        xd = dev(x).to(torch.bfloat16)
        xh = bf16_to_f64(xd)
    else:
        xd = dev(x)
        xh = x
    out = torch.empty((M, K), dtype=torch.uint8, device="cuda")
    q.qdit_quantize_act(ctx, xd, q.QDIT_BF16 if dtype == "bf16" else q.QDIT_F32, M, K, K, q.QDIT_QUANT_STATIC,
                        q.qparams(qp.scale, qp.zero_point, qp.qmin, qp.qmax), None, out, K)
    q.qdit_sync(ctx)
    with np.errstate(over="ignore"):
        want = quant.quantize(xh, qp)
    np.testing.assert_array_equal(host_codes(out, signed=qp.qmin < 0), want)


def test_quantize_act_strided_and_empty(q, ctx):
    M, K, ldx, ldq = 37, 40, 64, 48
    x = synth.normal(6, "xs", (M, ldx))
    xd = dev(x)
    out = torch.full((M, ldq), 99, dtype=torch.uint8, device="cuda")
    qp = QParams(0.02, 0, -127, 127)
    q.qdit_quantize_act(ctx, xd, q.QDIT_F32, M, K, ldx, q.QDIT_QUANT_STATIC, q.qparams(qp.scale), None, out, ldq)
    q.qdit_quantize_act(ctx, xd, q.QDIT_F32, 0, K, ldx, q.QDIT_QUANT_STATIC, q.qparams(qp.scale), None, out, ldq)
    q.qdit_sync(ctx)
    got = host_codes(out)
    np.testing.assert_array_equal(got[:, :K], quant.quantize(x[:, :K], qp))
    assert (got[:, K:] == 99).all()          # padding untouched


def test_quantize_act_dynamic(q, ctx):
    M, K = 300, 1152
    x = synth.outlier_activations(7, "xd", M, K)
    xd = dev(x).to(torch.bfloat16)
    xh = bf16_to_f64(xd)
    out = torch.empty((M, K), dtype=torch.uint8, device="cuda")
    s = torch.zeros(1, dtype=torch.float32, device="cuda")
    for _ in range(2):                        # second call: the accumulator is cleared again
        q.qdit_quantize_act(ctx, xd, q.QDIT_BF16, M, K, K, q.QDIT_QUANT_DYNAMIC, None, s, out, K)
    q.qdit_sync(ctx)
    qp = quant.qparams_symmetric(float(np.abs(xh).max()))
    assert float(s.item()) == qp.scale
    np.testing.assert_array_equal(host_codes(out), quant.quantize(xh, qp))
    z = torch.zeros((8, 16), dtype=torch.float32, device="cuda")
    o2 = torch.empty((8, 16), dtype=torch.uint8, device="cuda")
    q.qdit_quantize_act(ctx, z, q.QDIT_F32, 8, 16, 16, q.QDIT_QUANT_DYNAMIC, None, s, o2, 16)
    q.qdit_sync(ctx)
    assert float(s.item()) == 1.0 and not o2.any()


def test_quantize_act_rejects_bad_arguments(q, ctx):
    x = torch.zeros((4, 16), dtype=torch.float32, device="cuda")
    o = torch.zeros((4, 16), dtype=torch.uint8, device="cuda")
    L = q.lib
    qp = q.qparams(0.1)
    import ctypes as C
    assert L.qdit_quantize_act(ctx, None, q.QDIT_F32, 4, 16, 16, 0, C.byref(qp), None, o.data_ptr(), 16) == q.QDIT_ERR_INVALID_ARG
    assert L.qdit_quantize_act(ctx, x.data_ptr(), q.QDIT_F32, 4, 12, 16, 0, C.byref(qp), None, o.data_ptr(), 16) == q.QDIT_ERR_SHAPE
    assert L.qdit_quantize_act(ctx, x.data_ptr() + 4, q.QDIT_F32, 4, 8, 16, 0, C.byref(qp), None, o.data_ptr(), 16) == q.QDIT_ERR_ALIGN
    bad = q.qparams(0.0)
    assert L.qdit_quantize_act(ctx, x.data_ptr(), q.QDIT_F32, 4, 16, 16, 0, C.byref(bad), None, o.data_ptr(), 16) == q.QDIT_ERR_INVALID_ARG
    bad = q.qparams(0.1, 0, -300, 127)
    assert L.qdit_quantize_act(ctx, x.data_ptr(), q.QDIT_F32, 4, 16, 16, 0, C.byref(bad), None, o.data_ptr(), 16) == q.QDIT_ERR_INVALID_ARG
    assert L.qdit_quantize_act(ctx, x.data_ptr(), q.QDIT_F32, 4, 16, 16, 1, None, None, o.data_ptr(), 16) == q.QDIT_ERR_INVALID_ARG
    assert b"dyn_scale" in L.qdit_last_error(ctx)
    q.qdit_sync(ctx)


@pytest.mark.parametrize("N,K", [(7, 16), (384, 1536), (1152, 4608), (600, 1152)])
def test_quantize_weight_bit_exact(q, ctx, N, K):
    W = synth.normal(8, f"w{N}x{K}", (N, K), 0.02)
    W[min(3, N - 1)] = 0
    wd = dev(W)
    qo = torch.empty((N, K), dtype=torch.int8, device="cuda")
    so = torch.empty(N, dtype=torch.float32, device="cuda")
    co = torch.empty(N, dtype=torch.int32, device="cuda")
    q.qdit_quantize_weight(ctx, wd, N, K, qo, so, co)
    q.qdit_sync(ctx)
    wq, ws, wc = quant.quantize_weight_per_channel(W)
    np.testing.assert_array_equal(qo.cpu().numpy().astype(np.int32), wq)
    np.testing.assert_array_equal(so.cpu().numpy(), ws)
    np.testing.assert_array_equal(co.cpu().numpy().astype(np.int64), wc)


@pytest.mark.parametrize("M,K,dtype", [(300, 1152, "bf16"), (64, 4608, "f32"), (5, 8, "f32"), (1030, 384, "bf16")])
def test_quantize_act_per_token_bit_exact(q, ctx, M, K, dtype):
    """Per-token dynamic mode: one scale per row, codes and scales bit-exact against the oracle."""
    x = synth.outlier_activations(12, f"tok{M}x{K}", M, K) * (1.0 + np.arange(M, dtype=np.float32)[:, None] % 7)
    x[min(3, M - 1)] = 0
    if dtype == "bf16":
        xd = dev(x).to(torch.bfloat16)
        xh = xd.float().cpu().numpy()
        code = q.QDIT_BF16
    else:
        xd, xh, code = dev(x), x, q.QDIT_F32
    out = torch.empty((M, K), dtype=torch.uint8, device="cuda")
    sc = torch.empty(M, dtype=torch.float32, device="cuda")
    q.qdit_quantize_act(ctx, xd, code, M, K, K, q.QDIT_QUANT_DYNAMIC_TOKEN, None, sc, out, K)
    q.qdit_sync(ctx)
    want_q, want_s = quant.quantize_per_token(xh)
    np.testing.assert_array_equal(sc.cpu().numpy(), want_s)
    np.testing.assert_array_equal(host_codes(out), want_q)
    assert q.lib.qdit_quantize_act(ctx, xd.data_ptr(), code, M, K, K, q.QDIT_QUANT_DYNAMIC_TOKEN, None, None, out.data_ptr(), K) == q.QDIT_ERR_INVALID_ARG


@pytest.mark.parametrize("bits", [4, 6, 2])
def test_quantize_weight_bits_bit_exact(q, ctx, bits):
    """b-bit channel-wise weights (bits = 4: the W4A8 setting of Table 2): codes, scales and code sums."""
    N, K = 384, 1536
    W = synth.normal(8, f"w{bits}b", (N, K), 0.02)
    W[5] = 0
    qo = torch.empty((N, K), dtype=torch.int8, device="cuda")
    so = torch.empty(N, dtype=torch.float32, device="cuda")
    co = torch.empty(N, dtype=torch.int32, device="cuda")
    q.qdit_quantize_weight_bits(ctx, dev(W), N, K, bits, qo, so, co)
    q.qdit_sync(ctx)
    wq, ws, wc = quant.quantize_weight_per_channel(W, bits)
    top = (1 << (bits - 1)) - 1
    got = qo.cpu().numpy().astype(np.int32)
    np.testing.assert_array_equal(got, wq)
    np.testing.assert_array_equal(so.cpu().numpy(), ws)
    np.testing.assert_array_equal(co.cpu().numpy().astype(np.int64), wc)
    assert got.min() == -top and got.max() == top
    import ctypes as C
    assert q.lib.qdit_quantize_weight_bits(ctx, dev(W).data_ptr(), N, K, 9, qo.data_ptr(), so.data_ptr(), co.data_ptr()) == q.QDIT_ERR_INVALID_ARG
    assert q.lib.qdit_quantize_weight_bits(ctx, dev(W).data_ptr(), N, K, 1, qo.data_ptr(), so.data_ptr(), co.data_ptr()) == q.QDIT_ERR_INVALID_ARG
    q.qdit_sync(ctx)


@pytest.mark.parametrize("B,T,D", [(2, 256, 384), (3, 64, 1152), (2, 8, 144), (1, 5, 2048), (5, 7, 8)])
def test_adaln_modulate_float_outputs(q, ctx, B, T, D):
    M = B * T
    x = synth.normal(9, f"lnx{D}", (M, D), 1.7, 0.3)
    mod = synth.normal(9, f"lnm{D}", (B, 6 * D), 0.4)
    xd = dev(x).to(torch.bfloat16)
    xh = bf16_to_f64(xd)
    md = dev(mod)
    shift, scale = md[:, :D], md[:, D:2 * D]
    ref = dit.layer_norm_modulate(xh, mod[:, :D], mod[:, D:2 * D], T)
    of = torch.empty((M, D), dtype=torch.float32, device="cuda")
    q.qdit_adaln_modulate(ctx, xd, M, D, T, 1e-6, shift, scale, 6 * D, of, q.QDIT_F32)
    ob = torch.empty((M, D), dtype=torch.bfloat16, device="cuda")
    q.qdit_adaln_modulate(ctx, xd, M, D, T, 1e-6, shift, scale, 6 * D, ob, q.QDIT_BF16)
    q.qdit_sync(ctx)
    assert max_rel_err(of.cpu().numpy(), ref) < 1e-4   # f32 arithmetic incl. cancellation in (x-mean) and +shift
    np.testing.assert_array_equal(bf16_to_f64(ob), dit.round_bf16(of.cpu().numpy()))


@pytest.mark.parametrize("B,T,D", [(2, 256, 384), (4, 256, 1152)])
def test_adaln_modulate_fused_quantizer(q, ctx, B, T, D):
    M = B * T
    x = synth.normal(10, f"lqx{D}", (M, D), 1.2)
    mod = synth.normal(10, f"lqm{D}", (B, 6 * D), 0.4)
    xd = dev(x).to(torch.bfloat16)
    xh = bf16_to_f64(xd)
    md = dev(mod)
    ref = dit.layer_norm_modulate(xh, mod[:, 3 * D:4 * D], mod[:, 4 * D:5 * D], T)
    qp = quant.qparams_symmetric(float(np.abs(ref).max()) * 0.5)     # some saturation on purpose
    out = torch.empty((M, D), dtype=torch.uint8, device="cuda")
    q.qdit_adaln_modulate(ctx, xd, M, D, T, 1e-6, md[:, 3 * D:4 * D], md[:, 4 * D:5 * D], 6 * D, out, q.QDIT_I8,
                          q.qparams(qp.scale))
    q.qdit_sync(ctx)
    got = host_codes(out)
    want = quant.quantize(ref, qp)
    pre = ref.astype(np.float32).astype(np.float64) * float(qp.inv_scale)
    # the kernel value differs from the oracle by <= 1e-4 relative -> in code units:
    tol = 1e-4 * np.abs(pre).max() + 1e-6
    n_bad, ok = code_mismatch_report(got, want, pre, tol)
    assert ok and n_bad <= 1e-3 * got.size, (n_bad, got.size)
    assert np.abs(got).max() == 127 and (np.abs(want) == 127).sum() > 3


@pytest.mark.parametrize("B,T,D,asym", [(3, 5, 384, False), (7, 33, 768, True), (2, 100, 1024, False), (5, 64, 1152, True),
                                        (3, 64, 1152, False), (2, 8, 144, True)])
def test_adaln_modulate_fused_quantizer_ragged_and_unsigned(q, ctx, B, T, D, asym):
    """Row counts that leave ragged row ranges per CTA, ranges that straddle two samples, the other widths of the
    two-wide kernel (768, 1024), a width it does not take (144), and Eq. 1's unsigned codes with a zero point."""
    M = B * T
    x = synth.normal(12, f"lrx{D}_{T}", (M, D), 1.3, -0.2)
    mod = synth.normal(12, f"lrm{D}_{T}", (B, 6 * D), 0.4)
    xd = dev(x).to(torch.bfloat16)
    xh = bf16_to_f64(xd)
    md = dev(mod)
    ref = dit.layer_norm_modulate(xh, mod[:, :D], mod[:, D:2 * D], T)
    if asym:
        qp = quant.qparams_minmax(ref * 0.6)                              # Eq. 2-3 range, saturating at both ends
    else:
        qp = quant.qparams_symmetric(float(np.abs(ref).max()) * 0.6)
    out = torch.empty((M, D), dtype=torch.uint8, device="cuda")
    q.qdit_adaln_modulate(ctx, xd, M, D, T, 1e-6, md[:, :D], md[:, D:2 * D], 6 * D, out, q.QDIT_I8,
                          q.qparams(qp.scale, qp.zero_point, qp.qmin, qp.qmax))
    q.qdit_sync(ctx)
    got = host_codes(out, signed=not asym)
    want = quant.quantize(ref, qp)
    pre = ref.astype(np.float32).astype(np.float64) * float(qp.inv_scale)
    tol = 1e-4 * np.abs(pre).max() + 1e-6
    n_bad, ok = code_mismatch_report(got, want, pre, tol)
    assert ok and n_bad <= 2e-3 * got.size, (n_bad, got.size)
    assert got.min() == qp.qmin and got.max() == qp.qmax
