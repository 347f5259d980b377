"""GPU parity: W8A8 linear (tcgen05 int8 GEMM + de-quantising epilogue) vs the oracle."""
import os

import numpy as np
import pytest
import torch

import synth
from oracle import dit, linear, quant
from oracle.quant import QParams

from gpu_util import bf16_steps_err, bf16_to_f64, code_mismatch_report, dev, dev_i8, host_codes, max_rel_err

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


def _codes(seed, name, shape, lo, hi):
    return synth.uniform_int(seed, name, shape, lo, hi + 1)


def _run_i32(q, ctx, qa, qw, a_unsigned=False):
    M, K = qa.shape
    N = qw.shape[0]
    A, W = dev_i8(qa), dev_i8(qw)
    out = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    qp = q.qparams(1.0, 0, 0, 255) if a_unsigned else q.qparams(1.0)
    q.qdit_w8a8_linear(ctx, A, W, M, N, K, qp, None, q.QDIT_EPI_OUT_I32, None, out, N)
    q.qdit_sync(ctx)
    return out.cpu().numpy().astype(np.int64)


SHAPES = [(1, 8, 16), (128, 192, 128), (130, 200, 272), (256, 384, 1152), (517, 1152, 4608), (512, 1152, 384),
          (1000, 3456, 1152), (64, 6912, 1152), (2048, 64, 64), (129, 1536, 384)]


def _select_kernel(q, ctx, variant):
    """"NNN": token-major kernel with 128 x NNN tiles; "tNNN": channel-major kernel with 128 x NNN tiles; else automatic."""
    q.qdit_set_option(ctx, q.QDIT_OPT_GEMM_BN, 0)
    q.qdit_set_option(ctx, q.QDIT_OPT_GEMM_T, 0)
    if variant.startswith("t"):
        q.qdit_set_option(ctx, q.QDIT_OPT_GEMM_T, int(variant[1:]))
    elif variant.isdigit():
        q.qdit_set_option(ctx, q.QDIT_OPT_GEMM_BN, int(variant))


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("bn", ["auto", "64", "128", "192", "t128", "t256"])
def test_accumulators_bit_exact(q, ctx, M, N, K, bn):
    _select_kernel(q, ctx, bn)
    try:
        qa = _codes(31, f"a{M}.{K}", (M, K), -128, 127)
        qw = _codes(31, f"w{N}.{K}", (N, K), -127, 127)
        got = _run_i32(q, ctx, qa, qw)
    finally:
        _select_kernel(q, ctx, "auto")
    np.testing.assert_array_equal(got, linear.gemm_i8(qa, qw))


def test_accumulators_extremes_and_structure(q, ctx):
    K = 4608
    lo = np.full((130, K), -128)
    hi = np.full((200, K), 127)
    assert (_run_i32(q, ctx, lo, hi) == -128 * 127 * K).all()
    u8 = np.full((130, K), 255)
    assert (_run_i32(q, ctx, u8, hi, a_unsigned=True) == 255 * 127 * K).all()
    # identity weights return the activations; catches any K-offset / swizzle / transposition slip
    A = _codes(32, "aid", (300, 256), -128, 127)
    np.testing.assert_array_equal(_run_i32(q, ctx, A, np.eye(256, dtype=np.int64)), A)
    # one-hot rows pick single weights
    W = _codes(32, "wsel", (200, 1152), -127, 127)
    onehot = np.zeros((128, 1152), dtype=np.int64)
    ks = synth.uniform_int(32, "ks", (128,), 0, 1152)
    onehot[np.arange(128), ks] = 1
    np.testing.assert_array_equal(_run_i32(q, ctx, onehot, W), W[:, ks].T)


def test_unsigned_activations_bit_exact(q, ctx):
    qa = _codes(33, "au", (260, 1152), 0, 255)
    qw = _codes(33, "wu", (392, 1152), -127, 127)
    np.testing.assert_array_equal(_run_i32(q, ctx, qa, qw, a_unsigned=True), linear.gemm_i8(qa, qw))


def test_repeatable(q, ctx):
    qa = _codes(34, "ar", (1024, 1152), -128, 127)
    qw = _codes(34, "wr", (1152, 1152), -127, 127)
    a = _run_i32(q, ctx, qa, qw)
    b = _run_i32(q, ctx, qa, qw)
    np.testing.assert_array_equal(a, b)


def _layer(seed, M, N, K, T, a_qp):
    x = synth.outlier_activations(seed, "x", M, K, gain=6.0)
    Wf = synth.normal(seed, "W", (N, K), 0.02)
    bias = synth.normal(seed, "b", (N,), 0.02)
    gate = synth.normal(seed, "g", (-(-M // T), N), 0.35)
    resid = synth.normal(seed, "r", (M, N), 1.0)
    qw, s_w, cs = quant.quantize_weight_per_channel(Wf)
    qa = quant.quantize(x, a_qp)
    return dict(qa=qa, qw=qw, s_w=s_w, cs=cs, bias=bias, gate=gate, resid=resid)


@pytest.mark.parametrize("M,N,K,T", [(512, 384, 384, 256), (300, 200, 1152, 100), (1024, 1152, 4608, 256)])
@pytest.mark.parametrize("a_qp", [QParams(0.05, 0, -127, 127), QParams(0.047, 131, 0, 255)])
def test_dequant_bias_f32(q, ctx, M, N, K, T, a_qp):
    L = _layer(41, M, N, K, T, a_qp)
    A, W = dev_i8(L["qa"]), dev_i8(L["qw"])
    epi = q.epilogue(w_scale=dev(L["s_w"]), w_colsum=dev(L["cs"].astype(np.int32)), bias=dev(L["bias"]))
    keep = [epi]
    ws, wc, bi = dev(L["s_w"]), dev(L["cs"].astype(np.int32)), dev(L["bias"])
    epi = q.epilogue(w_scale=ws, w_colsum=wc, bias=bi)
    out = torch.empty((M, N), dtype=torch.float32, device="cuda")
    q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(a_qp.scale, a_qp.zero_point, a_qp.qmin, a_qp.qmax), None,
                       q.QDIT_EPI_BIAS | q.QDIT_EPI_OUT_F32, epi, out, N)
    q.qdit_sync(ctx)
    ref = linear.w8a8_linear(L["qa"], a_qp, L["qw"], L["s_w"], L["cs"], L["bias"])
    assert max_rel_err(out.cpu().numpy(), ref) < 1e-3      # the stated layer tolerance ...
    assert max_rel_err(out.cpu().numpy(), ref) < 1e-5      # ... and what f32 arithmetic actually gives


@pytest.fixture(params=["single", "192", "t128", "t256"])
def kernel_variant(request, q, ctx):
    _select_kernel(q, ctx, request.param)
    yield request.param
    _select_kernel(q, ctx, "auto")


def test_gate_residual_cache_epilogue(q, ctx, kernel_variant):
    M, N, K, T = 512, 1152, 1152, 256
    a_qp = QParams(0.05, 0, -127, 127)
    L = _layer(42, M, N, K, T, a_qp)
    A, W = dev_i8(L["qa"]), dev_i8(L["qw"])
    ws, bi, g = dev(L["s_w"]), dev(L["bias"]), dev(L["gate"])
    x = dev(L["resid"]).to(torch.bfloat16)
    xh = bf16_to_f64(x)
    cache = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    epi = q.epilogue(w_scale=ws, bias=bi, gate=g, ld_gate=N, tokens_per_sample=T, residual=x, cache_out=cache)
    flags = q.QDIT_EPI_BIAS | q.QDIT_EPI_GATE | q.QDIT_EPI_RESIDUAL | q.QDIT_EPI_CACHE_STORE | q.QDIT_EPI_OUT_BF16
    q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None, flags, epi, x, N)    # in place on x
    q.qdit_sync(ctx)
    f = linear.w8a8_linear(L["qa"], a_qp, L["qw"], L["s_w"], L["cs"], L["bias"])
    rows = np.arange(M) // T
    want_x = xh + L["gate"].astype(np.float64)[rows] * f
    # bf16 outputs: equal to the rounded oracle value up to one bf16 step where f32 and f64 straddle a tie
    got_c, got_x = bf16_to_f64(cache), bf16_to_f64(x)
    assert np.abs(got_c - dit.round_bf16(f)).max() <= 2.0 ** -8 * np.abs(f).max()
    assert (got_c != dit.round_bf16(f)).mean() < 1e-3
    assert (got_x != dit.round_bf16(want_x)).mean() < 1e-3
    assert max_rel_err(got_x, want_x) < 2.0 ** -8


def test_bias_bf16_epilogue(q, ctx, kernel_variant):
    # the QKV layer's epilogue, on ragged sizes (M, N not multiples of the tiles)
    M, N, K, T = 300, 1096, 384, 100
    a_qp = QParams(0.045, 0, -127, 127)
    L = _layer(45, M, N, K, T, a_qp)
    A, W = dev_i8(L["qa"]), dev_i8(L["qw"])
    ws, bi = dev(L["s_w"]), dev(L["bias"])
    out = torch.full((M, N), 7.0, dtype=torch.bfloat16, device="cuda")
    q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None, q.QDIT_EPI_BIAS | q.QDIT_EPI_OUT_BF16,
                       q.epilogue(w_scale=ws, bias=bi), out, N)
    q.qdit_sync(ctx)
    f = linear.w8a8_linear(L["qa"], a_qp, L["qw"], L["s_w"], L["cs"], L["bias"])
    got = bf16_to_f64(out)
    assert (got != dit.round_bf16(f)).mean() < 1e-3
    assert np.abs(got - f).max() <= 2.0 ** -8 * np.abs(f).max()


def test_gelu_requant_epilogue(q, ctx, kernel_variant):
    M, N, K, T = 384, 1536, 384, 128
    a_qp = QParams(0.04, 0, -127, 127)
    L = _layer(43, M, N, K, T, a_qp)
    A, W = dev_i8(L["qa"]), dev_i8(L["qw"])
    ws, bi = dev(L["s_w"]), dev(L["bias"])
    u = dit.gelu_tanh(linear.w8a8_linear(L["qa"], a_qp, L["qw"], L["s_w"], L["cs"], L["bias"]))
    o_qp = quant.qparams_symmetric(float(np.abs(u).max()) * 0.9)
    epi = q.epilogue(w_scale=ws, bias=bi, out_qp=q.qparams(o_qp.scale))
    out = torch.empty((M, N), dtype=torch.uint8, device="cuda")
    q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None,
                       q.QDIT_EPI_BIAS | q.QDIT_EPI_GELU | q.QDIT_EPI_QUANT_OUT, epi, out, N)
    outf = torch.empty((M, N), dtype=torch.float32, device="cuda")
    q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None,
                       q.QDIT_EPI_BIAS | q.QDIT_EPI_GELU | q.QDIT_EPI_OUT_F32, epi, outf, N)
    q.qdit_sync(ctx)
    assert max_rel_err(outf.cpu().numpy(), u) < 1e-3
    assert max_rel_err(outf.cpu().numpy(), u) < 2e-5
    got, want = host_codes(out), quant.quantize(u, o_qp)
    pre = u.astype(np.float32).astype(np.float64) * float(o_qp.inv_scale)
    n_bad, ok = code_mismatch_report(got, want, pre, 2e-5 * np.abs(pre).max() + 1e-6)
    assert ok and n_bad <= 1e-3 * got.size, (n_bad, got.size)
    # the fused codes are exactly the quantizer applied to the kernel's own f32 values
    np.testing.assert_array_equal(got, quant.quantize(outf.cpu().numpy(), o_qp))


@pytest.mark.parametrize("M,N,K", [(300, 384, 1152), (1024, 2304, 256)])
def test_per_token_scales(q, ctx, kernel_variant, M, N, K):
    """Per-token activation scales (QDIT_EPI_ROW_SCALE): quantizer in per-token mode, then the linear layer."""
    x = synth.outlier_activations(45, f"pt{M}", M, K) * (1.0 + (np.arange(M, dtype=np.float32)[:, None] % 5))
    W = synth.normal(45, f"ptw{N}", (N, K), 0.02)
    bias = synth.normal(45, f"ptb{N}", (N,), 0.02)
    wq, ws, wc = quant.quantize_weight_per_channel(W)
    qa, sa = quant.quantize_per_token(x)
    ref = linear.w8a8_linear_per_token(qa, sa, wq, ws, bias)
    a8 = torch.empty((M, K), dtype=torch.uint8, device="cuda")
    sc = torch.empty(M, dtype=torch.float32, device="cuda")
    q.qdit_quantize_act(ctx, dev(x), q.QDIT_F32, M, K, K, q.QDIT_QUANT_DYNAMIC_TOKEN, None, sc, a8, K)
    out = torch.empty((M, N), dtype=torch.float32, device="cuda")
    ws_d, bias_d, wq_d = dev(ws), dev(bias), dev_i8(wq)     # the epilogue struct holds raw addresses: keep the tensors alive
    epi = q.epilogue(w_scale=ws_d, bias=bias_d, a_scale_rows=sc)
    q.qdit_w8a8_linear(ctx, a8, wq_d, M, N, K, q.qparams(1.0), None,
                       q.QDIT_EPI_BIAS | q.QDIT_EPI_OUT_F32 | q.QDIT_EPI_ROW_SCALE, epi, out, N)
    q.qdit_sync(ctx)
    assert max_rel_err(out.cpu().numpy(), ref) < 1e-5
    # closer to the un-quantized product than one tensor-wide scale is, on rows of very different magnitude
    exact = x.astype(np.float64) @ W.astype(np.float64).T + bias
    qp = quant.qparams_symmetric(float(np.abs(x).max()))
    tens = linear.w8a8_linear(quant.quantize(x, qp), qp, wq, ws, wc, bias)
    small = np.arange(M) % 5 == 0
    assert np.abs(out.cpu().numpy()[small] - exact[small]).mean() < np.abs(tens[small] - exact[small]).mean()
    # the flag needs its scales and a symmetric quantizer
    L = q.lib
    import ctypes as C
    bad = q.epilogue(w_scale=ws_d, bias=bias_d)
    assert L.qdit_w8a8_linear(ctx, a8.data_ptr(), wq_d.data_ptr(), M, N, K, q.qparams(1.0), None,
                              q.QDIT_EPI_BIAS | q.QDIT_EPI_OUT_F32 | q.QDIT_EPI_ROW_SCALE, C.byref(bad), out.data_ptr(), N) == q.QDIT_ERR_INVALID_ARG


def test_device_scale_override(q, ctx):
    M, N, K = 256, 192, 256
    a_qp = QParams(0.05, 0, -127, 127)
    L = _layer(44, M, N, K, 256, a_qp)
    A, W, ws = dev_i8(L["qa"]), dev_i8(L["qw"]), dev(L["s_w"])
    sd = dev(np.array([a_qp.scale], dtype=np.float32))
    out = torch.empty((M, N), dtype=torch.float32, device="cuda")
    q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(123.0), sd, q.QDIT_EPI_OUT_F32, q.epilogue(w_scale=ws), out, N)
    q.qdit_sync(ctx)
    ref = linear.w8a8_linear(L["qa"], a_qp, L["qw"], L["s_w"], L["cs"], None)
    assert max_rel_err(out.cpu().numpy(), ref) < 1e-5


def test_rejects_bad_arguments(q, ctx):
    import ctypes as C
    A = torch.zeros((128, 64), dtype=torch.int8, device="cuda")
    W = torch.zeros((64, 64), dtype=torch.int8, device="cuda")
    o = torch.zeros((128, 64), dtype=torch.int32, device="cuda")
    L, qp = q.lib, q.qparams(1.0)
    f = L.qdit_w8a8_linear
    assert f(ctx, A.data_ptr(), W.data_ptr(), 128, 64, 24, qp, None, q.QDIT_EPI_OUT_I32, None, o.data_ptr(), 64) == q.QDIT_ERR_SHAPE
    assert f(ctx, A.data_ptr(), W.data_ptr(), 128, 60, 64, qp, None, q.QDIT_EPI_OUT_I32, None, o.data_ptr(), 64) == q.QDIT_ERR_SHAPE
    assert f(ctx, None, W.data_ptr(), 128, 64, 64, qp, None, q.QDIT_EPI_OUT_I32, None, o.data_ptr(), 64) == q.QDIT_ERR_INVALID_ARG
    assert f(ctx, A.data_ptr() + 1, W.data_ptr(), 128, 64, 64, qp, None, q.QDIT_EPI_OUT_I32, None, o.data_ptr(), 64) == q.QDIT_ERR_ALIGN
    assert f(ctx, A.data_ptr(), W.data_ptr(), 128, 64, 64, qp, None, 0, None, o.data_ptr(), 64) == q.QDIT_ERR_INVALID_ARG
    assert f(ctx, A.data_ptr(), W.data_ptr(), 128, 64, 64, qp, None, q.QDIT_EPI_OUT_F32 | q.QDIT_EPI_OUT_BF16, None, o.data_ptr(), 64) == q.QDIT_ERR_INVALID_ARG
    assert f(ctx, A.data_ptr(), W.data_ptr(), 128, 64, 64, qp, None, q.QDIT_EPI_OUT_F32, None, o.data_ptr(), 64) == q.QDIT_ERR_INVALID_ARG
    assert f(ctx, A.data_ptr(), W.data_ptr(), 0, 64, 64, qp, None, q.QDIT_EPI_OUT_I32, None, o.data_ptr(), 64) == q.QDIT_OK
    q.qdit_sync(ctx)


@pytest.mark.parametrize("M,T", [(192, 64), (300, 100), (1184, 32)])
def test_gated_epilogue_on_ragged_rows_with_an_exactly_sized_gate(q, ctx, kernel_variant, M, T):
    """The last tile is ragged (M % 128 != 0) and the gate tensor has exactly ceil(M / T) rows: no row past it may
    be read (the warps of a tile whose rows lie wholly past M have no sample)."""
    N, K = 1152, 384
    a_qp = QParams(0.05, 0, -127, 127)
    L = _layer(46, M, N, K, T, a_qp)
    B = -(-M // T)
    gate_h = synth.normal(46, "g2", (B, N), 0.35)
    A, W = dev_i8(L["qa"]), dev_i8(L["qw"])
    ws, bi = dev(L["s_w"]), dev(L["bias"])
    # the gate sits at the very end of its allocation, followed by a canary region that must stay untouched (reads
    # past the end cannot be seen directly; the exact size is what the kernels are given)
    g = dev(gate_h)
    x = dev(L["resid"]).to(torch.bfloat16)
    xh = bf16_to_f64(x)
    cache = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    epi = q.epilogue(w_scale=ws, bias=bi, gate=g, ld_gate=N, tokens_per_sample=T, residual=x, cache_out=cache)
    flags = q.QDIT_EPI_BIAS | q.QDIT_EPI_GATE | q.QDIT_EPI_RESIDUAL | q.QDIT_EPI_CACHE_STORE | q.QDIT_EPI_OUT_BF16
    q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None, flags, epi, x, N)
    q.qdit_sync(ctx)
    f = linear.w8a8_linear(L["qa"], a_qp, L["qw"], L["s_w"], L["cs"], L["bias"])
    rows = np.arange(M) // T
    want_x = xh + gate_h.astype(np.float64)[rows] * f
    got_c, got_x = bf16_to_f64(cache), bf16_to_f64(x)
    assert (got_c != dit.round_bf16(f)).mean() < 1e-3
    assert (got_x != dit.round_bf16(want_x)).mean() < 1e-3
    assert max_rel_err(got_x, want_x) < 2.0 ** -8


FULL_M = 8192   # tokens of the 50-step workload: network batch 32 x 256 tokens


@pytest.mark.parametrize("K,N,name", [(1152, 3456, "qkv"), (1152, 1152, "proj"), (1152, 4608, "fc1"), (4608, 1152, "fc2")])
def test_full_size_layers_element_by_element(q, ctx, K, N, name):
    """The four block-level layers at the full workload's size, in the kernels the model path selects: raw int32
    accumulators bit-exact, f32 outputs within 1e-3 (measured 1e-5), and each layer's own fused epilogue against the
    oracle on every element."""
    M, T = FULL_M, 256
    a_qp = QParams(0.05, 0, -127, 127)
    L = _layer(47, M, N, K, T, a_qp)
    A, W = dev_i8(L["qa"]), dev_i8(L["qw"])
    ws, bi, g = dev(L["s_w"]), dev(L["bias"]), dev(L["gate"])
    acc = linear.gemm_i8(L["qa"], L["qw"])
    f = linear.w8a8_linear(L["qa"], a_qp, L["qw"], L["s_w"], L["cs"], L["bias"])
    for variant in ("auto", "t256"):
        _select_kernel(q, ctx, variant)
        try:
            np.testing.assert_array_equal(_run_i32(q, ctx, L["qa"], L["qw"]), acc)
            outf = torch.empty((M, N), dtype=torch.float32, device="cuda")
            q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None, q.QDIT_EPI_BIAS | q.QDIT_EPI_OUT_F32,
                               q.epilogue(w_scale=ws, bias=bi), outf, N)
            q.qdit_sync(ctx)
            assert max_rel_err(outf.cpu().numpy(), f) < 1e-5
        finally:
            _select_kernel(q, ctx, "auto")
    if name == "qkv":
        out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None, q.QDIT_EPI_BIAS | q.QDIT_EPI_OUT_BF16,
                           q.epilogue(w_scale=ws, bias=bi), out, N)
        q.qdit_sync(ctx)
        got = bf16_to_f64(out)
        assert (got != dit.round_bf16(f)).mean() < 1e-4 and bf16_steps_err(got, f) <= 1.0
    elif name == "fc1":
        u = dit.gelu_tanh(f)
        o_qp = quant.qparams_symmetric(float(np.abs(u).max()) * 0.9)
        out = torch.empty((M, N), dtype=torch.uint8, device="cuda")
        q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None,
                           q.QDIT_EPI_BIAS | q.QDIT_EPI_GELU | q.QDIT_EPI_QUANT_OUT,
                           q.epilogue(w_scale=ws, bias=bi, out_qp=q.qparams(o_qp.scale)), out, N)
        q.qdit_sync(ctx)
        got, want = host_codes(out), quant.quantize(u, o_qp)
        pre = u.astype(np.float32).astype(np.float64) * float(o_qp.inv_scale)
        n_bad, ok = code_mismatch_report(got, want, pre, 2e-5 * np.abs(pre).max() + 1e-6)
        assert ok and n_bad <= 1e-3 * got.size, (n_bad, got.size)
    else:
        x = dev(L["resid"]).to(torch.bfloat16)
        xh = bf16_to_f64(x)
        cache = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
        epi = q.epilogue(w_scale=ws, bias=bi, gate=g, ld_gate=N, tokens_per_sample=T, residual=x, cache_out=cache)
        flags = q.QDIT_EPI_BIAS | q.QDIT_EPI_GATE | q.QDIT_EPI_RESIDUAL | q.QDIT_EPI_CACHE_STORE | q.QDIT_EPI_OUT_BF16
        q.qdit_w8a8_linear(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None, flags, epi, x, N)
        q.qdit_sync(ctx)
        want_x = xh + L["gate"].astype(np.float64)[np.arange(M) // T] * f
        got_c, got_x = bf16_to_f64(cache), bf16_to_f64(x)
        assert (got_c != dit.round_bf16(f)).mean() < 1e-4 and bf16_steps_err(got_c, f) <= 1.0
        assert (got_x != dit.round_bf16(want_x)).mean() < 1e-3 and bf16_steps_err(got_x, want_x) <= 1.0


def test_options_select_kernels_and_reject_bad_values(q, ctx):
    assert q.qdit_get_option(ctx, q.QDIT_OPT_PDL) == 1
    for opt, bad in ((q.QDIT_OPT_GEMM_BN, 96), (q.QDIT_OPT_GEMM_T, 64), (q.QDIT_OPT_ATTN, 3), (q.QDIT_OPT_PDL, 2), (99, 0)):
        assert q.lib.qdit_set_option(ctx, opt, bad) == q.QDIT_ERR_INVALID_ARG
    q.qdit_set_option(ctx, q.QDIT_OPT_GEMM_T, 128)
    assert q.qdit_get_option(ctx, q.QDIT_OPT_GEMM_T) == 128
    q.qdit_set_option(ctx, q.QDIT_OPT_GEMM_T, 0)
    # with and without programmatic dependent launch: same bits
    qa = _codes(35, "ap", (600, 384), -128, 127)
    qw = _codes(35, "wp", (384, 384), -127, 127)
    a = _run_i32(q, ctx, qa, qw)
    q.qdit_set_option(ctx, q.QDIT_OPT_PDL, 0)
    try:
        b = _run_i32(q, ctx, qa, qw)
    finally:
        q.qdit_set_option(ctx, q.QDIT_OPT_PDL, 1)
    np.testing.assert_array_equal(a, b)


# ----------------------------------------------------------------------------- packed 4-bit weights (W4A8, Table 2)
def _w4_codes(seed, name, N, K):
    return synth.uniform_int(seed, name, (N, K), -8, 8).astype(np.int64)


def test_w4_pack_unpack_match_the_oracle_bytes(q, ctx):
    N, K = 200, 1152
    codes = _w4_codes(51, "w4", N, K)
    codes[0, :4] = [-8, 7, -1, 0]
    w8 = dev_i8(codes)
    packed = torch.zeros((N, K // 2), dtype=torch.uint8, device="cuda")
    q.qdit_pack_weight_int4(ctx, w8, N, K, packed)
    q.qdit_sync(ctx)
    np.testing.assert_array_equal(packed.cpu().numpy(), quant.pack_int4(codes))
    back = torch.zeros((N, K), dtype=torch.uint8, device="cuda")
    q.qdit_unpack_weight_int4(ctx, packed, N, K, back)
    q.qdit_sync(ctx)
    np.testing.assert_array_equal(host_codes(back), codes)
    np.testing.assert_array_equal(host_codes(back), quant.unpack_int4(quant.pack_int4(codes)))
    # a code outside [-8, 7] cannot be stored
    bad = codes.copy()
    bad[3, 5] = 9
    assert q.lib.qdit_pack_weight_int4(ctx, dev_i8(bad).data_ptr(), N, K, packed.data_ptr()) == q.QDIT_ERR_INVALID_ARG
    assert q.lib.qdit_pack_weight_int4(ctx, w8.data_ptr(), N, 24, packed.data_ptr()) == q.QDIT_ERR_SHAPE


@pytest.mark.parametrize("M,N,K", [(64, 392, 1152), (1152, 1152, 1152), (300, 6912, 384), (2048, 256, 4608)])
@pytest.mark.parametrize("scratch", [False, True])
def test_w4a8_accumulators_bit_exact_and_stage_equals_the_codes(q, ctx, M, N, K, scratch):
    """The weight tile the tensor core reads must be the oracle's codes exactly: raw int32 accumulators on random
    activations equal the oracle's integer product, and one-hot activations (row m selects column m of W) return the
    widened codes themselves.  Both forms: widened inside the GEMM kernel, and widened into a scratch matrix first."""
    codes = _w4_codes(52, f"w4.{N}.{K}", N, K)
    packed = torch.from_numpy(quant.pack_int4(codes)).cuda()
    w8s = torch.empty((N, K), dtype=torch.uint8, device="cuda") if scratch else None
    qa = _codes(52, f"a4.{M}.{K}", (M, K), -128, 127)
    out = torch.empty((M, N), dtype=torch.int32, device="cuda")
    q.qdit_w4a8_linear(ctx, dev_i8(qa), packed, M, N, K, q.qparams(1.0), None, q.QDIT_EPI_OUT_I32, None, out, N, w8s)
    q.qdit_sync(ctx)
    np.testing.assert_array_equal(out.cpu().numpy().astype(np.int64), linear.gemm_i8(qa, codes))
    Ms = min(M, K)
    onehot = np.zeros((Ms, K), dtype=np.int64)
    ks = synth.uniform_int(52, f"ks{K}", (Ms,), 0, K)
    onehot[np.arange(Ms), ks] = 1
    out1 = torch.empty((Ms, N), dtype=torch.int32, device="cuda")
    q.qdit_w4a8_linear(ctx, dev_i8(onehot), packed, Ms, N, K, q.qparams(1.0), None, q.QDIT_EPI_OUT_I32, None, out1, N, w8s)
    q.qdit_sync(ctx)
    np.testing.assert_array_equal(out1.cpu().numpy(), quant.unpack_int4(quant.pack_int4(codes))[:, ks].T)


@pytest.mark.parametrize("M,T", [(512, 256), (96, 32)])
def test_w4a8_epilogues_equal_w8a8_on_the_same_codes(q, ctx, M, T):
    """Same codes, same arithmetic after the accumulator: the packed layer and the one-code-per-byte layer give the
    same bits for the f32, the GELU + re-quantised and the gated epilogue; and the f32 output matches the oracle."""
    N, K = 1152, 1152
    a_qp = QParams(0.05, 0, -127, 127)
    L = _layer(53, M, N, K, T, a_qp)
    Wf = synth.normal(53, "W", (N, K), 0.02)
    codes, s_w, cs = quant.quantize_weight_per_channel(Wf, bits=4)
    A = dev_i8(L["qa"])
    W8, W4 = dev_i8(codes), torch.from_numpy(quant.pack_int4(codes)).cuda()
    ws, bi, g = dev(s_w), dev(L["bias"]), dev(L["gate"])
    ref = linear.w8a8_linear(L["qa"], a_qp, codes, s_w, cs, L["bias"])
    outs = {}
    for name, fn, W in (("w8", q.qdit_w8a8_linear, W8), ("w4", q.qdit_w4a8_linear, W4)):
        of = torch.empty((M, N), dtype=torch.float32, device="cuda")
        fn(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None, q.QDIT_EPI_BIAS | q.QDIT_EPI_OUT_F32, q.epilogue(w_scale=ws, bias=bi), of, N)
        oq = torch.empty((M, N), dtype=torch.uint8, device="cuda")
        fn(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None, q.QDIT_EPI_BIAS | q.QDIT_EPI_GELU | q.QDIT_EPI_QUANT_OUT,
           q.epilogue(w_scale=ws, bias=bi, out_qp=q.qparams(0.01)), oq, N)
        x = dev(L["resid"]).to(torch.bfloat16)
        cache = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
        fn(ctx, A, W, M, N, K, q.qparams(a_qp.scale), None,
           q.QDIT_EPI_BIAS | q.QDIT_EPI_GATE | q.QDIT_EPI_RESIDUAL | q.QDIT_EPI_CACHE_STORE | q.QDIT_EPI_OUT_BF16,
           q.epilogue(w_scale=ws, bias=bi, gate=g, ld_gate=N, tokens_per_sample=T, residual=x, cache_out=cache), x, N)
        q.qdit_sync(ctx)
        outs[name] = (of.cpu().numpy(), oq.cpu().numpy(), x.float().cpu().numpy(), cache.float().cpu().numpy())
    assert max_rel_err(outs["w4"][0], ref) < 1e-5
    for a, b in zip(outs["w4"], outs["w8"]):
        np.testing.assert_array_equal(a, b)
