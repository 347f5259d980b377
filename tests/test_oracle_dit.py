"""Pins for oracle.dit: closed forms, invariants and an independent PyTorch composition."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import synth
from oracle import dit, calib


def test_round_bf16_matches_library_conversion():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(5000) * 10 ** rng.uniform(-6, 6, 5000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38]])
    want = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(dit.round_bf16(x), want)
    # ties to even on the 8th mantissa bit: 1 + 2^-8 -> 1, 1 + 3*2^-8 -> 1 + 2^-6
    assert dit.round_bf16(np.array([1 + 2.0 ** -8]))[0] == 1.0
    assert dit.round_bf16(np.array([1 + 3 * 2.0 ** -8]))[0] == 1 + 2.0 ** -6


def test_layer_norm_modulate_pins():
    rng = np.random.default_rng(1)
    T, B, D = 4, 3, 64
    x = rng.standard_normal((B * T, D)) * 3 + 1.5
    shift = rng.standard_normal((B, D))
    scale = rng.standard_normal((B, D))
    z = np.zeros((B, D))
    y0 = dit.layer_norm_modulate(x, z, z, T)
    assert np.abs(y0.mean(axis=1)).max() < 1e-12
    np.testing.assert_allclose(y0.var(axis=1), 1.0, atol=2e-6)           # eps = 1e-6 keeps it just under 1
    want = F.layer_norm(torch.tensor(x), (D,), eps=1e-6).numpy()
    np.testing.assert_allclose(y0, want, atol=1e-12)
    # modulation uses the sample index row // T and the (1 + scale) form
    y = dit.layer_norm_modulate(x, shift, scale, T)
    b = np.repeat(np.arange(B), T)
    np.testing.assert_allclose(y, want * (1 + scale[b]) + shift[b], atol=1e-12)
    # a constant row normalises to 0 -> output is the shift alone
    xc = np.full((B * T, D), 7.25)
    np.testing.assert_allclose(dit.layer_norm_modulate(xc, shift, scale, T), shift[b], atol=1e-9)


def test_gelu_silu_pins():
    x = np.linspace(-8, 8, 4001)
    np.testing.assert_allclose(dit.gelu_tanh(x), F.gelu(torch.tensor(x), approximate="tanh").numpy(), atol=1e-14)
    np.testing.assert_allclose(dit.gelu_tanh(x) - dit.gelu_tanh(-x), x, atol=1e-14)
    assert abs(dit.gelu_tanh(np.array([1.0]))[0] - 0.8411919906082768) < 1e-12
    np.testing.assert_allclose(dit.silu(x), F.silu(torch.tensor(x)).numpy(), atol=1e-14)


def test_attention_pins():
    rng = np.random.default_rng(2)
    B, T, H, dh = 2, 9, 3, 8
    q, k, v = (rng.standard_normal((B, T, H, dh)) for _ in range(3))
    o = dit.attention(q, k, v)
    tq, tk, tv = (torch.tensor(a).permute(0, 2, 1, 3) for a in (q, k, v))
    want = F.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(o, want, atol=1e-12)
    # zero queries -> uniform weights -> mean of V over tokens
    np.testing.assert_allclose(dit.attention(np.zeros_like(q), k, v),
                               np.broadcast_to(v.mean(axis=1, keepdims=True), v.shape), atol=1e-14)
    # single token -> V
    np.testing.assert_allclose(dit.attention(q[:, :1], k[:, :1], v[:, :1]), v[:, :1], atol=1e-14)
    # permuting the tokens permutes the output (no mask, no position dependence)
    perm = rng.permutation(T)
    np.testing.assert_allclose(dit.attention(q[:, perm], k[:, perm], v[:, perm]), o[:, perm], atol=1e-13)
    # permuting only keys/values leaves the output unchanged
    np.testing.assert_allclose(dit.attention(q, k[:, perm], v[:, perm]), o, atol=1e-13)


def test_timestep_features_closed_form():
    f = dit.timestep_features(np.array([0.0, 1.0]), 8)
    np.testing.assert_allclose(f[0], [1, 1, 1, 1, 0, 0, 0, 0], atol=0)
    np.testing.assert_allclose(f[1, :4], np.cos(10000.0 ** (-np.arange(4) / 4)), atol=1e-15)
    np.testing.assert_allclose(f[1, 4:], np.sin(10000.0 ** (-np.arange(4) / 4)), atol=1e-15)


# ------------------------------------------------------------------ independent library composition
def torch_dit_forward(cfg, w, latent, t, y):
    """Un-quantized DiT written only with torch library ops (float64)."""
    tt = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    D, H, p = cfg.hidden, cfg.heads, cfg.patch
    x = F.conv2d(tt(latent), tt(w["w_patch"]).reshape(D, cfg.channels, p, p), tt(w["b_patch"]), stride=p)
    B = x.shape[0]
    x = x.flatten(2).transpose(1, 2) + tt(w["pos"])[None]
    half = cfg.freq_dim // 2
    freqs = torch.exp(-np.log(10000.0) * torch.arange(half, dtype=torch.float64) / half)
    args = tt(t)[:, None] * freqs[None]
    temb = torch.cat([torch.cos(args), torch.sin(args)], dim=-1)
    c = F.linear(F.silu(F.linear(temb, tt(w["w_t1"]), tt(w["b_t1"]))), tt(w["w_t2"]), tt(w["b_t2"]))
    c = c + F.embedding(torch.tensor(np.asarray(y), dtype=torch.long), tt(w["y_table"]))
    mod = lambda v, sh, sc: v * (1 + sc[:, None]) + sh[:, None]
    for bw in w["blocks"]:
        m = F.linear(F.silu(c), tt(bw["w_ada"]), tt(bw["b_ada"])).chunk(6, dim=1)
        h = mod(F.layer_norm(x, (D,), eps=1e-6), m[0], m[1])
        qkv = F.linear(h, tt(bw["w_qkv"]), tt(bw["b_qkv"])).reshape(B, -1, 3, H, D // H).permute(2, 0, 3, 1, 4)
        a = F.scaled_dot_product_attention(qkv[0], qkv[1], qkv[2]).transpose(1, 2).reshape(B, -1, D)
        x = x + m[2][:, None] * F.linear(a, tt(bw["w_proj"]), tt(bw["b_proj"]))
        h = mod(F.layer_norm(x, (D,), eps=1e-6), m[3], m[4])
        h = F.linear(F.gelu(F.linear(h, tt(bw["w_fc1"]), tt(bw["b_fc1"])), approximate="tanh"),
                     tt(bw["w_fc2"]), tt(bw["b_fc2"]))
        x = x + m[5][:, None] * h
    m = F.linear(F.silu(c), tt(w["w_ada_f"]), tt(w["b_ada_f"])).chunk(2, dim=1)
    o = F.linear(mod(F.layer_norm(x, (D,), eps=1e-6), m[0], m[1]), tt(w["w_out"]), tt(w["b_out"]))
    g, co = cfg.grid, 2 * cfg.channels
    o = o.reshape(B, g, g, p, p, co)
    o = torch.einsum("nhwpqc->nchpwq", o).reshape(B, co, g * p, g * p)
    return o.numpy()


@pytest.fixture(scope="module")
def tiny():
    cfg = synth.DIT_TINY
    w = synth.model_weights(11, cfg)
    latent = synth.normal(11, "latent", (3, cfg.channels, cfg.latent_side, cfg.latent_side))
    t = np.array([999.0, 500.0, 3.0])
    y = np.array([5, 999, 1000])
    return cfg, w, latent, t, y


def test_unquantized_network_matches_library_composition(tiny):
    cfg, w, latent, t, y = tiny
    model = dit.make_qmodel(cfg, w)
    ctx = dit.Context(quant="off", storage=dit.Storage.exact())
    got = dit.forward(model, ctx, latent, t, y)
    want = torch_dit_forward(cfg, w, latent, t, y)
    assert got.shape == want.shape == (3, 8, cfg.latent_side, cfg.latent_side)
    np.testing.assert_allclose(got, want, rtol=1e-9, atol=1e-11)


def test_quantized_network_tracks_unquantized(tiny):
    cfg, w, latent, t, y = tiny
    model = dit.make_qmodel(cfg, w)
    ref = dit.forward(model, dit.Context(quant="off", storage=dit.Storage.exact()), latent, t, y)
    scales = calib.calibrate_model(model, [(latent, t, y)], storage=dit.Storage.exact())
    got = dit.forward(model, dit.Context(quant="static", scales=scales, storage=dit.Storage.exact()), latent, t, y)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert 0 < rel < 0.05            # 8-bit: close, but not identical
    got16 = dit.forward(model, dit.Context(quant="static", scales=scales), latent, t, y)
    rel16 = np.linalg.norm(got16 - got) / np.linalg.norm(got)
    assert 0 < rel16 < 0.02          # bf16 storage: a further small perturbation


def test_static_scales_reproduce_dynamic_pass_on_the_calibration_input(tiny):
    cfg, w, latent, t, y = tiny
    model = dit.make_qmodel(cfg, w)
    taps = {}
    ctx_d = dit.Context(quant="dynamic", tap=lambda n, a: taps.__setitem__(n, np.array(a)))
    out_d = dit.forward(model, ctx_d, latent, t, y)
    scales = calib.calibrate_model(model, [(latent, t, y)])
    # calibrated scale = absmax of the tapped float32 input / 127
    for i in range(cfg.depth):
        for n in ("qkv", "proj", "fc1", "fc2"):
            amax = np.float32(np.abs(taps[f"blk{i}.{n}.in"].astype(np.float32)).max())
            assert scales.blocks[i][n].scale == float(amax / np.float32(127))
            assert (scales.blocks[i][n].zero_point, scales.blocks[i][n].qmin, scales.blocks[i][n].qmax) == (0, -127, 127)
            assert np.abs(taps[f"blk{i}.{n}.qa"]).max() == 127
    out_s = dit.forward(model, dit.Context(quant="static", scales=scales), latent, t, y)
    np.testing.assert_array_equal(out_s, out_d)
    # more calibration inputs can only widen the ranges
    lat2 = synth.normal(12, "latent2", latent.shape) * 2
    scales2 = calib.calibrate_model(model, [(latent, t, y), (lat2, t, y)])
    for i in range(cfg.depth):
        for n in ("qkv", "proj", "fc1", "fc2"):
            assert scales2.blocks[i][n].scale >= scales.blocks[i][n].scale


def test_block_samples_are_independent(tiny):
    # static tensor-wise scales: a sample's result does not depend on its batch-mates
    cfg, w, latent, t, y = tiny
    model = dit.make_qmodel(cfg, w)
    scales = calib.calibrate_model(model, [(latent, t, y)])
    ctx = dit.Context(quant="static", scales=scales)
    full = dit.forward(model, ctx, latent, t, y)
    one = dit.forward(model, ctx, latent[1:2], t[1:2], y[1:2])
    np.testing.assert_allclose(full[1:2], one, rtol=0, atol=1e-6)   # up to summation order and rare code flips
    assert np.abs(full[1:2] - one).mean() < 1e-9


def test_quantized_linear_with_cached_codes_is_the_integer_definition(tiny):
    """The layer evaluation keeps a float64 copy of the weight codes (made once): its output must be, bit for bit, the
    definition on the integer codes - brute-force int64 products, then the affine de-quantisation."""
    from oracle import linear, quant
    cfg, w, *_ = tiny
    lin = dit.make_qlinear(w["blocks"][0]["w_fc1"], w["blocks"][0]["b_fc1"])
    x = synth.normal(12, "cached.x", (7, lin.q.shape[1]), 1.3)
    qp = quant.qparams_symmetric(float(np.abs(x.astype(np.float32)).max()))
    ctx = dit.Context(quant="static")
    got1 = dit._qlinear_apply(ctx, lin, x, qp, "t")
    got2 = dit._qlinear_apply(ctx, lin, x, qp, "t")            # second call: the cached copy
    qa = quant.quantize(x, qp).astype(np.int64)
    acc = np.zeros((7, lin.q.shape[0]), dtype=np.int64)
    for k in range(qa.shape[1]):                                # integer accumulation, no floating point involved
        acc += qa[:, k:k + 1] * lin.q[:, k].astype(np.int64)[None, :]
    want = linear.dequant_affine(acc, qp, lin.scale, lin.colsum, lin.bias)
    np.testing.assert_array_equal(got1, want)
    np.testing.assert_array_equal(got2, want)
    assert lin.q.dtype == np.int8                               # the stored codes themselves are untouched
