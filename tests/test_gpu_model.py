"""GPU parity of the composed path: a DiT block from the primitives, whole-network evaluation,
on-device calibration, and the cached sampler, all against the oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import synth
from oracle import calib, dit, quant, sampler
from oracle.quant import QParams

from gpu_util import (bf16_steps_err, bf16_to_f64, bf16_view_to_f64, code_mismatch_report, dev, host_codes, max_rel_err, rel_l2,
                      scales_to_arrays, view)

pytestmark = pytest.mark.gpu

LINEAR_IDS = {"ada": 0, "qkv": 1, "proj": 2, "fc1": 3, "fc2": 4}


@pytest.fixture(scope="module")
def q():
    import paper_2503_02508_b200 as q
    return q


@pytest.fixture(scope="module")
def ctx(q):
    c = q.qdit_create(0, None)
    yield c
    q.qdit_destroy(c)


class Rig:
    """GPU model + oracle model built from the same seeded float weights."""

    def __init__(self, q, ctx, cfg, seed, weight_bits=8):
        self.q, self.ctx, self.cfg = q, ctx, cfg
        self.w = synth.model_weights(seed, cfg)
        self.om = dit.make_qmodel(cfg, self.w, weight_bits)
        self.gm = q.qdit_model_create(ctx, cfg, self.w, weight_bits)
        self.samplers = []

    def set_scales(self, scales):
        ada, blk = scales_to_arrays(scales, self.cfg.depth)
        self.q.qdit_model_set_act_scales(self.ctx, self.gm, ada, blk)

    def sampler(self, **kw):
        s = self.q.qdit_sampler_create(self.ctx, self.gm, **kw)
        self.samplers.append(s)
        return s

    def forward(self, s, latent, t, y, flags=0):
        B = latent.shape[0]
        out = torch.empty((B, 2 * self.cfg.channels, self.cfg.latent_side, self.cfg.latent_side), dtype=torch.float32,
                          device="cuda")
        self.q.qdit_forward(self.ctx, s, dev(latent), dev(np.asarray(t, dtype=np.float32)),
                            dev(np.asarray(y, dtype=np.int32)), B, out, flags)
        self.q.qdit_sync(self.ctx)
        return out.cpu().numpy().astype(np.float64)

    def close(self):
        for s in self.samplers:
            self.q.qdit_sampler_destroy(s)
        self.q.qdit_model_destroy(self.gm)


def _inputs(cfg, seed, B):
    latent = synth.normal(seed, "latent", (B, cfg.channels, cfg.latent_side, cfg.latent_side))
    t = synth.uniform_int(seed, "t", (B,), 0, 1000).astype(np.float64)
    y = synth.uniform_int(seed, "y", (B,), 0, cfg.num_classes)
    return latent, t, y


# ----------------------------------------------------------------------------- weights
@pytest.mark.parametrize("cfg", [synth.DIT_TINY, synth.DIT_S2_BLOCK], ids=["tiny", "s2"])
def test_model_weights_quantized_bit_exact(q, ctx, cfg):
    rig = Rig(q, ctx, cfg, 71)
    try:
        for i, blk in enumerate(rig.om.blocks):
            for name, wid in LINEAR_IDS.items():
                L = q.qdit_model_linear(rig.gm, i, wid)
                lin = getattr(blk, name)
                assert (L["N"], L["K"]) == lin.q.shape
                np.testing.assert_array_equal(view(L["w_q"], lin.q.shape, "|i1").cpu().numpy(), lin.q)
                np.testing.assert_array_equal(view(L["w_scale"], (L["N"],), "<f4").cpu().numpy(), lin.scale)
                np.testing.assert_array_equal(view(L["w_colsum"], (L["N"],), "<i4").cpu().numpy(), lin.colsum)
                np.testing.assert_array_equal(view(L["bias"], (L["N"],), "<f4").cpu().numpy(), lin.bias)
    finally:
        rig.close()


# ----------------------------------------------------------------------------- one block from the primitives
def test_block_s2_from_primitives(q, ctx):
    """Single DiT-S/2-shaped block, W8A8, batch 2, 256 tokens; activation scales from a seeded calibration batch."""
    cfg = synth.DIT_S2_BLOCK
    seed = synth.CONFIG_SEEDS["block_s2"]
    D, H, F, T, B = cfg.hidden, cfg.heads, cfg.mlp, cfg.tokens, 2
    M = B * T
    rig = Rig(q, ctx, cfg, seed)
    try:
        blk = rig.om.blocks[0]
        x0 = synth.normal(seed, "tokens", (M, D))
        c = synth.normal(seed, "cond", (B, D))
        cal = [(synth.normal(seed, f"cal_tokens{i}", (M, D)), synth.normal(seed, f"cal_cond{i}", (B, D))) for i in range(8)]
        scales = calib.calibrate_block(blk, cal, T, H)
        taps = {}
        octx = dit.Context(quant="static", scales=scales, tap=lambda n, a: taps.__setitem__(n, np.array(a)))
        x_ref = dit.block_forward(octx, blk, dit.store(x0, "bf16"), c, T, H, 0)

        lin = {n: q.qdit_model_linear(rig.gm, 0, i) for n, i in LINEAR_IDS.items()}
        sq = lambda n: q.qparams((scales.ada if n == "ada" else scales.blocks[0][n]).scale)

        def linear(A, name, flags, out, **epi):
            L = lin[name]
            e = q.epilogue(w_scale=L["w_scale"], w_colsum=L["w_colsum"], bias=L["bias"], **epi)
            q.qdit_w8a8_linear(ctx, A, L["w_q"], M if name != "ada" else B, L["N"], L["K"], sq(name), None,
                               flags | q.QDIT_EPI_BIAS, e, out, L["N"])

        x = dev(x0).to(torch.bfloat16)
        sc = dev(dit.silu(c.astype(np.float64)).astype(np.float32))
        ca = torch.empty((B, D), dtype=torch.uint8, device="cuda")
        q.qdit_quantize_act(ctx, sc, q.QDIT_F32, B, D, D, q.QDIT_QUANT_STATIC, sq("ada"), None, ca, D)
        mod = torch.empty((B, 6 * D), dtype=torch.float32, device="cuda")
        linear(ca, "ada", q.QDIT_EPI_OUT_F32, mod)
        h = torch.empty((M, D), dtype=torch.uint8, device="cuda")
        q.qdit_adaln_modulate(ctx, x, M, D, T, 1e-6, mod[:, 0:], mod[:, D:], 6 * D, h, q.QDIT_I8, sq("qkv"))
        qkv = torch.empty((M, 3 * D), dtype=torch.bfloat16, device="cuda")
        linear(h, "qkv", q.QDIT_EPI_OUT_BF16, qkv)
        a = torch.empty((M, D), dtype=torch.uint8, device="cuda")
        p = qkv.data_ptr()
        q.qdit_attention(ctx, p, p + 2 * D, p + 4 * D, 3 * D, B, H, T, D // H, 1.0 / np.sqrt(D // H), a, q.QDIT_I8, sq("proj"))
        gflags = q.QDIT_EPI_GATE | q.QDIT_EPI_RESIDUAL | q.QDIT_EPI_OUT_BF16
        linear(a, "proj", gflags, x, gate=mod[:, 2 * D:], ld_gate=6 * D, tokens_per_sample=T, residual=x)
        h2 = torch.empty((M, D), dtype=torch.uint8, device="cuda")
        q.qdit_adaln_modulate(ctx, x, M, D, T, 1e-6, mod[:, 3 * D:], mod[:, 4 * D:], 6 * D, h2, q.QDIT_I8, sq("fc1"))
        u = torch.empty((M, F), dtype=torch.uint8, device="cuda")
        linear(h2, "fc1", q.QDIT_EPI_GELU | q.QDIT_EPI_QUANT_OUT, u, out_qp=sq("fc2"))
        linear(u, "fc2", gflags, x, gate=mod[:, 5 * D:], ld_gate=6 * D, tokens_per_sample=T, residual=x)
        q.qdit_sync(ctx)

        # modulation: a de-quantized layer output -> max relative error 1e-3
        assert max_rel_err(mod.cpu().numpy(), taps["blk0.mod"]) < 1e-3
        np.testing.assert_array_equal(host_codes(ca), taps["blk0.ada.qa"])
        # fused LN quantizer: codes equal the oracle's except where the oracle's pre-rounding value lies within 2e-3 code
        # units of a rounding boundary (f32 statistics and products against f64: a few 1e-7 of |pre| <= 127, plus the
        # 1e-5 relative difference of the modulation the kernel was given)
        pre = taps["blk0.qkv.in"].astype(np.float32).astype(np.float64) * float(scales.blocks[0]["qkv"].inv_scale)
        n_bad, ok = code_mismatch_report(host_codes(h), taps["blk0.qkv.qa"], pre, 2e-3)
        assert ok and n_bad < 2e-3 * h.numel(), n_bad
        # QKV in bf16: oracle value rounded to bf16, up to one step at ties
        got_qkv = bf16_to_f64(qkv)
        assert bf16_steps_err(got_qkv, taps["blk0.qkv.out"]) <= 1.0
        assert rel_l2(got_qkv, taps["blk0.qkv.out"]) < 2e-3
        # block output (bf16 residual stream)
        got = bf16_to_f64(x)
        assert rel_l2(got, x_ref) < 2e-3, rel_l2(got, x_ref)
        assert bf16_steps_err(got, x_ref) <= 2.0          # bf16 residual stream: a couple of rounding flips at most
    finally:
        rig.close()


# ----------------------------------------------------------------------------- whole network
def _forward_case(q, ctx, cfg, seed, B, depth_note=""):
    rig = Rig(q, ctx, cfg, seed)
    latent, t, y = _inputs(cfg, seed, B)
    scales = calib.calibrate_model(rig.om, [(latent, t, y)])
    rig.set_scales(scales)
    return rig, latent, t, y, scales


def test_forward_tiny_matches_oracle(q, ctx):
    cfg = synth.DIT_TINY
    rig, latent, t, y, scales = _forward_case(q, ctx, cfg, 72, 3)
    try:
        s = rig.sampler(batch=3, num_steps=4)
        got = rig.forward(s, latent, t, y)
        taps = {}
        octx = dit.Context(quant="static", scales=scales, tap=lambda n, a: taps.__setitem__(n, np.array(a)))
        ref = dit.forward(rig.om, octx, latent, t, y)
        M, D = 3 * cfg.tokens, cfg.hidden
        assert max_rel_err(view(q.qdit_sampler_buffer(s, "c"), (3, D), "<f4").cpu().numpy(), taps["c"]) < 1e-4
        assert max_rel_err(view(q.qdit_sampler_buffer(s, "mod"), (3, cfg.depth * 6 * D), "<f4").cpu().numpy(),
                           np.concatenate([taps[f"blk{i}.mod"] for i in range(cfg.depth)], axis=1)) < 1e-3
        assert rel_l2(bf16_view_to_f64(q.qdit_sampler_buffer(s, "x"), (M, D)), taps["x_final"]) < 3e-3
        assert rel_l2(got, ref) < 5e-3, rel_l2(got, ref)
        assert max_rel_err(got, ref) < 5e-2
        # a smaller batch through the same workspace gives the same per-sample result
        got1 = rig.forward(s, latent[1:2], t[1:2], y[1:2])
        np.testing.assert_array_equal(got1, got[1:2])
    finally:
        rig.close()


def test_forward_tiny_w4a8_matches_oracle(q, ctx):
    """4-bit channel-wise weights, 8-bit activations (the W4A8 setting of Table 2) through the same kernels."""
    cfg = synth.DIT_TINY
    rig = Rig(q, ctx, cfg, 74, weight_bits=4)
    try:
        latent, t, y = _inputs(cfg, 74, 3)
        scales = calib.calibrate_model(rig.om, [(latent, t, y)])
        rig.set_scales(scales)
        s = rig.sampler(batch=3, num_steps=2)
        got = rig.forward(s, latent, t, y)
        ref = dit.forward(rig.om, dit.Context(quant="static", scales=scales), latent, t, y)
        assert rel_l2(got, ref) < 5e-3, rel_l2(got, ref)
        # the 4-bit model is a different function from the 8-bit one (the option is not silently ignored) ...
        rig8 = Rig(q, ctx, cfg, 74)
        try:
            rig8.set_scales(scales)
            got8 = rig8.forward(rig8.sampler(batch=3, num_steps=2), latent, t, y)
        finally:
            rig8.close()
        d = rel_l2(got, got8)
        assert 1e-3 < d < 0.5, d
        # ... whose weight codes stay inside the 4-bit range (this width, 144, is not a multiple of 32: one code per byte)
        assert q.qdit_model_weights_packed(rig.gm) == 0
        lin = q.qdit_model_linear(rig.gm, 0, LINEAR_IDS["fc1"])
        codes = host_codes(view(lin["w_q"], (lin["N"], lin["K"]), "|i1"))
        assert codes.min() >= -7 and codes.max() <= 7 and np.abs(codes).max() == 7
    finally:
        rig.close()


def test_forward_w4a8_packed_weights_match_oracle(q, ctx):
    """W4A8 with the weights stored two codes per byte (widths that are multiples of 32): the stored bytes are the
    oracle's packed codes, and the network evaluation on them matches the oracle (few rows: widened inside the GEMM
    kernel; 512 rows per block layer here)."""
    cfg = synth.DiTConfig(hidden=384, heads=6, mlp=1536, depth=2, grid=16)
    rig = Rig(q, ctx, cfg, 75, weight_bits=4)
    try:
        assert q.qdit_model_weights_packed(rig.gm) == 1
        for i, blk in enumerate(rig.om.blocks):
            for name, wid in LINEAR_IDS.items():
                L = q.qdit_model_linear(rig.gm, i, wid)
                lin = getattr(blk, name)
                got = view(L["w_q"], (L["N"], L["K"] // 2), "|u1").cpu().numpy()
                np.testing.assert_array_equal(got, quant.pack_int4(lin.q.astype(np.int32)))
        latent, t, y = _inputs(cfg, 75, 2)
        scales = calib.calibrate_model(rig.om, [(latent, t, y)])
        rig.set_scales(scales)
        got = rig.forward(rig.sampler(batch=2, num_steps=2), latent, t, y)
        ref = dit.forward(rig.om, dit.Context(quant="static", scales=scales), latent, t, y)
        assert rel_l2(got, ref) < 5e-3, rel_l2(got, ref)
        # many rows (8 images x 256 tokens = 2048 per block layer): the weights are widened into the scratch matrix
        # and the W8A8 kernels run; each image's result is what the few-row path gives for it alone
        lat8, t8, y8 = _inputs(cfg, 79, 8)
        s8 = rig.sampler(batch=8, num_steps=2)
        got8 = rig.forward(s8, lat8, t8, y8)
        got1 = rig.forward(s8, lat8[3:4], t8[3:4], y8[3:4])
        assert rel_l2(got8[3:4], got1) < 1e-6
        ref8 = dit.forward(rig.om, dit.Context(quant="static", scales=scales), lat8[3:4], t8[3:4], y8[3:4])
        assert rel_l2(got8[3:4], ref8) < 5e-3
    finally:
        rig.close()


def test_forward_xl_width_two_blocks(q, ctx):
    cfg = synth.DiTConfig(hidden=1152, heads=16, mlp=4608, depth=2, grid=16)
    rig, latent, t, y, scales = _forward_case(q, ctx, cfg, 73, 2)
    try:
        s = rig.sampler(batch=2, num_steps=2)
        got = rig.forward(s, latent, t, y)
        ref = dit.forward(rig.om, dit.Context(quant="static", scales=scales), latent, t, y)
        assert rel_l2(got, ref) < 5e-3, rel_l2(got, ref)
    finally:
        rig.close()


def test_on_device_calibration_matches_oracle(q, ctx):
    cfg = synth.DIT_TINY
    rig = Rig(q, ctx, cfg, 74)
    try:
        batches = [_inputs(cfg, 74 + i, 2) for i in range(3)]
        want = calib.calibrate_model(rig.om, batches)
        s = rig.sampler(batch=2, num_steps=2)
        q.qdit_model_begin_calibration(ctx, rig.gm)
        for latent, t, y in batches:
            rig.forward(s, latent, t, y, q.QDIT_FWD_CALIBRATE)
        q.qdit_model_finish_calibration(ctx, rig.gm)
        q.qdit_sync(ctx)
        ada, blk = q.qdit_model_get_act_scales(ctx, rig.gm, cfg.depth)
        w_ada, w_blk = scales_to_arrays(want, cfg.depth)
        assert abs(ada - w_ada) <= 1e-5 * w_ada
        np.testing.assert_allclose(blk, w_blk, rtol=5e-3)        # ranges are maxima of values that agree to ~1e-3
        # the calibrated model then runs the static path
        latent, t, y = batches[0]
        got = rig.forward(s, latent, t, y)
        ref = dit.forward(rig.om, dit.Context(quant="static", scales=want), latent, t, y)
        assert rel_l2(got, ref) < 1e-2
    finally:
        rig.close()


def test_forward_requires_scales(q, ctx):
    cfg = synth.DIT_TINY
    rig = Rig(q, ctx, cfg, 75)
    try:
        s = rig.sampler(batch=1, num_steps=2)
        latent, t, y = _inputs(cfg, 75, 1)
        with pytest.raises(q.QditError) as e:
            rig.forward(s, latent, t, y)
        assert e.value.status == q.QDIT_ERR_STATE
    finally:
        rig.close()


# ----------------------------------------------------------------------------- sampler
def _run_sampler(rig, latent, labels, **kw):
    q, ctx = rig.q, rig.ctx
    s = rig.sampler(batch=latent.shape[0], **kw)
    out = np.empty_like(latent, dtype=np.float32)
    lat = np.ascontiguousarray(latent, dtype=np.float32)
    lab = np.ascontiguousarray(labels, dtype=np.int32)
    q.qdit_sample(ctx, s, lat, lab, out)
    return out.astype(np.float64), s


@pytest.mark.parametrize("interval,guidance,use_vc", [(1, None, False), (2, 1.5, True), (3, None, True), (20, 1.5, False)])
def test_sampler_tiny_matches_oracle(q, ctx, interval, guidance, use_vc):
    cfg = synth.DIT_TINY
    S, B = 10, 3
    rig, latent, t, y, scales = _forward_case(q, ctx, cfg, 76, B)
    try:
        K = (1.0 + 0.03 * synth.normal(76, "K", (S, cfg.channels))).astype(np.float32) if use_vc else None
        got, s = _run_sampler(rig, latent, y, num_steps=S, cache_interval=interval, use_cfg=guidance is not None,
                              guidance=guidance or 1.0, vc_mode=q.QDIT_VC_K_TABLE if use_vc else q.QDIT_VC_NONE, vc_table=K)
        ref = sampler.sample(rig.om, dit.Context(quant="static", scales=scales),
                             sampler.SamplerConfig(S, cache_interval=interval, guidance=guidance, vc_table=K), latent, y)
        assert rel_l2(got, ref) < 2e-2, rel_l2(got, ref)       # the stated end-to-end tolerance
        assert rel_l2(got, ref) < 5e-3, rel_l2(got, ref)       # and the margin this path actually has
        # steps out of order are refused
        assert q.lib.qdit_sample_step(ctx, s, 3) == q.QDIT_ERR_STATE
    finally:
        rig.close()


@pytest.mark.parametrize("which", ["tiny", "xl_width_two_blocks"])
def test_distance_to_the_oracle_without_storage_rounding(q, ctx, which):
    """The default oracle rounds the residual stream, Q/K/V and the cache to bfloat16 where the CUDA path stores them
    in bfloat16, and accumulates a fully skipped step once.  This test measures the CUDA path against the oracle with
    neither: float64 storage throughout (Storage.exact) and the skipped step walked block by block.  Both distances
    are printed; the stated end-to-end bound (relative L2 2e-2) is asserted against the un-rounded oracle."""
    if which == "tiny":
        cfg, seed, B, S = synth.DIT_TINY, 77, 3, 10
    else:
        cfg, seed, B, S = synth.DiTConfig(hidden=1152, heads=16, mlp=4608, depth=2, grid=16), 78, 2, 6
    rig = Rig(q, ctx, cfg, seed)
    try:
        latent, t, y = _inputs(cfg, seed, B)
        # activation ranges from the un-rounded network, so that the yardstick owes nothing to the storage formats
        scales = calib.calibrate_model(rig.om, [(latent, t, y)], storage=dit.Storage.exact())
        rig.set_scales(scales)
        mirrored = dit.Context(quant="static", scales=scales)
        plain = dit.Context(quant="static", scales=scales, storage=dit.Storage.exact(), reuse_walk=True)
        # one network evaluation
        got = rig.forward(rig.sampler(batch=B, num_steps=2), latent, t, y)
        d_m = rel_l2(got, dit.forward(rig.om, mirrored, latent, t, y))
        d_p = rel_l2(got, dit.forward(rig.om, plain, latent, t, y))
        print(f"{which}: forward rel-L2 vs bf16-storage oracle {d_m:.3e}, vs float64-storage oracle {d_p:.3e}")
        assert d_p < 2e-2 and d_m < 2e-2
        # a cached, guided trajectory with VC
        K = (1.0 + 0.03 * synth.normal(seed, "K", (S, cfg.channels))).astype(np.float32)
        kw = dict(num_steps=S, cache_interval=2, use_cfg=True, guidance=1.5, vc_mode=q.QDIT_VC_K_TABLE, vc_table=K)
        got_s, _ = _run_sampler(rig, latent, y, **kw)
        scfg = sampler.SamplerConfig(S, cache_interval=2, guidance=1.5, vc_table=K)
        s_m = rel_l2(got_s, sampler.sample(rig.om, mirrored, scfg, latent, y))
        s_p = rel_l2(got_s, sampler.sample(rig.om, plain, scfg, latent, y))
        print(f"{which}: {S}-step cached guided trajectory rel-L2 vs bf16-storage oracle {s_m:.3e}, "
              f"vs float64-storage, block-by-block oracle {s_p:.3e}")
        assert s_p < 2e-2 and s_m < 2e-2
    finally:
        rig.close()


def test_sampler_per_branch_schedule_matches_oracle(q, ctx):
    """Per-block, per-branch reuse schedule ([steps, blocks, 2]) against the oracle, and its two reductions."""
    cfg = synth.DIT_TINY
    S, B = 8, 2
    rig, latent, t, y, scales = _forward_case(q, ctx, cfg, 78, B)
    try:
        sched = synth.uniform_int(78, "schedule", (S, cfg.depth, 2), 0, 2).astype(bool)
        sched[0] = False            # the first step fills the cache
        sched[3] = True             # one fully skipped step
        sched[5] = False            # one full refresh
        assert sched[1].any() and not sched[1].all()
        K = (1.0 + 0.03 * synth.normal(78, "K", (S, cfg.channels))).astype(np.float32)

        def run(schedule, interval=1):
            sm = rig.sampler(batch=B, num_steps=S, cache_interval=interval, use_cfg=True, guidance=1.5,
                             vc_mode=q.QDIT_VC_K_TABLE, vc_table=K)
            q.qdit_sampler_set_schedule(ctx, sm, schedule)
            out = np.empty_like(latent, dtype=np.float32)
            l0 = q.qdit_launch_count(ctx)
            q.qdit_sample(ctx, sm, np.ascontiguousarray(latent, dtype=np.float32), np.ascontiguousarray(y, dtype=np.int32), out)
            return out.astype(np.float64), q.qdit_launch_count(ctx) - l0

        got, launches = run(sched)
        ref = sampler.sample(rig.om, dit.Context(quant="static", scales=scales),
                             sampler.SamplerConfig(S, guidance=1.5, vc_table=K, schedule=sched), latent, y)
        assert rel_l2(got, ref) < 5e-3, rel_l2(got, ref)
        # launch accounting: 6 for the trajectory's conditioning; per step embed + final + DDIM + VC; a fully skipped
        # step one kernel; otherwise 4 kernels per computed attention branch, 3 per computed MLP branch, 1 per reused
        want = 6
        for i in range(S):
            want += 4
            if sched[i].all():
                want += 1
            else:
                want += int((~sched[i, :, 0]).sum()) * 4 + int((~sched[i, :, 1]).sum()) * 3 + int(sched[i].sum())
        assert launches == want
        # the global rule written as a schedule gives the same bits as the built-in rule
        glob = np.zeros((S, cfg.depth, 2), dtype=bool)
        glob[1::2] = True
        a, _ = run(glob)
        b, _ = run(None, interval=2)
        np.testing.assert_array_equal(a, b)
        # NULL schedule returns to the global rule; an all-compute schedule equals interval 1
        c, _ = run(np.zeros((S, cfg.depth, 2), dtype=bool), interval=2)
        d, _ = run(None, interval=1)
        np.testing.assert_array_equal(c, d)
        # reusing an entry that was never stored is refused
        bad = np.zeros((S, cfg.depth, 2), dtype=bool)
        bad[0, 1, 0] = True
        sm = rig.sampler(batch=B, num_steps=S)
        q.qdit_sampler_set_schedule(ctx, sm, bad)
        q.qdit_sampler_reset(ctx, sm, dev(latent), dev(y.astype(np.int32)))
        assert q.lib.qdit_sample_step(ctx, sm, 0) == q.QDIT_ERR_STATE
        q.qdit_sync(ctx)
    finally:
        rig.close()


@pytest.mark.parametrize("guidance", [None, 1.5])
def test_ddpm_sampler_tiny_matches_oracle(q, ctx, guidance):
    """Stochastic sampler with learned variance; the noise of every step is an input shared with the oracle."""
    cfg = synth.DIT_TINY
    S, B = 8, 3
    rig, latent, t, y, scales = _forward_case(q, ctx, cfg, 79, B)
    try:
        noise = synth.normal(79, "ddpm_noise", (S,) + latent.shape)
        K = (1.0 + 0.03 * synth.normal(79, "K", (S, cfg.channels))).astype(np.float32)
        nd = dev(noise)

        def run(noise_dev):
            sm = rig.sampler(batch=B, num_steps=S, cache_interval=2, use_cfg=guidance is not None, guidance=guidance or 1.0,
                             vc_mode=q.QDIT_VC_K_TABLE, vc_table=K)
            q.qdit_sampler_set_ddpm(ctx, sm, noise_dev)
            out = np.empty_like(latent, dtype=np.float32)
            q.qdit_sample(ctx, sm, np.ascontiguousarray(latent, dtype=np.float32), np.ascontiguousarray(y, dtype=np.int32), out)
            return out.astype(np.float64)

        got = run(nd)
        ref = sampler.sample(rig.om, dit.Context(quant="static", scales=scales),
                             sampler.SamplerConfig(S, cache_interval=2, guidance=guidance, vc_table=K, kind="ddpm", noise=noise),
                             latent, y)
        assert rel_l2(got, ref) < 5e-3, rel_l2(got, ref)
        # NULL noise returns to the deterministic sampler
        ddim = run(None)
        ref_ddim = sampler.sample(rig.om, dit.Context(quant="static", scales=scales),
                                  sampler.SamplerConfig(S, cache_interval=2, guidance=guidance, vc_table=K), latent, y)
        assert rel_l2(ddim, ref_ddim) < 5e-3 and rel_l2(got, ddim) > 1e-2
        # the last step draws no noise
        n2 = noise.copy()
        n2[-1] = 1e6
        np.testing.assert_array_equal(run(dev(n2)), got)
        # a one-step trajectory has no stochastic form
        s1 = rig.sampler(batch=B, num_steps=1)
        assert q.lib.qdit_sampler_set_ddpm(ctx, s1, nd.data_ptr()) == q.QDIT_ERR_INVALID_ARG
    finally:
        rig.close()


def test_conditioning_chunks_give_the_same_trajectory(q, ctx):
    """The conditioning of a trajectory is evaluated for many steps at once; chunk size (all steps, 3 steps, one
    step at a time inside the network evaluation) must not change a bit of the result."""
    cfg = synth.DIT_TINY
    S, B = 10, 2
    rig, latent, t, y, scales = _forward_case(q, ctx, cfg, 80, B)
    try:
        kw = dict(num_steps=S, cache_interval=2, use_cfg=True, guidance=1.5)
        a, _ = _run_sampler(rig, latent, y, **kw)
        q.qdit_set_option(ctx, q.QDIT_OPT_CONDITIONING_CHUNK, 3)
        l0 = q.qdit_launch_count(ctx)
        b, _ = _run_sampler(rig, latent, y, **kw)
        n_chunked = q.qdit_launch_count(ctx) - l0
        q.qdit_set_option(ctx, q.QDIT_OPT_CONDITIONING_CHUNK, -1)
        c, _ = _run_sampler(rig, latent, y, **kw)
        q.qdit_set_option(ctx, q.QDIT_OPT_CONDITIONING_CHUNK, 0)
        np.testing.assert_array_equal(a, b)
        assert rel_l2(c, a) < 5e-3          # the per-step path sums the small f32 linears in another order (code flips)
        # 4 chunks of conditioning (6 kernels each): steps 0, 3, 6, 9
        per_refresh, per_reuse = 1 + 7 * cfg.depth + 1 + 1, 1 + 1 + 1 + 1
        assert n_chunked == 4 * 6 + 5 * per_refresh + 5 * per_reuse
    finally:
        q.qdit_set_option(ctx, q.QDIT_OPT_CONDITIONING_CHUNK, 0)
        rig.close()


def test_sampler_step_by_step_and_cache_effect(q, ctx):
    cfg = synth.DIT_TINY
    S, B = 6, 2
    rig, latent, t, y, scales = _forward_case(q, ctx, cfg, 77, B)
    try:
        a, _ = _run_sampler(rig, latent, y, num_steps=S, cache_interval=1)
        b, _ = _run_sampler(rig, latent, y, num_steps=S, cache_interval=2)
        assert not np.array_equal(a, b) and rel_l2(b, a) < 0.2
        # same trajectory twice: deterministic
        b2, _ = _run_sampler(rig, latent, y, num_steps=S, cache_interval=2)
        np.testing.assert_array_equal(b, b2)
        # explicit stepping from device buffers equals the host-buffer convenience call
        s = rig.sampler(batch=B, num_steps=S, cache_interval=2)
        q.qdit_sampler_reset(ctx, s, dev(latent), dev(y.astype(np.int32)))
        for i in range(S):
            q.qdit_sample_step(ctx, s, i)
        q.qdit_sync(ctx)
        got = view(q.qdit_sampler_latent(s), latent.shape, "<f4").cpu().numpy().astype(np.float64)
        np.testing.assert_array_equal(got, b)
    finally:
        rig.close()


GLUE_CASES = [
    # tensor-core embedding and final layer: full groups of four samples, a short last group, a single sample
    ("xl", dict(hidden=1152, heads=16, mlp=4608, depth=1, grid=16), 4),
    ("xl", dict(hidden=1152, heads=16, mlp=4608, depth=1, grid=16), 7),
    ("xl", dict(hidden=1152, heads=16, mlp=4608, depth=1, grid=16), 1),
    ("xl_1024_tokens", dict(hidden=1152, heads=16, mlp=4608, depth=1, grid=32), 2),
    ("width_768", dict(hidden=768, heads=12, mlp=3072, depth=1, grid=16), 5),
    # tensor-core embedding, scalar final layer (width below the tensor-core form's range)
    ("s", dict(hidden=384, heads=6, mlp=1536, depth=1, grid=16), 5),
    # scalar kernels (width 144, 64 tokens)
    ("tiny", None, 3),
]


@pytest.mark.parametrize("name,shape,B", GLUE_CASES)
def test_patch_embed_and_final_layer_element_by_element(q, ctx, name, shape, B):
    """The floating-point layers around the blocks as calls of their own.  Embedding: every stored bf16 value is the
    rounding of the oracle's value, up to the f32 / split-operand error of the product (1e-5 of the sum of the terms'
    magnitudes: a missing remainder product would be 2e-3).  Final layer: f32-level agreement with the oracle."""
    cfg = synth.DIT_TINY if shape is None else synth.DiTConfig(**shape)
    rig = Rig(q, ctx, cfg, 91)
    try:
        D, T, C, side = cfg.hidden, cfg.tokens, cfg.channels, cfg.latent_side
        M = B * T
        w = rig.om.w
        # ---- embedding
        latent = synth.normal(92, f"glue.latent.{name}.{B}", (B, C, side, side))
        xg = torch.empty((M, D), dtype=torch.bfloat16, device="cuda")
        q.qdit_patch_embed(ctx, rig.gm, dev(latent), B, xg)
        q.qdit_sync(ctx)
        got = bf16_to_f64(xg)
        patches = dit.patchify(cfg, latent.astype(np.float32).astype(np.float64))
        ref = patches @ w["w_patch"].T + w["b_patch"] + np.tile(w["pos"], (B, 1))
        mag = np.abs(patches) @ np.abs(w["w_patch"]).T + np.abs(w["b_patch"]) + np.tile(np.abs(w["pos"]), (B, 1))
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref), 1e-30))) - 7)
        assert np.all(np.abs(got - ref) <= 0.5 * ulp + 1e-5 * mag + 1e-12)
        assert np.mean(got == dit.round_bf16(ref)) > 0.995          # flips only where the value sits within that error of a rounding boundary
        # ---- final layer
        x = synth.normal(93, f"glue.x.{name}.{B}", (M, D), 1.7, 0.3)
        xd = dev(x).to(torch.bfloat16)
        mod = synth.normal(93, f"glue.mod.{name}.{B}", (B, 2 * D), 0.4)
        out = torch.empty((B, 2 * C, side, side), dtype=torch.float32, device="cuda")
        q.qdit_final_layer(ctx, rig.gm, xd, dev(mod), B, out)
        q.qdit_sync(ctx)
        h = dit.layer_norm_modulate(bf16_to_f64(xd), mod[:, :D].astype(np.float32).astype(np.float64),
                                    mod[:, D:].astype(np.float32).astype(np.float64), T)
        ref_o = dit.unpatchify(cfg, h @ w["w_out"].T + w["b_out"], B)
        got_o = out.cpu().numpy().astype(np.float64)
        # f32 statistics (1e-4 under this metric, as for LayerNorm alone) plus a D-term product accumulated in f32 by the
        # tensor core, whose adds may truncate: up to D * 2^-24 * mean|term| = 1152 * 6e-8 * 0.04 = 3e-6 absolute on outputs
        # of rms 1, i.e. 3e-4 against the metric's floor of 1e-2 rms.  In the norm the agreement is 1e-6.
        assert max_rel_err(got_o, ref_o) < 4e-4, max_rel_err(got_o, ref_o)
        assert rel_l2(got_o, ref_o) < 5e-6, rel_l2(got_o, ref_o)
        # misaligned pointers are refused before any launch
        assert q.lib.qdit_patch_embed(ctx, rig.gm, dev(latent).data_ptr(), B, xg.data_ptr() + 2) == q.QDIT_ERR_ALIGN
        assert q.lib.qdit_final_layer(ctx, rig.gm, xd.data_ptr() + 2, dev(mod).data_ptr(), B, out.data_ptr()) == q.QDIT_ERR_ALIGN
    finally:
        rig.close()
