"""GPU parity at the full workload sizes: DiT-XL/2 forward (batch 8), the 50-step guided sampler (batch 16,
cache interval 2, VC) and the 100-step 512x512 sampler (batch 8, cache interval 3, VC).

The CPU oracle cannot run these workloads whole in test time, so it computes a sample of them: because
activation scales are static and tensor-wise, VC statistics per sample and the cache per sample, every image's
trajectory is independent of its batch-mates.  The oracle therefore follows ONE image (with its unconditional
twin under guidance): through ALL 50 steps of the 256x256 workload (about five minutes of CPU), so that the final
latent of a full sampling run is compared, and through the first 7 of the 100 steps of the 512x512 workload (three
cache refreshes; a refresh step at 1024 tokens costs the oracle close to a minute, all 34 would take half an hour).
The full-batch CUDA run must match the oracle on that image; the rest of the batch and of the trajectory is
covered by properties that hold at any size (batch independence bit for bit, determinism, finiteness, the
schedule's launch counts).
"""
import numpy as np
import pytest
import torch

import synth
from oracle import calib, dit, sampler

from gpu_util import dev, rel_l2, scales_to_arrays, view

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


class XLRig:
    def __init__(self, q, ctx, cfg, seed, weight_bits=8):
        self.q, self.ctx, self.cfg = q, ctx, cfg
        w = synth.model_weights(seed, cfg)
        self.om = dit.make_qmodel(cfg, w, weight_bits)
        self.gm = q.qdit_model_create(ctx, cfg, w, weight_bits)
        del w
        self.samplers = []

    def set_scales(self, scales):
        ada, blk = scales_to_arrays(scales, self.cfg.depth)
        self.q.qdit_model_set_act_scales(self.ctx, self.gm, ada, blk)

    def sampler(self, **kw):
        s = self.q.qdit_sampler_create(self.ctx, self.gm, **kw)
        self.samplers.append(s)
        return s

    def close(self):
        for s in self.samplers:
            self.q.qdit_sampler_destroy(s)
        self.q.qdit_model_destroy(self.gm)


@pytest.fixture(scope="module")
def xl256(q, ctx):
    rig = XLRig(q, ctx, synth.DIT_XL2, synth.CONFIG_SEEDS["forward_xl2"])
    yield rig
    rig.close()


def test_forward_xl2_batch8_matches_oracle_on_sampled_images(q, ctx, xl256):
    """Full DiT-XL/2 forward, W8A8, 28 blocks, 256 tokens, batch 8, no cache."""
    cfg, seed, B = xl256.cfg, synth.CONFIG_SEEDS["forward_xl2"], 8
    latent = synth.normal(seed, "latent", (B, cfg.channels, cfg.latent_side, cfg.latent_side))
    t = synth.uniform_int(seed, "t", (B,), 0, 1000).astype(np.float64)
    y = synth.uniform_int(seed, "y", (B,), 0, cfg.num_classes)
    pick = [0, 5]
    scales = calib.calibrate_model(xl256.om, [(latent[pick], t[pick], y[pick])])
    xl256.set_scales(scales)
    s = xl256.sampler(batch=B, num_steps=2)
    out = torch.empty((B, 2 * cfg.channels, cfg.latent_side, cfg.latent_side), dtype=torch.float32, device="cuda")
    l0 = q.qdit_launch_count(ctx)
    q.qdit_forward(ctx, s, dev(latent), dev(t.astype(np.float32)), dev(y.astype(np.int32)), B, out, 0)
    q.qdit_sync(ctx)
    assert q.qdit_launch_count(ctx) - l0 == 6 + 7 * cfg.depth + 2     # embed/cond (4) + quant + modulation GEMM, 7 per block, final (2)
    got = out.cpu().numpy().astype(np.float64)
    ref = dit.forward(xl256.om, dit.Context(quant="static", scales=scales), latent[pick], t[pick], y[pick])
    err = rel_l2(got[pick], ref)
    # 28 blocks deep: bf16 probabilities in attention, one-step code flips and bf16 residual flips accumulate
    # to about 1e-2; the stated bound for an end-to-end result is 2e-2
    assert err < 2e-2, err
    print(f"forward_xl2 rel-L2 vs oracle: {err:.3e}")
    assert np.isfinite(got).all() and got.std() > 1e-3
    # the other images: same result when evaluated alone (batch independence, bit for bit)
    out1 = torch.empty((1,) + tuple(out.shape[1:]), dtype=torch.float32, device="cuda")
    q.qdit_forward(ctx, s, dev(latent[3:4]), dev(t[3:4].astype(np.float32)), dev(y[3:4].astype(np.int32)), 1, out1, 0)
    q.qdit_sync(ctx)
    np.testing.assert_array_equal(out1.cpu().numpy(), out[3:4].cpu().numpy())


def _oracle_prefix(rig, scales, latent1, label1, steps, n_prefix, interval, guidance, vc_table):
    snaps = []

    class Stop(Exception):
        pass

    def on_step(i, x, reuse):
        snaps.append(x.copy())
        if i + 1 >= n_prefix:
            raise Stop

    try:
        sampler.sample(rig.om, dit.Context(quant="static", scales=scales),
                       sampler.SamplerConfig(steps, cache_interval=interval, guidance=guidance, vc_table=vc_table),
                       latent1, label1, on_step=on_step)
    except Stop:
        pass
    return snaps


def _gpu_trajectory(q, ctx, rig, latent, labels, steps, interval, guidance, vc_table, snapshot_steps):
    B = latent.shape[0]
    s = rig.sampler(batch=B, num_steps=steps, cache_interval=interval, use_cfg=guidance is not None,
                    guidance=guidance or 1.0, vc_mode=q.QDIT_VC_K_TABLE, vc_table=vc_table)
    q.qdit_sampler_reset(ctx, s, dev(latent), dev(labels.astype(np.int32)))
    snaps = {}
    l0 = q.qdit_launch_count(ctx)
    for i in range(steps):
        q.qdit_sample_step(ctx, s, i)
        if i in snapshot_steps:
            q.qdit_sync(ctx)
            snaps[i] = view(q.qdit_sampler_latent(s), latent.shape, "<f4").cpu().numpy().astype(np.float64)
    q.qdit_sync(ctx)
    final = view(q.qdit_sampler_latent(s), latent.shape, "<f4").cpu().numpy().astype(np.float64)
    launches = q.qdit_launch_count(ctx) - l0
    q.qdit_sampler_destroy(s)
    rig.samplers.remove(s)
    return snaps, final, launches


def test_ddim50_guided_cached_sampler_batch16(q, ctx, xl256):
    """50-step DDIM at 256x256, batch 16, guidance 1.5 (network batch 32), cache interval 2, VC every step."""
    cfg, seed = xl256.cfg, synth.CONFIG_SEEDS["ddim50_xl2"]
    S, B, interval, guidance, n_prefix = 50, 16, 2, 1.5, 50     # the oracle follows image 0 through ALL steps
    latent = synth.normal(seed, "latent", (B, cfg.channels, cfg.latent_side, cfg.latent_side))
    labels = synth.uniform_int(seed, "labels", (B,), 0, cfg.num_classes)
    K = (1.0 + 0.02 * synth.normal(seed, "vc_table", (S, cfg.channels))).astype(np.float32)
    cal_lat = np.concatenate([latent[:1], latent[:1]])
    scales = calib.calibrate_model(xl256.om, [(cal_lat, np.full(2, 980.0), np.array([labels[0], cfg.num_classes]))])
    xl256.set_scales(scales)
    ref = _oracle_prefix(xl256, scales, latent[:1], labels[:1], S, n_prefix, interval, guidance, K)
    snaps, final, launches = _gpu_trajectory(q, ctx, xl256, latent, labels, S, interval, guidance, K, set(range(n_prefix)))
    worst = 0.0
    for i in range(n_prefix):                      # steps 0, 1, 2, ... = refresh, reuse, refresh, ...
        err = rel_l2(snaps[i][:1], ref[i])
        worst = max(worst, err)
        if i < 4 or i % 10 == 9:
            print(f"ddim50 step {i} latent rel-L2 vs oracle: {err:.3e}")
        assert err < 2e-2, (i, err)
    # the benchmark spec's bound: the FINAL latent of the full 50-step run
    err_final = rel_l2(final[:1], ref[S - 1])
    print(f"ddim50 final latent (after step {S - 1}) rel-L2 vs oracle: {err_final:.3e}; worst step {worst:.3e}")
    assert err_final < 2e-2, err_final
    assert np.isfinite(final).all()
    # launch accounting: the conditioning of all steps is evaluated once (6 kernels); refresh steps run 7 kernels
    # per block, reuse steps one kernel for all blocks
    per_refresh = 1 + 7 * cfg.depth + 1 + 2          # embed + blocks + final layer + guidance/DDIM + VC
    per_reuse = 1 + 1 + 1 + 2
    assert launches == 6 + 25 * per_refresh + 25 * per_reuse
    # batch independence over the WHOLE trajectory: image 7 alone gives bit-identical latents
    _, final1, _ = _gpu_trajectory(q, ctx, xl256, latent[7:8], labels[7:8], S, interval, guidance, K, set())
    np.testing.assert_array_equal(final1, final[7:8])
    # the cache changes the result (it is not silently disabled), but mildly
    _, nocache, _ = _gpu_trajectory(q, ctx, xl256, latent[7:8], labels[7:8], S, 1, guidance, K, set())
    d = rel_l2(final1, nocache)
    assert 0 < d < 0.5, d


def test_forward_xl2_w4a8_matches_oracle(q, ctx):
    """Full DiT-XL/2 forward with 4-bit channel-wise weights and 8-bit activations (the W4A8 setting of Table 2)."""
    cfg, seed, B = synth.DIT_XL2, synth.CONFIG_SEEDS["forward_xl2"], 2
    rig = XLRig(q, ctx, cfg, seed, weight_bits=4)
    try:
        latent = synth.normal(seed, "latent", (B, cfg.channels, cfg.latent_side, cfg.latent_side))
        t = synth.uniform_int(seed, "t", (B,), 0, 1000).astype(np.float64)
        y = synth.uniform_int(seed, "y", (B,), 0, cfg.num_classes)
        scales = calib.calibrate_model(rig.om, [(latent, t, y)])
        rig.set_scales(scales)
        s = rig.sampler(batch=B, num_steps=2)
        out = torch.empty((B, 2 * cfg.channels, cfg.latent_side, cfg.latent_side), dtype=torch.float32, device="cuda")
        q.qdit_forward(ctx, s, dev(latent), dev(t.astype(np.float32)), dev(y.astype(np.int32)), B, out, 0)
        q.qdit_sync(ctx)
        got = out.cpu().numpy().astype(np.float64)
        ref = dit.forward(rig.om, dit.Context(quant="static", scales=scales), latent, t, y)
        err = rel_l2(got, ref)
        print(f"forward_xl2 W4A8 rel-L2 vs oracle: {err:.3e}")
        assert err < 2e-2, err
    finally:
        rig.close()


def test_ddim100_512_cached_sampler_batch8(q, ctx):
    """100-step DDIM at 512x512 (1024 tokens), batch 8, cache interval 3, VC every step, no guidance."""
    cfg, seed = synth.DIT_XL2_512, synth.CONFIG_SEEDS["ddim100_xl2_512"]
    S, B, interval, n_prefix = 100, 8, 3, 25     # steps 0..24: nine refreshes (0, 3, .., 24) and the reuse steps between them
    rig = XLRig(q, ctx, cfg, seed)
    try:
        latent = synth.normal(seed, "latent", (B, cfg.channels, cfg.latent_side, cfg.latent_side))
        labels = synth.uniform_int(seed, "labels", (B,), 0, cfg.num_classes)
        K = (1.0 + 0.02 * synth.normal(seed, "vc_table", (S, cfg.channels))).astype(np.float32)
        scales = calib.calibrate_model(rig.om, [(latent[:1], np.full(1, 990.0), labels[:1])])
        rig.set_scales(scales)
        ref = _oracle_prefix(rig, scales, latent[:1], labels[:1], S, n_prefix, interval, None, K)
        snaps, final, launches = _gpu_trajectory(q, ctx, rig, latent, labels, S, interval, None, K, set(range(n_prefix)))
        for i in range(n_prefix):                  # refresh, reuse, reuse, refresh, ...
            err = rel_l2(snaps[i][:1], ref[i])
            print(f"ddim100_512 step {i} latent rel-L2 vs oracle: {err:.3e}")
            assert err < 2e-2, (i, err)
        assert np.isfinite(final).all()
        assert launches == 6 + 34 * (1 + 7 * cfg.depth + 1 + 2) + 66 * (1 + 1 + 1 + 2)
        _, final1, _ = _gpu_trajectory(q, ctx, rig, latent[2:3], labels[2:3], S, interval, None, K, set())
        np.testing.assert_array_equal(final1, final[2:3])
    finally:
        rig.close()
