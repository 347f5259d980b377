"""Pins for oracle.sampler and oracle.vc: cache schedule, DDIM identities, VC identities and fit."""
import numpy as np
import pytest

import synth
from oracle import calib, dit, sampler, vc


def test_cache_schedule():
    assert all(sampler.should_refresh(i, 1) for i in range(10))
    assert [sampler.should_refresh(i, 2) for i in range(5)] == [True, False, True, False, True]
    assert [i for i in range(50) if sampler.should_refresh(i, 100)] == [0]
    assert sum(sampler.should_refresh(i, 2) for i in range(50)) == 25
    assert sum(sampler.should_refresh(i, 3) for i in range(100)) == 34
    with pytest.raises(ValueError):
        sampler.should_refresh(0, 0)


def test_ddim_table_and_identities():
    tab = sampler.ddim_table(50)
    assert [r[0] for r in tab[:3]] == [980, 960, 940] and tab[-1][0] == 0
    for r in tab:
        assert abs(r[1] ** 2 + r[2] ** 2 - 1) < 1e-12 and abs(r[3] ** 2 + r[4] ** 2 - 1) < 1e-12
    assert abs(tab[-1][1] ** 2 - (1 - 1e-4)) < 1e-15          # alpha_bar_0 = 1 - beta_0
    assert tab[-1][3] == 1.0 and tab[-1][4] == 0.0            # after the last step alpha_bar_prev = 1
    for a, b in zip(tab[:-1], tab[1:]):
        assert a[3] == b[1] and a[1] < b[1]                    # prev of step i is t of step i+1; alpha_bar grows
    # closed form of alpha_bar at t = 980: prod_{j<=980} (1 - beta_j)
    betas = [1e-4 + (2e-2 - 1e-4) * j / 999 for j in range(1000)]
    ab = 1.0
    for j in range(981):
        ab *= 1 - betas[j]
    assert abs(tab[0][1] - np.sqrt(ab)) < 1e-12
    # if eps is the true noise, the update lands exactly on the same (x0, eps) at the previous level
    rng = np.random.default_rng(0)
    x0, eps = rng.standard_normal((2, 4, 8, 8)), rng.standard_normal((2, 4, 8, 8))
    for row in (tab[0], tab[17], tab[-1]):
        xt = row[1] * x0 + row[2] * eps
        np.testing.assert_allclose(sampler.ddim_update(xt, eps, row), row[3] * x0 + row[4] * eps, atol=1e-12)
    np.testing.assert_allclose(sampler.ddim_update(tab[-1][1] * x0 + tab[-1][2] * eps, eps, tab[-1]), x0, atol=1e-12)
    # equivalent textbook form: x_prev = sqrt(ab_p/ab_t) x + (sqrt(1-ab_p) - sqrt(ab_p (1-ab_t)/ab_t)) eps
    row = tab[5]
    xt = rng.standard_normal((2, 4, 8, 8))
    alt = row[3] / row[1] * xt + (row[4] - row[3] * row[2] / row[1]) * eps
    np.testing.assert_allclose(sampler.ddim_update(xt, eps, row), alt, atol=1e-12)


def test_ddpm_table_and_posterior_identities():
    """The stochastic step against the Gaussian algebra it comes from (cited DDPM papers): re-derived betas,
    posterior mean and variance of q(x_{k-1} | x_k, x0), the log-domain variance interpolation, the last step."""
    # all 1000 steps kept: the re-derived betas are the original linear schedule
    full = sampler.ddpm_table(1000)
    betas = np.linspace(1e-4, 2e-2, 1000)
    np.testing.assert_allclose([np.exp(r[5]) for r in full], betas[::-1], rtol=1e-12)
    tab = sampler.ddpm_table(50)
    assert [r[0] for r in tab[:3]] == [980, 960, 940] and tab[-1][0] == 0       # same timestep subset as DDIM
    ddim = sampler.ddim_table(50)
    ab = np.array([r[1] ** 2 for r in ddim])            # alpha_bar of the kept steps, descending t
    ab_prev = np.array([r[3] ** 2 for r in ddim])
    for i, r in enumerate(tab):
        _, sr, srm1, c0, ct, lb, lp, nz = r
        a, ap = ab[i], ab_prev[i]
        beta = 1 - a / ap
        assert abs(sr - 1 / np.sqrt(a)) < 1e-12 and abs(srm1 - np.sqrt(1 / a - 1)) < 1e-9
        assert abs(np.exp(lb) - beta) < 1e-14
        # q(x_{k-1} | x_k, x0) from the joint Gaussian: x_{k-1} = sqrt(ap) x0 + sqrt(1-ap) e1,  x_k = sqrt(1-beta) x_{k-1} + sqrt(beta) e2
        #   precision = (1-beta)/beta + 1/(1-ap);  mean = var * (sqrt(1-beta)/beta x_k + sqrt(ap)/(1-ap) x0)
        if i < len(tab) - 1:
            var = 1.0 / ((1 - beta) / beta + 1.0 / (1 - ap))
            assert abs(np.exp(lp) - var) < 1e-12 * var + 1e-18
            assert abs(ct - var * np.sqrt(1 - beta) / beta) < 1e-10 and abs(c0 - var * np.sqrt(ap) / (1 - ap)) < 1e-10
            assert nz == 1.0
        else:
            assert nz == 0.0 and abs(c0 - 1.0) < 1e-12 and abs(ct) < 1e-12      # alpha_bar_prev = 1: the mean is x0
            assert lp == tab[-2][6]                                              # clipped log variance
        # a noise-free x0 maps to the mean of q(x_{k-1} | x0): coef_x0 + coef_xt sqrt(ab) = sqrt(ab_prev)
        assert abs(c0 + ct * np.sqrt(a) - np.sqrt(ap)) < 1e-12
    # update rule: true noise in -> exact x0 and its posterior mean; v = +1 / -1 select beta' / posterior variance
    rng = np.random.default_rng(11)
    x0 = rng.standard_normal((2, 4, 8, 8))
    e = rng.standard_normal(x0.shape)
    z = rng.standard_normal(x0.shape)
    r = tab[7]
    a = ab[7]
    xk = np.sqrt(a) * x0 + np.sqrt(1 - a) * e
    mean = r[3] * x0 + r[4] * xk
    up = sampler.ddpm_update(xk, e, np.ones_like(x0), r, z)
    np.testing.assert_allclose(up, mean + np.sqrt(np.exp(r[5])) * z, rtol=1e-10, atol=1e-10)
    lo = sampler.ddpm_update(xk, e, -np.ones_like(x0), r, z)
    np.testing.assert_allclose(lo, mean + np.sqrt(np.exp(r[6])) * z, rtol=1e-10, atol=1e-10)
    mid = sampler.ddpm_update(xk, e, np.zeros_like(x0), r, z)
    np.testing.assert_allclose(mid, mean + np.exp(0.25 * (r[5] + r[6])) * z, rtol=1e-10, atol=1e-10)   # geometric mean
    last = sampler.ddpm_update(xk, e, np.zeros_like(x0), tab[-1], z)
    x0_last = tab[-1][1] * xk - tab[-1][2] * e
    np.testing.assert_allclose(last, x0_last, rtol=1e-12, atol=1e-12)            # no noise at the last step
    with pytest.raises(ValueError):
        sampler.ddpm_table(1)


def test_ddpm_sampler_runs_and_uses_the_noise(tiny):
    cfg, model, latent, labels, scales = tiny
    ctx = dit.Context(quant="static", scales=scales)
    S = 5
    rng = np.random.default_rng(12)
    noise = rng.standard_normal((S,) + latent.shape)
    a = sampler.sample(model, ctx, sampler.SamplerConfig(S, cache_interval=2, guidance=1.5, kind="ddpm", noise=noise), latent, labels)
    b = sampler.sample(model, ctx, sampler.SamplerConfig(S, cache_interval=2, guidance=1.5, kind="ddpm", noise=noise), latent, labels)
    np.testing.assert_array_equal(a, b)                                           # deterministic given the noise
    c = sampler.sample(model, ctx, sampler.SamplerConfig(S, cache_interval=2, guidance=1.5, kind="ddpm", noise=-noise), latent, labels)
    assert np.isfinite(a).all() and not np.allclose(a, c)
    # the last step's noise is never used
    n2 = noise.copy()
    n2[-1] = 0
    d = sampler.sample(model, ctx, sampler.SamplerConfig(S, cache_interval=2, guidance=1.5, kind="ddpm", noise=n2), latent, labels)
    np.testing.assert_array_equal(a, d)


def test_cfg_combine():
    rng = np.random.default_rng(1)
    e = rng.standard_normal((6, 4, 2, 2))
    np.testing.assert_array_equal(sampler.cfg_combine(e, 1.0), e[3:] + 1.0 * (e[:3] - e[3:]))
    np.testing.assert_allclose(sampler.cfg_combine(e, 1.0), e[:3], atol=1e-15)      # g = 1: conditional
    np.testing.assert_allclose(sampler.cfg_combine(e, 0.0), e[3:], atol=0)          # g = 0: unconditional
    np.testing.assert_allclose(sampler.cfg_combine(e, 1.5), 1.5 * e[:3] - 0.5 * e[3:], atol=1e-15)


@pytest.fixture(scope="module")
def tiny():
    cfg = synth.DIT_TINY
    model = dit.make_qmodel(cfg, synth.model_weights(21, cfg))
    latent = synth.normal(21, "latent", (2, cfg.channels, cfg.latent_side, cfg.latent_side))
    labels = np.array([3, 77])
    scales = calib.calibrate_model(model, [(latent, np.array([500.0, 500.0]), labels)])
    return cfg, model, latent, labels, scales


def test_interval_one_equals_uncached_bit_for_bit(tiny):
    cfg, model, latent, labels, scales = tiny
    ctx = dit.Context(quant="static", scales=scales)
    a = sampler.sample(model, ctx, sampler.SamplerConfig(6, cache_interval=1, guidance=1.5), latent, labels)
    b = sampler.sample(model, ctx, sampler.SamplerConfig(6, use_cache=False, guidance=1.5), latent, labels)
    np.testing.assert_array_equal(a, b)
    c = sampler.sample(model, ctx, sampler.SamplerConfig(6, cache_interval=2, guidance=1.5), latent, labels)
    assert not np.array_equal(a, c)           # the cache changes the trajectory ...
    assert np.linalg.norm(a - c) / np.linalg.norm(a) < 0.2     # ... but only mildly


def test_large_interval_computes_only_step_zero(tiny):
    cfg, model, latent, labels, scales = tiny
    ctx = dit.Context(quant="static", scales=scales)
    flags = []
    sampler.sample(model, ctx, sampler.SamplerConfig(5, cache_interval=9), latent, labels,
                   on_step=lambda i, x, reuse: flags.append(reuse))
    assert flags == [False, True, True, True, True]


def test_reuse_step_closed_form_and_state_error(tiny):
    cfg, model, latent, labels, scales = tiny
    ctx = dit.Context(quant="static", scales=scales, storage=dit.Storage.exact())
    t0, t1 = np.full(2, 900.0), np.full(2, 800.0)
    with pytest.raises(KeyError):
        dit.forward(model, ctx, latent, t1, labels, cache={}, reuse=True)
    cache = {}
    dit.forward(model, ctx, latent, t0, labels, cache=cache)
    assert sorted(cache) == sorted((i, b) for i in range(cfg.depth) for b in ("attn", "mlp"))
    taps = {}
    ctx2 = dit.Context(quant="static", scales=scales, storage=dit.Storage.exact(),
                       tap=lambda n, a: taps.__setitem__(n, np.array(a)))
    lat1 = latent * 0.9 + 0.05
    dit.forward(model, ctx2, lat1, t1, labels, cache=cache, reuse=True)
    # x_final = x_embed + sum_b (gate_msa_b * A_b + gate_mlp_b * Mo_b) with gates of the CURRENT step
    rows = np.arange(2 * cfg.tokens) // cfg.tokens
    want = taps["x_embed"].copy()
    D = cfg.hidden
    for i in range(cfg.depth):
        mod = taps[f"blk{i}.mod"]
        want += mod[rows, 2 * D:3 * D] * cache[(i, "attn")] + mod[rows, 5 * D:6 * D] * cache[(i, "mlp")]
    np.testing.assert_allclose(taps["x_final"], want, rtol=1e-13, atol=1e-13)
    # no attention / MLP linear ran on the reuse step
    assert not any(k.endswith((".qkv.in", ".fc1.in", ".proj.in", ".fc2.in")) for k in taps)
    # the cached tensors are the pre-gate branch outputs of the refresh step
    taps0 = {}
    ctx3 = dit.Context(quant="static", scales=scales, storage=dit.Storage.exact(),
                       tap=lambda n, a: taps0.__setitem__(n, np.array(a)))
    dit.forward(model, ctx3, latent, t0, labels, cache={})
    np.testing.assert_array_equal(cache[(1, "attn")], taps0["blk1.attn_branch"])
    np.testing.assert_array_equal(cache[(1, "mlp")], taps0["blk1.mlp_branch"])


# ----------------------------------------------------------------------------- VC
def test_per_branch_schedule_reduces_to_the_global_rule_and_to_its_closed_form(tiny):
    """A [steps, blocks, 2] reuse schedule: the global rule written as a schedule gives the same trajectory bit for
    bit; an all-compute schedule equals the un-cached loop; a mixed step obeys its block-by-block definition."""
    cfg, model, latent, labels, scales = tiny
    ctx = dit.Context(quant="static", scales=scales)
    S, N = 6, 2
    glob = np.zeros((S, cfg.depth, 2), dtype=bool)
    for i in range(S):
        glob[i] = not sampler.should_refresh(i, N)
    a = sampler.sample(model, ctx, sampler.SamplerConfig(S, cache_interval=N, guidance=1.5), latent, labels)
    b = sampler.sample(model, ctx, sampler.SamplerConfig(S, cache_interval=1, guidance=1.5, schedule=glob), latent, labels)
    np.testing.assert_array_equal(a, b)
    none = np.zeros((S, cfg.depth, 2), dtype=bool)
    c = sampler.sample(model, ctx, sampler.SamplerConfig(S, guidance=1.5, schedule=none), latent, labels)
    d = sampler.sample(model, ctx, sampler.SamplerConfig(S, use_cache=False, guidance=1.5), latent, labels)
    np.testing.assert_array_equal(c, d)
    # mixed mask in exact storage: reusing only block 1's attention branch replaces exactly that branch output
    ex = dit.Context(quant="static", scales=scales, storage=dit.Storage.exact())
    t0, t1 = np.full(2, 900.0), np.full(2, 800.0)
    cache = {}
    dit.forward(model, ex, latent, t0, labels, cache=cache)
    kept = cache[(1, "attn")].copy()
    mask = np.zeros((cfg.depth, 2), dtype=bool)
    mask[1, 0] = True
    taps = {}
    ex2 = dit.Context(quant="static", scales=scales, storage=dit.Storage.exact(),
                      tap=lambda n, v: taps.__setitem__(n, np.array(v)))
    lat1 = latent * 0.9 + 0.05
    dit.forward(model, ex2, lat1, t1, labels, cache=cache, mask=mask)
    np.testing.assert_array_equal(cache[(1, "attn")], kept)                       # a reused entry is not rewritten
    assert "blk1.attn_branch" not in taps and "blk0.attn_branch" in taps and "blk1.mlp_branch" in taps
    rows = np.arange(2 * cfg.tokens) // cfg.tokens
    D = cfg.hidden
    want_mid = taps["blk0.x_out"] + taps["blk1.mod"][rows, 2 * D:3 * D] * kept    # x + gate_msa(current step) * cached A
    np.testing.assert_allclose(taps["blk1.x_mid"], want_mid, rtol=1e-13, atol=1e-13)
    # the other entries were refreshed with this step's values
    np.testing.assert_array_equal(cache[(1, "mlp")], taps["blk1.mlp_branch"])
    # a branch that was never stored cannot be reused
    with pytest.raises(KeyError):
        dit.forward(model, ex, latent, t1, labels, cache={}, mask=mask)


def test_vc_apply_identities():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((3, 4, 8, 8)) * np.array([0.5, 1, 2, 3]).reshape(1, 4, 1, 1) + 0.7
    np.testing.assert_allclose(vc.apply(x, np.ones(4)), x, atol=1e-15)
    K = np.array([0.9, 1.0, 1.1, 1.3])
    y = vc.apply(x, K)
    np.testing.assert_allclose(y.mean(axis=(2, 3)), x.mean(axis=(2, 3)), atol=1e-14)      # mean preserved
    np.testing.assert_allclose(y.var(axis=(2, 3)), x.var(axis=(2, 3)) * K ** 2, rtol=1e-12)  # variance scaled by K^2
    # rescaling identity: var_ratio mode reaches the target variance; factor 1 when variances already match
    tgt = np.array([0.3, 1.0, 2.5, 4.0])
    z = vc.apply(x, tgt, mode="var_ratio", eps=0.0)
    np.testing.assert_allclose(z.var(axis=(2, 3)), np.broadcast_to(tgt, (3, 4)), rtol=1e-12)
    same = vc.apply(x[:1], x[0].var(axis=(1, 2)), mode="var_ratio", eps=0.0)
    np.testing.assert_allclose(same, x[:1], atol=1e-13)
    z6 = vc.apply(x, tgt, mode="var_ratio", eps=1e-6)
    np.testing.assert_allclose(z6.var(axis=(2, 3)), np.broadcast_to(tgt, (3, 4)), rtol=1e-5)


def _objective(K, xh, xt, eps):
    mu = xh.mean(axis=(2, 3), keepdims=True)
    xtil = mu + K.reshape(1, -1, 1, 1) * (xh - mu)
    d = xtil - xt
    return (d ** 2 / (xt ** 2 + eps)).sum(axis=(0, 2, 3)) + (d ** 2).sum(axis=(0, 2, 3))


def test_vc_fit_closed_form():
    rng = np.random.default_rng(4)
    xt = rng.standard_normal((5, 4, 6, 6)) + 0.3
    # x^ = mu + r (x' - mu)  =>  K = 1/r ;  x^ = x'  =>  K = 1
    np.testing.assert_allclose(vc.fit(xt, xt), np.ones(4), atol=1e-13)
    r = np.array([0.8, 0.9, 1.25, 2.0]).reshape(1, 4, 1, 1)
    mu = xt.mean(axis=(2, 3), keepdims=True)
    xh = mu + r * (xt - mu)
    np.testing.assert_allclose(vc.fit(xh, xt), 1 / r.ravel(), rtol=1e-12)
    # general case: the closed form is the minimiser of rQNSR^2 + MSE (checked by bracketing)
    xh = xt * 0.9 + 0.2 * rng.standard_normal(xt.shape)
    K = vc.fit(xh, xt, eps=1e-6)
    f0 = _objective(K, xh, xt, 1e-6)
    for d in (1e-3, -1e-3, 0.05, -0.05):
        assert (_objective(K + d, xh, xt, 1e-6) > f0).all()
    # the form as printed coincides with the derived one when mu = 0 and eps = 0
    xh0 = xh - xh.mean(axis=(2, 3), keepdims=True)
    np.testing.assert_allclose(vc.fit(xh0, xt, eps=0.0, form="printed"), vc.fit(xh0, xt, eps=0.0), rtol=1e-10)


def test_sampler_applies_vc_every_step(tiny):
    cfg, model, latent, labels, scales = tiny
    ctx = dit.Context(quant="static", scales=scales)
    S = 4
    base = sampler.sample(model, ctx, sampler.SamplerConfig(S, cache_interval=2), latent, labels)
    ones = sampler.sample(model, ctx, sampler.SamplerConfig(S, cache_interval=2, vc_table=np.ones((S, 4))), latent, labels)
    np.testing.assert_allclose(ones, base, atol=1e-6)         # K = 1 is the identity (up to float32 storage)
    K = np.full((S, 4), 1.05)
    seen = []
    out = sampler.sample(model, ctx, sampler.SamplerConfig(S, cache_interval=2, vc_table=K), latent, labels,
                         on_step=lambda i, x, r: seen.append(x.copy()))
    assert len(seen) == S and not np.allclose(out, base)
    # first step by hand: DDIM update of the un-corrected run, then mu + K (x - mu)
    first = []
    sampler.sample(model, ctx, sampler.SamplerConfig(1 * S, cache_interval=2), latent, labels,
                   on_step=lambda i, x, r: first.append(x.copy()))
    np.testing.assert_allclose(seen[0], vc.apply(first[0], K[0]), atol=1e-6)


def test_skipped_step_walked_block_by_block_equals_the_accumulated_form(tiny):
    """The fully skipped step has two spellings: every block adds its cached branches in turn (the cache rule
    taken literally), or all of them are accumulated and stored once.  In exact storage they are the same sum;
    with a bfloat16 residual stream the walked form rounds after each of the 2 * depth additions, so the two may
    differ by a few bfloat16 steps per element (at most depth steps: 2 * depth roundings of half a step each)."""
    cfg, model, latent, labels, scales = tiny
    t0, t1 = np.full(2, 900.0), np.full(2, 800.0)
    lat1 = latent * 0.9 + 0.05
    for storage, exact in ((dit.Storage.exact(), True), (dit.Storage(), False)):
        outs, finals = [], []
        for walk in (False, True):
            taps = {}
            ctx = dit.Context(quant="static", scales=scales, storage=storage, reuse_walk=walk,
                              tap=lambda n, a, taps=taps: taps.__setitem__(n, np.array(a)))
            cache = {}
            dit.forward(model, ctx, latent, t0, labels, cache=cache)
            outs.append(dit.forward(model, ctx, lat1, t1, labels, cache=cache, reuse=True))
            finals.append(taps["x_final"])
        acc, walk = finals
        if exact:
            np.testing.assert_allclose(walk, acc, rtol=1e-13, atol=1e-13)
            np.testing.assert_allclose(outs[1], outs[0], rtol=1e-11, atol=1e-12)
        else:
            # one bfloat16 step at the largest magnitude any partial sum of the element can reach
            rows = np.arange(2 * cfg.tokens) // cfg.tokens
            D = cfg.hidden
            bound = np.abs(taps["x_embed"])
            for i in range(cfg.depth):
                mod = taps[f"blk{i}.mod"]
                bound = bound + np.abs(mod[rows, 2 * D:3 * D] * cache[(i, "attn")]) + np.abs(mod[rows, 5 * D:6 * D] * cache[(i, "mlp")])
            step = 2.0 ** (np.floor(np.log2(bound)) - 7)
            steps = np.abs(walk - acc) / step
            assert steps.max() <= cfg.depth + 1
            assert np.mean(steps > 0) > 0.01                 # the two spellings do differ, by rounding only
            rel = np.linalg.norm(outs[1] - outs[0]) / np.linalg.norm(outs[0])
            print(f"walked vs accumulated skipped step, bf16 residual: max {steps.max():.1f} bf16 steps, output rel-L2 {rel:.2e}")
            assert rel < 1e-2
