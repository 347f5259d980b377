"""GPU parity: block-output cache kernels and the variance-compensation kernel vs the oracle."""
import numpy as np
import pytest
import torch

import synth
from oracle import dit, vc

from gpu_util import bf16_to_f64, dev

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


def test_cache_schedule_host():
    import paper_2503_02508_b200 as q
    from oracle import sampler
    for interval in (1, 2, 3, 7):
        for i in range(20):
            assert q.qdit_cache_should_refresh(i, interval) == int(sampler.should_refresh(i, interval))
    assert q.qdit_cache_should_refresh(0, 0) == q.QDIT_ERR_INVALID_ARG
    assert q.qdit_cache_should_refresh(-1, 2) == q.QDIT_ERR_INVALID_ARG


def test_cache_store_reuse_and_state(q, ctx):
    blocks, B, T, D = 3, 2, 64, 144
    M = B * T
    cache = q.qdit_cache_create(ctx, blocks, M, D)
    try:
        x0 = synth.normal(61, "x", (M, D))
        xd = dev(x0).to(torch.bfloat16)
        mod = synth.normal(61, "mod", (B, blocks * 6 * D), 0.35)
        md = dev(mod)
        # reuse before any store is a state error, not a read of uninitialised memory
        assert q.lib.qdit_cache_reuse(ctx, cache, 0, 0, md.data_ptr(), blocks * 6 * D, T, xd.data_ptr()) == q.QDIT_ERR_STATE
        assert q.lib.qdit_cache_reuse_all(ctx, cache, md.data_ptr(), blocks * 6 * D, T, xd.data_ptr()) == q.QDIT_ERR_STATE
        ys = {}
        for b in range(blocks):
            for br in (0, 1):
                y = dev(synth.normal(61, f"y{b}.{br}", (M, D))).to(torch.bfloat16)
                ys[(b, br)] = bf16_to_f64(y)
                q.qdit_cache_store(ctx, cache, b, br, y)
        rows = np.arange(M) // T
        # one fused pass == the closed form of a fully skipped step
        x1 = xd.clone()
        q.qdit_cache_reuse_all(ctx, cache, md, blocks * 6 * D, T, x1)
        q.qdit_sync(ctx)
        want = bf16_to_f64(xd).copy()
        for b in range(blocks):
            want += mod[rows, b * 6 * D + 2 * D:b * 6 * D + 3 * D].astype(np.float64) * ys[(b, 0)]
            want += mod[rows, b * 6 * D + 5 * D:b * 6 * D + 6 * D].astype(np.float64) * ys[(b, 1)]
        got = bf16_to_f64(x1)
        assert (got != dit.round_bf16(want)).mean() < 2e-3                     # f32 vs f64 sums straddling a bf16 tie
        assert np.abs(got - want).max() <= 2.0 ** -8 * np.abs(want).max()
        # single-slot reuse: x + gate * slot
        x2 = xd.clone()
        g = md[:, 2 * D:3 * D]
        q.qdit_cache_reuse(ctx, cache, 0, q.QDIT_BRANCH_ATTN, g, blocks * 6 * D, T, x2)
        q.qdit_sync(ctx)
        want2 = bf16_to_f64(xd) + mod[rows, 2 * D:3 * D].astype(np.float64) * ys[(0, 0)]
        assert (bf16_to_f64(x2) != dit.round_bf16(want2)).mean() < 2e-3
        # invalidation empties the cache again
        q.qdit_cache_invalidate(cache)
        assert q.lib.qdit_cache_reuse(ctx, cache, 0, 0, md.data_ptr(), blocks * 6 * D, T, xd.data_ptr()) == q.QDIT_ERR_STATE
        assert q.qdit_cache_slot(cache, blocks, 0) is None and q.qdit_cache_slot(cache, 0, 2) is None
    finally:
        q.qdit_cache_destroy(cache)


@pytest.mark.parametrize("N,C,HW", [(4, 4, 1024), (2, 4, 4096), (1, 3, 64), (5, 2, 100)])
def test_vc_fit_matches_the_closed_form(q, ctx, N, C, HW):
    """K of one step fitted on the device against oracle.vc.fit (both forms), incl. targets that pass through zero."""
    side = int(np.sqrt(HW))
    xt = synth.normal(63, f"fit_t{HW}", (N, C, HW)) * np.array([0.5, 1.0, 2.0, 3.0][:C], dtype=np.float32).reshape(1, C, 1)
    r = np.array([1.1, 0.9, 1.3, 0.8][:C], dtype=np.float32).reshape(1, C, 1)
    xh = (xt.mean(axis=2, keepdims=True) + r * (xt - xt.mean(axis=2, keepdims=True)) +
          0.05 * synth.normal(63, f"fit_n{HW}", (N, C, HW))).astype(np.float32)
    ws = torch.empty(4 * N * C, dtype=torch.float64, device="cuda")
    for form, name in ((q.QDIT_VC_FIT_DERIVED, "derived"), (q.QDIT_VC_FIT_PRINTED, "printed")):
        kd = torch.empty(C, dtype=torch.float32, device="cuda")
        q.qdit_vc_fit(ctx, dev(xh), dev(xt), N, C, HW, 1e-6, form, ws, kd)
        q.qdit_sync(ctx)
        want = vc.fit(xh.reshape(N, C, side, side), xt.reshape(N, C, side, side), eps=1e-6, form=name)
        # f64 sums on both sides; what is left is the summation order and the final rounding of K to f32
        np.testing.assert_allclose(kd.cpu().numpy(), want, rtol=2e-6)
    # a trajectory that already matches its target needs no compensation
    kd = torch.empty(C, dtype=torch.float32, device="cuda")
    q.qdit_vc_fit(ctx, dev(xt), dev(xt), N, C, HW, 1e-6, q.QDIT_VC_FIT_DERIVED, ws, kd)
    q.qdit_sync(ctx)
    np.testing.assert_allclose(kd.cpu().numpy(), np.ones(C), rtol=1e-6)
    # the fitted K minimises the objective sum (K a - b)^2 (1 + w) per channel: lower than K = 1 and than K +- 1 %
    kd = torch.empty(C, dtype=torch.float32, device="cuda")
    q.qdit_vc_fit(ctx, dev(xh), dev(xt), N, C, HW, 1e-6, q.QDIT_VC_FIT_DERIVED, ws, kd)
    q.qdit_sync(ctx)
    kf = kd.cpu().numpy().astype(np.float64).reshape(1, C, 1)
    x64, t64 = xh.astype(np.float64), xt.astype(np.float64)
    a = x64 - x64.mean(axis=2, keepdims=True)
    b = t64 - x64.mean(axis=2, keepdims=True)
    w1 = 1.0 + 1.0 / (t64 ** 2 + 1e-6)

    def objective(k):
        return (np.square(k * a - b) * w1).sum(axis=(0, 2))

    j = objective(kf)
    assert (j <= objective(np.ones_like(kf))).all()
    assert (j <= objective(kf * 1.01)).all() and (j <= objective(kf * 0.99)).all()


@pytest.mark.parametrize("n,d,alpha,e", [(64, 4096, 0.7, 0.5), (200, 1024, 0.3, -0.5), (4, 16, 1.0, 0.5)])
def test_tap_laplacian_matches_oracle(q, ctx, n, d, alpha, e):
    """Similarity matrix and degree normalisation of Algorithm 1 for one subsample."""
    from oracle import tap
    x = synth.normal(65, f"tap{n}x{d}", (n, d)) + 0.5          # a common offset: cosines well away from zero
    if n > 8:
        x[5] = 0                                               # a zero feature vector
        x[7] = 3 * x[2]
    t = synth.uniform_int(65, f"tapt{n}", (n,), 0, 20).astype(np.float32)
    ws = torch.empty(n * d + 2 * n, dtype=torch.float32, device="cuda")
    L = torch.empty((n, n), dtype=torch.float32, device="cuda")
    q.qdit_tap_laplacian(ctx, dev(x), dev(t), n, d, alpha, e, ws, L)
    q.qdit_sync(ctx)
    want = tap.laplacian(tap.affinity(x, t, alpha), e)
    got = L.cpu().numpy().astype(np.float64)
    assert np.abs(got - want).max() <= 2e-5 * np.abs(want).max()
    np.testing.assert_allclose(got, got.T, rtol=1e-5, atol=1e-6 * np.abs(want).max())
    assert q.lib.qdit_tap_laplacian(ctx, dev(x).data_ptr(), dev(t).data_ptr(), n + 1, d, alpha, e, ws.data_ptr(), L.data_ptr()) == q.QDIT_ERR_SHAPE
    q.qdit_sync(ctx)


def test_bounded_wait_times_out_and_context_stays_usable(q, ctx):
    """The time-out path of the pipelined kernels, exercised without hanging anything: a wait with a small poll
    limit on a barrier that nobody signals runs out, a second waiter leaves through the abort flag, the kernel
    ends normally, qdit_sync reports the time-out once, and the context keeps working."""
    q.qdit_sync(ctx)
    obs = torch.zeros(2, dtype=torch.int32, device="cuda")
    q.qdit_selftest_wait_timeout(ctx, 4096, obs)
    assert q.lib.qdit_sync(ctx) == q.QDIT_ERR_TIMEOUT
    assert b"wait" in q.lib.qdit_last_error(ctx)
    assert obs.cpu().tolist() == [1, 1]
    assert q.lib.qdit_sync(ctx) == q.QDIT_OK
    x = synth.normal(64, "after_timeout", (64, 128))
    out = torch.empty((64, 128), dtype=torch.uint8, device="cuda")
    q.qdit_quantize_act(ctx, dev(x), q.QDIT_F32, 64, 128, 128, q.QDIT_QUANT_STATIC, q.qparams(0.02), None, out, 128)
    q.qdit_sync(ctx)
    want = np.clip(np.rint(x * (np.float32(1.0) / np.float32(0.02))), -127, 127).astype(np.int32)
    got = out.cpu().numpy().view(np.int8).astype(np.int32)
    np.testing.assert_array_equal(got, want)
    assert q.lib.qdit_selftest_wait_timeout(ctx, 0, obs.data_ptr()) == q.QDIT_ERR_INVALID_ARG
    assert q.lib.qdit_selftest_wait_timeout(ctx, 1 << 21, obs.data_ptr()) == q.QDIT_ERR_INVALID_ARG


def test_vc_fit_rejects_bad_arguments(q, ctx):
    import ctypes as C
    x = torch.zeros(4 * 64, dtype=torch.float32, device="cuda")
    ws = torch.zeros(16, dtype=torch.float64, device="cuda")
    k = torch.zeros(4, dtype=torch.float32, device="cuda")
    L = q.lib
    assert L.qdit_vc_fit(ctx, x.data_ptr(), x.data_ptr(), 0, 4, 64, 1e-6, 0, ws.data_ptr(), k.data_ptr()) == q.QDIT_ERR_SHAPE
    assert L.qdit_vc_fit(ctx, x.data_ptr(), x.data_ptr(), 1, 4, 64, 1e-6, 7, ws.data_ptr(), k.data_ptr()) == q.QDIT_ERR_INVALID_ARG
    assert L.qdit_vc_fit(ctx, x.data_ptr(), None, 1, 4, 64, 1e-6, 0, ws.data_ptr(), k.data_ptr()) == q.QDIT_ERR_INVALID_ARG
    assert L.qdit_vc_fit(ctx, x.data_ptr(), x.data_ptr(), 1, 4, 64, 1e-6, 0, None, k.data_ptr()) == q.QDIT_ERR_INVALID_ARG
    q.qdit_sync(ctx)


@pytest.mark.parametrize("B,C,HW", [(3, 4, 1024), (2, 4, 4096), (1, 3, 64)])
def test_vc_correct(q, ctx, B, C, HW):
    S = 5
    x = synth.normal(62, f"lat{HW}", (B, C, HW)) * np.array([0.5, 1.0, 2.0, 3.0][:C], dtype=np.float32).reshape(1, C, 1) + 0.4
    K = (1.0 + 0.1 * synth.normal(62, "K", (S, C))).astype(np.float32)
    kd = dev(K)
    side = int(np.sqrt(HW))
    for step in (0, 3):
        xd = dev(x)
        q.qdit_vc_correct(ctx, xd, B, C, HW, step, q.QDIT_VC_K_TABLE, kd, 1e-6)
        q.qdit_sync(ctx)
        want = vc.apply(x.reshape(B, C, side, side), K[step]).reshape(B, C, HW)
        np.testing.assert_allclose(xd.cpu().numpy(), want, rtol=2e-6, atol=2e-6)
    tgt = np.abs(synth.normal(62, "tgt", (S, C))).astype(np.float32) + 0.2
    xd = dev(x)
    q.qdit_vc_correct(ctx, xd, B, C, HW, 2, q.QDIT_VC_VAR_RATIO, dev(tgt), 1e-6)
    q.qdit_sync(ctx)
    got = xd.cpu().numpy().astype(np.float64)
    want = vc.apply(x.reshape(B, C, side, side), tgt[2], mode="var_ratio", eps=1e-6).reshape(B, C, HW)
    np.testing.assert_allclose(got, want, rtol=5e-6, atol=5e-6)
    np.testing.assert_allclose(got.var(axis=2), np.broadcast_to(tgt[2], (B, C)), rtol=1e-4)   # reaches the target variance
    np.testing.assert_allclose(got.mean(axis=2), x.astype(np.float64).mean(axis=2), atol=1e-5)  # mean preserved
    # K = 1 leaves the latent unchanged up to f32 rounding of mu + (x - mu)
    xd = dev(x)
    q.qdit_vc_correct(ctx, xd, B, C, HW, 0, q.QDIT_VC_K_TABLE, dev(np.ones((S, C), dtype=np.float32)), 1e-6)
    q.qdit_sync(ctx)
    np.testing.assert_allclose(xd.cpu().numpy(), x, rtol=0, atol=1e-6)


def test_mma_probe_runs_and_scales_with_the_work(q, ctx):
    """The tensor-pipe probe: both modes end by themselves with a clean status, the time grows with the number of
    instruction groups, and bad arguments are refused before any launch."""
    operands = torch.randint(-127, 128, (1024, 1024), dtype=torch.int8, device="cuda")
    torch.cuda.synchronize()
    for mode in (0, 1):
        for n in (64, 256):
            q.qdit_probe_mma_rate(ctx, mode, n, 256, operands, 1024)       # warm-up
            short = min(q.qdit_probe_mma_rate(ctx, mode, n, 512, operands, 1024) for _ in range(3))
            long_ = min(q.qdit_probe_mma_rate(ctx, mode, n, 4096, operands, 1024) for _ in range(3))
            assert 0.0 < short < long_ < 50.0, (mode, n, short, long_)
            assert long_ > 3.0 * short - 0.05, (mode, n, short, long_)      # 8 x the groups, minus the fixed launch cost
    q.qdit_sync(ctx)                                                       # no wait ran out
    import ctypes as C
    ms = C.c_float()
    for bad in ((2, 128, 16, 1024), (0, 100, 16, 1024), (0, 128, 0, 1024), (0, 128, 1 << 17, 1024), (0, 128, 16, 100)):
        mode, n, iters, rows = bad
        assert q.lib.qdit_probe_mma_rate(ctx, mode, n, iters, operands.data_ptr(), rows, C.byref(ms)) < 0, bad
