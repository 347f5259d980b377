"""The allocation-free dynamic quantizer gives exactly what the regular dynamic quantizer gives.

qdit_quantize_act_dynamic_static exists for callers that may not allocate device memory (they own only
their input and output tensors).  It reduces max|x| through a fixed array inside the library instead of
borrowed or allocated scratch.  This file is collected last on purpose: it must pass on its own in a
fresh process and also after every other GPU test has run in the same process.
"""
import numpy as np
import pytest
import torch

import synth
from oracle import quant

pytestmark = pytest.mark.gpu


def _both(q, ctx, x, dtype):
    M, K = x.shape
    xd = torch.from_numpy(x).cuda()
    code = q.QDIT_F32
    if dtype == "bf16":
        xd, code = xd.to(torch.bfloat16), q.QDIT_BF16
    ref_q = torch.empty((M, K), dtype=torch.uint8, device="cuda")
    ref_s = torch.zeros(1, dtype=torch.float32, device="cuda")
    q.qdit_quantize_act(ctx, xd, code, M, K, K, q.QDIT_QUANT_DYNAMIC, None, ref_s, ref_q, K)
    new_q = torch.full((M, K), 0x55, dtype=torch.uint8, device="cuda")
    new_s = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
    q.qdit_quantize_act_dynamic_static(ctx, xd, code, M, K, K, new_s, new_q, K)
    q.qdit_sync(ctx)
    return ref_q.cpu().numpy(), float(ref_s.item()), new_q.cpu().numpy(), float(new_s.item())


def test_static_scratch_quantizer_matches_regular_entry_point_twice_in_a_row():
    import paper_2503_02508_b200 as q
    ctx = q.qdit_create(0, None)
    try:
        # first call: large, fills many scratch slots with large maxima (outlier channels x20)
        x1 = synth.outlier_activations(91, "noalloc1", 4096, 1152)
        # second call: smaller and much smaller in magnitude; stale slots of the first call must not leak in
        x2 = (synth.normal(91, "noalloc2", (37, 384)) * 1e-3).astype(np.float32)
        for x, dtype in ((x1, "bf16"), (x2, "f32"), (x1[:300], "f32"), (np.zeros((8, 16), dtype=np.float32), "f32")):
            ref_q, ref_s, new_q, new_s = _both(q, ctx, x, dtype)
            assert new_s == ref_s                       # same scale, bit for bit (a maximum has no rounding order)
            np.testing.assert_array_equal(new_q, ref_q)  # same codes
            # and both are the CPU oracle's dynamic quantizer (Eq. 1 with s = max|x| / 127) on the same input bits
            xin = x if dtype == "f32" else torch.from_numpy(x).to(torch.bfloat16).float().numpy()
            qp = quant.qparams_symmetric(float(np.abs(xin).max()))
            assert new_s == np.float32(qp.scale)
            np.testing.assert_array_equal(new_q.view(np.int8).astype(np.int32), quant.quantize(xin, qp))
        assert _both(q, ctx, np.zeros((8, 16), dtype=np.float32), "f32")[3] == 1.0
        # beyond the built-in scratch: refused with a clear message, nothing launched
        big_m = 65536 * 2048 // 1152 + 2
        st = q.lib.qdit_quantize_act_dynamic_static(ctx, 256, q.QDIT_F32, big_m, 1152, 1152, 256, 256, 1152)
        assert st == q.QDIT_ERR_SHAPE and b"built-in scratch" in q.lib.qdit_last_error(ctx)
        # sizes whose product would wrap a 64-bit integer are refused the same way
        st = q.lib.qdit_quantize_act_dynamic_static(ctx, 256, q.QDIT_F32, 2 ** 40, 2 ** 40, 2 ** 40, 256, 256, 2 ** 40)
        assert st == q.QDIT_ERR_SHAPE and b"built-in scratch" in q.lib.qdit_last_error(ctx)
        # the one-time set-up leaves the caller's current device as it was
        assert torch.cuda.current_device() == 0
        q.qdit_sync(ctx)
    finally:
        q.qdit_destroy(ctx)
