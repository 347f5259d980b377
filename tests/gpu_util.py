"""Helpers for the GPU parity tests: context fixture plumbing, host<->device moves, error metrics."""
import numpy as np
import torch


def dev(a, dtype=None):
    t = torch.as_tensor(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda().contiguous()


def dev_i8(codes):
    """Integer codes in [-128,255] -> device bytes (two's complement / unsigned share the byte)."""
    a = (np.asarray(codes).astype(np.int64) & 0xFF).astype(np.uint8)
    return torch.from_numpy(a).cuda().contiguous()


def host_codes(t, signed=True):
    a = t.cpu().numpy().view(np.uint8).astype(np.int32)
    if signed:
        a = np.where(a > 127, a - 256, a)
    return a


def bf16_to_f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def max_rel_err(got, ref):
    """max_i |got_i - ref_i| / max(|ref_i|, 1e-2 * rms(ref))."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    floor = 1e-2 * np.sqrt(np.mean(ref ** 2)) + 1e-30
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), floor)))


def code_mismatch_report(q_gpu, q_ref, pre_round_ref, tol):
    """Fused producers: codes may differ from the oracle by one step, and only where the oracle's
    pre-rounding value x/s lies within `tol` of a half-integer.  Returns (n_mismatch, ok)."""
    d = q_gpu.astype(np.int64) - q_ref.astype(np.int64)
    bad = d != 0
    if not bad.any():
        return 0, True
    frac = np.abs(pre_round_ref - np.floor(pre_round_ref) - 0.5)
    ok = (np.abs(d[bad]) <= 1).all() and (frac[bad] <= tol).all()
    return int(bad.sum()), bool(ok)


class _DevView:
    def __init__(self, ptr, shape, typestr):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (int(ptr), False), "version": 2}


def view(ptr, shape, typestr):
    """Torch tensor aliasing raw device memory (typestr: '|i1', '|u1', '<f4', '<i4', '<u2' ...)."""
    return torch.as_tensor(_DevView(ptr, shape, typestr), device="cuda")


def bf16_view_to_f64(ptr, shape):
    u = view(ptr, shape, "<i2").clone()
    return u.view(torch.bfloat16).float().cpu().numpy().astype(np.float64)


def scales_to_arrays(scales, depth):
    """oracle ActScales -> (ada_scale, [depth,4] array) in the library's order qkv, proj, fc1, fc2."""
    blk = np.array([[scales.blocks[i][n].scale for n in ("qkv", "proj", "fc1", "fc2")] for i in range(depth)],
                   dtype=np.float32)
    return np.float32(scales.ada.scale), blk


def rel_l2(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.linalg.norm(got - ref) / (np.linalg.norm(ref) + 1e-30))


def bf16_steps_err(got, ref):
    """max_i |got_i - ref_i| / (bf16 step at max(|ref_i|, rms(ref))): how many bf16 steps apart a bf16-stored
    result is from the oracle's value (1 = a single rounding flip)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    mag = np.maximum(np.abs(ref), np.sqrt(np.mean(ref ** 2)) + 1e-30)
    step = 2.0 ** (np.floor(np.log2(mag)) - 7)
    return float(np.max(np.abs(got - ref) / step))
