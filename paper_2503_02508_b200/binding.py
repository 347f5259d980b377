"""ctypes binding of libqdit.so: same names as the C ABI, arguments marshalled only."""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqdit.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python paper_2503_02508_b200/build.py` "
        "(needs nvcc; the library targets sm_100a and has no CPU fallback)")
lib = C.CDLL(LIB_PATH)

# ----------------------------------------------------------------------------- constants (qdit.h)
QDIT_OK = 0
QDIT_ERR_INVALID_ARG, QDIT_ERR_SHAPE, QDIT_ERR_ALIGN, QDIT_ERR_UNSUPPORTED = -1, -2, -3, -4
QDIT_ERR_CUDA, QDIT_ERR_STATE, QDIT_ERR_TIMEOUT, QDIT_ERR_NOMEM = -5, -6, -7, -8
QDIT_BF16, QDIT_F32, QDIT_I8, QDIT_I32 = 0, 1, 2, 3
QDIT_QUANT_STATIC, QDIT_QUANT_DYNAMIC, QDIT_QUANT_DYNAMIC_TOKEN = 0, 1, 2
QDIT_EPI_BIAS, QDIT_EPI_GELU, QDIT_EPI_GATE, QDIT_EPI_RESIDUAL = 1, 2, 4, 8
QDIT_EPI_CACHE_STORE, QDIT_EPI_QUANT_OUT, QDIT_EPI_OUT_BF16, QDIT_EPI_OUT_F32, QDIT_EPI_OUT_I32 = 16, 32, 64, 128, 256
QDIT_EPI_ROW_SCALE = 512
QDIT_BRANCH_ATTN, QDIT_BRANCH_MLP = 0, 1
QDIT_VC_NONE, QDIT_VC_K_TABLE, QDIT_VC_VAR_RATIO = 0, 1, 2
QDIT_VC_FIT_DERIVED, QDIT_VC_FIT_PRINTED = 0, 1
QDIT_FWD_STORE_CACHE, QDIT_FWD_REUSE, QDIT_FWD_CALIBRATE = 1, 2, 4
(QDIT_OPT_PDL, QDIT_OPT_GEMM_BN, QDIT_OPT_GEMM_T, QDIT_OPT_GEMM_GENERIC_EPILOGUE, QDIT_OPT_ATTN,
 QDIT_OPT_CONDITIONING_CHUNK, QDIT_OPT_ATTN_STAGGER_NS) = range(7)

_vp, _i32, _i64, _u32, _f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_float
_int = C.c_int


class qdit_qparams(C.Structure):
    _fields_ = [("scale", _f32), ("zero_point", _i32), ("qmin", _i32), ("qmax", _i32)]


class qdit_epilogue(C.Structure):
    _fields_ = [("w_scale", _vp), ("w_colsum", _vp), ("bias", _vp), ("gate", _vp), ("ld_gate", _i64),
                ("tokens_per_sample", _i64), ("residual", _vp), ("cache_out", _vp), ("out_qp", qdit_qparams),
                ("out_scale_dev", _vp), ("a_scale_rows", _vp)]


class qdit_model_shape(C.Structure):
    _fields_ = [(n, _i32) for n in ("hidden", "heads", "mlp", "depth", "grid", "patch", "channels", "num_classes",
                                    "freq_dim", "weight_bits")]


class qdit_block_weights(C.Structure):
    _fields_ = [(n, _vp) for n in ("w_ada", "b_ada", "w_qkv", "b_qkv", "w_proj", "b_proj", "w_fc1", "b_fc1",
                                   "w_fc2", "b_fc2")]


class qdit_model_desc(C.Structure):
    _fields_ = [("shape", qdit_model_shape)] + [(n, _vp) for n in (
        "w_patch", "b_patch", "pos", "w_t1", "b_t1", "w_t2", "b_t2", "y_table", "w_ada_f", "b_ada_f", "w_out",
        "b_out")] + [("blocks", C.POINTER(qdit_block_weights))]


class qdit_sampler_desc(C.Structure):
    _fields_ = [("batch", _i32), ("num_steps", _i32), ("cache_interval", _i32), ("use_cfg", _i32),
                ("guidance", _f32), ("vc_mode", _i32), ("vc_table", _vp), ("vc_eps", _f32)]


_SIGNATURES = {
    "qdit_create": (_i32, [C.POINTER(_vp), _int, _vp]),
    "qdit_destroy": (_i32, [_vp]),
    "qdit_sync": (_i32, [_vp]),
    "qdit_status_string": (C.c_char_p, [_i32]),
    "qdit_last_error": (C.c_char_p, [_vp]),
    "qdit_launch_count": (_i64, [_vp]),
    "qdit_set_option": (_i32, [_vp, _int, _int]),
    "qdit_get_option": (_i32, [_vp, _int, _vp]),
    "qdit_profile_enable": (_i32, [_vp, _int]),
    "qdit_profile_read": (_i32, [_vp, _int, C.POINTER(_i64), C.POINTER(C.c_double), C.POINTER(C.c_double)]),
    "qdit_quantize_act": (_i32, [_vp, _vp, _int, _i64, _i64, _i64, _int, C.POINTER(qdit_qparams), _vp, _vp, _i64]),
    "qdit_quantize_act_dynamic_static": (_i32, [_vp, _vp, _int, _i64, _i64, _i64, _vp, _vp, _i64]),
    "qdit_w8a8_linear": (_i32, [_vp, _vp, _vp, _i64, _i64, _i64, qdit_qparams, _vp, _u32, C.POINTER(qdit_epilogue),
                                _vp, _i64]),
    "qdit_quantize_weight": (_i32, [_vp, _vp, _i64, _i64, _vp, _vp, _vp]),
    "qdit_quantize_weight_bits": (_i32, [_vp, _vp, _i64, _i64, _int, _vp, _vp, _vp]),
    "qdit_attention": (_i32, [_vp, _vp, _vp, _vp, _i64, _int, _int, _int, _int, _f32, _vp, _int,
                              C.POINTER(qdit_qparams), _vp]),
    "qdit_adaln_modulate": (_i32, [_vp, _vp, _i64, _i64, _i64, _f32, _vp, _vp, _i64, _vp, _int,
                                   C.POINTER(qdit_qparams), _vp]),
    "qdit_cache_create": (_i32, [_vp, _int, _i64, _i64, C.POINTER(_vp)]),
    "qdit_cache_destroy": (_i32, [_vp]),
    "qdit_cache_should_refresh": (_i32, [_int, _int]),
    "qdit_cache_invalidate": (_i32, [_vp]),
    "qdit_cache_store": (_i32, [_vp, _vp, _int, _int, _vp]),
    "qdit_cache_slot": (_vp, [_vp, _int, _int, _int]),
    "qdit_cache_reuse": (_i32, [_vp, _vp, _int, _int, _vp, _i64, _i64, _vp]),
    "qdit_cache_reuse_all": (_i32, [_vp, _vp, _vp, _i64, _i64, _vp]),
    "qdit_selftest_wait_timeout": (_i32, [_vp, C.c_uint32, _vp]),
    "qdit_patch_embed": (_i32, [_vp, _vp, _vp, _int, _vp]),
    "qdit_final_layer": (_i32, [_vp, _vp, _vp, _vp, _int, _vp]),
    "qdit_probe_mma_rate": (_i32, [_vp, _int, _int, _int, _vp, _i64, C.POINTER(C.c_float)]),
    "qdit_vc_correct": (_i32, [_vp, _vp, _int, _int, _int, _int, _int, _vp, _f32]),
    "qdit_tap_laplacian": (_i32, [_vp, _vp, _vp, _int, _int, _f32, _f32, _vp, _vp]),
    "qdit_tap_cluster_workspace": (_i64, [_int, _int, _int, _int]),
    "qdit_tap_cluster": (_i32, [_vp, _vp, _vp, _int, _int, _int, _f32, _f32, _int, _int, _int, _vp, _vp, _vp, _vp]),
    "qdit_tap_aggregate_workspace": (_i64, [_int, _int, _int, _int, _i64]),
    "qdit_tap_aggregate": (_i32, [_vp, _vp, _vp, _vp, _int, _int, _int, _int, _f32, _vp, _vp, _i64, _vp, _vp, _vp, _vp]),
    "qdit_vc_fit": (_i32, [_vp, _vp, _vp, _int, _int, _int, _f32, _int, _vp, _vp]),
    "qdit_model_create": (_i32, [_vp, C.POINTER(qdit_model_desc), C.POINTER(_vp)]),
    "qdit_model_destroy": (_i32, [_vp]),
    "qdit_model_set_act_scales": (_i32, [_vp, _vp, _vp, _vp]),
    "qdit_model_get_act_scales": (_i32, [_vp, _vp, _vp, _vp]),
    "qdit_model_weights_packed": (_i32, [_vp]),
    "qdit_w4a8_linear": (_i32, [_vp, _vp, _vp, _i64, _i64, _i64, qdit_qparams, _vp, _u32, C.POINTER(qdit_epilogue), _vp, _i64, _vp]),
    "qdit_pack_weight_int4": (_i32, [_vp, _vp, _i64, _i64, _vp]),
    "qdit_unpack_weight_int4": (_i32, [_vp, _vp, _i64, _i64, _vp]),
    "qdit_model_linear": (_i32, [_vp, _int, _int, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp),
                                 C.POINTER(_i64), C.POINTER(_i64)]),
    "qdit_sampler_create": (_i32, [_vp, _vp, C.POINTER(qdit_sampler_desc), C.POINTER(_vp)]),
    "qdit_sampler_destroy": (_i32, [_vp]),
    "qdit_sampler_reset": (_i32, [_vp, _vp, _vp, _vp]),
    "qdit_sampler_latent": (_vp, [_vp]),
    "qdit_sampler_set_schedule": (_i32, [_vp, _vp, _vp]),
    "qdit_sampler_set_ddpm": (_i32, [_vp, _vp, _vp]),
    "qdit_sample_step": (_i32, [_vp, _vp, _int]),
    "qdit_sample": (_i32, [_vp, _vp, _vp, _vp, _vp]),
    "qdit_forward": (_i32, [_vp, _vp, _vp, _vp, _vp, _int, _vp, _u32]),
    "qdit_model_begin_calibration": (_i32, [_vp, _vp]),
    "qdit_model_finish_calibration": (_i32, [_vp, _vp]),
    "qdit_sampler_buffer": (_vp, [_vp, C.c_char_p]),
    "qdit_sampler_cache": (_vp, [_vp]),
}

EXPORTS = tuple(_SIGNATURES)

for _name, (_res, _args) in _SIGNATURES.items():
    _fn = getattr(lib, _name)          # AttributeError here = the library lacks a declared symbol
    _fn.restype = _res
    _fn.argtypes = _args


class QditError(RuntimeError):
    def __init__(self, status, detail=""):
        self.status = status
        name = lib.qdit_status_string(status).decode()
        super().__init__(f"qdit status {status} ({name}){': ' + detail if detail else ''}")


def ptr(t):
    """Device/host address of a torch tensor or numpy array; ints and None pass through."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        return t.ctypes.data
    raise TypeError(type(t))


def check(ctx, status):
    if status != QDIT_OK:
        detail = lib.qdit_last_error(ctx).decode() if ctx else ""
        raise QditError(status, detail)
    return status


def qparams(scale, zero_point=0, qmin=-127, qmax=127):
    return qdit_qparams(float(scale), int(zero_point), int(qmin), int(qmax))


# ----------------------------------------------------------------------------- thin wrappers, same names
def qdit_create(device=0, stream=None):
    out = _vp()
    st = lib.qdit_create(C.byref(out), int(device), ptr(stream))
    if st != QDIT_OK:
        raise QditError(st, "qdit_create (needs an sm_100 device)")
    return out.value


def qdit_destroy(ctx):
    return lib.qdit_destroy(ctx)


def qdit_sync(ctx):
    return check(ctx, lib.qdit_sync(ctx))


def qdit_launch_count(ctx):
    return lib.qdit_launch_count(ctx)


def qdit_set_option(ctx, option, value):
    return check(ctx, lib.qdit_set_option(ctx, option, value))


def qdit_get_option(ctx, option):
    v = C.c_int(0)
    check(ctx, lib.qdit_get_option(ctx, option, C.byref(v)))
    return v.value


QDIT_PROF_GEMM, QDIT_PROF_ATTENTION, QDIT_PROF_LN_MODULATE, QDIT_PROF_ACT_QUANT = 0, 1, 2, 3
QDIT_PROF_CACHE_REUSE, QDIT_PROF_OTHER, QDIT_PROF_KINDS = 4, 5, 6


def qdit_profile_enable(ctx, enable):
    return check(ctx, lib.qdit_profile_enable(ctx, int(enable)))


def qdit_profile_read(ctx, kind):
    """-> (launches, ms, work)"""
    n, ms, w = _i64(), C.c_double(), C.c_double()
    check(ctx, lib.qdit_profile_read(ctx, kind, C.byref(n), C.byref(ms), C.byref(w)))
    return n.value, ms.value, w.value


def qdit_quantize_act(ctx, x, x_dtype, M, K, ldx, mode, qp, dyn_scale, q, ldq):
    return check(ctx, lib.qdit_quantize_act(ctx, ptr(x), x_dtype, M, K, ldx, mode,
                                            C.byref(qp) if qp is not None else None, ptr(dyn_scale), ptr(q), ldq))


def qdit_quantize_act_dynamic_static(ctx, x, x_dtype, M, K, ldx, dyn_scale, q, ldq):
    return check(ctx, lib.qdit_quantize_act_dynamic_static(ctx, ptr(x), x_dtype, M, K, ldx, ptr(dyn_scale), ptr(q), ldq))


def epilogue(w_scale=None, w_colsum=None, bias=None, gate=None, ld_gate=0, tokens_per_sample=0, residual=None,
             cache_out=None, out_qp=None, out_scale_dev=None, a_scale_rows=None):
    return qdit_epilogue(ptr(w_scale), ptr(w_colsum), ptr(bias), ptr(gate), ld_gate, tokens_per_sample,
                         ptr(residual), ptr(cache_out), out_qp if out_qp is not None else qparams(1.0),
                         ptr(out_scale_dev), ptr(a_scale_rows))


def qdit_w8a8_linear(ctx, A, W, M, N, K, a_qp, a_scale_dev, flags, epi, out, ldo):
    return check(ctx, lib.qdit_w8a8_linear(ctx, ptr(A), ptr(W), M, N, K, a_qp, ptr(a_scale_dev), flags,
                                           C.byref(epi) if epi is not None else None, ptr(out), ldo))


def qdit_w4a8_linear(ctx, A, W_packed, M, N, K, a_qp, a_scale_dev, flags, epi, out, ldo, w8_scratch=None):
    return check(ctx, lib.qdit_w4a8_linear(ctx, ptr(A), ptr(W_packed), M, N, K, a_qp, ptr(a_scale_dev), flags,
                                           C.byref(epi) if epi is not None else None, ptr(out), ldo, ptr(w8_scratch)))


def qdit_pack_weight_int4(ctx, w8, N, K, packed):
    return check(ctx, lib.qdit_pack_weight_int4(ctx, ptr(w8), N, K, ptr(packed)))


def qdit_unpack_weight_int4(ctx, packed, N, K, w8):
    return check(ctx, lib.qdit_unpack_weight_int4(ctx, ptr(packed), N, K, ptr(w8)))


def qdit_model_weights_packed(model):
    return lib.qdit_model_weights_packed(model)


def qdit_quantize_weight(ctx, w, N, K, q, w_scale, w_colsum):
    return check(ctx, lib.qdit_quantize_weight(ctx, ptr(w), N, K, ptr(q), ptr(w_scale), ptr(w_colsum)))


def qdit_quantize_weight_bits(ctx, w, N, K, bits, q, w_scale, w_colsum):
    return check(ctx, lib.qdit_quantize_weight_bits(ctx, ptr(w), N, K, bits, ptr(q), ptr(w_scale), ptr(w_colsum)))


def qdit_attention(ctx, q, k, v, ld, B, H, T, dh, softmax_scale, out, out_dtype, out_qp=None, out_scale_dev=None):
    return check(ctx, lib.qdit_attention(ctx, ptr(q), ptr(k), ptr(v), ld, B, H, T, dh, softmax_scale, ptr(out),
                                         out_dtype, C.byref(out_qp) if out_qp is not None else None,
                                         ptr(out_scale_dev)))


def qdit_adaln_modulate(ctx, x, M, D, T, eps, shift, scale, ld_mod, out, out_dtype, out_qp=None, out_scale_dev=None):
    return check(ctx, lib.qdit_adaln_modulate(ctx, ptr(x), M, D, T, eps, ptr(shift), ptr(scale), ld_mod, ptr(out),
                                              out_dtype, C.byref(out_qp) if out_qp is not None else None,
                                              ptr(out_scale_dev)))


def qdit_cache_create(ctx, blocks, M, D):
    out = _vp()
    check(ctx, lib.qdit_cache_create(ctx, blocks, M, D, C.byref(out)))
    return out.value


def qdit_cache_destroy(cache):
    return lib.qdit_cache_destroy(cache)


def qdit_cache_should_refresh(step_index, interval):
    return lib.qdit_cache_should_refresh(step_index, interval)


def qdit_cache_invalidate(cache):
    return lib.qdit_cache_invalidate(cache)


def qdit_cache_store(ctx, cache, block, branch, y):
    return check(ctx, lib.qdit_cache_store(ctx, cache, block, branch, ptr(y)))


def qdit_cache_slot(cache, block, branch, mark_filled=0):
    return lib.qdit_cache_slot(cache, block, branch, mark_filled)


def qdit_cache_reuse(ctx, cache, block, branch, gate, ld_gate, T, x):
    return check(ctx, lib.qdit_cache_reuse(ctx, cache, block, branch, ptr(gate), ld_gate, T, ptr(x)))


def qdit_cache_reuse_all(ctx, cache, mod_all, ld_mod, T, x):
    return check(ctx, lib.qdit_cache_reuse_all(ctx, cache, ptr(mod_all), ld_mod, T, ptr(x)))


def qdit_selftest_wait_timeout(ctx, polls, observed):
    return check(ctx, lib.qdit_selftest_wait_timeout(ctx, polls, ptr(observed)))


def qdit_patch_embed(ctx, model, latent, B, x):
    return check(ctx, lib.qdit_patch_embed(ctx, model, ptr(latent), B, ptr(x)))


def qdit_final_layer(ctx, model, x, mod, B, out):
    return check(ctx, lib.qdit_final_layer(ctx, model, ptr(x), ptr(mod), B, ptr(out)))


def qdit_probe_mma_rate(ctx, mode, n, iters, operands, rows):
    """Kernel duration in milliseconds."""
    ms = C.c_float(0.0)
    check(ctx, lib.qdit_probe_mma_rate(ctx, mode, n, iters, ptr(operands), rows, C.byref(ms)))
    return ms.value


def qdit_vc_correct(ctx, latent, B, Cc, HW, step_index, mode, table, eps):
    return check(ctx, lib.qdit_vc_correct(ctx, ptr(latent), B, Cc, HW, step_index, mode, ptr(table), eps))


def qdit_tap_cluster_workspace(m, n, d, k):
    return lib.qdit_tap_cluster_workspace(m, n, d, k)


def qdit_tap_cluster(ctx, x, t, m, n, d, alpha, exponent, k, power_iters, kmeans_iters, workspace, eigvals, eigvecs, labels):
    return check(ctx, lib.qdit_tap_cluster(ctx, ptr(x), ptr(t), m, n, d, alpha, exponent, k, power_iters, kmeans_iters,
                                           ptr(workspace), ptr(eigvals), ptr(eigvecs), ptr(labels)))


def qdit_tap_aggregate_workspace(m, n, d, k, N):
    return lib.qdit_tap_aggregate_workspace(m, n, d, k, N)


def qdit_tap_aggregate(ctx, x, t, labels, m, n, d, k, alpha, x_all, t_all, N, workspace, labels_all, centroids, tau):
    return check(ctx, lib.qdit_tap_aggregate(ctx, ptr(x), ptr(t), ptr(labels), m, n, d, k, alpha, ptr(x_all), ptr(t_all), N,
                                             ptr(workspace), ptr(labels_all), ptr(centroids), ptr(tau)))


def qdit_tap_laplacian(ctx, x, t, n, d, alpha, exponent, workspace, L):
    return check(ctx, lib.qdit_tap_laplacian(ctx, ptr(x), ptr(t), n, d, alpha, exponent, ptr(workspace), ptr(L)))


def qdit_vc_fit(ctx, x_hat, x_target, N, Cc, HW, eps, form, workspace, K):
    return check(ctx, lib.qdit_vc_fit(ctx, ptr(x_hat), ptr(x_target), N, Cc, HW, eps, form, ptr(workspace), ptr(K)))


def qdit_model_create(ctx, cfg, weights, weight_bits=8):
    """cfg: object with hidden, heads, mlp, depth, grid, patch, channels, num_classes, freq_dim;
    weights: dict of contiguous float32 numpy arrays laid out as qdit_model_desc documents;
    weight_bits: code width of the quantized linears' weights (8 = W8A8, 4 = W4A8)."""
    import numpy as np

    keep = []

    def hp(a):
        a = np.ascontiguousarray(a, dtype=np.float32)
        keep.append(a)
        return a.ctypes.data

    blocks = (qdit_block_weights * cfg.depth)()
    for i, bw in enumerate(weights["blocks"]):
        for n, _ in qdit_block_weights._fields_:
            setattr(blocks[i], n, hp(bw[n]))
    desc = qdit_model_desc()
    desc.shape = qdit_model_shape(cfg.hidden, cfg.heads, cfg.mlp, cfg.depth, cfg.grid, cfg.patch, cfg.channels,
                                  cfg.num_classes, cfg.freq_dim, weight_bits)
    for n in ("w_patch", "b_patch", "pos", "w_t1", "b_t1", "w_t2", "b_t2", "y_table", "w_ada_f", "b_ada_f", "w_out",
              "b_out"):
        setattr(desc, n, hp(weights[n]))
    desc.blocks = blocks
    out = _vp()
    check(ctx, lib.qdit_model_create(ctx, C.byref(desc), C.byref(out)))
    return out.value


def qdit_model_destroy(model):
    return lib.qdit_model_destroy(model)


def qdit_model_set_act_scales(ctx, model, ada_scale, block_scales):
    import numpy as np
    a = np.asarray([ada_scale], dtype=np.float32)
    b = np.ascontiguousarray(block_scales, dtype=np.float32)
    return check(ctx, lib.qdit_model_set_act_scales(ctx, model, a.ctypes.data, b.ctypes.data))


def qdit_model_get_act_scales(ctx, model, depth):
    import numpy as np
    a = np.zeros(1, dtype=np.float32)
    b = np.zeros(depth * 4, dtype=np.float32)
    check(ctx, lib.qdit_model_get_act_scales(ctx, model, a.ctypes.data, b.ctypes.data))
    return float(a[0]), b.reshape(depth, 4)


def qdit_model_linear(model, block, which):
    """-> dict(w_q, w_scale, w_colsum, bias: device addresses; N, K)."""
    wq, ws, wc, bi = _vp(), _vp(), _vp(), _vp()
    N, K = _i64(), _i64()
    st = lib.qdit_model_linear(model, block, which, C.byref(wq), C.byref(ws), C.byref(wc), C.byref(bi), C.byref(N),
                               C.byref(K))
    if st != QDIT_OK:
        raise QditError(st)
    return dict(w_q=wq.value, w_scale=ws.value, w_colsum=wc.value, bias=bi.value, N=N.value, K=K.value)


def qdit_sampler_create(ctx, model, batch, num_steps, cache_interval=1, use_cfg=False, guidance=1.0,
                        vc_mode=QDIT_VC_NONE, vc_table=None, vc_eps=1e-6):
    import numpy as np
    tab = None if vc_table is None else np.ascontiguousarray(vc_table, dtype=np.float32)
    desc = qdit_sampler_desc(batch, num_steps, cache_interval, int(bool(use_cfg)), guidance, vc_mode,
                             None if tab is None else tab.ctypes.data, vc_eps)
    out = _vp()
    check(ctx, lib.qdit_sampler_create(ctx, model, C.byref(desc), C.byref(out)))
    return out.value


def qdit_sampler_destroy(s):
    return lib.qdit_sampler_destroy(s)


def qdit_sampler_reset(ctx, s, latent, labels):
    return check(ctx, lib.qdit_sampler_reset(ctx, s, ptr(latent), ptr(labels)))


def qdit_sampler_latent(s):
    return lib.qdit_sampler_latent(s)


def qdit_sampler_set_ddpm(ctx, s, noise):
    """noise: device tensor [num_steps, batch, C, Hl, Wl] f32 (kept alive by the caller), or None for DDIM."""
    return check(ctx, lib.qdit_sampler_set_ddpm(ctx, s, ptr(noise)))


def qdit_sampler_set_schedule(ctx, s, schedule):
    """schedule: array-like [num_steps, blocks, 2] of reuse flags, or None for the global rule."""
    import numpy as np
    if schedule is None:
        return check(ctx, lib.qdit_sampler_set_schedule(ctx, s, None))
    a = np.ascontiguousarray(np.asarray(schedule) != 0, dtype=np.uint8)
    return check(ctx, lib.qdit_sampler_set_schedule(ctx, s, a.ctypes.data))


def qdit_sample_step(ctx, s, step_index):
    return check(ctx, lib.qdit_sample_step(ctx, s, step_index))


def qdit_sample(ctx, s, latent_host, labels_host, out_host):
    return check(ctx, lib.qdit_sample(ctx, s, ptr(latent_host), ptr(labels_host), ptr(out_host)))


def qdit_forward(ctx, s, latent, t, y, B, out, flags=0):
    return check(ctx, lib.qdit_forward(ctx, s, ptr(latent), ptr(t), ptr(y), B, ptr(out), flags))


def qdit_model_begin_calibration(ctx, model):
    return check(ctx, lib.qdit_model_begin_calibration(ctx, model))


def qdit_model_finish_calibration(ctx, model):
    return check(ctx, lib.qdit_model_finish_calibration(ctx, model))


def qdit_sampler_buffer(s, name):
    return lib.qdit_sampler_buffer(s, name.encode())


def qdit_sampler_cache(s):
    return lib.qdit_sampler_cache(s)


__all__ = [n for n in dir() if n.startswith(("qdit_", "QDIT_"))] + [
    "lib", "LIB_PATH", "EXPORTS", "QditError", "ptr", "check", "qparams", "epilogue"]
