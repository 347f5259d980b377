/*
 * qdit.h - C ABI of libqdit: the quantized-and-cached DiT denoising step of
 * Q&C ("When Quantization Meets Cache in Efficient Image Generation") as
 * hand-written CUDA kernels for NVIDIA B200 (sm_100a).
 *
 * Conventions
 *   - Every call returns an int32 status: QDIT_OK (0) or a negative QDIT_ERR_*.
 *     qdit_status_string() names a code; qdit_last_error() gives the detail of
 *     the last failing call on a context.  No call throws, traps or aborts.
 *   - Unless a parameter says "host", every tensor pointer is DEVICE memory owned
 *     by the caller, 16-byte aligned, row-major with the stated leading
 *     dimension in ELEMENTS.  The library allocates only inside *_create calls
 *     and frees in the matching *_destroy.
 *   - Work is enqueued on the context's CUDA stream and is asynchronous.
 *     Argument errors are reported before anything is launched.  Every wait
 *     inside a kernel is bounded; a wait that runs out sets a device status word
 *     that the next qdit_sync() returns as QDIT_ERR_TIMEOUT.
 *   - Rows of a token matrix are ordered sample-major: row m belongs to sample
 *     m / tokens_per_sample.
 *   - There is no CPU fallback: on a machine without an sm_100 device
 *     qdit_create fails with QDIT_ERR_CUDA.
 */
#ifndef QDIT_H_
#define QDIT_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  QDIT_OK = 0,
  QDIT_ERR_INVALID_ARG = -1, /* null pointer, bad enum, bad flag combination */
  QDIT_ERR_SHAPE = -2,       /* size not supported (e.g. K not a multiple of 16) */
  QDIT_ERR_ALIGN = -3,       /* pointer or leading dimension not 16-byte aligned */
  QDIT_ERR_UNSUPPORTED = -4,
  QDIT_ERR_CUDA = -5,        /* a CUDA runtime/driver call failed; see qdit_last_error */
  QDIT_ERR_STATE = -6,       /* e.g. cache reuse before any store, step out of order */
  QDIT_ERR_TIMEOUT = -7,     /* a bounded device-side wait ran out */
  QDIT_ERR_NOMEM = -8
};

enum { QDIT_BF16 = 0, QDIT_F32 = 1, QDIT_I8 = 2, QDIT_I32 = 3 };

typedef struct qdit_ctx qdit_ctx;

/* Context = device + borrowed stream + tensor-map cache + device status word.
 * cuda_stream is a cudaStream_t (NULL = the legacy default stream). */
int32_t qdit_create(qdit_ctx** out, int device, void* cuda_stream);
int32_t qdit_destroy(qdit_ctx* ctx);
/* Waits for the stream; returns QDIT_ERR_TIMEOUT / QDIT_ERR_CUDA if work since the last sync failed. */
int32_t qdit_sync(qdit_ctx* ctx);
/* Self-test of the device-side time-out path (the paper has no counterpart): launches one small kernel in which
 * a bounded wait of `polls` polls (1..2^20) on a barrier that nobody signals runs out, and a second waiting
 * thread leaves through the CTA's abort flag, exactly as the roles of the pipelined kernels do.  The kernel ends
 * normally; the next qdit_sync returns QDIT_ERR_TIMEOUT once and the context stays usable.
 * observed_dev: device int[2], set to {1, 1} when both threads left their wait the intended way. */
int32_t qdit_selftest_wait_timeout(qdit_ctx* ctx, uint32_t polls, int* observed_dev);
/* Tensor-pipe probe (the paper has no counterpart; bench.py --workload mma_probe reports it): every SM runs
 * `iters` groups of four tcgen05.mma kind::i8 instructions (M 128, N = n in {64, 128, 192, 256}, K 32 each), the
 * products are discarded.  mode 0: the operands stay in shared memory (the instruction path's own rate); mode 1: a TMA
 * producer refills a four-stage ring of 128 + n rows of 128 bytes per group from `operands` and the issuer frees each
 * stage with a commit, as the GEMM kernels' main loop does, with no epilogue.  operands: int8 [rows][1024], rows a
 * multiple of 256, values arbitrary.  Synchronous: returns the kernel's duration in milliseconds in *ms_host (host
 * pointer); int-ops performed = SMs x iters x 4 x 2 x 128 x n x 32.  iters in 1..65536. */
int32_t qdit_probe_mma_rate(qdit_ctx* ctx, int mode, int n, int iters, const void* operands, int64_t rows, float* ms_host);
const char* qdit_status_string(int32_t status);
const char* qdit_last_error(const qdit_ctx* ctx);
/* Number of kernels this context has launched since creation (for launch accounting). */
int64_t qdit_launch_count(const qdit_ctx* ctx);

/* Kernel-selection options of a context (tuning and test aid; the paper has no counterpart).  Every option chooses
 * among kernels that compute the same values.  A new context takes its initial values from the environment
 * variables of the same names (QDIT_PDL, QDIT_GEMM_BN, QDIT_GEMM_T, QDIT_GEMM_GENERIC_EPILOGUE, QDIT_ATTN,
 * QDIT_CONDITIONING_CHUNK, QDIT_ATTN_STAGGER_NS), read once inside qdit_create; afterwards only qdit_set_option changes
 * them.
 *   QDIT_OPT_PDL                    1 (default): kernels are launched with programmatic stream serialization, so that
 *                                   a kernel's preamble overlaps the tail of the kernel before it; 0: plain launches
 *   QDIT_OPT_GEMM_BN                0 (default): automatic; 64 | 128 | 192: token-major GEMM kernel with 128 x BN tiles
 *   QDIT_OPT_GEMM_T                 0 (default): automatic; 128 | 256: channel-major GEMM kernel with 128 x BT tiles
 *   QDIT_OPT_GEMM_GENERIC_EPILOGUE  1: the GEMM kernels' run-time-flag epilogue instead of the specialised classes
 *   QDIT_OPT_ATTN                   0 (default): automatic; 1: the mma.sync attention kernel for every token count;
 *                                   2: the online-softmax tcgen05 kernel also at 256 tokens
 *   QDIT_OPT_CONDITIONING_CHUNK     sampling steps whose conditioning a sampler evaluates at once: 0 (default) as many
 *                                   as fit a 4 GB modulation table, -1 step by step, n > 0 at most n (read by
 *                                   qdit_sampler_create)
 *   QDIT_OPT_ATTN_STAGGER_NS        256-token attention: the CTAs that become the second resident of an SM in the first
 *                                   wave start this many nanoseconds late (default 2000; 0 = together), so that the two
 *                                   CTAs of an SM do not run their phases in lockstep; 0..20000 */
enum {
  QDIT_OPT_PDL = 0, QDIT_OPT_GEMM_BN = 1, QDIT_OPT_GEMM_T = 2, QDIT_OPT_GEMM_GENERIC_EPILOGUE = 3, QDIT_OPT_ATTN = 4,
  QDIT_OPT_CONDITIONING_CHUNK = 5, QDIT_OPT_ATTN_STAGGER_NS = 6, QDIT_OPT_COUNT = 7
};
int32_t qdit_set_option(qdit_ctx* ctx, int option, int value);
int32_t qdit_get_option(const qdit_ctx* ctx, int option, int* value);

/* Per-kernel timing for measurement (the paper has no counterpart): while enabled, every kernel launch of
 * this context is bracketed by CUDA events on the context's stream.  qdit_profile_read synchronises the
 * stream and returns, for one kernel kind, the launches since profiling was enabled, their summed device
 * time in ms and their summed algorithmic work (integer ops for QDIT_PROF_GEMM, flops for
 * QDIT_PROF_ATTENTION, bytes that must cross HBM for the others).  Enabling resets the counters.
 * The events cost a few microseconds per launch: leave profiling off when timing end to end. */
enum {
  QDIT_PROF_GEMM = 0, QDIT_PROF_ATTENTION = 1, QDIT_PROF_LN_MODULATE = 2, QDIT_PROF_ACT_QUANT = 3,
  QDIT_PROF_CACHE_REUSE = 4, QDIT_PROF_OTHER = 5, QDIT_PROF_KINDS = 6
};
int32_t qdit_profile_enable(qdit_ctx* ctx, int enable);
int32_t qdit_profile_read(qdit_ctx* ctx, int kind, int64_t* launches, double* ms, double* work);

/* ------------------------------------------------------------------------------------------------
 * Uniform quantizer, Eq. 1:  Q(X|b) = clip(round(X/s) + z, qmin, qmax).
 * round = nearest, ties to even; X/s is evaluated as the float32 product X * (1/s).
 * Eq. 1's range is [0, 2^b-1] (codes stored as unsigned bytes when qmin >= 0); the symmetric
 * signed range [-127,127] with z = 0 is the default of the DiT path.  Activations are quantized
 * tensor-wise, weights channel-wise (Comparison on Performance). */
typedef struct {
  float scale;        /* s > 0 */
  int32_t zero_point; /* z */
  int32_t qmin, qmax; /* clip range; either within [-128,127] or within [0,255] */
} qdit_qparams;

enum { QDIT_QUANT_STATIC = 0, QDIT_QUANT_DYNAMIC = 1, QDIT_QUANT_DYNAMIC_TOKEN = 2 };

/* q[m,k] = Q(x[m,k]).  x: [M,K] bf16 or f32 (x_dtype), ldx elements per row; q: [M,K] bytes, ldq
 * (8-byte alignment of q and ldq suffices).
 * STATIC : *qp (host) gives s, z and the range.
 * DYNAMIC: symmetric range [-127,127]; s = max|x| / 127 is reduced on the device first (s = 1 if the
 *          tensor is all zero) and left in dyn_scale (device, 1 float, required); qp is ignored.
 * DYNAMIC_TOKEN: the same per row (per token): s[m] = max_k|x[m,k]| / 127 left in dyn_scale (device,
 *          M floats); the linear layer takes these scales with QDIT_EPI_ROW_SCALE.  (The paper quantizes
 *          activations tensor-wise, Experimental Settings; the per-token form is the variant of the
 *          quantization baselines it compares with.)
 * K must be a multiple of 8; M or K of 0 is a no-op. */
int32_t qdit_quantize_act(qdit_ctx* ctx, const void* x, int x_dtype, int64_t M, int64_t K, int64_t ldx,
                          int mode, const qdit_qparams* qp, float* dyn_scale, void* q, int64_t ldq);

/* Dynamic quantizer for callers that cannot allocate device memory (the paper has no counterpart; this
 * is a deployment convenience).  Same result as qdit_quantize_act in QDIT_QUANT_DYNAMIC mode: symmetric
 * codes in q and s = max|x| / 127 (1 for an all-zero tensor) in dyn_scale.  The difference is where the
 * reduction's intermediate values live: in a fixed 256 KB array inside the library's device image instead
 * of memory somebody had to cudaMalloc, so the call (and everything it calls) allocates nothing.  Use it
 * from code that is handed only its tensors and must not touch the allocator: a plug-in inside another
 * framework's memory plan, a process with a fixed memory budget, a region being recorded for replay.
 *  - Limit: M*K <= 134,217,728 elements per call (65536 partial maxima of 2048 elements each); larger
 *    inputs are refused with QDIT_ERR_SHAPE before anything is launched.
 *  - The first call on a device looks up the array's device address (cudaGetSymbolAddress) with that
 *    device made current for the lookup (the caller's current device is put back); make that first call
 *    outside any stream capture.  The lookup is serialised, so first calls from several threads are safe.
 *  - The array is shared by every call on the device and keeps the last call's values.  Each call
 *    overwrites all slots it later reads, so nothing needs clearing; two calls that overlap on the GPU
 *    (different streams, no ordering) race on it and must be serialised by the caller.
 * x, q, ldx, ldq, K % 8 == 0 and alignment as for qdit_quantize_act; dyn_scale: device, 1 float, required. */
int32_t qdit_quantize_act_dynamic_static(qdit_ctx* ctx, const void* x, int x_dtype, int64_t M, int64_t K,
                                         int64_t ldx, float* dyn_scale, void* q, int64_t ldq);

/* ------------------------------------------------------------------------------------------------
 * W8A8 linear layer (8-bit weights and activations, Table 1) on quantized activations:
 *   acc[m,n] = sum_k A[m,k] * W[n,k]                       exact int32 (tcgen05 kind::i8, TMEM)
 *   f        = (acc - z_a * w_colsum[n]) * (s_a * w_scale[n])
 *   f       += bias[n]                 QDIT_EPI_BIAS
 *   f        = GELU_tanh(f)            QDIT_EPI_GELU
 *   cache_out[m,n] = bf16(f)           QDIT_EPI_CACHE_STORE  (the block-output cache of the cache
 *                                      mechanism: the branch output BEFORE the adaLN gate)
 *   f       *= gate[m / tokens, n]     QDIT_EPI_GATE
 *   f       += residual[m,n]           QDIT_EPI_RESIDUAL
 *   out[m,n] = f as bf16 / f32, or Q(f | out_qp) as bytes with QDIT_EPI_QUANT_OUT (Eq. 1 again,
 *              fusing the next layer's activation quantizer), or acc itself with QDIT_EPI_OUT_I32.
 * Exactly one of OUT_BF16, OUT_F32, OUT_I32, QUANT_OUT must be set.
 * A: [M,K] bytes (signed, or unsigned when a_qp.qmin >= 0 and a_qp.qmax > 127), W: [N,K] signed bytes,
 * both K-contiguous with leading dimension K.  K % 16 == 0 and N % 8 == 0 are required; M, N, K are
 * otherwise free (ragged tiles are handled; with QDIT_EPI_GATE the gate needs one row per started sample,
 * ceil(M / tokens_per_sample) rows, and no row beyond them is read).  a_scale_dev, if non-NULL, is a device float that
 * overrides a_qp.scale at run time (used when the scale was just reduced on the device). */
enum {
  QDIT_EPI_BIAS = 1u << 0,
  QDIT_EPI_GELU = 1u << 1,
  QDIT_EPI_GATE = 1u << 2,
  QDIT_EPI_RESIDUAL = 1u << 3,
  QDIT_EPI_CACHE_STORE = 1u << 4,
  QDIT_EPI_QUANT_OUT = 1u << 5,
  QDIT_EPI_OUT_BF16 = 1u << 6,
  QDIT_EPI_OUT_F32 = 1u << 7,
  QDIT_EPI_OUT_I32 = 1u << 8,
  QDIT_EPI_ROW_SCALE = 1u << 9 /* activation scale per row: epi->a_scale_rows[m] replaces a_qp.scale (a_qp.zero_point must be 0) */
};

typedef struct {
  const float* w_scale;       /* [N] channel-wise weight scales */
  const int32_t* w_colsum;    /* [N] sum_k W[n,k]; may be NULL when a_qp.zero_point == 0 */
  const float* bias;          /* [N] f32 */
  const float* gate;          /* f32, row b at gate + b*ld_gate, [n] within the row */
  int64_t ld_gate;
  int64_t tokens_per_sample;  /* T in b = m / T */
  const void* residual;       /* [M,N] bf16, leading dimension ldo; may alias out */
  void* cache_out;            /* [M,N] bf16, leading dimension N */
  qdit_qparams out_qp;        /* for QDIT_EPI_QUANT_OUT */
  const float* out_scale_dev; /* optional device override of out_qp.scale */
  const float* a_scale_rows;  /* [M] f32 device, per-token activation scales for QDIT_EPI_ROW_SCALE
                                 (as written by qdit_quantize_act in QDIT_QUANT_DYNAMIC_TOKEN mode) */
} qdit_epilogue;

int32_t qdit_w8a8_linear(qdit_ctx* ctx, const void* A, const void* W, int64_t M, int64_t N, int64_t K,
                         qdit_qparams a_qp, const float* a_scale_dev, uint32_t flags,
                         const qdit_epilogue* epi, void* out, int64_t ldo);

/* W4A8 linear layer (Table 2, the 512 x 512 setting): the same operation on 4-bit channel-wise weight codes stored
 * two per byte.  W_packed: [N, K/2] bytes, row n holds codes W[n, 2j] in the low nibble and W[n, 2j+1] in the high
 * nibble of byte j, each a 4-bit two's-complement number in [-8, 7] (the byte layout is this library's; the paper
 * fixes only the code width).  K % 32 == 0; QDIT_EPI_ROW_SCALE is not available; everything else as
 * qdit_w8a8_linear, with identical results for identical codes.  The weights cross HBM at half the bytes: with
 * few rows (M < 1024, or no scratch given) they are widened to int8 inside the GEMM kernel in front of the tensor
 * core; with many rows and w8_scratch != NULL (device, N*K bytes, 16-byte aligned, overwritten) they are widened
 * into the scratch first and the W8A8 kernels run on it.
 * qdit_pack_weight_int4 / qdit_unpack_weight_int4 convert between [N, K] int8 codes and the packed form
 * (K % 16 == 0; packing refuses codes outside [-8, 7] with QDIT_ERR_INVALID_ARG and synchronises the stream). */
int32_t qdit_w4a8_linear(qdit_ctx* ctx, const void* A, const void* W_packed, int64_t M, int64_t N, int64_t K,
                         qdit_qparams a_qp, const float* a_scale_dev, uint32_t flags,
                         const qdit_epilogue* epi, void* out, int64_t ldo, void* w8_scratch);
int32_t qdit_pack_weight_int4(qdit_ctx* ctx, const void* w8, int64_t N, int64_t K, void* packed);
int32_t qdit_unpack_weight_int4(qdit_ctx* ctx, const void* packed, int64_t N, int64_t K, void* w8);

/* Channel-wise symmetric weight quantizer (the weight side of Eq. 1): for each output row n of
 * w[N,K] (f32, device), s[n] = max_k|w| / 127 (1 if the row is zero), q = clip(round(w * (1/s)),-127,127),
 * colsum[n] = sum_k q[n,k].  q: [N,K] bytes, w_scale: [N] f32, w_colsum: [N] int32.  K % 4 == 0.
 * qdit_quantize_weight_bits is the same with b-bit codes (2 <= bits <= 8): top = 2^(bits-1) - 1 replaces 127.
 * With bits = 4 this is the weight side of the paper's W4A8 setting (Table 2); this call leaves the codes one per
 * byte (qdit_pack_weight_int4 packs them two per byte for qdit_w4a8_linear). */
int32_t qdit_quantize_weight(qdit_ctx* ctx, const float* w, int64_t N, int64_t K, void* q, float* w_scale,
                             int32_t* w_colsum);
int32_t qdit_quantize_weight_bits(qdit_ctx* ctx, const float* w, int64_t N, int64_t K, int bits, void* q,
                                  float* w_scale, int32_t* w_colsum);

/* ------------------------------------------------------------------------------------------------
 * Self-attention between the quantized linears (kept in bf16, not quantized):
 *   out[b,t,h,:] = softmax_s(q[b,t,h,:] . k[b,s,h,:] * softmax_scale) v[b,s,h,:]     (non-causal)
 * q, k, v: bf16, token-major; element (b,t,h,d) at ptr[(b*T + t)*ld + h*dh + d] (so the three may
 * point into one packed [B*T, 3*H*dh] QKV matrix).  dh in {64, 72}; T a multiple of 64.
 * out: [B*T, H*dh] with leading dimension H*dh, as bf16, f32, or bytes Q(. | out_qp) when
 * out_dtype == QDIT_I8 (fused quantizer of the projection's input).  Softmax statistics in f32. */
int32_t qdit_attention(qdit_ctx* ctx, const void* q, const void* k, const void* v, int64_t ld, int B, int H,
                       int T, int dh, float softmax_scale, void* out, int out_dtype,
                       const qdit_qparams* out_qp, const float* out_scale_dev);

/* LayerNorm (no affine, biased variance, eps) followed by the adaLN modulation of the DiT block:
 *   y[m,:] = (x[m,:] - mean) / sqrt(var + eps) * (1 + scale[b,:]) + shift[b,:],   b = m / T
 * x: [M,D] bf16 (leading dimension D).  shift/scale: f32, row b at ptr + b*ld_mod.
 * out: [M,D] bf16, f32, or bytes Q(y | out_qp) when out_dtype == QDIT_I8 (fused activation quantizer
 * of the following linear).  D a multiple of 8, D <= 2048. */
int32_t qdit_adaln_modulate(qdit_ctx* ctx, const void* x, int64_t M, int64_t D, int64_t T, float eps,
                            const float* shift, const float* scale, int64_t ld_mod, void* out,
                            int out_dtype, const qdit_qparams* out_qp, const float* out_scale_dev);

/* ------------------------------------------------------------------------------------------------
 * Block-output cache (Background, "Quantization and Cache"): with cache interval N the model
 * recomputes and refreshes the cache at sampling steps i with i mod N == 0 (i = 0 is the first step,
 * which fills it) and reuses it for the following N-1 steps.  Cached per block: the outputs of the
 * self-attention branch and of the MLP branch, before the adaLN gate, as bf16 [M,D]. */
typedef struct qdit_cache qdit_cache;
enum { QDIT_BRANCH_ATTN = 0, QDIT_BRANCH_MLP = 1 };

int32_t qdit_cache_create(qdit_ctx* ctx, int blocks, int64_t M, int64_t D, qdit_cache** out);
int32_t qdit_cache_destroy(qdit_cache* cache);
/* Pure host function: 1 if step_index refreshes the cache, 0 if it reuses, <0 on bad arguments. */
int32_t qdit_cache_should_refresh(int step_index, int interval);
/* Marks every slot empty (start of a new trajectory). */
int32_t qdit_cache_invalidate(qdit_cache* cache);
/* Copies y [M,D] bf16 into slot (block, branch) and marks it filled. */
int32_t qdit_cache_store(qdit_ctx* ctx, qdit_cache* cache, int block, int branch, const void* y);
/* Device address of a slot, for a producer that writes it directly (QDIT_EPI_CACHE_STORE);
 * mark_filled != 0 records the slot as filled.  NULL on bad arguments. */
void* qdit_cache_slot(qdit_cache* cache, int block, int branch, int mark_filled);
/* x[m,:] = bf16(x[m,:] + gate[b,:] * slot[m,:]).  QDIT_ERR_STATE if the slot was never stored. */
int32_t qdit_cache_reuse(qdit_ctx* ctx, qdit_cache* cache, int block, int branch, const float* gate,
                         int64_t ld_gate, int64_t T, void* x);
/* A fully skipped step in one pass over the cache:
 *   x = bf16(x + sum_blocks gate_msa_b * A_b + gate_mlp_b * Mo_b)   (f32 accumulation, one rounding)
 * mod_all: f32 [B, blocks*6*D]; block b's gate_msa at column b*6D + 2D, gate_mlp at b*6D + 5D. */
int32_t qdit_cache_reuse_all(qdit_ctx* ctx, qdit_cache* cache, const float* mod_all, int64_t ld_mod,
                             int64_t T, void* x);

/* ------------------------------------------------------------------------------------------------
 * Variance compensation (section "Variance Align for Exposure Bias"):
 *   x~ = mu + K[step,c] * (x^ - mu),  mu = spatial mean of x^ per (sample, channel).
 * QDIT_VC_K_TABLE  : table[step*C + c] is K.
 * QDIT_VC_VAR_RATIO: table[step*C + c] is a target variance; K = sqrt(target / (var(x^) + eps))
 *                    with var the spatial variance per (sample, channel) (the rescaling identity
 *                    Y = mu + (sigma_new/sigma)(f - mu)).
 * latent: f32 [B,C,HW] updated in place; table: device f32 [steps, C]; HW % 4 == 0. */
enum { QDIT_VC_NONE = 0, QDIT_VC_K_TABLE = 1, QDIT_VC_VAR_RATIO = 2 };
int32_t qdit_vc_correct(qdit_ctx* ctx, float* latent, int B, int C, int HW, int step_index, int mode,
                        const float* table, float eps);
/* Fitting the factor of one step (same section, the closed form for K that follows the correction formula): from
 * N calibration samples x^ (accelerated trajectory) and targets x' (reference
 * trajectory), both device f32 [N, C, HW], with mu = spatial mean of x^ per (sample, channel), a = x^ - mu,
 * b = x' - mu, w = 1 / (x'^2 + eps), sums over the samples and positions of channel c:
 *   QDIT_VC_FIT_DERIVED : K[c] = (sum a b + sum a b w) / (sum a^2 + sum a^2 w)   (d/dK of rQNSR^2 + MSE = 0)
 *   QDIT_VC_FIT_PRINTED : the numerator's second term as the paper prints it, sum a / x'.
 * workspace: caller-owned device scratch of 4 * N * C doubles (overwritten); K: device f32 [C] (one row of the
 * K table).  Sums are taken in f64 and combined in a fixed order: the result is reproducible. */
enum { QDIT_VC_FIT_DERIVED = 0, QDIT_VC_FIT_PRINTED = 1 };
int32_t qdit_vc_fit(qdit_ctx* ctx, const float* x_hat, const float* x_target, int N, int C, int HW, float eps, int form,
                    double* workspace, float* K);

/* ------------------------------------------------------------------------------------------------
 * Matrix steps of Temporal-Aware Parallel Clustering for one subsample (section "Temporal-Aware Parallel
 * Clustering for Calibration", Algorithm 1): from the n samples' features x [n,d] and timestamps t [n] (device f32)
 *   A_spatial[k,h] = x_k.x_h / (|x_k||x_h|),  A_temporal[k,h] = exp(-|t_k - t_h|),
 *   A = alpha A_spatial + (1 - alpha) A_temporal,   L = D^e A D^e,  D = diag(row sums of A)
 * (A is symmetric, so the paper's row and column degree matrices coincide; the paper prints e = +1/2, the usual
 * normalised adjacency is e = -1/2: `exponent` selects).  L: device f32 [n,n].  workspace: device f32, n*d + 2n
 * floats, overwritten.  n % 4 == 0, d % 16 == 0. */
int32_t qdit_tap_laplacian(qdit_ctx* ctx, const float* x, const float* t, int n, int d, float alpha, float exponent,
                           float* workspace, float* L);
/* Spectral step of Algorithm 1 for the m subsamples as one batch: for each subsample the matrix L above, its top k
 * eigenvectors (largest eigenvalues; L is symmetric positive semi-definite when the degrees are positive) and
 * k-means on the rows of the n x k eigenvector matrix.  x [m, n, d], t [m, n] (device f32).
 *   eigvals [m, k] descending, eigvecs [m, n, k] (column j = eigenvector j, unit length; its sign and, inside a
 *   repeated eigenvalue, its rotation are arbitrary), labels [m, n] int32 in [0, k).
 * Eigenvectors by orthogonal iteration on a block of k + 8 vectors (power_iters multiplications by L, each followed by
 * re-orthonormalisation) and a Rayleigh-Ritz step; the gap between eigenvalue k and k + 9 sets how many iterations
 * are needed.  k-means: Lloyd's iterations (at most kmeans_iters, stops when no label changes) from the
 * farthest-point start: centre 0 = row 0, each further centre = the row farthest from the centres so far (ties to
 * the lowest index); nearest centre with ties to the lowest centre; an emptied cluster keeps its centre.  (The
 * paper fixes none of these details.)  n % 16 == 0, d % 16 == 0, k + 8 <= min(n, 128), n <= 8192.
 * workspace: device f32, qdit_tap_cluster_workspace(m, n, d, k) floats, overwritten. */
int64_t qdit_tap_cluster_workspace(int m, int n, int d, int k);
int32_t qdit_tap_cluster(qdit_ctx* ctx, const float* x, const float* t, int m, int n, int d, float alpha, float exponent,
                         int k, int power_iters, int kmeans_iters, float* workspace, float* eigvals, float* eigvecs,
                         int32_t* labels);
/* Last step of Algorithm 1, "aggregate cluster assignments from all subsamples" (the paper does not say how; this is
 * the reading taken): every cluster of a subsample is summarised by the mean of its members' unit-length features
 * and the mean of their timestamps; the clusters of subsamples 2..m are matched one-to-one to those of subsample 1,
 * greedily by the similarity alpha cos + (1 - alpha) exp(-|dt|) of the summaries (largest remaining entry first);
 * matched summaries are averaged with the cluster sizes as weights; every sample of the whole dataset
 * (x_all [N, d], t_all [N]) is assigned to the aggregated cluster it is most similar to (ties to the lowest).
 * labels [m, n] as written by qdit_tap_cluster.  Outputs: labels_all [N] int32, centroids [k, d], tau [k] (device).
 * The matching of the m k summaries runs on the host inside this call (it synchronises the stream twice).
 * d % 16 == 0, k % 4 == 0.  workspace: device f32, qdit_tap_aggregate_workspace(m, n, d, k, N) floats. */
int64_t qdit_tap_aggregate_workspace(int m, int n, int d, int k, int64_t N);
int32_t qdit_tap_aggregate(qdit_ctx* ctx, const float* x, const float* t, const int32_t* labels, int m, int n, int d, int k,
                           float alpha, const float* x_all, const float* t_all, int64_t N, float* workspace,
                           int32_t* labels_all, float* centroids, float* tau);

/* ------------------------------------------------------------------------------------------------
 * Whole model and sampler.  The DiT architecture (adaLN-Zero blocks, patch 2, learned-sigma output)
 * is the one the paper evaluates (Experimental Settings); quantized layers are each block's
 * modulation linear, QKV, projection, fc1 and fc2; embedders and the final layer stay in f32. */
typedef struct {
  int32_t hidden, heads, mlp, depth, grid, patch, channels, num_classes, freq_dim;
  int32_t weight_bits; /* code width of the quantized linears' weights: 0 or 8 = W8A8; 4 = W4A8 (Table 2), stored two
                          codes per byte (half the weight memory); 2..7 other widths, stored one code per byte */
} qdit_model_shape;

typedef struct { /* HOST f32 arrays, each linear [out_features, in_features] row-major */
  const float *w_ada, *b_ada;   /* [6D, D], [6D]: shift_msa, scale_msa, gate_msa, shift_mlp, scale_mlp, gate_mlp */
  const float *w_qkv, *b_qkv;   /* [3D, D]: output laid out [3, heads, head_dim] */
  const float *w_proj, *b_proj; /* [D, D] */
  const float *w_fc1, *b_fc1;   /* [mlp, D] */
  const float *w_fc2, *b_fc2;   /* [D, mlp] */
} qdit_block_weights;

typedef struct { /* HOST pointers */
  qdit_model_shape shape;
  const float *w_patch, *b_patch; /* [D, C*p*p] (patch vector ordered c, py, px), [D] */
  const float* pos;               /* [tokens, D] position table */
  const float *w_t1, *b_t1;       /* [D, freq_dim] */
  const float *w_t2, *b_t2;       /* [D, D] */
  const float* y_table;           /* [num_classes + 1, D]; last row = "no class" */
  const float *w_ada_f, *b_ada_f; /* [2D, D]: shift, scale of the final layer */
  const float *w_out, *b_out;     /* [p*p*2C, D] (output vector ordered py, px, c) */
  const qdit_block_weights* blocks; /* [depth] */
} qdit_model_desc;

typedef struct qdit_model qdit_model;
/* Uploads the weights and quantizes the five linears of every block on the device
 * (qdit_quantize_weight).  Activation scales start unset. */
int32_t qdit_model_create(qdit_ctx* ctx, const qdit_model_desc* desc, qdit_model** out);
int32_t qdit_model_destroy(qdit_model* model);
/* Static tensor-wise activation scales (symmetric, z = 0, range [-127,127]), HOST arrays:
 * ada_scale: 1 float (input SiLU(c) shared by all modulation linears);
 * block_scales: [depth*4] = per block the inputs of qkv, proj, fc1, fc2. */
int32_t qdit_model_set_act_scales(qdit_ctx* ctx, qdit_model* model, const float* ada_scale,
                                  const float* block_scales);
int32_t qdit_model_get_act_scales(qdit_ctx* ctx, qdit_model* model, float* ada_scale, float* block_scales);
/* Device views of a quantized linear, for tests and for driving the primitives by hand.
 * which: 0 ada (of `block`; all blocks are stacked block-major in one [depth*6D, D] matrix),
 * 1 qkv, 2 proj, 3 fc1, 4 fc2.  Any out pointer may be NULL.  w_q is [N, K] bytes, or the packed form [N, K/2] of
 * qdit_w4a8_linear when the model stores 4-bit weights two per byte (weight_bits = 4 with hidden and mlp multiples
 * of 32; qdit_model_weights_packed tells). */
int32_t qdit_model_linear(qdit_model* model, int block, int which, const void** w_q, const float** w_scale,
                          const int32_t** w_colsum, const float** bias, int64_t* N, int64_t* K);

/* 1 if the model keeps its quantized weights as two 4-bit codes per byte, else 0. */
int32_t qdit_model_weights_packed(const qdit_model* model);

typedef struct {
  int32_t batch;          /* images per trajectory batch */
  int32_t num_steps;      /* S: DDIM steps, evenly spaced over 1000 training steps, eta = 0 */
  int32_t cache_interval; /* N of the cache rule; 1 = recompute every step */
  int32_t use_cfg;        /* classifier-free guidance: network batch = 2*batch ([cond; uncond]) */
  float guidance;         /* eps = eps_u + guidance * (eps_c - eps_u) */
  int32_t vc_mode;        /* QDIT_VC_* */
  const float* vc_table;  /* HOST f32 [num_steps, channels] (copied) or NULL */
  float vc_eps;
} qdit_sampler_desc;

typedef struct qdit_sampler qdit_sampler;
/* Allocates the activation workspace, the modulation table, the cache and the latent state. */
int32_t qdit_sampler_create(qdit_ctx* ctx, qdit_model* model, const qdit_sampler_desc* desc, qdit_sampler** out);
int32_t qdit_sampler_destroy(qdit_sampler* s);
/* Starts a trajectory: copies latent [batch,C,Hl,Wl] f32 and labels [batch] int32 (DEVICE pointers)
 * into the sampler, empties the cache. */
int32_t qdit_sampler_reset(qdit_ctx* ctx, qdit_sampler* s, const float* latent, const int32_t* labels);
/* Device pointer to the current latent [batch,C,Hl,Wl] f32 (owned by the sampler). */
float* qdit_sampler_latent(qdit_sampler* s);
/* One denoising step i (0-based; must be called in order 0..S-1 after a reset):
 * embed -> modulation for all blocks -> blocks computed (i mod N == 0, cache refreshed) or served
 * from the cache -> final layer -> guidance -> DDIM update -> VC. */
int32_t qdit_sample_step(qdit_ctx* ctx, qdit_sampler* s, int step_index);
/* Per-block, per-branch cache schedule in place of the global rule (the layer-wise schedules of the cache
 * methods the paper compares with and builds on, Related Work "Cache"): schedule is a HOST byte array
 * [num_steps][blocks][2] (attention branch, MLP branch), non-zero = serve that branch's cached output under the
 * current step's gate, zero = evaluate the branch and refresh its cache entry.  A step whose entries are all
 * non-zero is the fused skipped step, all zero the refresh step; a mixed step walks the blocks in order.
 * The array is copied; NULL returns to the global rule.  Reusing an entry that was never stored makes the step
 * fail with QDIT_ERR_STATE. */
int32_t qdit_sampler_set_schedule(qdit_ctx* ctx, qdit_sampler* s, const uint8_t* schedule);
/* The stochastic sampler of the Experimental Settings ("DDPM") in place of the deterministic update: the
 * ancestral step of the cited DDPM papers on the same evenly spaced timestep subset, betas re-derived for the
 * subset (beta'_k = 1 - ab_k / ab_{k-1}):
 *   x0 = x / sqrt(ab_k) - sqrt(1/ab_k - 1) eps,   mean = coef_x0 x0 + coef_xt x   (posterior q(x_{k-1} | x_k, x0)),
 *   log var = f log beta'_k + (1 - f) log beta~_k,  f = (v + 1)/2,  v = the network's second output group
 *   (learned variance; of the conditional half under guidance),   x <- mean + [k > 0] exp(log var / 2) * noise.
 * noise: DEVICE f32 [num_steps, batch, C, Hl*Wl] standard-normal numbers supplied by the caller (borrowed: must
 * stay valid while the sampler steps; the last step's slice is not read); NULL returns to DDIM.  Needs
 * num_steps >= 2.  Guidance, cache schedule and VC apply as with DDIM. */
int32_t qdit_sampler_set_ddpm(qdit_ctx* ctx, qdit_sampler* s, const float* noise);
/* Whole trajectory from HOST buffers: copies latent_host/labels_host in, runs steps 0..S-1, copies the
 * final latent to out_host, and synchronises. */
int32_t qdit_sample(qdit_ctx* ctx, qdit_sampler* s, const float* latent_host, const int32_t* labels_host,
                    float* out_host);

/* The un-quantized layers around the blocks (the paper takes them from the DiT architecture it cites and leaves them
 * in floating point), as calls of their own:
 *   qdit_patch_embed: x[m,:] = bf16(W_patch . patch(m) + b_patch + pos[m mod T,:]) for the B*T tokens of B samples;
 *     a patch vector holds the p x p x C latent values of a token in (channel, row, column) order.
 *     latent f32 [B,C,Hl,Wl], x bf16 [B*T, D] (both DEVICE, 16-byte aligned).
 *   qdit_final_layer: out = unpatchify(W_out . (LN(x[m,:]) * (1 + scale_b) + shift_b) + b_out): LayerNorm without
 *     affine (eps 1e-6, biased variance), the sample's modulation mod[b] = (shift | scale), a D -> p*p*2C linear in f32
 *     accuracy, output vector ordered (row, column, channel).  x bf16 [B*T, D], mod f32 [B, 2D], out f32 [B,2C,Hl,Wl].
 * Both return QDIT_ERR_ALIGN for a misaligned pointer and launch nothing then. */
int32_t qdit_patch_embed(qdit_ctx* ctx, qdit_model* model, const float* latent, int B, void* x);
int32_t qdit_final_layer(qdit_ctx* ctx, qdit_model* model, const void* x, const float* mod, int B, float* out);

/* One network evaluation on B <= (use_cfg ? 2 : 1) * batch samples, no sampler update:
 * latent [B,C,Hl,Wl] f32, t [B] f32 timesteps, y [B] int32 labels, out [B,2C,Hl,Wl] f32 (all DEVICE).
 * flags: QDIT_FWD_STORE_CACHE writes the cache, QDIT_FWD_REUSE serves all blocks from it,
 * QDIT_FWD_CALIBRATE runs every activation quantizer in dynamic mode and widens the model's
 * recorded activation ranges (then call qdit_model_finish_calibration). */
enum { QDIT_FWD_STORE_CACHE = 1, QDIT_FWD_REUSE = 2, QDIT_FWD_CALIBRATE = 4 };
int32_t qdit_forward(qdit_ctx* ctx, qdit_sampler* s, const float* latent, const float* t, const int32_t* y,
                     int B, float* out, uint32_t flags);
/* Activation-range calibration (text after Eq. 3): begin clears the recorded ranges, forwards with
 * QDIT_FWD_CALIBRATE widen them, finish turns them into the static scales (s = absmax / 127). */
int32_t qdit_model_begin_calibration(qdit_ctx* ctx, qdit_model* model);
int32_t qdit_model_finish_calibration(qdit_ctx* ctx, qdit_model* model);

/* Device buffers of the sampler's last network evaluation, for layer-level tests.
 * name: "x" residual stream bf16 [M,D]; "mod" f32 [B, depth*6D]; "c" f32 [B,D]; "qkv" bf16 [M,3D];
 * "h" bytes [M,D]; "a" bytes [M,D]; "u" bytes [M,mlp].  Returns NULL for an unknown name. */
void* qdit_sampler_buffer(qdit_sampler* s, const char* name);
qdit_cache* qdit_sampler_cache(qdit_sampler* s);

#ifdef __cplusplus
}
#endif
#endif /* QDIT_H_ */
