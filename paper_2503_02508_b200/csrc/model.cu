// Model (quantized weights + activation scales) and sampler (workspace, cache, trajectory state):
// host-side orchestration of one network evaluation and of one denoising step.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include <cuda_bf16.h>

#include "internal.h"
#include "kernels.h"

namespace {

struct DeviceArena {  // owns cudaMalloc'd blocks
  std::vector<void*> blocks;
  template <typename T>
  T* alloc(size_t n) {
    void* p = nullptr;
    if (n == 0) n = 1;
    if (cudaMalloc(&p, n * sizeof(T)) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    blocks.push_back(p);
    return static_cast<T*>(p);
  }
  void release() {
    for (void* p : blocks) cudaFree(p);
    blocks.clear();
  }
};

struct QLinearDev {
  int8_t* q = nullptr;   // codes: [N, K] one per byte, or [N, K/2] two 4-bit codes per byte when `packed4`
  float* scale = nullptr;
  int32_t* colsum = nullptr;
  float* bias = nullptr;
  int64_t N = 0, K = 0;
  bool packed4 = false;
};

}  // namespace

struct qdit_model {
  int device;
  qdit_model_shape s;
  DeviceArena mem;
  QLinearDev ada_all;                     // [depth*6D, D], block-major
  std::vector<QLinearDev> qkv, proj, fc1, fc2;
  float *w_patch, *b_patch, *pos, *w_t1, *b_t1, *w_t2, *b_t2, *y_table, *w_ada_f, *b_ada_f, *w_out, *b_out;
  uint8_t* w_patch_frag = nullptr;   // patch-embedding weights in tensor-core fragment order (patch vectors of 16 values)
  float* d_scales;      // [1 + 4*depth] static activation scales: [0] ada input, then per block qkv, proj, fc1, fc2
  float* d_absmax_run;  // [1 + 4*depth] widest range seen during calibration
  bool scales_set;
  bool packed4;         // 4-bit weights stored two codes per byte (weight_bits == 4 and every K a multiple of 32)
  int64_t max_block_weight;  // largest N*K among the block-level linears (size of the widening scratch)
  int n_scales() const { return 1 + 4 * s.depth; }
};

struct qdit_sampler {
  qdit_model* model;
  qdit_sampler_desc d;
  DeviceArena mem;
  int Beff;
  int64_t M;
  void *x, *qkv;                 // bf16
  uint8_t *h, *a, *u, *ca;       // activation codes
  float *c, *sc, *hidden, *feat, *mod, *modf, *net, *latent, *t_all, *tmpf;   // t_all: [S, Beff] timestep of every step
  int32_t *y, *labels;
  float* dyn_absmax;             // [1 + 4*depth] this pass's ranges (calibration)
  float* dyn_scale;              // [1 + 4*depth] and the scales derived from them
  int8_t* w8_scratch;            // [max N*K] int8: a packed block-level weight matrix widened for the many-row kernels
  float* vc_table;               // device [S, C] or null
  // Conditioning of the whole trajectory, evaluated at step 0: the conditioning vector, and with it every block's
  // modulation, depends on the timestep and the label only, never on the latent.  Rows are (step, sample).
  float *traj_c, *traj_sc, *traj_hidden, *traj_feat, *traj_mod, *traj_modf;
  uint8_t* traj_ca;
  int traj_chunk;                // steps whose conditioning is evaluated together (0: per step, inside forward_impl)
  qdit_cache* cache;
  std::vector<DdimCoef> ddim;
  std::vector<DdpmCoef> ddpm;    // filled when the stochastic sampler is selected
  const float* noise;            // device [S, batch, C, HW] standard-normal noise of the stochastic sampler, or null
  std::vector<float> t_host;
  std::vector<uint8_t> schedule;  // [S][depth][2] per-branch reuse flags; empty = global rule
  int next_step;
};

namespace {

int32_t upload(qdit_ctx* ctx, DeviceArena& mem, const float* host, size_t n, float** out) {
  if (!host) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "a weight pointer in the model description is NULL");
  float* d = mem.alloc<float>(n);
  if (!d) return qdit_fail(ctx, QDIT_ERR_NOMEM, "out of device memory");
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(d, host, n * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
  *out = d;
  return QDIT_OK;
}

int32_t alloc_qlinear(qdit_ctx* ctx, DeviceArena& mem, int64_t N, int64_t K, bool packed4, QLinearDev* l) {
  l->N = N;
  l->K = K;
  l->packed4 = packed4;
  l->q = mem.alloc<int8_t>(static_cast<size_t>(N) * K / (packed4 ? 2 : 1));
  l->scale = mem.alloc<float>(N);
  l->colsum = mem.alloc<int32_t>(N);
  l->bias = mem.alloc<float>(N);
  if (!l->q || !l->scale || !l->colsum || !l->bias) return qdit_fail(ctx, QDIT_ERR_NOMEM, "out of device memory");
  return QDIT_OK;
}

// Uploads one f32 linear through the staging buffer and quantizes rows [row0, row0+N) of `l` on the device
// (`codes8`: N*K bytes of scratch for the one-per-byte codes of a layer that is stored packed).
int32_t quantize_into(qdit_ctx* ctx, float* staging, int8_t* codes8, const float* w, const float* b, int64_t N, int64_t K,
                      QLinearDev* l, int64_t row0, int bits) {
  if (!w || !b) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "a block weight pointer is NULL");
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(staging, w, static_cast<size_t>(N) * K * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
  if (l->packed4) {
    QDIT_TRY(qdit_quantize_weight_bits(ctx, staging, N, K, bits, codes8, l->scale + row0, l->colsum + row0));
    QDIT_TRY(qdit_pack_weight_int4(ctx, codes8, N, K, l->q + row0 * K / 2));
  } else {
    QDIT_TRY(qdit_quantize_weight_bits(ctx, staging, N, K, bits, l->q + row0 * K, l->scale + row0, l->colsum + row0));
  }
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(l->bias + row0, b, static_cast<size_t>(N) * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
  return QDIT_OK;
}

int32_t build_model(qdit_ctx* ctx, const qdit_model_desc* desc, qdit_model* m) {
  const qdit_model_shape& s = desc->shape;
  const int64_t D = s.hidden, F = s.mlp, T = static_cast<int64_t>(s.grid) * s.grid;
  const int pd = s.channels * s.patch * s.patch, od = 2 * s.channels * s.patch * s.patch;
  {
    // the embedding kernel reads the patch weights transposed: [pd][D]
    if (!desc->w_patch) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "a weight pointer in the model description is NULL");
    std::vector<float> wt(static_cast<size_t>(D) * pd);
    for (int64_t d = 0; d < D; ++d)
      for (int j = 0; j < pd; ++j) wt[static_cast<size_t>(j) * D + d] = desc->w_patch[d * pd + j];
    QDIT_TRY(upload(ctx, m->mem, wt.data(), D * pd, &m->w_patch));
    if (pd == 16 && D % 8 == 0) {
      m->w_patch_frag = m->mem.alloc<uint8_t>(static_cast<size_t>(D / 8) * 512);
      if (!m->w_patch_frag) return qdit_fail(ctx, QDIT_ERR_NOMEM, "out of device memory");
      QDIT_TRY(launch_embed_fragments(ctx, m->w_patch, D, m->w_patch_frag));
    }
    QDIT_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));  // `wt` is a host temporary
  }
  QDIT_TRY(upload(ctx, m->mem, desc->b_patch, D, &m->b_patch));
  QDIT_TRY(upload(ctx, m->mem, desc->pos, T * D, &m->pos));
  QDIT_TRY(upload(ctx, m->mem, desc->w_t1, D * s.freq_dim, &m->w_t1));
  QDIT_TRY(upload(ctx, m->mem, desc->b_t1, D, &m->b_t1));
  QDIT_TRY(upload(ctx, m->mem, desc->w_t2, D * D, &m->w_t2));
  QDIT_TRY(upload(ctx, m->mem, desc->b_t2, D, &m->b_t2));
  QDIT_TRY(upload(ctx, m->mem, desc->y_table, static_cast<size_t>(s.num_classes + 1) * D, &m->y_table));
  QDIT_TRY(upload(ctx, m->mem, desc->w_ada_f, 2 * D * D, &m->w_ada_f));
  QDIT_TRY(upload(ctx, m->mem, desc->b_ada_f, 2 * D, &m->b_ada_f));
  QDIT_TRY(upload(ctx, m->mem, desc->w_out, od * D, &m->w_out));
  QDIT_TRY(upload(ctx, m->mem, desc->b_out, od, &m->b_out));

  const int wbits = s.weight_bits == 0 ? 8 : s.weight_bits;
  // 4-bit codes are stored two per byte when every reduction length allows it (packed rows must be multiples of 16 bytes)
  const bool packed4 = wbits == 4 && D % 32 == 0 && F % 32 == 0;
  m->packed4 = packed4;
  m->max_block_weight = (6 * D > F ? 6 * D : F) * D;   // the modulation linear of one block is the largest (6D x D) unless mlp > 6D
  const int64_t big = 6 * D > F ? 6 * D : F;
  float* staging = nullptr;
  if (cudaMalloc(&staging, static_cast<size_t>(big) * (D > F ? D : F) * (sizeof(float) + (packed4 ? 1 : 0))) != cudaSuccess) {
    cudaGetLastError();
    return qdit_fail(ctx, QDIT_ERR_NOMEM, "out of device memory (staging)");
  }
  int8_t* codes8 = reinterpret_cast<int8_t*>(staging + static_cast<size_t>(big) * (D > F ? D : F));
  int32_t st = alloc_qlinear(ctx, m->mem, static_cast<int64_t>(s.depth) * 6 * D, D, packed4, &m->ada_all);
  m->qkv.resize(s.depth);
  m->proj.resize(s.depth);
  m->fc1.resize(s.depth);
  m->fc2.resize(s.depth);
  for (int i = 0; i < s.depth && st == QDIT_OK; ++i) {
    const qdit_block_weights& b = desc->blocks[i];
    if ((st = alloc_qlinear(ctx, m->mem, 3 * D, D, packed4, &m->qkv[i])) != QDIT_OK) break;
    if ((st = alloc_qlinear(ctx, m->mem, D, D, packed4, &m->proj[i])) != QDIT_OK) break;
    if ((st = alloc_qlinear(ctx, m->mem, F, D, packed4, &m->fc1[i])) != QDIT_OK) break;
    if ((st = alloc_qlinear(ctx, m->mem, D, F, packed4, &m->fc2[i])) != QDIT_OK) break;
    if ((st = quantize_into(ctx, staging, codes8, b.w_ada, b.b_ada, 6 * D, D, &m->ada_all, static_cast<int64_t>(i) * 6 * D, wbits)) != QDIT_OK) break;
    if ((st = quantize_into(ctx, staging, codes8, b.w_qkv, b.b_qkv, 3 * D, D, &m->qkv[i], 0, wbits)) != QDIT_OK) break;
    if ((st = quantize_into(ctx, staging, codes8, b.w_proj, b.b_proj, D, D, &m->proj[i], 0, wbits)) != QDIT_OK) break;
    if ((st = quantize_into(ctx, staging, codes8, b.w_fc1, b.b_fc1, F, D, &m->fc1[i], 0, wbits)) != QDIT_OK) break;
    if ((st = quantize_into(ctx, staging, codes8, b.w_fc2, b.b_fc2, D, F, &m->fc2[i], 0, wbits)) != QDIT_OK) break;
  }
  if (st == QDIT_OK) {
    m->d_scales = m->mem.alloc<float>(m->n_scales());
    m->d_absmax_run = m->mem.alloc<float>(m->n_scales());
    if (!m->d_scales || !m->d_absmax_run) st = qdit_fail(ctx, QDIT_ERR_NOMEM, "out of device memory");
  }
  if (st == QDIT_OK && cudaMemsetAsync(m->d_absmax_run, 0, m->n_scales() * sizeof(float), ctx->stream) != cudaSuccess)
    st = qdit_fail(ctx, QDIT_ERR_CUDA, "memset failed");
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
  cudaFree(staging);
  if (st == QDIT_OK && e != cudaSuccess) st = qdit_fail(ctx, QDIT_ERR_CUDA, "model upload failed: %s", cudaGetErrorString(e));
  return st;
}

qdit_qparams sym_qp() { return qdit_qparams{1.0f, 0, -127, 127}; }

// One quantized linear of the fused (static-scale) path.
// `w8_scratch`: for a layer stored packed, the matrix its weights are widened into when the layer has many rows
// (NULL: always widened inside the GEMM kernel, which is the form for the weight-streaming modulation GEMM).
int32_t run_linear(qdit_ctx* ctx, const void* A, const QLinearDev& l, int64_t M, const float* a_scale_dev, uint32_t flags,
                   qdit_epilogue epi, void* out, void* w8_scratch = nullptr) {
  epi.w_scale = l.scale;
  epi.w_colsum = l.colsum;
  epi.bias = l.bias;
  if (l.packed4)
    return qdit_w4a8_linear(ctx, A, l.q, M, l.N, l.K, sym_qp(), a_scale_dev, flags | QDIT_EPI_BIAS, &epi, out, l.N, w8_scratch);
  return qdit_w8a8_linear(ctx, A, l.q, M, l.N, l.K, sym_qp(), a_scale_dev, flags | QDIT_EPI_BIAS, &epi, out, l.N);
}

// The modulation linears of all blocks on `rows` conditioning rows: out[rows, depth * 6D].  One stacked GEMM; with
// packed 4-bit weights and many rows (the whole trajectory's conditioning) block by block instead, each block's
// 6D x D weights widened into the scratch matrix first (the stacked matrix would need a scratch of its own size).
int32_t run_modulation(qdit_ctx* ctx, const qdit_model* m, const void* A, int64_t rows, const float* a_scale_dev, float* out,
                       void* w8_scratch) {
  qdit_epilogue epi{};
  if (!(m->ada_all.packed4 && w8_scratch && rows >= 1024)) return run_linear(ctx, A, m->ada_all, rows, a_scale_dev, QDIT_EPI_OUT_F32, epi, out);
  const int64_t D = m->s.hidden, n6 = 6 * D, ld = static_cast<int64_t>(m->s.depth) * n6;
  for (int i = 0; i < m->s.depth; ++i) {
    const int64_t r0 = i * n6;
    epi.w_scale = m->ada_all.scale + r0;
    epi.w_colsum = m->ada_all.colsum + r0;
    epi.bias = m->ada_all.bias + r0;
    QDIT_TRY(qdit_w4a8_linear(ctx, A, m->ada_all.q + r0 * D / 2, rows, n6, D, sym_qp(), a_scale_dev, QDIT_EPI_BIAS | QDIT_EPI_OUT_F32,
                              &epi, out + r0, ld, w8_scratch));
  }
  return QDIT_OK;
}

// Calibration helper: range of an f32 tensor -> this pass's scale slot (and the running range), then codes.
int32_t dyn_quant(qdit_ctx* ctx, qdit_sampler* s, int slot, const float* x, int64_t M, int64_t K, uint8_t* q) {
  QDIT_CUDA_CHECK(ctx, cudaMemsetAsync(s->dyn_absmax + slot, 0, sizeof(float), ctx->stream));
  QDIT_TRY(launch_absmax(ctx, x, QDIT_F32, M, K, K, s->dyn_absmax + slot));
  QDIT_TRY(launch_absmax_to_scale(ctx, s->dyn_absmax + slot, s->dyn_scale + slot, s->model->d_absmax_run + slot, 1));
  // the quantizer reads the scale from the device slot
  qdit_qparams qp = sym_qp();
  // static mode validates qp->scale > 0 on the host; the device scale is what is used
  return qdit_quantize_act_dev(ctx, x, M, K, qp, s->dyn_scale + slot, q);
}

}  // namespace

// `pre_mod` / `pre_modf`: modulation [B, depth*6D] and final-layer modulation [B, 2D] evaluated beforehand for this
// step (both or neither); without them the conditioning path runs here.
// `mask`: [depth][2] per-branch reuse flags of a mixed step (needs STORE_CACHE; a flagged branch is not evaluated,
// its cached output enters the residual under this step's gate).
static int32_t forward_impl(qdit_ctx* ctx, qdit_sampler* s, const float* latent, int latent_batch, const float* t,
                            const int32_t* y, int B, float* out, uint32_t flags, const float* pre_mod = nullptr,
                            const float* pre_modf = nullptr, const uint8_t* mask = nullptr) {
  qdit_model* m = s->model;
  const qdit_model_shape& sh = m->s;
  const int D = sh.hidden, F = sh.mlp, T = sh.grid * sh.grid, depth = sh.depth;
  const int64_t M = static_cast<int64_t>(B) * T;
  const int64_t ld_mod = static_cast<int64_t>(depth) * 6 * D;
  const bool calib = (flags & QDIT_FWD_CALIBRATE) != 0;
  const bool reuse = (flags & QDIT_FWD_REUSE) != 0;
  const bool store = (flags & QDIT_FWD_STORE_CACHE) != 0;
  if (!calib && !m->scales_set) return qdit_fail(ctx, QDIT_ERR_STATE, "activation scales are not set (set them or calibrate)");
  if (reuse && (store || calib)) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "REUSE cannot be combined with STORE_CACHE or CALIBRATE");
  const float* scales = calib ? s->dyn_scale : m->d_scales;

  QDIT_TRY(launch_embed(ctx, latent, latent_batch, m->w_patch, m->w_patch_frag, m->b_patch, m->pos, s->x, M, D, sh.grid, sh.patch, sh.channels));
  const float* mod_all = pre_mod;
  if (!pre_mod) {
    QDIT_TRY(launch_cond1(ctx, t, m->w_t1, m->b_t1, s->feat, s->hidden, B, D, sh.freq_dim));
    QDIT_TRY(launch_small_linear(ctx, s->hidden, m->w_t2, m->b_t2, m->y_table, y, s->c, s->sc, B, D, D, 0, 0, 0));
    // modulation of every block in one stacked GEMM (the conditioning does not depend on the tokens)
    if (calib) {
      QDIT_TRY(dyn_quant(ctx, s, 0, s->sc, B, D, s->ca));
    } else {
      QDIT_TRY(qdit_quantize_act_dev(ctx, s->sc, B, D, sym_qp(), scales + 0, s->ca));
    }
    QDIT_TRY(run_modulation(ctx, m, s->ca, B, scales + 0, s->mod, s->w8_scratch));
    mod_all = s->mod;
  }

  if (reuse) {
    QDIT_TRY(qdit_cache_reuse_all(ctx, s->cache, mod_all, ld_mod, T, s->x));
  } else {
    for (int i = 0; i < depth; ++i) {
      const float* mod = mod_all + static_cast<int64_t>(i) * 6 * D;
      const float* sc_qkv = scales + 1 + 4 * i;
      const float* sc_proj = sc_qkv + 1;
      const float* sc_fc1 = sc_qkv + 2;
      const float* sc_fc2 = sc_qkv + 3;
      const float att_scale = 1.0f / sqrtf(static_cast<float>(D / sh.heads));
      qdit_qparams qp = sym_qp();
      qdit_epilogue gated{};
      gated.ld_gate = ld_mod;
      gated.tokens_per_sample = T;
      gated.residual = s->x;
      uint32_t gflags = QDIT_EPI_GATE | QDIT_EPI_RESIDUAL | QDIT_EPI_OUT_BF16 | (store ? QDIT_EPI_CACHE_STORE : 0u);
      if (!calib) {
        // ---- attention branch, fused quantizers
        if (mask && mask[2 * i]) {
          QDIT_TRY(qdit_cache_reuse(ctx, s->cache, i, QDIT_BRANCH_ATTN, mod + 2 * D, ld_mod, T, s->x));
        } else {
          QDIT_TRY(qdit_adaln_modulate(ctx, s->x, M, D, T, 1e-6f, mod, mod + D, ld_mod, s->h, QDIT_I8, &qp, sc_qkv));
          qdit_epilogue e0{};
          QDIT_TRY(run_linear(ctx, s->h, m->qkv[i], M, sc_qkv, QDIT_EPI_OUT_BF16, e0, s->qkv, s->w8_scratch));
          const __nv_bfloat16* qkv = static_cast<const __nv_bfloat16*>(s->qkv);
          QDIT_TRY(qdit_attention(ctx, qkv, qkv + D, qkv + 2 * D, 3 * D, B, sh.heads, T, D / sh.heads, att_scale, s->a,
                                  QDIT_I8, &qp, sc_proj));
          gated.gate = mod + 2 * D;
          gated.cache_out = store ? qdit_cache_slot(s->cache, i, QDIT_BRANCH_ATTN, 1) : nullptr;
          QDIT_TRY(run_linear(ctx, s->a, m->proj[i], M, sc_proj, gflags, gated, s->x, s->w8_scratch));
        }
        // ---- MLP branch
        if (mask && mask[2 * i + 1]) {
          QDIT_TRY(qdit_cache_reuse(ctx, s->cache, i, QDIT_BRANCH_MLP, mod + 5 * D, ld_mod, T, s->x));
        } else {
          QDIT_TRY(qdit_adaln_modulate(ctx, s->x, M, D, T, 1e-6f, mod + 3 * D, mod + 4 * D, ld_mod, s->h, QDIT_I8, &qp, sc_fc1));
          qdit_epilogue e1{};
          e1.out_qp = qp;
          e1.out_scale_dev = sc_fc2;
          QDIT_TRY(run_linear(ctx, s->h, m->fc1[i], M, sc_fc1, QDIT_EPI_GELU | QDIT_EPI_QUANT_OUT, e1, s->u, s->w8_scratch));
          gated.gate = mod + 5 * D;
          gated.cache_out = store ? qdit_cache_slot(s->cache, i, QDIT_BRANCH_MLP, 1) : nullptr;
          QDIT_TRY(run_linear(ctx, s->u, m->fc2[i], M, sc_fc2, gflags, gated, s->x, s->w8_scratch));
        }
      } else {
        // ---- calibration: every quantizer input is materialised in f32, its range reduced, then quantized
        QDIT_TRY(qdit_adaln_modulate(ctx, s->x, M, D, T, 1e-6f, mod, mod + D, ld_mod, s->tmpf, QDIT_F32, nullptr, nullptr));
        QDIT_TRY(dyn_quant(ctx, s, 1 + 4 * i, s->tmpf, M, D, s->h));
        qdit_epilogue e0{};
        QDIT_TRY(run_linear(ctx, s->h, m->qkv[i], M, sc_qkv, QDIT_EPI_OUT_BF16, e0, s->qkv, s->w8_scratch));
        const __nv_bfloat16* qkv = static_cast<const __nv_bfloat16*>(s->qkv);
        QDIT_TRY(qdit_attention(ctx, qkv, qkv + D, qkv + 2 * D, 3 * D, B, sh.heads, T, D / sh.heads, att_scale, s->tmpf,
                                QDIT_F32, nullptr, nullptr));
        QDIT_TRY(dyn_quant(ctx, s, 2 + 4 * i, s->tmpf, M, D, s->a));
        gated.gate = mod + 2 * D;
        gated.cache_out = store ? qdit_cache_slot(s->cache, i, QDIT_BRANCH_ATTN, 1) : nullptr;
        QDIT_TRY(run_linear(ctx, s->a, m->proj[i], M, sc_proj, gflags, gated, s->x, s->w8_scratch));
        QDIT_TRY(qdit_adaln_modulate(ctx, s->x, M, D, T, 1e-6f, mod + 3 * D, mod + 4 * D, ld_mod, s->tmpf, QDIT_F32, nullptr, nullptr));
        QDIT_TRY(dyn_quant(ctx, s, 3 + 4 * i, s->tmpf, M, D, s->h));
        qdit_epilogue e1{};
        QDIT_TRY(run_linear(ctx, s->h, m->fc1[i], M, sc_fc1, QDIT_EPI_GELU | QDIT_EPI_OUT_F32, e1, s->tmpf, s->w8_scratch));
        QDIT_TRY(dyn_quant(ctx, s, 4 + 4 * i, s->tmpf, M, F, s->u));
        gated.gate = mod + 5 * D;
        gated.cache_out = store ? qdit_cache_slot(s->cache, i, QDIT_BRANCH_MLP, 1) : nullptr;
        QDIT_TRY(run_linear(ctx, s->u, m->fc2[i], M, sc_fc2, gflags, gated, s->x, s->w8_scratch));
      }
    }
  }
  // final layer (f32): modulation from SiLU(c), LayerNorm, linear, un-patchify
  if (!pre_modf) QDIT_TRY(launch_small_linear(ctx, s->c, m->w_ada_f, m->b_ada_f, nullptr, nullptr, s->modf, nullptr, B, 2 * D, D, 1, 0, 0));
  QDIT_TRY(launch_final(ctx, s->x, M, D, T, 1e-6f, pre_modf ? pre_modf : s->modf, m->w_out, m->b_out, out, sh.grid, sh.patch,
                        2 * sh.channels * sh.patch * sh.patch));
  return QDIT_OK;
}

// Conditioning and modulation of `n_steps` steps of the trajectory, from step `first`, in one batch of
// n_steps * Beff rows (step-major).
static int32_t trajectory_conditioning(qdit_ctx* ctx, qdit_sampler* s, int first, int n_steps) {
  qdit_model* m = s->model;
  const qdit_model_shape& sh = m->s;
  const int D = sh.hidden, rows = n_steps * s->Beff;
  if (!m->scales_set) return qdit_fail(ctx, QDIT_ERR_STATE, "activation scales are not set (set them or calibrate)");
  const float* t = s->t_all + static_cast<int64_t>(first) * s->Beff;
  QDIT_TRY(launch_timestep_features(ctx, t, s->traj_feat, rows, sh.freq_dim));
  QDIT_TRY(launch_batched_linear(ctx, s->traj_feat, m->w_t1, m->b_t1, nullptr, nullptr, s->traj_hidden, nullptr, rows, D,
                                 sh.freq_dim, 0, 1, 0));
  QDIT_TRY(launch_batched_linear(ctx, s->traj_hidden, m->w_t2, m->b_t2, m->y_table, s->y, s->traj_c, s->traj_sc, rows, D, D, 0, 0,
                                 s->Beff));
  QDIT_TRY(qdit_quantize_act_dev(ctx, s->traj_sc, rows, D, sym_qp(), m->d_scales + 0, s->traj_ca));
  QDIT_TRY(run_modulation(ctx, m, s->traj_ca, rows, m->d_scales + 0, s->traj_mod, s->w8_scratch));
  return launch_batched_linear(ctx, s->traj_c, m->w_ada_f, m->b_ada_f, nullptr, nullptr, s->traj_modf, nullptr, rows, 2 * D, D, 1, 0, 0);
}

extern "C" {

int32_t qdit_model_create(qdit_ctx* ctx, const qdit_model_desc* desc, qdit_model** out) {
  if (!ctx || !out) return QDIT_ERR_INVALID_ARG;
  *out = nullptr;
  if (!desc || !desc->blocks) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "model description or its blocks are NULL");
  const qdit_model_shape& s = desc->shape;
  if (s.hidden <= 0 || s.heads <= 0 || s.mlp <= 0 || s.depth <= 0 || s.grid <= 0 || s.patch <= 0 || s.channels <= 0 ||
      s.num_classes <= 0 || s.freq_dim <= 0)
    return qdit_fail(ctx, QDIT_ERR_SHAPE, "model shape fields must be positive");
  if (s.weight_bits != 0 && (s.weight_bits < 2 || s.weight_bits > 8))
    return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "weight_bits = %d outside 2..8 (0 = 8)", s.weight_bits);
  if (s.hidden % s.heads != 0 || (s.hidden / s.heads != 64 && s.hidden / s.heads != 72))
    return qdit_fail(ctx, QDIT_ERR_SHAPE, "head_dim must be 64 or 72");
  if (s.hidden % 16 != 0 || s.mlp % 16 != 0 || s.hidden > 1536) return qdit_fail(ctx, QDIT_ERR_SHAPE, "hidden (<= 1536) and mlp must be multiples of 16");
  if ((s.grid * s.grid) % 64 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "tokens per image must be a multiple of 64");
  if (s.freq_dim % 2 != 0 || s.freq_dim % 4 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "freq_dim must be a multiple of 4");
  if ((s.grid * s.patch * s.grid * s.patch) % 4 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "latent size must be a multiple of 4");
  qdit_model* m = new (std::nothrow) qdit_model();
  if (!m) return QDIT_ERR_NOMEM;
  m->device = ctx->device;
  m->s = s;
  m->scales_set = false;
  m->d_scales = m->d_absmax_run = nullptr;
  int32_t st = build_model(ctx, desc, m);
  if (st != QDIT_OK) {
    m->mem.release();
    delete m;
    return st;
  }
  *out = m;
  return QDIT_OK;
}

int32_t qdit_model_destroy(qdit_model* m) {
  if (!m) return QDIT_ERR_INVALID_ARG;
  m->mem.release();
  delete m;
  return QDIT_OK;
}

int32_t qdit_model_set_act_scales(qdit_ctx* ctx, qdit_model* m, const float* ada_scale, const float* block_scales) {
  if (!ctx || !m) return QDIT_ERR_INVALID_ARG;
  if (!ada_scale || !block_scales) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "scale arrays are NULL");
  std::vector<float> h(m->n_scales());
  h[0] = *ada_scale;
  std::memcpy(h.data() + 1, block_scales, sizeof(float) * 4 * m->s.depth);
  for (float v : h)
    if (!(v > 0.0f)) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "activation scales must be > 0");
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(m->d_scales, h.data(), h.size() * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
  QDIT_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
  m->scales_set = true;
  return QDIT_OK;
}

int32_t qdit_model_get_act_scales(qdit_ctx* ctx, qdit_model* m, float* ada_scale, float* block_scales) {
  if (!ctx || !m) return QDIT_ERR_INVALID_ARG;
  if (!ada_scale || !block_scales) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "scale arrays are NULL");
  if (!m->scales_set) return qdit_fail(ctx, QDIT_ERR_STATE, "activation scales are not set");
  std::vector<float> h(m->n_scales());
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(h.data(), m->d_scales, h.size() * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
  QDIT_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
  *ada_scale = h[0];
  std::memcpy(block_scales, h.data() + 1, sizeof(float) * 4 * m->s.depth);
  return QDIT_OK;
}

int32_t qdit_model_begin_calibration(qdit_ctx* ctx, qdit_model* m) {
  if (!ctx || !m) return QDIT_ERR_INVALID_ARG;
  QDIT_CUDA_CHECK(ctx, cudaMemsetAsync(m->d_absmax_run, 0, m->n_scales() * sizeof(float), ctx->stream));
  return QDIT_OK;
}

int32_t qdit_model_finish_calibration(qdit_ctx* ctx, qdit_model* m) {
  if (!ctx || !m) return QDIT_ERR_INVALID_ARG;
  QDIT_TRY(launch_absmax_to_scale(ctx, m->d_absmax_run, m->d_scales, nullptr, m->n_scales()));
  m->scales_set = true;
  return QDIT_OK;
}

int32_t qdit_model_weights_packed(const qdit_model* m) { return m && m->packed4 ? 1 : 0; }

int32_t qdit_model_linear(qdit_model* m, int block, int which, const void** w_q, const float** w_scale,
                          const int32_t** w_colsum, const float** bias, int64_t* N, int64_t* K) {
  if (!m || block < 0 || block >= m->s.depth || which < 0 || which > 4) return QDIT_ERR_INVALID_ARG;
  QLinearDev l;
  if (which == 0) {
    const int64_t D = m->s.hidden, r0 = static_cast<int64_t>(block) * 6 * D;
    l = m->ada_all;
    l.q += r0 * D / (l.packed4 ? 2 : 1);
    l.scale += r0;
    l.colsum += r0;
    l.bias += r0;
    l.N = 6 * D;
  } else {
    l = which == 1 ? m->qkv[block] : which == 2 ? m->proj[block] : which == 3 ? m->fc1[block] : m->fc2[block];
  }
  if (w_q) *w_q = l.q;
  if (w_scale) *w_scale = l.scale;
  if (w_colsum) *w_colsum = l.colsum;
  if (bias) *bias = l.bias;
  if (N) *N = l.N;
  if (K) *K = l.K;
  return QDIT_OK;
}

int32_t qdit_sampler_create(qdit_ctx* ctx, qdit_model* m, const qdit_sampler_desc* d, qdit_sampler** out) {
  if (!ctx || !out) return QDIT_ERR_INVALID_ARG;
  *out = nullptr;
  if (!m || !d) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "model or description is NULL");
  if (d->batch <= 0 || d->num_steps <= 0 || d->num_steps > 1000 || d->cache_interval < 1)
    return qdit_fail(ctx, QDIT_ERR_SHAPE, "batch, num_steps (1..1000) and cache_interval (>= 1) must be positive");
  if (d->vc_mode != QDIT_VC_NONE && d->vc_mode != QDIT_VC_K_TABLE && d->vc_mode != QDIT_VC_VAR_RATIO)
    return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "unknown VC mode");
  if (d->vc_mode != QDIT_VC_NONE && !d->vc_table) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "VC mode set but vc_table is NULL");
  qdit_sampler* s = new (std::nothrow) qdit_sampler();
  if (!s) return QDIT_ERR_NOMEM;
  s->model = m;
  s->d = *d;
  s->d.vc_table = nullptr;
  s->cache = nullptr;
  s->vc_table = nullptr;
  s->next_step = -1;
  s->noise = nullptr;
  const qdit_model_shape& sh = m->s;
  const int D = sh.hidden, F = sh.mlp, T = sh.grid * sh.grid, C = sh.channels;
  const int HW = sh.grid * sh.patch * sh.grid * sh.patch;
  s->Beff = d->use_cfg ? 2 * d->batch : d->batch;
  s->M = static_cast<int64_t>(s->Beff) * T;
  const int64_t M = s->M, B = s->Beff;
  DeviceArena& a = s->mem;
  s->x = a.alloc<uint16_t>(M * D);
  s->qkv = a.alloc<uint16_t>(M * 3 * D);
  s->h = a.alloc<uint8_t>(M * D);
  s->a = a.alloc<uint8_t>(M * D);
  s->u = a.alloc<uint8_t>(M * F);
  s->ca = a.alloc<uint8_t>(B * D);
  s->c = a.alloc<float>(B * D);
  s->sc = a.alloc<float>(B * D);
  s->hidden = a.alloc<float>(B * D);
  s->feat = a.alloc<float>(B * sh.freq_dim);
  s->mod = a.alloc<float>(B * sh.depth * 6 * D);
  s->modf = a.alloc<float>(B * 2 * D);
  s->net = a.alloc<float>(B * 2 * C * HW);
  s->latent = a.alloc<float>(static_cast<int64_t>(d->batch) * C * HW);
  s->t_all = a.alloc<float>(B * d->num_steps);
  s->y = a.alloc<int32_t>(B);
  s->labels = a.alloc<int32_t>(d->batch);
  s->tmpf = a.alloc<float>(M * F);
  s->w8_scratch = m->packed4 ? a.alloc<int8_t>(m->max_block_weight) : nullptr;
  s->dyn_absmax = a.alloc<float>(m->n_scales());
  s->dyn_scale = a.alloc<float>(m->n_scales());
  // conditioning of as many steps at once as a 4 GB modulation table holds (all of them for the paper's 50- and
  // 100-step settings; a 250-step trajectory at network batch 32 goes in chunks of 173 steps)
  bool traj_ok = true;
  {
    const int64_t per_step = B * sh.depth * 6 * D * static_cast<int64_t>(sizeof(float));
    int64_t chunk = (int64_t(4) << 30) / per_step;
    if (chunk > d->num_steps) chunk = d->num_steps;
    const int want = ctx->opt[QDIT_OPT_CONDITIONING_CHUNK];  // -1: per step; n > 0: at most n steps at once (memory, tests)
    if (want < 0) chunk = 0;
    if (want > 0 && want < chunk) chunk = want;
    s->traj_chunk = static_cast<int>(chunk);
    s->traj_c = s->traj_sc = s->traj_hidden = s->traj_feat = s->traj_mod = s->traj_modf = nullptr;
    s->traj_ca = nullptr;
    if (s->traj_chunk > 0) {
      const int64_t rows = B * s->traj_chunk;
      s->traj_c = a.alloc<float>(rows * D);
      s->traj_sc = a.alloc<float>(rows * D);
      s->traj_hidden = a.alloc<float>(rows * D);
      s->traj_feat = a.alloc<float>(rows * sh.freq_dim);
      s->traj_mod = a.alloc<float>(rows * sh.depth * 6 * D);
      s->traj_modf = a.alloc<float>(rows * 2 * D);
      s->traj_ca = a.alloc<uint8_t>(rows * D);
      if (!s->traj_c || !s->traj_sc || !s->traj_hidden || !s->traj_feat || !s->traj_mod || !s->traj_modf || !s->traj_ca) traj_ok = false;
    }
  }
  bool ok = traj_ok && s->x && s->qkv && s->h && s->a && s->u && s->ca && s->c && s->sc && s->hidden && s->feat && s->mod && s->modf && s->net &&
            s->latent && s->t_all && s->y && s->labels && s->tmpf && s->dyn_absmax && s->dyn_scale && (!m->packed4 || s->w8_scratch);
  if (ok && d->vc_mode != QDIT_VC_NONE) {
    s->vc_table = a.alloc<float>(static_cast<int64_t>(d->num_steps) * C);
    ok = s->vc_table && cudaMemcpy(s->vc_table, d->vc_table, sizeof(float) * d->num_steps * C, cudaMemcpyHostToDevice) == cudaSuccess;
  }
  int32_t st = ok ? QDIT_OK : qdit_fail(ctx, QDIT_ERR_NOMEM, "out of device memory (sampler workspace)");
  if (st == QDIT_OK) st = qdit_cache_create(ctx, sh.depth, M, D, &s->cache);
  if (st != QDIT_OK) {
    cudaGetLastError();
    if (s->cache) qdit_cache_destroy(s->cache);
    a.release();
    delete s;
    return st;
  }
  // DDIM (eta = 0) over a 1000-step linear-beta schedule, evenly spaced timesteps, alpha_bar_prev = 1 at the end
  std::vector<double> ab(1000);
  double prod = 1.0;
  for (int j = 0; j < 1000; ++j) {
    const double beta = 1e-4 + (2e-2 - 1e-4) * static_cast<double>(j) / 999.0;
    prod *= 1.0 - beta;
    ab[j] = prod;
  }
  const int stride = 1000 / d->num_steps;
  s->ddim.resize(d->num_steps);
  s->t_host.resize(d->num_steps);
  for (int i = 0; i < d->num_steps; ++i) {
    const int ti = (d->num_steps - 1 - i) * stride;
    const double abt = ab[ti];
    const double abp = i + 1 < d->num_steps ? ab[(d->num_steps - 2 - i) * stride] : 1.0;
    s->ddim[i] = DdimCoef{static_cast<float>(std::sqrt(abt)), static_cast<float>(std::sqrt(1.0 - abt)),
                          static_cast<float>(std::sqrt(abp)), static_cast<float>(std::sqrt(1.0 - abp))};
    s->t_host[i] = static_cast<float>(ti);
  }
  {
    std::vector<float> tv(static_cast<size_t>(B) * d->num_steps);
    for (int i = 0; i < d->num_steps; ++i)
      for (int64_t b = 0; b < B; ++b) tv[i * B + b] = s->t_host[i];
    std::vector<int32_t> yv(B, sh.num_classes);  // second half stays the "no class" label under guidance
    if (cudaMemcpy(s->t_all, tv.data(), tv.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(s->y, yv.data(), yv.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess) {
      cudaGetLastError();
      qdit_cache_destroy(s->cache);
      a.release();
      delete s;
      return qdit_fail(ctx, QDIT_ERR_CUDA, "sampler table upload failed");
    }
  }
  *out = s;
  return QDIT_OK;
}

int32_t qdit_sampler_destroy(qdit_sampler* s) {
  if (!s) return QDIT_ERR_INVALID_ARG;
  if (s->cache) qdit_cache_destroy(s->cache);
  s->mem.release();
  delete s;
  return QDIT_OK;
}

float* qdit_sampler_latent(qdit_sampler* s) { return s ? s->latent : nullptr; }
qdit_cache* qdit_sampler_cache(qdit_sampler* s) { return s ? s->cache : nullptr; }

void* qdit_sampler_buffer(qdit_sampler* s, const char* name) {
  if (!s || !name) return nullptr;
  if (!strcmp(name, "x")) return s->x;
  if (!strcmp(name, "mod")) return s->mod;
  if (!strcmp(name, "c")) return s->c;
  if (!strcmp(name, "qkv")) return s->qkv;
  if (!strcmp(name, "h")) return s->h;
  if (!strcmp(name, "a")) return s->a;
  if (!strcmp(name, "u")) return s->u;
  return nullptr;
}

int32_t qdit_forward(qdit_ctx* ctx, qdit_sampler* s, const float* latent, const float* t, const int32_t* y, int B,
                     float* out, uint32_t flags) {
  if (!ctx || !s) return QDIT_ERR_INVALID_ARG;
  if (!latent || !t || !y || !out) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  if (B <= 0 || B > s->Beff) return qdit_fail(ctx, QDIT_ERR_SHAPE, "B = %d outside 1..%d", B, s->Beff);
  if ((flags & (QDIT_FWD_STORE_CACHE | QDIT_FWD_REUSE)) && B != s->Beff)
    return qdit_fail(ctx, QDIT_ERR_SHAPE, "cache flags need the sampler's full batch (%d)", s->Beff);
  return forward_impl(ctx, s, latent, B, t, y, B, out, flags);
}

int32_t qdit_patch_embed(qdit_ctx* ctx, qdit_model* m, const float* latent, int B, void* x) {
  if (!ctx || !m) return QDIT_ERR_INVALID_ARG;
  if (!latent || !x) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  if (B <= 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "B = %d", B);
  if (!aligned16(x) || !aligned16(latent)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "latent and x must be 16-byte aligned");
  const qdit_model_shape& sh = m->s;
  const int64_t M = static_cast<int64_t>(B) * sh.grid * sh.grid;
  return launch_embed(ctx, latent, B, m->w_patch, m->w_patch_frag, m->b_patch, m->pos, x, M, sh.hidden, sh.grid, sh.patch, sh.channels);
}

int32_t qdit_final_layer(qdit_ctx* ctx, qdit_model* m, const void* x, const float* mod, int B, float* out) {
  if (!ctx || !m) return QDIT_ERR_INVALID_ARG;
  if (!x || !mod || !out) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  if (B <= 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "B = %d", B);
  if (!aligned16(x) || !aligned16(mod) || !aligned16(out)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "x, mod and out must be 16-byte aligned");
  const qdit_model_shape& sh = m->s;
  const int T = sh.grid * sh.grid;
  return launch_final(ctx, x, static_cast<int64_t>(B) * T, sh.hidden, T, 1e-6f, mod, m->w_out, m->b_out, out, sh.grid, sh.patch,
                      2 * sh.channels * sh.patch * sh.patch);
}

int32_t qdit_sampler_reset(qdit_ctx* ctx, qdit_sampler* s, const float* latent, const int32_t* labels) {
  if (!ctx || !s) return QDIT_ERR_INVALID_ARG;
  if (!latent || !labels) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "latent or labels is NULL");
  const qdit_model_shape& sh = s->model->s;
  const int HW = sh.grid * sh.patch * sh.grid * sh.patch, B = s->d.batch;
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(s->latent, latent, sizeof(float) * B * sh.channels * HW, cudaMemcpyDefault, ctx->stream));
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(s->y, labels, sizeof(int32_t) * B, cudaMemcpyDefault, ctx->stream));
  qdit_cache_invalidate(s->cache);
  s->next_step = 0;
  return QDIT_OK;
}

int32_t qdit_sampler_set_ddpm(qdit_ctx* ctx, qdit_sampler* s, const float* noise) {
  if (!ctx || !s) return QDIT_ERR_INVALID_ARG;
  s->noise = noise;
  if (!noise) return QDIT_OK;
  const int S = s->d.num_steps;
  if (S < 2) {
    s->noise = nullptr;
    return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "the stochastic sampler needs at least two steps");
  }
  // alpha_bar of the kept timesteps (ascending), betas re-derived for the subset, posterior q(x_{k-1} | x_k, x0)
  std::vector<double> ab_full(1000);
  double prod = 1.0;
  for (int j = 0; j < 1000; ++j) {
    prod *= 1.0 - (1e-4 + (2e-2 - 1e-4) * static_cast<double>(j) / 999.0);
    ab_full[j] = prod;
  }
  const int stride = 1000 / S;
  std::vector<double> ab(S), beta(S), post(S);
  for (int k = 0; k < S; ++k) {
    ab[k] = ab_full[k * stride];
    const double abp = k > 0 ? ab[k - 1] : 1.0;
    beta[k] = 1.0 - ab[k] / abp;
    post[k] = beta[k] * (1.0 - abp) / (1.0 - ab[k]);
  }
  s->ddpm.resize(S);
  for (int i = 0; i < S; ++i) {
    const int k = S - 1 - i;
    const double abp = k > 0 ? ab[k - 1] : 1.0;
    DdpmCoef c;
    c.rs = static_cast<float>(1.0 / std::sqrt(ab[k]));
    c.rsm1 = static_cast<float>(std::sqrt(1.0 / ab[k] - 1.0));
    c.c_x0 = static_cast<float>(beta[k] * std::sqrt(abp) / (1.0 - ab[k]));
    c.c_xt = static_cast<float>((1.0 - abp) * std::sqrt(1.0 - beta[k]) / (1.0 - ab[k]));
    c.log_beta = static_cast<float>(std::log(beta[k]));
    c.log_post = static_cast<float>(std::log(post[k > 0 ? k : 1]));
    c.nz = k > 0 ? 1.0f : 0.0f;
    s->ddpm[i] = c;
  }
  return QDIT_OK;
}

int32_t qdit_sampler_set_schedule(qdit_ctx* ctx, qdit_sampler* s, const uint8_t* schedule) {
  if (!ctx || !s) return QDIT_ERR_INVALID_ARG;
  if (!schedule) {
    s->schedule.clear();
    return QDIT_OK;
  }
  const size_t n = static_cast<size_t>(s->d.num_steps) * s->model->s.depth * 2;
  s->schedule.assign(schedule, schedule + n);
  return QDIT_OK;
}

int32_t qdit_sample_step(qdit_ctx* ctx, qdit_sampler* s, int i) {
  if (!ctx || !s) return QDIT_ERR_INVALID_ARG;
  if (s->next_step < 0) return qdit_fail(ctx, QDIT_ERR_STATE, "qdit_sampler_reset has not been called");
  if (i != s->next_step || i >= s->d.num_steps) return qdit_fail(ctx, QDIT_ERR_STATE, "step %d out of order (expected %d of %d)", i, s->next_step, s->d.num_steps);
  const qdit_model_shape& sh = s->model->s;
  const int HW = sh.grid * sh.patch * sh.grid * sh.patch, B = s->d.batch;
  uint32_t flags = 0;
  if (s->d.cache_interval > 1) flags = qdit_cache_should_refresh(i, s->d.cache_interval) ? QDIT_FWD_STORE_CACHE : QDIT_FWD_REUSE;
  const uint8_t* mask = nullptr;
  if (!s->schedule.empty()) {
    // per-branch schedule: all flags set = the fused skipped step, none = the refresh step, else a mixed step
    const uint8_t* row = s->schedule.data() + static_cast<size_t>(i) * sh.depth * 2;
    int set = 0;
    for (int j = 0; j < 2 * sh.depth; ++j) set += row[j] != 0;
    if (set == 2 * sh.depth) {
      flags = QDIT_FWD_REUSE;
    } else {
      flags = QDIT_FWD_STORE_CACHE;
      if (set > 0) mask = row;
    }
  }
  const float *pre_mod = nullptr, *pre_modf = nullptr;
  if (s->traj_chunk > 0) {
    const int in_chunk = i % s->traj_chunk;
    if (in_chunk == 0) {
      const int left = s->d.num_steps - i;
      QDIT_TRY(trajectory_conditioning(ctx, s, i, left < s->traj_chunk ? left : s->traj_chunk));
    }
    const int64_t row0 = static_cast<int64_t>(in_chunk) * s->Beff;
    pre_mod = s->traj_mod + row0 * sh.depth * 6 * sh.hidden;
    pre_modf = s->traj_modf + row0 * 2 * sh.hidden;
  }
  QDIT_TRY(forward_impl(ctx, s, s->latent, B, s->t_all + static_cast<int64_t>(i) * s->Beff, s->y, s->Beff, s->net, flags, pre_mod,
                        pre_modf, mask));
  if (s->noise) {
    QDIT_TRY(launch_cfg_ddpm(ctx, s->latent, s->net, s->noise + static_cast<int64_t>(i) * B * sh.channels * HW, B, sh.channels,
                             HW, s->d.use_cfg, s->d.guidance, s->ddpm[i]));
  } else {
    QDIT_TRY(launch_cfg_ddim(ctx, s->latent, s->net, B, sh.channels, HW, s->d.use_cfg, s->d.guidance, s->ddim[i]));
  }
  if (s->d.vc_mode != QDIT_VC_NONE)
    QDIT_TRY(qdit_vc_correct(ctx, s->latent, B, sh.channels, HW, i, s->d.vc_mode, s->vc_table, s->d.vc_eps));
  s->next_step = i + 1;
  return QDIT_OK;
}

int32_t qdit_sample(qdit_ctx* ctx, qdit_sampler* s, const float* latent_host, const int32_t* labels_host, float* out_host) {
  if (!ctx || !s) return QDIT_ERR_INVALID_ARG;
  if (!latent_host || !labels_host || !out_host) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  const qdit_model_shape& sh = s->model->s;
  const size_t n = static_cast<size_t>(s->d.batch) * sh.channels * sh.grid * sh.patch * sh.grid * sh.patch;
  QDIT_TRY(qdit_sampler_reset(ctx, s, latent_host, labels_host));
  for (int i = 0; i < s->d.num_steps; ++i) QDIT_TRY(qdit_sample_step(ctx, s, i));
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(out_host, s->latent, n * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
  return qdit_sync(ctx);
}

}  // extern "C"
