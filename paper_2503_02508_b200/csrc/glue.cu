// Small HBM-/latency-bound kernels around the blocks: block-output cache, variance compensation,
// guidance + DDIM update, patch embedding, conditioning MLP, final layer.
#include <cmath>
#include <new>

#include "common.cuh"
#include "internal.h"
#include "kernels.h"

namespace {

using namespace qd;

// ----------------------------------------------------------------------------- block-output cache
// x[m, 8 cols] = bf16(x + gate[b] * slot)
__global__ void __launch_bounds__(256) cache_reuse_kernel(__nv_bfloat16* __restrict__ x,
                                                          const __nv_bfloat16* __restrict__ slot,
                                                          const float* __restrict__ gate, int64_t ld_gate, int64_t M,
                                                          int D, int64_t T) {
  const int vec_per_row = D >> 3;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= M * vec_per_row) return;
  const int64_t row = idx / vec_per_row;
  const int col = static_cast<int>(idx - row * vec_per_row) * 8;
  float xv[8], sv[8], gv[8];
  Load8<__nv_bfloat16>::load(x + row * D + col, xv);
  Load8<__nv_bfloat16>::load(slot + row * D + col, sv);
  Load8<float>::load(gate + (row / T) * ld_gate + col, gv);
#pragma unroll
  for (int i = 0; i < 8; ++i) xv[i] = fmaf(gv[i], sv[i], xv[i]);
  *reinterpret_cast<uint4*>(x + row * D + col) = pack_bf16x8(xv);
}

// Fully skipped step: x = bf16(x + sum_b gate_msa_b * A_b + gate_mlp_b * Mo_b), one pass over the cache.
// Slot (b, branch) starts at cache + (2*b + branch) * M * D.
__global__ void __launch_bounds__(256) cache_reuse_all_kernel(__nv_bfloat16* __restrict__ x,
                                                              const __nv_bfloat16* __restrict__ cache,
                                                              const float* __restrict__ mod, int64_t ld_mod, int64_t M,
                                                              int D, int64_t T, int blocks) {
  const int vec_per_row = D >> 3;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= M * vec_per_row) return;
  const int64_t row = idx / vec_per_row;
  const int col = static_cast<int>(idx - row * vec_per_row) * 8;
  const int64_t off = row * D + col;
  const int64_t slot_stride = M * D;
  const float* mrow = mod + (row / T) * ld_mod + col;
  float acc[8];
  Load8<__nv_bfloat16>::load(x + off, acc);
#pragma unroll 4
  for (int b = 0; b < blocks; ++b) {
    float av[8], mv[8], ga[8], gm[8];
    Load8<__nv_bfloat16>::load(cache + (2 * b) * slot_stride + off, av);
    Load8<__nv_bfloat16>::load(cache + (2 * b + 1) * slot_stride + off, mv);
    Load8<float>::load(mrow + static_cast<int64_t>(b) * 6 * D + 2 * D, ga);
    Load8<float>::load(mrow + static_cast<int64_t>(b) * 6 * D + 5 * D, gm);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] += ga[i] * av[i] + gm[i] * mv[i];
  }
  *reinterpret_cast<uint4*>(x + off) = pack_bf16x8(acc);
}

// ----------------------------------------------------------------------------- block reductions
__device__ __forceinline__ float block_sum(float v, float* sm) {
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.0f;
  for (int i = 0; i < (blockDim.x >> 5); ++i) t += sm[i];
  return t;
}

// ----------------------------------------------------------------------------- variance compensation
// One CTA per (sample, channel): mean (and variance) over HW, then x = mu + K (x - mu) in place.
__global__ void __launch_bounds__(256) vc_kernel(float* __restrict__ latent, int C, int HW, int mode,
                                                 const float* __restrict__ row, float eps) {
  __shared__ float sm[8];
  float* x = latent + static_cast<int64_t>(blockIdx.x) * HW;
  const int c = blockIdx.x % C;
  float s = 0.0f;
  for (int i = threadIdx.x * 4; i < HW; i += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(x + i);
    s += (v.x + v.y) + (v.z + v.w);
  }
  const float mu = block_sum(s, sm) / static_cast<float>(HW);
  float K = row[c];
  if (mode == QDIT_VC_VAR_RATIO) {
    float ss = 0.0f;
    for (int i = threadIdx.x * 4; i < HW; i += blockDim.x * 4) {
      const float4 v = *reinterpret_cast<const float4*>(x + i);
      const float a = v.x - mu, b = v.y - mu, cc = v.z - mu, d = v.w - mu;
      ss += (a * a + b * b) + (cc * cc + d * d);
    }
    const float var = block_sum(ss, sm) / static_cast<float>(HW);
    K = sqrtf(K / (var + eps));
  }
  for (int i = threadIdx.x * 4; i < HW; i += blockDim.x * 4) {
    float4 v = *reinterpret_cast<const float4*>(x + i);
    v.x = mu + K * (v.x - mu);
    v.y = mu + K * (v.y - mu);
    v.z = mu + K * (v.z - mu);
    v.w = mu + K * (v.w - mu);
    *reinterpret_cast<float4*>(x + i) = v;
  }
}

// ----------------------------------------------------------------------------- guidance + DDIM update
// net: [Beff, 2C, HW]; eps = first C channels; with guidance, sample b's unconditional twin is b + B.
__global__ void __launch_bounds__(256) cfg_ddim_kernel(float* __restrict__ latent, const float* __restrict__ net, int B,
                                                       int C, int HW, int use_cfg, float guidance, DdimCoef k) {
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t per_sample = static_cast<int64_t>(C) * HW;
  if (idx >= B * per_sample) return;
  const int64_t b = idx / per_sample;
  const int64_t r = idx - b * per_sample;  // c*HW + i
  float eps = net[b * 2 * per_sample + r];
  if (use_cfg) {
    const float eu = net[(b + B) * 2 * per_sample + r];
    eps = eu + guidance * (eps - eu);
  }
  const float x = latent[idx];
  const float x0 = (x - k.sqrt_1mab_t * eps) / k.sqrt_ab_t;
  latent[idx] = k.sqrt_ab_prev * x0 + k.sqrt_1mab_prev * eps;
}

// ----------------------------------------------------------------------------- patch embedding
// One CTA per token row: x[m,:] = bf16(W_patch . patch(m) + b_patch + pos[t,:]); patch vector (c,py,px).
__global__ void __launch_bounds__(128) embed_kernel(const float* __restrict__ latent, int latent_batch,
                                                    const float* __restrict__ w, const float* __restrict__ bias,
                                                    const float* __restrict__ pos, __nv_bfloat16* __restrict__ x,
                                                    int D, int grid, int patch, int C) {
  extern __shared__ float sp[];  // patch vector, C*patch*patch
  const int T = grid * grid;
  const int64_t m = blockIdx.x;
  const int b = static_cast<int>(m / T) % latent_batch;
  const int t = static_cast<int>(m % T);
  const int gy = t / grid, gx = t % grid;
  const int side = grid * patch;
  const int pd = C * patch * patch;
  for (int j = threadIdx.x; j < pd; j += blockDim.x) {
    const int c = j / (patch * patch), py = (j / patch) % patch, px = j % patch;
    sp[j] = latent[((static_cast<int64_t>(b) * C + c) * side + gy * patch + py) * side + gx * patch + px];
  }
  __syncthreads();
  for (int d = threadIdx.x; d < D; d += blockDim.x) {
    float acc = 0.0f;
    const float* wr = w + static_cast<int64_t>(d) * pd;
    for (int j = 0; j < pd; ++j) acc = fmaf(wr[j], sp[j], acc);
    x[m * D + d] = __float2bfloat16_rn(acc + bias[d] + pos[static_cast<int64_t>(t) * D + d]);
  }
}

// ----------------------------------------------------------------------------- conditioning
// Warp per output.  h[b,d] = SiLU(W1[d,:] . feat(t_b) + b1[d]); features [cos(t f_j), sin(t f_j)],
// f_j = 10000^(-j/half), evaluated in double so that large arguments keep their phase.
__global__ void __launch_bounds__(256) cond1_kernel(const float* __restrict__ t, const float* __restrict__ w1,
                                                    const float* __restrict__ b1, float* __restrict__ h, int B, int D,
                                                    int F) {
  const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (gw >= B * D) return;
  const int b = gw / D, d = gw % D;
  const int half = F / 2;
  const double tv = static_cast<double>(t[b]);
  float acc = 0.0f;
  for (int j = lane; j < F; j += 32) {
    const int jj = j < half ? j : j - half;
    const double arg = tv * exp(-9.210340371976184 * static_cast<double>(jj) / static_cast<double>(half));
    const float f = static_cast<float>(j < half ? cos(arg) : sin(arg));
    acc = fmaf(w1[static_cast<int64_t>(d) * F + j], f, acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) h[gw] = silu_f(acc + b1[d]);
}

// out[b,n] = W[n,:] . in[b,:] + bias[n] (+ table[y[b], n]); optionally also SiLU(out) to out_silu.
__global__ void __launch_bounds__(256) small_linear_kernel(const float* __restrict__ in, const float* __restrict__ w,
                                                           const float* __restrict__ bias,
                                                           const float* __restrict__ table, const int32_t* __restrict__ y,
                                                           float* __restrict__ out, float* __restrict__ out_silu, int B,
                                                           int N, int K, int silu_input) {
  const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (gw >= B * N) return;
  const int b = gw / N, n = gw % N;
  float acc = 0.0f;
  const float* wr = w + static_cast<int64_t>(n) * K;
  const float* xr = in + static_cast<int64_t>(b) * K;
  for (int k = lane * 4; k < K; k += 128) {
    const float4 wv = *reinterpret_cast<const float4*>(wr + k);
    float4 xv = *reinterpret_cast<const float4*>(xr + k);
    if (silu_input) {
      xv.x = silu_f(xv.x); xv.y = silu_f(xv.y); xv.z = silu_f(xv.z); xv.w = silu_f(xv.w);
    }
    acc = fmaf(wv.x, xv.x, acc);
    acc = fmaf(wv.y, xv.y, acc);
    acc = fmaf(wv.z, xv.z, acc);
    acc = fmaf(wv.w, xv.w, acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) {
    float v = acc + bias[n];
    if (table) v += table[static_cast<int64_t>(y[b]) * N + n];
    out[gw] = v;
    if (out_silu) out_silu[gw] = silu_f(v);
  }
}

// ----------------------------------------------------------------------------- final layer
// Warp per token row: LayerNorm + modulate in registers, then the D -> OUT linear and un-patchify
// (output vector ordered (py, px, c)) into net[b, c, gy*p+py, gx*p+px].
template <int NV>
__global__ void __launch_bounds__(256) final_kernel(const __nv_bfloat16* __restrict__ x, int64_t M, int D, int T,
                                                    float eps, const float* __restrict__ modf,
                                                    const float* __restrict__ w, const float* __restrict__ bias,
                                                    float* __restrict__ net, int grid, int patch, int OUT) {
  const int lane = threadIdx.x & 31;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= M) return;
  const int nvec = D >> 3;
  float v[NV][8];
  float sum = 0.0f;
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int vi = lane + 32 * j;
    if (vi < nvec) {
      Load8<__nv_bfloat16>::load(x + row * D + vi * 8, v[j]);
#pragma unroll
      for (int i = 0; i < 8; ++i) sum += v[j][i];
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[j][i] = 0.0f;
    }
  }
  const float mean = warp_sum(sum) / static_cast<float>(D);
  float ss = 0.0f;
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    if (lane + 32 * j < nvec) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float d = v[j][i] - mean;
        ss += d * d;
      }
    }
  }
  const float rstd = 1.0f / sqrtf(warp_sum(ss) / static_cast<float>(D) + eps);
  const int b = static_cast<int>(row / T), t = static_cast<int>(row % T);
  const float* sh = modf + static_cast<int64_t>(b) * 2 * D;
  const float* sc = sh + D;
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int vi = lane + 32 * j;
    if (vi < nvec) {
      float shv[8], scv[8];
      Load8<float>::load(sh + vi * 8, shv);
      Load8<float>::load(sc + vi * 8, scv);
#pragma unroll
      for (int i = 0; i < 8; ++i) v[j][i] = (v[j][i] - mean) * rstd * (1.0f + scv[i]) + shv[i];
    }
  }
  const int gy = t / grid, gx = t % grid, side = grid * patch, co = OUT / (patch * patch);
  for (int o = 0; o < OUT; ++o) {
    float acc = 0.0f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      const int vi = lane + 32 * j;
      if (vi < nvec) {
        float wv[8];
        Load8<float>::load(w + static_cast<int64_t>(o) * D + vi * 8, wv);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc = fmaf(wv[i], v[j][i], acc);
      }
    }
    acc = warp_sum(acc);
    if (lane == 0) {
      const int c = o % co, px = (o / co) % patch, py = o / (co * patch);
      net[((static_cast<int64_t>(b) * co + c) * side + gy * patch + py) * side + gx * patch + px] = acc + bias[o];
    }
  }
}

}  // namespace

// ================================================================================ launchers
int32_t launch_embed(qdit_ctx* ctx, const float* latent, int latent_batch, const float* w, const float* bias,
                     const float* pos, void* x, int64_t M, int D, int grid, int patch, int C) {
  embed_kernel<<<static_cast<unsigned>(M), 128, C * patch * patch * sizeof(float), ctx->stream>>>(
      latent, latent_batch, w, bias, pos, static_cast<__nv_bfloat16*>(x), D, grid, patch, C);
  return qdit_after_launch(ctx, "embed_kernel");
}

int32_t launch_cond1(qdit_ctx* ctx, const float* t, const float* w1, const float* b1, float* h, int B, int D, int F) {
  const int64_t threads = static_cast<int64_t>(B) * D * 32;
  cond1_kernel<<<static_cast<unsigned>((threads + 255) / 256), 256, 0, ctx->stream>>>(t, w1, b1, h, B, D, F);
  return qdit_after_launch(ctx, "cond1_kernel");
}

int32_t launch_small_linear(qdit_ctx* ctx, const float* in, const float* w, const float* bias, const float* table,
                            const int32_t* y, float* out, float* out_silu, int B, int N, int K, int silu_input) {
  const int64_t threads = static_cast<int64_t>(B) * N * 32;
  small_linear_kernel<<<static_cast<unsigned>((threads + 255) / 256), 256, 0, ctx->stream>>>(
      in, w, bias, table, y, out, out_silu, B, N, K, silu_input);
  return qdit_after_launch(ctx, "small_linear_kernel");
}

int32_t launch_final(qdit_ctx* ctx, const void* x, int64_t M, int D, int T, float eps, const float* modf,
                     const float* w, const float* bias, float* net, int grid, int patch, int OUT) {
  const int warps = 8;
  const unsigned g = static_cast<unsigned>((M + warps - 1) / warps);
  const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
  const int nv = (D / 8 + 31) / 32;
#define QDIT_FINAL_CASE(NV) \
  case NV: final_kernel<NV><<<g, warps * 32, 0, ctx->stream>>>(xb, M, D, T, eps, modf, w, bias, net, grid, patch, OUT); break;
  switch (nv) {
    QDIT_FINAL_CASE(1) QDIT_FINAL_CASE(2) QDIT_FINAL_CASE(3) QDIT_FINAL_CASE(4) QDIT_FINAL_CASE(5) QDIT_FINAL_CASE(6)
    QDIT_FINAL_CASE(7)
    default: final_kernel<8><<<g, warps * 32, 0, ctx->stream>>>(xb, M, D, T, eps, modf, w, bias, net, grid, patch, OUT); break;
  }
#undef QDIT_FINAL_CASE
  return qdit_after_launch(ctx, "final_kernel");
}

int32_t launch_cfg_ddim(qdit_ctx* ctx, float* latent, const float* net, int B, int C, int HW, int use_cfg,
                        float guidance, const DdimCoef& k) {
  const int64_t n = static_cast<int64_t>(B) * C * HW;
  cfg_ddim_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, ctx->stream>>>(latent, net, B, C, HW, use_cfg,
                                                                                  guidance, k);
  return qdit_after_launch(ctx, "cfg_ddim_kernel");
}

// ================================================================================ cache object
struct qdit_cache {
  int device;
  int blocks;
  int64_t M, D;
  __nv_bfloat16* data;
  std::vector<uint8_t> filled;
};

extern "C" {

int32_t qdit_cache_should_refresh(int step_index, int interval) {
  if (step_index < 0 || interval < 1) return QDIT_ERR_INVALID_ARG;
  return step_index % interval == 0 ? 1 : 0;
}

int32_t qdit_cache_create(qdit_ctx* ctx, int blocks, int64_t M, int64_t D, qdit_cache** out) {
  if (!ctx || !out) return QDIT_ERR_INVALID_ARG;
  *out = nullptr;
  if (blocks <= 0 || M <= 0 || D <= 0 || D % 8 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "cache needs blocks, M > 0 and D a positive multiple of 8");
  qdit_cache* c = new (std::nothrow) qdit_cache();
  if (!c) return QDIT_ERR_NOMEM;
  c->device = ctx->device;
  c->blocks = blocks;
  c->M = M;
  c->D = D;
  c->filled.assign(static_cast<size_t>(blocks) * 2, 0);
  const size_t bytes = static_cast<size_t>(blocks) * 2 * M * D * sizeof(__nv_bfloat16);
  if (cudaMalloc(&c->data, bytes) != cudaSuccess) {
    cudaGetLastError();
    delete c;
    return qdit_fail(ctx, QDIT_ERR_NOMEM, "cannot allocate %zu bytes of cache", bytes);
  }
  *out = c;
  return QDIT_OK;
}

int32_t qdit_cache_destroy(qdit_cache* c) {
  if (!c) return QDIT_ERR_INVALID_ARG;
  cudaFree(c->data);
  delete c;
  return QDIT_OK;
}

int32_t qdit_cache_invalidate(qdit_cache* c) {
  if (!c) return QDIT_ERR_INVALID_ARG;
  std::fill(c->filled.begin(), c->filled.end(), 0);
  return QDIT_OK;
}

void* qdit_cache_slot(qdit_cache* c, int block, int branch, int mark_filled) {
  if (!c || block < 0 || block >= c->blocks || branch < 0 || branch > 1) return nullptr;
  if (mark_filled) c->filled[2 * block + branch] = 1;
  return c->data + static_cast<int64_t>(2 * block + branch) * c->M * c->D;
}

int32_t qdit_cache_store(qdit_ctx* ctx, qdit_cache* c, int block, int branch, const void* y) {
  if (!ctx || !c) return QDIT_ERR_INVALID_ARG;
  if (!y) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "y is NULL");
  void* dst = qdit_cache_slot(c, block, branch, 0);
  if (!dst) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "no slot (block %d, branch %d)", block, branch);
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(dst, y, static_cast<size_t>(c->M) * c->D * sizeof(__nv_bfloat16),
                                       cudaMemcpyDeviceToDevice, ctx->stream));
  c->filled[2 * block + branch] = 1;
  return QDIT_OK;
}

int32_t qdit_cache_reuse(qdit_ctx* ctx, qdit_cache* c, int block, int branch, const float* gate, int64_t ld_gate,
                         int64_t T, void* x) {
  if (!ctx || !c) return QDIT_ERR_INVALID_ARG;
  if (!gate || !x || T <= 0) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "gate or x is NULL, or T <= 0");
  const void* slot = qdit_cache_slot(c, block, branch, 0);
  if (!slot) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "no slot (block %d, branch %d)", block, branch);
  if (!c->filled[2 * block + branch]) return qdit_fail(ctx, QDIT_ERR_STATE, "cache slot (block %d, branch %d) reused before any store", block, branch);
  if (!aligned16(gate) || !aligned16(x) || ld_gate % 4 != 0) return qdit_fail(ctx, QDIT_ERR_ALIGN, "gate and x must be 16-byte aligned, ld_gate a multiple of 4");
  const int64_t n = c->M * (c->D / 8);
  cache_reuse_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, ctx->stream>>>(
      static_cast<__nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(slot), gate, ld_gate, c->M, static_cast<int>(c->D), T);
  return qdit_after_launch(ctx, "cache_reuse_kernel");
}

int32_t qdit_cache_reuse_all(qdit_ctx* ctx, qdit_cache* c, const float* mod_all, int64_t ld_mod, int64_t T, void* x) {
  if (!ctx || !c) return QDIT_ERR_INVALID_ARG;
  if (!mod_all || !x || T <= 0) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "mod_all or x is NULL, or T <= 0");
  for (size_t i = 0; i < c->filled.size(); ++i)
    if (!c->filled[i]) return qdit_fail(ctx, QDIT_ERR_STATE, "cache slot (block %zu, branch %zu) reused before any store", i / 2, i % 2);
  if (!aligned16(mod_all) || !aligned16(x) || ld_mod % 4 != 0) return qdit_fail(ctx, QDIT_ERR_ALIGN, "mod_all and x must be 16-byte aligned, ld_mod a multiple of 4");
  const int64_t n = c->M * (c->D / 8);
  ProfScope prof(ctx, QDIT_PROF_CACHE_REUSE, static_cast<double>(c->M) * c->D * 2.0 * (2.0 * c->blocks + 2.0));
  cache_reuse_all_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, ctx->stream>>>(
      static_cast<__nv_bfloat16*>(x), c->data, mod_all, ld_mod, c->M, static_cast<int>(c->D), T, c->blocks);
  return qdit_after_launch(ctx, "cache_reuse_all_kernel");
}

int32_t qdit_vc_correct(qdit_ctx* ctx, float* latent, int B, int C, int HW, int step_index, int mode,
                        const float* table, float eps) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (mode == QDIT_VC_NONE) return QDIT_OK;
  if (mode != QDIT_VC_K_TABLE && mode != QDIT_VC_VAR_RATIO) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "unknown VC mode %d", mode);
  if (B < 0 || C <= 0 || HW <= 0 || step_index < 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "bad sizes");
  if (B == 0) return QDIT_OK;
  if (!latent || !table) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "latent or table is NULL");
  if (HW % 4 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "HW must be a multiple of 4");
  if (!aligned16(latent)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "latent must be 16-byte aligned");
  vc_kernel<<<static_cast<unsigned>(B) * C, 256, 0, ctx->stream>>>(latent, C, HW, mode,
                                                                  table + static_cast<int64_t>(step_index) * C, eps);
  return qdit_after_launch(ctx, "vc_kernel");
}

}  // extern "C"
