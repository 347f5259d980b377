// Small HBM-/latency-bound kernels around the blocks: block-output cache, variance compensation (correction and
// the closed-form fit of its factors), guidance + DDIM update, patch embedding, conditioning MLP (per call and
// batched over a whole trajectory), final layer.
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
// Slot (b, branch) starts at cache + (2*b + branch) * M * D.  A thread owns 8 columns of R consecutive rows of one
// sample, so the two gate vectors of a block are loaded once per R rows (with R = 1 they are as many bytes from
// L2 as the cache itself is from HBM) and 2 R independent 16-byte cache loads are in flight per block.
template <int R>
__global__ void __launch_bounds__(256, 2) cache_reuse_all_kernel(__nv_bfloat16* __restrict__ x,
                                                                 const __nv_bfloat16* __restrict__ cache,
                                                                 const float* __restrict__ mod, int64_t ld_mod, int64_t M,
                                                                 int D, int64_t T, int blocks) {
  const int vec_per_row = D >> 3;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t groups = M / R;  // the launcher picks R with M % R == 0 and T % R == 0
  if (idx >= groups * vec_per_row) return;
  const int64_t row = (idx / vec_per_row) * R;
  const int col = static_cast<int>(idx % vec_per_row) * 8;
  const int64_t off = row * D + col;
  const int64_t slot_stride = M * D;
  const float* mrow = mod + (row / T) * ld_mod + col;
  float acc[R][8];
#pragma unroll
  for (int r = 0; r < R; ++r) Load8<__nv_bfloat16>::load(x + off + static_cast<int64_t>(r) * D, acc[r]);
#pragma unroll(R >= 4 ? 1 : 2)
  for (int b = 0; b < blocks; ++b) {
    float ga[8], gm[8];
    Load8<float>::load(mrow + static_cast<int64_t>(b) * 6 * D + 2 * D, ga);
    Load8<float>::load(mrow + static_cast<int64_t>(b) * 6 * D + 5 * D, gm);
    float av[R][8], mv[R][8];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      Load8<__nv_bfloat16>::load(cache + (2 * b) * slot_stride + off + static_cast<int64_t>(r) * D, av[r]);
      Load8<__nv_bfloat16>::load(cache + (2 * b + 1) * slot_stride + off + static_cast<int64_t>(r) * D, mv[r]);
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[r][i] += ga[i] * av[r][i] + gm[i] * mv[r][i];
  }
#pragma unroll
  for (int r = 0; r < R; ++r) *reinterpret_cast<uint4*>(x + off + static_cast<int64_t>(r) * D) = pack_bf16x8(acc[r]);
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

// ----------------------------------------------------------------------------- variance compensation: fitting K
// Closed-form factor of one step from calibration samples x^ (quantized + cached trajectory) and targets x'
// (reference trajectory): with mu = spatial mean of x^ per (sample, channel), a = x^ - mu, b = x' - mu and
// w = 1 / (x'^2 + eps), minimising rQNSR^2 + MSE over K gives
//   K[c] = (sum a b + sum a b w) / (sum a^2 + sum a^2 w)        (sums over samples and positions of channel c);
// the form as printed in the paper has sum a / x' in place of sum a b w.
// Pass 1: one CTA per (sample, channel) writes its four partial sums (f64: w reaches 1/eps where x' passes
// through zero).  Pass 2: one thread per channel adds the samples' partials in order and divides, so the result
// does not depend on scheduling.
__device__ __forceinline__ double block_sum_f64(double v, double* sm) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
  for (int i = 0; i < (blockDim.x >> 5); ++i) t += sm[i];
  return t;
}

__global__ void __launch_bounds__(256) vc_fit_partial_kernel(const float* __restrict__ x_hat, const float* __restrict__ x_tgt,
                                                             int HW, double eps, int printed_form,
                                                             double* __restrict__ partial) {
  __shared__ double sm[8];
  const float* xh = x_hat + static_cast<int64_t>(blockIdx.x) * HW;
  const float* xt = x_tgt + static_cast<int64_t>(blockIdx.x) * HW;
  double s = 0.0;
  for (int i = threadIdx.x; i < HW; i += blockDim.x) s += static_cast<double>(xh[i]);
  const double mu = block_sum_f64(s, sm) / static_cast<double>(HW);
  double ab = 0.0, aa = 0.0, abw = 0.0, aaw = 0.0;
  for (int i = threadIdx.x; i < HW; i += blockDim.x) {
    const double t = static_cast<double>(xt[i]);
    const double a = static_cast<double>(xh[i]) - mu, b = t - mu;
    const double w = 1.0 / (t * t + eps);
    ab += a * b;
    aa += a * a;
    abw += printed_form ? a / t : a * b * w;
    aaw += a * a * w;
  }
  ab = block_sum_f64(ab, sm);
  aa = block_sum_f64(aa, sm);
  abw = block_sum_f64(abw, sm);
  aaw = block_sum_f64(aaw, sm);
  if (threadIdx.x == 0) {
    double* o = partial + static_cast<int64_t>(blockIdx.x) * 4;
    o[0] = ab;
    o[1] = aa;
    o[2] = abw;
    o[3] = aaw;
  }
}

__global__ void vc_fit_finish_kernel(const double* __restrict__ partial, int N, int C, float* __restrict__ K) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  double num = 0.0, den = 0.0;
  for (int n = 0; n < N; ++n) {
    const double* o = partial + (static_cast<int64_t>(n) * C + c) * 4;
    num += o[0] + o[2];
    den += o[1] + o[3];
  }
  K[c] = static_cast<float>(num / den);
}

// ----------------------------------------------------------------------------- TAP: similarity matrix and its normalisation
// Matrix steps of Algorithm 1 for one subsample of n samples (features x [n,d], timestamps t [n]):
//   xn = x / |x| (rows; a zero row stays zero)            tap_normalize_kernel, one CTA per row
//   S  = xn xn^T                                            batched_linear_kernel (the register-tiled f32 GEMM)
//   A  = alpha S + (1 - alpha) exp(-|t_k - t_h|), deg = row sums of A   tap_combine_kernel, one CTA per row
//   L  = deg_k^e A_kh deg_h^e                               tap_scale_kernel
// A is symmetric, so the row-sum and column-sum degrees of the paper coincide.
__global__ void __launch_bounds__(256) tap_normalize_kernel(const float* __restrict__ x, int d, float* __restrict__ xn) {
  __shared__ float sm[8];
  const float* row = x + static_cast<int64_t>(blockIdx.x) * d;
  float* out = xn + static_cast<int64_t>(blockIdx.x) * d;
  float s = 0.0f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) s = fmaf(row[i], row[i], s);
  const float norm = sqrtf(block_sum(s, sm));
  const float inv = norm > 0.0f ? 1.0f / norm : 0.0f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) out[i] = row[i] * inv;
}

__global__ void __launch_bounds__(256) tap_combine_kernel(float* __restrict__ A, const float* __restrict__ t, int n, float alpha,
                                                          float* __restrict__ deg) {
  __shared__ float sm[8];
  float* row = A + static_cast<int64_t>(blockIdx.x) * n;
  const float tk = t[blockIdx.x];
  float s = 0.0f;
  for (int h = threadIdx.x; h < n; h += blockDim.x) {
    const float a = alpha * row[h] + (1.0f - alpha) * expf(-fabsf(tk - t[h]));
    row[h] = a;
    s += a;
  }
  s = block_sum(s, sm);
  if (threadIdx.x == 0) deg[blockIdx.x] = s;
}

__global__ void __launch_bounds__(256) tap_scale_kernel(float* __restrict__ A, const float* __restrict__ deg, int n, float e) {
  float* row = A + static_cast<int64_t>(blockIdx.x) * n;
  const float dk = powf(deg[blockIdx.x], e);
  for (int h = threadIdx.x; h < n; h += blockDim.x) row[h] = dk * row[h] * powf(deg[h], e);
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

// Stochastic (ancestral) step with learned variance: the network's second output group v in [-1, 1] interpolates
// the log variance between beta' and the posterior variance; v comes from the conditional half under guidance.
__global__ void __launch_bounds__(256) cfg_ddpm_kernel(float* __restrict__ latent, const float* __restrict__ net,
                                                       const float* __restrict__ noise, int B, int C, int HW, int use_cfg,
                                                       float guidance, DdpmCoef k) {
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t per_sample = static_cast<int64_t>(C) * HW;
  if (idx >= B * per_sample) return;
  const int64_t b = idx / per_sample;
  const int64_t r = idx - b * per_sample;  // c*HW + i
  float eps = net[b * 2 * per_sample + r];
  const float v = net[b * 2 * per_sample + per_sample + r];
  if (use_cfg) {
    const float eu = net[(b + B) * 2 * per_sample + r];
    eps = eu + guidance * (eps - eu);
  }
  const float x = latent[idx];
  const float x0 = k.rs * x - k.rsm1 * eps;
  const float mean = k.c_x0 * x0 + k.c_xt * x;
  const float f = (v + 1.0f) * 0.5f;
  const float logvar = f * k.log_beta + (1.0f - f) * k.log_post;
  latent[idx] = k.nz != 0.0f ? mean + expf(0.5f * logvar) * noise[idx] : mean;  // the last step draws no noise
}

// ----------------------------------------------------------------------------- patch embedding
// x[m,:] = bf16(W_patch . patch(m) + b_patch + pos[t,:]); patch vector ordered (c, py, px).
// CTA = 32 token rows x 512 columns.  The weights come TRANSPOSED (wT[j][d], made once when the model is
// built), so a thread reads the PD weights of its two columns with coalesced 8-byte loads and keeps them
// in registers while it walks the rows; patch values are broadcast from shared memory; the bf16 stores of
// a warp are 128 contiguous bytes.
constexpr int EMB_ROWS = 32;
template <int PD>
__global__ void __launch_bounds__(256) embed_kernel(const float* __restrict__ latent, int latent_batch,
                                                    const float* __restrict__ wT, const float* __restrict__ bias,
                                                    const float* __restrict__ pos, __nv_bfloat16* __restrict__ x,
                                                    int64_t M, int D, int grid, int patch, int C) {
  __shared__ float sp[EMB_ROWS][PD];
  const int T = grid * grid, side = grid * patch, pp = patch * patch;
  const int64_t m0 = static_cast<int64_t>(blockIdx.x) * EMB_ROWS;
  for (int i = threadIdx.x; i < EMB_ROWS * PD; i += blockDim.x) {
    const int r = i / PD, j = i % PD;
    const int64_t m = m0 + r;
    float v = 0.0f;
    if (m < M) {
      const int b = static_cast<int>(m / T) % latent_batch, t = static_cast<int>(m % T);
      const int gy = t / grid, gx = t % grid;
      const int c = j / pp, py = (j / patch) % patch, px = j % patch;
      v = latent[((static_cast<int64_t>(b) * C + c) * side + gy * patch + py) * side + gx * patch + px];
    }
    sp[r][j] = v;
  }
  __syncthreads();
  const int d = (blockIdx.y * blockDim.x + threadIdx.x) * 2;
  if (d >= D) return;
  float2 w[PD];
#pragma unroll
  for (int j = 0; j < PD; ++j) w[j] = *reinterpret_cast<const float2*>(wT + static_cast<int64_t>(j) * D + d);
  const float2 bv = *reinterpret_cast<const float2*>(bias + d);
  int t = static_cast<int>(m0 % T);
  const int rows = M - m0 < EMB_ROWS ? static_cast<int>(M - m0) : EMB_ROWS;
  for (int r = 0; r < rows; ++r) {
    float a0 = bv.x, a1 = bv.y;
#pragma unroll
    for (int j = 0; j < PD; ++j) {
      const float pv = sp[r][j];
      a0 = fmaf(w[j].x, pv, a0);
      a1 = fmaf(w[j].y, pv, a1);
    }
    const float2 ps = *reinterpret_cast<const float2*>(pos + static_cast<int64_t>(t) * D + d);
    *reinterpret_cast<uint32_t*>(x + (m0 + r) * D + d) = pack_bf16x2(a0 + ps.x, a1 + ps.y);
    if (++t == T) t = 0;
  }
}

// ----------------------------------------------------------------------------- conditioning
// Sinusoidal timestep features feat[b, :] = [cos(t f_j), sin(t f_j)], f_j = 10000^(-j/half), evaluated in
// double so that arguments of hundreds of radians keep their phase.
__global__ void timestep_features_kernel(const float* __restrict__ t, float* __restrict__ feat, int B, int F) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * F) return;
  const int b = i / F, j = i % F, half = F / 2;
  const int jj = j < half ? j : j - half;
  const double arg = static_cast<double>(t[b]) * exp(-9.210340371976184 * static_cast<double>(jj) / static_cast<double>(half));
  feat[i] = static_cast<float>(j < half ? cos(arg) : sin(arg));
}

// out[b,n] = W[n,:] . f(in[b,:]) + bias[n] (+ table[y[b % y_period],n]), optionally passed through SiLU, and optionally
// SiLU(out) as a second output.  One CTA per 8 output features: the inputs of up to `bc` samples are copied
// into shared memory with cp.async (all copies in flight at once: the copy is one L2 latency, not one per
// loop trip), f is applied in place, then a warp keeps its weight row in registers and walks the samples.
constexpr int SL_MAXV = 16;  // float4 per lane: K <= 2048
__global__ void __launch_bounds__(256) small_linear_kernel(const float* __restrict__ in, const float* __restrict__ w,
                                                           const float* __restrict__ bias,
                                                           const float* __restrict__ table, const int32_t* __restrict__ y,
                                                           float* __restrict__ out, float* __restrict__ out_silu, int B,
                                                           int N, int K, int bc, int silu_input, int silu_output,
                                                           int y_period) {
  extern __shared__ float s_in[];  // [bc][K]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = blockIdx.x * (blockDim.x >> 5) + warp;
  float4 wv[SL_MAXV];
  if (n < N) {
#pragma unroll
    for (int j = 0; j < SL_MAXV; ++j) {
      const int k = lane * 4 + 128 * j;
      wv[j] = k < K ? *reinterpret_cast<const float4*>(w + static_cast<int64_t>(n) * K + k) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  const uint32_t s_base = smem_u32(s_in);
  for (int b0 = 0; b0 < B; b0 += bc) {
    const int nb = B - b0 < bc ? B - b0 : bc;
    __syncthreads();  // the previous group has been consumed
    for (int i = threadIdx.x * 4; i < nb * K; i += blockDim.x * 4)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s_base + i * 4), "l"(in + static_cast<int64_t>(b0) * K + i) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (silu_input) {  // own elements only: no barrier needed before
      for (int i = threadIdx.x * 4; i < nb * K; i += blockDim.x * 4) {
        float4 v = *reinterpret_cast<float4*>(s_in + i);
        v.x = silu_f(v.x); v.y = silu_f(v.y); v.z = silu_f(v.z); v.w = silu_f(v.w);
        *reinterpret_cast<float4*>(s_in + i) = v;
      }
    }
    __syncthreads();
    if (n < N) {
      for (int b = 0; b < nb; ++b) {
        float acc = 0.0f;
#pragma unroll
        for (int j = 0; j < SL_MAXV; ++j) {
          const int k = lane * 4 + 128 * j;
          if (k < K) {
            const float4 xv = *reinterpret_cast<const float4*>(s_in + b * K + k);
            acc = fmaf(wv[j].x, xv.x, acc);
            acc = fmaf(wv[j].y, xv.y, acc);
            acc = fmaf(wv[j].z, xv.z, acc);
            acc = fmaf(wv[j].w, xv.w, acc);
          }
        }
        acc = warp_sum(acc);
        if (lane == 0) {
          const int64_t o = static_cast<int64_t>(b0 + b) * N + n;
          float v = acc + bias[n];
          if (table) v += table[static_cast<int64_t>(y[(b0 + b) % y_period]) * N + n];
          if (silu_output) v = silu_f(v);
          out[o] = v;
          if (out_silu) out_silu[o] = silu_f(v);
        }
      }
    }
  }
}

// The same linear for many rows (the conditioning of a whole trajectory): a register-tiled f32 GEMM,
// out[r, n] = g(sum_k f(in[r, k]) W[n, k] + bias[n] (+ table[y[r % y_period], n])).  Tiles of 128 rows x 64 features
// x 16 k; each thread owns 8 x 4 outputs and sums over k in ascending order, so an output's value does not
// depend on how many rows the call has or where the row sits.
constexpr int BL_BM = 128, BL_BN = 64, BL_BK = 16;
__global__ void __launch_bounds__(256) batched_linear_kernel(const float* __restrict__ in, const float* __restrict__ w,
                                                             const float* __restrict__ bias, const float* __restrict__ table,
                                                             const int32_t* __restrict__ y, float* __restrict__ out,
                                                             float* __restrict__ out_silu, int R, int N, int K, int silu_input,
                                                             int silu_output, int y_period) {
  __shared__ __align__(16) float sA[2][BL_BK][BL_BM + 4];
  __shared__ __align__(16) float sW[2][BL_BK][BL_BN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int r0 = blockIdx.y * BL_BM, n0 = blockIdx.x * BL_BN;
  const int lr = tid >> 2, lk = (tid & 3) * 4;  // loader coordinates: row (or feature) within the tile, k offset
  float4 ra[2], rw;
  auto load = [&](int k0) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int r = r0 + lr + 64 * j;
      ra[j] = r < R ? *reinterpret_cast<const float4*>(in + static_cast<int64_t>(r) * K + k0 + lk) : make_float4(0.f, 0.f, 0.f, 0.f);
      if (silu_input) { ra[j].x = silu_f(ra[j].x); ra[j].y = silu_f(ra[j].y); ra[j].z = silu_f(ra[j].z); ra[j].w = silu_f(ra[j].w); }
    }
    const int n = n0 + lr;
    rw = n < N ? *reinterpret_cast<const float4*>(w + static_cast<int64_t>(n) * K + k0 + lk) : make_float4(0.f, 0.f, 0.f, 0.f);
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      sA[buf][lk + 0][lr + 64 * j] = ra[j].x;
      sA[buf][lk + 1][lr + 64 * j] = ra[j].y;
      sA[buf][lk + 2][lr + 64 * j] = ra[j].z;
      sA[buf][lk + 3][lr + 64 * j] = ra[j].w;
    }
    sW[buf][lk + 0][lr] = rw.x;
    sW[buf][lk + 1][lr] = rw.y;
    sW[buf][lk + 2][lr] = rw.z;
    sW[buf][lk + 3][lr] = rw.w;
  };
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
  load(0);
  stash(0);
  __syncthreads();
  const int nk = K / BL_BK;
  for (int kb = 0; kb < nk; ++kb) {
    const int buf = kb & 1;
    if (kb + 1 < nk) load((kb + 1) * BL_BK);
#pragma unroll
    for (int k = 0; k < BL_BK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&sA[buf][k][ty * 8]);
      const float4 a1 = *reinterpret_cast<const float4*>(&sA[buf][k][ty * 8 + 4]);
      const float4 b = *reinterpret_cast<const float4*>(&sW[buf][k][tx * 4]);
      const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    if (kb + 1 < nk) {
      stash(buf ^ 1);  // the other buffer was last read before the previous barrier
      __syncthreads();
    }
  }
  const int n = n0 + tx * 4;
  if (n >= N) return;
  const float4 bz = *reinterpret_cast<const float4*>(bias + n);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = r0 + ty * 8 + i;
    if (r >= R) break;
    float v[4] = {acc[i][0] + bz.x, acc[i][1] + bz.y, acc[i][2] + bz.z, acc[i][3] + bz.w};
    if (table) {
      const float4 tv = *reinterpret_cast<const float4*>(table + static_cast<int64_t>(y[r % y_period]) * N + n);
      v[0] += tv.x; v[1] += tv.y; v[2] += tv.z; v[3] += tv.w;
    }
    if (silu_output) {
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = silu_f(v[j]);
    }
    const int64_t o = static_cast<int64_t>(r) * N + n;
    *reinterpret_cast<float4*>(out + o) = make_float4(v[0], v[1], v[2], v[3]);
    if (out_silu) *reinterpret_cast<float4*>(out_silu + o) = make_float4(silu_f(v[0]), silu_f(v[1]), silu_f(v[2]), silu_f(v[3]));
  }
}

// ----------------------------------------------------------------------------- final layer
// LayerNorm + modulate, then the D -> OUT linear (OUT = 32 for patch 2, 8 channels) and un-patchify (output
// vector ordered (py, px, c)) into net[b, c, gy*p+py, gx*p+px].  Persistent CTAs keep the whole weight
// matrix in shared memory (laid out so that a lane's 16-byte reads are conflict-free); a warp normalises
// two token rows in registers, accumulates all OUT partial dot products per lane and finishes with a
// transposing butterfly (31 shuffles per row) after which lane o holds output o.
constexpr int FIN_OUT = 32;
template <int NV>
__global__ void __launch_bounds__(512, 1) final_kernel(const __nv_bfloat16* __restrict__ x, int64_t M, int D, int T,
                                                       float eps, const float* __restrict__ modf,
                                                       const float* __restrict__ w, const float* __restrict__ bias,
                                                       float* __restrict__ net, int grid, int patch) {
  extern __shared__ float4 s_w[];  // [FIN_OUT][NV][2][32] float4: (o, j, h, lane) = w[o][(lane + 32 j) * 8 + 4 h ..]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int nvec = D >> 3;
  for (int i = threadIdx.x; i < FIN_OUT * NV * 2 * 32; i += blockDim.x) {
    const int l = i & 31, h = (i >> 5) & 1, j = (i >> 6) % NV, o = i / (64 * NV);
    const int vi = l + 32 * j;
    s_w[i] = vi < nvec ? *reinterpret_cast<const float4*>(w + static_cast<int64_t>(o) * D + vi * 8 + 4 * h)
                       : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  __syncthreads();
  const int side = grid * patch, co = FIN_OUT / (patch * patch);
  for (int64_t row0 = (static_cast<int64_t>(blockIdx.x) * nwarps + warp) * 2; row0 < M;
       row0 += static_cast<int64_t>(gridDim.x) * nwarps * 2) {
    float y[2][NV][8];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int64_t row = row0 + r;
      const bool live = row < M;
      float sum = 0.0f;
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        const int vi = lane + 32 * j;
        if (live && vi < nvec) {
          Load8<__nv_bfloat16>::load(x + row * D + vi * 8, y[r][j]);
#pragma unroll
          for (int i = 0; i < 8; ++i) sum += y[r][j][i];
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) y[r][j][i] = 0.0f;
        }
      }
      const float mean = warp_sum(sum) / static_cast<float>(D);
      float ss = 0.0f;
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        if (lane + 32 * j < nvec) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float d = y[r][j][i] - mean;
            ss += d * d;
          }
        }
      }
      const float rstd = 1.0f / sqrtf(warp_sum(ss) / static_cast<float>(D) + eps);
      const int b = live ? static_cast<int>(row / T) : 0;
      const float* sh = modf + static_cast<int64_t>(b) * 2 * D;
      const float* sc = sh + D;
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        const int vi = lane + 32 * j;
        if (live && vi < nvec) {
          float shv[8], scv[8];
          Load8<float>::load(sh + vi * 8, shv);
          Load8<float>::load(sc + vi * 8, scv);
#pragma unroll
          for (int i = 0; i < 8; ++i) y[r][j][i] = (y[r][j][i] - mean) * rstd * (1.0f + scv[i]) + shv[i];
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) y[r][j][i] = 0.0f;
        }
      }
    }
    float p0[FIN_OUT], p1[FIN_OUT];
#pragma unroll
    for (int o = 0; o < FIN_OUT; ++o) {
      float a0 = 0.0f, a1 = 0.0f;
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        const float4 wl = s_w[((o * NV + j) * 2 + 0) * 32 + lane], wh = s_w[((o * NV + j) * 2 + 1) * 32 + lane];
        a0 = fmaf(wl.x, y[0][j][0], a0); a0 = fmaf(wl.y, y[0][j][1], a0); a0 = fmaf(wl.z, y[0][j][2], a0); a0 = fmaf(wl.w, y[0][j][3], a0);
        a0 = fmaf(wh.x, y[0][j][4], a0); a0 = fmaf(wh.y, y[0][j][5], a0); a0 = fmaf(wh.z, y[0][j][6], a0); a0 = fmaf(wh.w, y[0][j][7], a0);
        a1 = fmaf(wl.x, y[1][j][0], a1); a1 = fmaf(wl.y, y[1][j][1], a1); a1 = fmaf(wl.z, y[1][j][2], a1); a1 = fmaf(wl.w, y[1][j][3], a1);
        a1 = fmaf(wh.x, y[1][j][4], a1); a1 = fmaf(wh.y, y[1][j][5], a1); a1 = fmaf(wh.z, y[1][j][6], a1); a1 = fmaf(wh.w, y[1][j][7], a1);
      }
      p0[o] = a0;
      p1[o] = a1;
    }
    // transposing reduction: after the round with stride s, a lane with bit s set keeps the upper half
#pragma unroll
    for (int sft = 16; sft >= 1; sft >>= 1) {
      const bool up = (lane & sft) != 0;
#pragma unroll
      for (int i = 0; i < sft; ++i) {
        const float send0 = up ? p0[i] : p0[i + sft], keep0 = up ? p0[i + sft] : p0[i];
        const float send1 = up ? p1[i] : p1[i + sft], keep1 = up ? p1[i + sft] : p1[i];
        p0[i] = keep0 + __shfl_xor_sync(0xffffffffu, send0, sft);
        p1[i] = keep1 + __shfl_xor_sync(0xffffffffu, send1, sft);
      }
    }
    const int o = lane;  // lane o now holds output o of both rows
    const int c = o % co, px = (o / co) % patch, py = o / (co * patch);
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int64_t row = row0 + r;
      if (row < M) {
        const int b = static_cast<int>(row / T), t = static_cast<int>(row % T);
        const int gy = t / grid, gx = t % grid;
        net[((static_cast<int64_t>(b) * co + c) * side + gy * patch + py) * side + gx * patch + px] =
            (r == 0 ? p0[0] : p1[0]) + bias[o];
      }
    }
  }
}

// ----------------------------------------------------------------------------- final layer on the tensor cores
// The same operation for the widths the DiT blocks use (D a multiple of 128, 64 rows of one sample per CTA), with the
// D -> 32 linear on mma.sync (bf16 operands, f32 accumulation).  The row statistics are taken out of the product,
//   out[o] = rstd (S[o] - mean c1[o]) + c2[o] + bias[o],   S[o] = sum_k x_k W'[o,k],   W'[o,k] = (1 + scale_k) W[o,k],
//   c1[o] = sum_k W'[o,k],   c2[o] = sum_k shift_k W[o,k],
// so the bf16 activations go to the tensor cores as they are (exactly), and are read once.  W' is specific to the
// sample: the CTA forms it chunk by chunk in f32 and splits it into three bf16 parts, head + remainder + second
// remainder, which together hold all 24 bits of the f32 value; the three products are accumulated in f32, so the
// result has the accuracy of an f32 dot product (with two parts the 2^-18 truncation per term showed as 7e-6 of the
// output's rms).  The statistics (sum x, sum x^2 in f32) are
// accumulated from the same fragments on the ordinary pipes: mma.sync issues one m16n8k16 per 16 cycles and scheduler
// here, which is the kernel's limit, so nothing that the other pipes can do goes to it.  The CTA's 64 rows are one contiguous piece of memory; they are fetched whole, one bulk copy per
// row (whole rows keep DRAM pages streaming; column chunks of 256 bytes per row ran at a third of the bandwidth), into
// rows padded by 16 bytes.  Thirty-two warps: (row tile 0..3) x (k-step 0..7 of a 128-column chunk), so that each
// scheduler has eight warps to hide the mma and ldmatrix latencies; W' chunks are double-buffered; the partial sums of
// the eight k-step groups meet in shared memory at the end.
constexpr int FT_ROWS = 64, FT_KC = 128, FT_THREADS = 1024, FT_KG = 8, FT_PITCH = FT_KC * 2 + 16, FT_DMAX = 1152, FT_RED_PITCH = 68;
constexpr int FT_WBUF_BYTES = 3 * FIN_OUT * FT_PITCH;   // weight heads, remainders, second remainders of one chunk
constexpr int ft_smem_bytes(int D) {
  return (2 * D + FT_KG * FT_ROWS * 2 + 2 * FIN_OUT) * 4 + 16 + 2 * FT_WBUF_BYTES + FT_ROWS * (2 * D + 16);
}
static_assert(ft_smem_bytes(FT_DMAX) <= 227 * 1024, "final layer: shared memory");
constexpr int FT_DMIN = 5 * FT_KC;
static_assert(FT_ROWS * (2 * FT_DMIN + 16) >= FT_KG * FIN_OUT * FT_RED_PITCH * 4, "the partial products reuse the activation tile");

__device__ __forceinline__ void bulk_load_row(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(smem_dst)),
               "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// (z0, z1) -> packed bf16 heads and packed bf16 remainders
__device__ __forceinline__ void split_pair(float z0, float z1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(z0, z1);
  const __nv_bfloat162 l = __floats2bfloat162_rn(z0 - __low2float(h), z1 - __high2float(h));
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}
// (z0, z1) -> three packed bf16 pairs with hi + lo + lo2 == z (8 + 8 + 8 mantissa bits: all of an f32 value)
__device__ __forceinline__ void split_triple(float z0, float z1, uint32_t& hi, uint32_t& lo, uint32_t& lo2) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(z0, z1);
  const float r0 = z0 - __low2float(h), r1 = z1 - __high2float(h);
  const __nv_bfloat162 l = __floats2bfloat162_rn(r0, r1);
  const __nv_bfloat162 m = __floats2bfloat162_rn(r0 - __low2float(l), r1 - __high2float(l));
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
  lo2 = *reinterpret_cast<const uint32_t*>(&m);
}

__global__ void __launch_bounds__(FT_THREADS) final_tc_kernel(const __nv_bfloat16* __restrict__ x, int64_t M, int D, int T, float eps,
                                                              const float* __restrict__ modf, const float* __restrict__ w,
                                                              const float* __restrict__ bias, float* __restrict__ net, int grid, int patch,
                                                              int* status) {
  extern __shared__ __align__(16) uint8_t ft_smem[];
  float* s_mul = reinterpret_cast<float*>(ft_smem);   // [D] 1 + scale
  float* s_add = s_mul + D;                             // [D] shift
  float* s_stat = s_add + D;                            // [8 k-step groups][64 rows][2] sum x, sum x^2; then [64][2] mean, rstd
  float* s_c = s_stat + FT_KG * FT_ROWS * 2;                // [2][32] c1, c2
  uint64_t* bar = reinterpret_cast<uint64_t*>(s_c + 2 * FIN_OUT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar + 1);
  uint8_t* wring = reinterpret_cast<uint8_t*>(bar + 2);   // [2] W' chunks
  uint8_t* xt = wring + 2 * FT_WBUF_BYTES;                // [64][2 D + 16] activations; the partial products afterwards
  const int xp = 2 * D + 16;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int kg = warp & 7, rt = warp >> 3;             // k-step (group), row tile
  const int g = lane >> 2, t4 = lane & 3;
  const int64_t row0 = static_cast<int64_t>(blockIdx.x) * FT_ROWS;   // the CTA's rows lie inside one sample (T % 64 == 0)
  const int nc = D / FT_KC;
  const float* sh = modf + (row0 / T) * 2 * D;
  float2 mod_pre[2] = {make_float2(0.0f, 0.0f), make_float2(0.0f, 0.0f)};   // (shift, scale) of columns tid, tid + 1024: in flight during set-up
#pragma unroll
  for (int i = 0; i < 2; ++i)
    if (tid + i * FT_THREADS < D) mod_pre[i] = make_float2(sh[tid + i * FT_THREADS], sh[D + tid + i * FT_THREADS]);
  if (tid == 0) {
    mbar_init(bar, FT_ROWS);
    *abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  if (tid < FT_ROWS) {
    const int64_t row = row0 + tid < M ? row0 + tid : M - 1;   // rows past M repeat the last row (never stored)
    mbar_expect_tx(bar, static_cast<uint32_t>(2 * D));
    bulk_load_row(xt + tid * xp, x + row * D, static_cast<uint32_t>(2 * D), bar);
  }
#pragma unroll
  for (int i = 0; i < 2; ++i)
    if (tid + i * FT_THREADS < D) s_add[tid + i * FT_THREADS] = mod_pre[i].x, s_mul[tid + i * FT_THREADS] = 1.0f + mod_pre[i].y;
  // W' of a chunk: thread -> output wo (= its warp), four consecutive columns from wk
  const int wo = warp, wk = lane * 4;
  const float* wrow = w + static_cast<int64_t>(wo) * D + wk;
  float4 wa = *reinterpret_cast<const float4*>(wrow);
  float c1 = 0.0f, c2 = 0.0f;
  auto store_w = [&](int c) {   // wa holds W[wo, c * 128 + wk ..]
    const float4 ma = *reinterpret_cast<const float4*>(s_mul + c * FT_KC + wk), da = *reinterpret_cast<const float4*>(s_add + c * FT_KC + wk);
    const float z0 = wa.x * ma.x, z1 = wa.y * ma.y, z2 = wa.z * ma.z, z3 = wa.w * ma.w;
    c1 += (z0 + z1) + (z2 + z3);
    c2 = fmaf(wa.x, da.x, fmaf(wa.y, da.y, fmaf(wa.z, da.z, fmaf(wa.w, da.w, c2))));
    uint32_t h0, h1, l0, l1, m0, m1;
    split_triple(z0, z1, h0, l0, m0);
    split_triple(z2, z3, h1, l1, m1);
    uint8_t* dst = wring + (c & 1) * FT_WBUF_BYTES + wo * FT_PITCH + wk * 2;
    *reinterpret_cast<uint2*>(dst) = make_uint2(h0, h1);
    *reinterpret_cast<uint2*>(dst + FIN_OUT * FT_PITCH) = make_uint2(l0, l1);
    *reinterpret_cast<uint2*>(dst + 2 * FIN_OUT * FT_PITCH) = make_uint2(m0, m1);
  };
  __syncthreads();   // the modulation table is complete
  store_w(0);
  if (nc > 1) wa = *reinterpret_cast<const float4*>(wrow + FT_KC);
  float acc[4][4], s1a = 0.0f, s2a = 0.0f, s1b = 0.0f, s2b = 0.0f;
#pragma unroll
  for (int n = 0; n < 4; ++n)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[n][i] = 0.0f;
  const bool landed = mbar_wait(bar, 0, abort_flag, status);
  if (!__syncthreads_and(landed)) return;   // bounded wait ran out: the status word is set, the whole CTA leaves together
  const uint32_t xs = smem_u32(xt);
  for (int c = 0; c < nc; ++c) {
    if (c > 0) __syncthreads();   // W' of chunk c is there for everybody, and everybody is done with chunk c - 1
    const uint32_t whs = smem_u32(wring + (c & 1) * FT_WBUF_BYTES), wls = whs + FIN_OUT * FT_PITCH, wms = wls + FIN_OUT * FT_PITCH;
    {
      const int ks = kg;
      uint32_t a[4];   // a[0] row g, a[1] row g + 8 (columns 2 t4, + 1 of the k-step); a[2], a[3] the same rows, columns + 8
      ldmatrix_x4(xs + (16 * rt + (lane & 15)) * xp + (c * FT_KC + ks * 16 + (lane >> 4) * 8) * 2, a);
#pragma unroll
      for (int i = 0; i < 4; ++i) {   // statistics of rows g (even i) and g + 8 (odd i)
        float v0, v1;
        unpack_bf16x2(a[i], v0, v1);
        if (i & 1) {
          s1b += v0 + v1;
          s2b = fmaf(v0, v0, fmaf(v1, v1, s2b));
        } else {
          s1a += v0 + v1;
          s2a = fmaf(v0, v0, fmaf(v1, v1, s2a));
        }
      }
#pragma unroll
      for (int n2 = 0; n2 < 2; ++n2) {   // two output tiles of 8 per ldmatrix
        const uint32_t off = (n2 * 16 + (lane & 7) + ((lane >> 4) << 3)) * FT_PITCH + (ks * 16 + ((lane >> 3) & 1) * 8) * 2;
        uint32_t bh[4], bl[4], bm[4];
        ldmatrix_x4(whs + off, bh);
        ldmatrix_x4(wls + off, bl);
        ldmatrix_x4(wms + off, bm);
        mma_bf16_16816(acc[2 * n2], a, bm[0], bm[1]);   // smallest parts first
        mma_bf16_16816(acc[2 * n2 + 1], a, bm[2], bm[3]);
        mma_bf16_16816(acc[2 * n2], a, bl[0], bl[1]);
        mma_bf16_16816(acc[2 * n2 + 1], a, bl[2], bl[3]);
        mma_bf16_16816(acc[2 * n2], a, bh[0], bh[1]);
        mma_bf16_16816(acc[2 * n2 + 1], a, bh[2], bh[3]);
      }
    }
    if (c + 1 < nc) {   // while the tensor pipe works through this chunk: W' of the next one, into the buffer of chunk c - 1
      store_w(c + 1);
      if (c + 2 < nc) wa = *reinterpret_cast<const float4*>(wrow + (c + 2) * FT_KC);
    }
  }
  __syncthreads();   // the activation tile is free: it now holds the partial products [8 k-step groups][32 outputs][64 rows, padded]
  float* red = reinterpret_cast<float*>(xt);
  {
    float* mine = red + (static_cast<size_t>(kg) * FIN_OUT + 2 * t4) * FT_RED_PITCH + 16 * rt + g;
#pragma unroll
    for (int n = 0; n < 4; ++n) {   // acc[n][0..1]: row g, outputs 8 n + 2 t4, + 1; acc[n][2..3]: row g + 8
      mine[(8 * n) * FT_RED_PITCH] = acc[n][0];
      mine[(8 * n + 1) * FT_RED_PITCH] = acc[n][1];
      mine[(8 * n) * FT_RED_PITCH + 8] = acc[n][2];
      mine[(8 * n + 1) * FT_RED_PITCH + 8] = acc[n][3];
    }
    float* st = s_stat + (kg * FT_ROWS + 16 * rt + g) * 2;
#pragma unroll
    for (int o = 1; o < 4; o <<= 1) {   // the four lanes of a row
      s1a += __shfl_xor_sync(0xffffffffu, s1a, o);
      s2a += __shfl_xor_sync(0xffffffffu, s2a, o);
      s1b += __shfl_xor_sync(0xffffffffu, s1b, o);
      s2b += __shfl_xor_sync(0xffffffffu, s2b, o);
    }
    if (t4 == 0) st[0] = s1a, st[1] = s2a, st[16] = s1b, st[17] = s2b;
    c1 = warp_sum(c1);
    c2 = warp_sum(c2);
    if (lane == 0) s_c[wo] = c1, s_c[FIN_OUT + wo] = c2;
  }
  __syncthreads();
  float mean = 0.0f, rstd = 0.0f;
  if (tid < FT_ROWS) {
    float s1 = 0.0f, s2 = 0.0f;
#pragma unroll
    for (int k = 0; k < FT_KG; ++k) s1 += s_stat[(k * FT_ROWS + tid) * 2], s2 += s_stat[(k * FT_ROWS + tid) * 2 + 1];
    mean = s1 / static_cast<float>(D);
    rstd = 1.0f / sqrtf(fmaxf(s2 / static_cast<float>(D) - mean * mean, 0.0f) + eps);
  }
  __syncthreads();   // every partial sum of the statistics has been read
  if (tid < FT_ROWS) s_stat[2 * tid] = mean, s_stat[2 * tid + 1] = rstd;
  __syncthreads();
  // un-patchify: output o = (py, px, c); consecutive threads take consecutive tokens of one output
  const int side = grid * patch, co = FIN_OUT / (patch * patch);
  const int b = static_cast<int>(row0 / T), tok0 = static_cast<int>(row0 % T);
  for (int i = tid; i < FT_ROWS * FIN_OUT; i += FT_THREADS) {
    const int o = i / FT_ROWS, r = i % FT_ROWS;
    if (row0 + r >= M) continue;
    float sum = 0.0f;
#pragma unroll
    for (int k = 0; k < FT_KG; ++k) sum += red[(k * FIN_OUT + o) * FT_RED_PITCH + r];
    const float v = fmaf(s_stat[2 * r + 1], sum - s_stat[2 * r] * s_c[o], s_c[FIN_OUT + o]) + bias[o];
    const int t = tok0 + r, gy = t / grid, gx = t % grid;
    const int cc = o % co, px = (o / co) % patch, py = o / (co * patch);
    net[((static_cast<int64_t>(b) * co + cc) * side + gy * patch + py) * side + gx * patch + px] = v;
  }
}

// ----------------------------------------------------------------------------- patch embedding on the tensor cores
// The same operation for a patch vector of 16 values (4 latent channels, 2 x 2 patches): the reduction is exactly one
// k-step of mma.sync m16n8k16.  f32 operands are split into a bf16 head and remainder and three products are
// accumulated (hi.hi + lo.hi + hi.lo; what is dropped is below 2^-17 relative).  The weights are split and laid out in
// fragment order once, when the model is built: one 16-byte load per lane and column tile.  A CTA owns the same 16
// token positions of four samples (four 16-row tiles) and half of the columns, so a position row and a weight fragment
// are fetched once for four tiles (position rows in f32 are twice the bytes of the output).  Every thread builds the
// A fragments straight from the latent (a fragment pair is two horizontally adjacent latent values); a warp walks its
// column tiles three at a time, with all of a batch's loads (weights, bias, position rows) issued before the first
// use, adds bias and position, and stages bf16 pairs in shared memory; the rows then leave by bulk copies.
constexpr int ET_TOK = 16, ET_SAMPLES = 4, ET_ROWS = ET_TOK * ET_SAMPLES, ET_THREADS = 256, ET_SPLIT = 2, ET_BATCH = 3;

__device__ __forceinline__ void bulk_store_row(void* gdst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(reinterpret_cast<uint64_t>(gdst)),
               "r"(smem_u32(smem_src)), "r"(bytes)
               : "memory");
}

// frag[n][lane] = (head(j, j+1), remainder(j, j+1), head(j+8, j+9), remainder(j+8, j+9)) of W[d = 8 n + lane / 4][.],
// j = 2 (lane % 4): the B fragment of column tile n, from the transposed weights wT[j][d].
__global__ void embed_fragments_kernel(const float* __restrict__ wT, int D, uint4* __restrict__ frag) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (D >> 3) * 32) return;
  const int n = i >> 5, lane = i & 31, g = lane >> 2, t4 = lane & 3;
  const float* wc = wT + 8 * n + g;
  uint4 f;
  split_pair(wc[static_cast<int64_t>(2 * t4) * D], wc[static_cast<int64_t>(2 * t4 + 1) * D], f.x, f.y);
  split_pair(wc[static_cast<int64_t>(2 * t4 + 8) * D], wc[static_cast<int64_t>(2 * t4 + 9) * D], f.z, f.w);
  frag[i] = f;
}

__global__ void __launch_bounds__(ET_THREADS, 2) embed_tc_kernel(const float* __restrict__ latent, int latent_batch,
                                                                 const uint4* __restrict__ frag, const float* __restrict__ bias,
                                                                 const float* __restrict__ pos, __nv_bfloat16* __restrict__ x, int B,
                                                                 int D, int grid, int C) {
  extern __shared__ __align__(16) uint8_t et_smem[];   // [4 samples][16 tokens][D + 16 bytes]: the CTA's half of the bf16 rows, padded
  const int dh = D / ET_SPLIT, xp = 2 * dh + 16;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t4 = lane & 3;
  const int T = grid * grid, side = 2 * grid;
  const int t0 = blockIdx.x * ET_TOK, b0 = blockIdx.y * ET_SAMPLES, d0 = blockIdx.z * dh;
  // A fragments: value pair (j, j + 1) of a token with j = 2 t4 (+ 8) is latent[b, c, 2 gy + py, 2 gx .. 2 gx + 1],
  // c = t4 / 2 (+ 2), py = t4 % 2.  Fragment registers of a 16-row tile: 0 row g, 1 row g + 8 (columns 2 t4, + 1);
  // 2, 3 the same rows, columns + 8.
  uint32_t ah[ET_SAMPLES][4], al[ET_SAMPLES][4];
  {
    const int64_t plane = static_cast<int64_t>(side) * side;
    int off[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int t = t0 + g + 8 * i, gy = t / grid, gx = t % grid;
      off[i] = (2 * gy + (t4 & 1)) * side + 2 * gx;
    }
    float2 pv[ET_SAMPLES][4];
#pragma unroll
    for (int sidx = 0; sidx < ET_SAMPLES; ++sidx) {
      const float* base = latent + (static_cast<int64_t>((b0 + sidx) % latent_batch) * C + (t4 >> 1)) * plane;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        pv[sidx][i] = *reinterpret_cast<const float2*>(base + off[i]);
        pv[sidx][2 + i] = *reinterpret_cast<const float2*>(base + 2 * plane + off[i]);
      }
    }
#pragma unroll
    for (int sidx = 0; sidx < ET_SAMPLES; ++sidx)
#pragma unroll
      for (int r = 0; r < 4; ++r) split_pair(pv[sidx][r].x, pv[sidx][r].y, ah[sidx][r], al[sidx][r]);
  }
  const float* prow0 = pos + static_cast<int64_t>(t0 + g) * D + 2 * t4;   // position rows of tokens g and g + 8, at column 2 t4
  const float* prow1 = prow0 + static_cast<int64_t>(8) * D;
  const int n_end = (d0 + dh) >> 3;
  for (int nb = (d0 >> 3) + warp; nb < n_end; nb += ET_BATCH * (ET_THREADS / 32)) {
    uint4 f[ET_BATCH];
    float2 bv[ET_BATCH], pa[ET_BATCH], pb[ET_BATCH];
#pragma unroll
    for (int u = 0; u < ET_BATCH; ++u) {
      const int n = nb + u * (ET_THREADS / 32);
      if (n < n_end) {
        f[u] = frag[n * 32 + lane];
        bv[u] = *reinterpret_cast<const float2*>(bias + 8 * n + 2 * t4);
        pa[u] = *reinterpret_cast<const float2*>(prow0 + 8 * n);
        pb[u] = *reinterpret_cast<const float2*>(prow1 + 8 * n);
      }
    }
#pragma unroll
    for (int u = 0; u < ET_BATCH; ++u) {
      const int n = nb + u * (ET_THREADS / 32);
      if (n < n_end) {
        const int col = (8 * n - d0 + 2 * t4) * 2;   // byte offset inside a staged row
#pragma unroll
        for (int sidx = 0; sidx < ET_SAMPLES; ++sidx) {
          float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
          mma_bf16_16816(acc, ah[sidx], f[u].x, f[u].z);
          mma_bf16_16816(acc, al[sidx], f[u].x, f[u].z);
          mma_bf16_16816(acc, ah[sidx], f[u].y, f[u].w);
          *reinterpret_cast<uint32_t*>(et_smem + (ET_TOK * sidx + g) * xp + col) = pack_bf16x2((acc[0] + bv[u].x) + pa[u].x, (acc[1] + bv[u].y) + pa[u].y);
          *reinterpret_cast<uint32_t*>(et_smem + (ET_TOK * sidx + g + 8) * xp + col) = pack_bf16x2((acc[2] + bv[u].x) + pb[u].x, (acc[3] + bv[u].y) + pb[u].y);
        }
      }
    }
  }
  fence_async_smem();   // the staged rows are read by the bulk copies
  __syncthreads();
  if (tid < ET_ROWS && b0 + tid / ET_TOK < B) {   // the last group of samples may be short (its extra tiles repeat valid latents)
    const int64_t m = static_cast<int64_t>(b0 + tid / ET_TOK) * T + t0 + tid % ET_TOK;
    bulk_store_row(x + m * D + d0, et_smem + tid * xp, static_cast<uint32_t>(2 * dh));
    tma_store_commit();
    tma_store_wait_all();   // shared memory must outlive the copy
  }
}

}  // namespace

// ================================================================================ launchers
int32_t launch_embed_fragments(qdit_ctx* ctx, const float* wT, int D, void* frag) {
  embed_fragments_kernel<<<(D / 8 * 32 + 255) / 256, 256, 0, ctx->stream>>>(wT, D, static_cast<uint4*>(frag));
  return qdit_after_launch(ctx, "embed_fragments_kernel");
}

int32_t launch_embed(qdit_ctx* ctx, const float* latent, int latent_batch, const float* wT, const void* frag, const float* bias,
                     const float* pos, void* x, int64_t M, int D, int grid, int patch, int C) {
  const int pd = C * patch * patch;
  dim3 g(static_cast<unsigned>((M + EMB_ROWS - 1) / EMB_ROWS), static_cast<unsigned>((D / 2 + 255) / 256));
  __nv_bfloat16* xb = static_cast<__nv_bfloat16*>(x);
  ProfScope prof(ctx, QDIT_PROF_OTHER, static_cast<double>(M) * D * 2.0);
  const int64_t T = static_cast<int64_t>(grid) * grid;
  if (frag && pd == 16 && patch == 2 && D % (16 * ET_SPLIT) == 0 && D <= 2048 && T % ET_TOK == 0 && M % T == 0 &&
      reinterpret_cast<uintptr_t>(x) % 16 == 0 && reinterpret_cast<uintptr_t>(latent) % 8 == 0) {   // the tensor-core form
    const int smem = ET_ROWS * (D + 16);
    QDIT_TRY(qdit_allow_smem(ctx, embed_tc_kernel, ET_ROWS * (2048 + 16)));
    const int B = static_cast<int>(M / T);
    embed_tc_kernel<<<dim3(static_cast<unsigned>(T / ET_TOK), static_cast<unsigned>((B + ET_SAMPLES - 1) / ET_SAMPLES), ET_SPLIT), ET_THREADS, smem,
                      ctx->stream>>>(latent, latent_batch, static_cast<const uint4*>(frag), bias, pos, xb, B, D, grid, C);
    return qdit_after_launch(ctx, "embed_tc_kernel");
  }
  switch (pd) {
    case 16: embed_kernel<16><<<g, 256, 0, ctx->stream>>>(latent, latent_batch, wT, bias, pos, xb, M, D, grid, patch, C); break;
    case 4: embed_kernel<4><<<g, 256, 0, ctx->stream>>>(latent, latent_batch, wT, bias, pos, xb, M, D, grid, patch, C); break;
    case 64: embed_kernel<64><<<g, 256, 0, ctx->stream>>>(latent, latent_batch, wT, bias, pos, xb, M, D, grid, patch, C); break;
    default: return qdit_fail(ctx, QDIT_ERR_SHAPE, "patch vector length %d not supported (4, 16 or 64)", pd);
  }
  return qdit_after_launch(ctx, "embed_kernel");
}

int32_t launch_small_linear(qdit_ctx* ctx, const float* in, const float* w, const float* bias, const float* table,
                            const int32_t* y, float* out, float* out_silu, int B, int N, int K, int silu_input,
                            int silu_output, int y_period) {
  if (K % 4 != 0 || K > 128 * SL_MAXV) return qdit_fail(ctx, QDIT_ERR_SHAPE, "small linear needs K %% 4 == 0 and K <= %d", 128 * SL_MAXV);
  if (!aligned16(in) || !aligned16(w)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "small linear operands must be 16-byte aligned");
  const int smem_budget = 160 * 1024;
  int bc = smem_budget / (K * static_cast<int>(sizeof(float)));
  if (bc > B) bc = B;
  if (bc < 1) bc = 1;
  const size_t smem = static_cast<size_t>(bc) * K * sizeof(float);
  QDIT_TRY(qdit_allow_smem(ctx, small_linear_kernel, smem_budget));
  ProfScope prof(ctx, QDIT_PROF_OTHER, static_cast<double>(N) * K * 4.0);
  small_linear_kernel<<<static_cast<unsigned>((N + 7) / 8), 256, smem, ctx->stream>>>(in, w, bias, table, y, out, out_silu, B, N,
                                                                                    K, bc, silu_input, silu_output,
                                                                                    y_period > 0 ? y_period : B);
  return qdit_after_launch(ctx, "small_linear_kernel");
}

int32_t launch_batched_linear(qdit_ctx* ctx, const float* in, const float* w, const float* bias, const float* table,
                              const int32_t* y, float* out, float* out_silu, int R, int N, int K, int silu_input,
                              int silu_output, int y_period) {
  if (K % BL_BK != 0 || N % 4 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "batched linear needs K %% 16 == 0 and N %% 4 == 0");
  if (!aligned16(in) || !aligned16(w) || !aligned16(bias) || !aligned16(out) || (table && !aligned16(table)) ||
      (out_silu && !aligned16(out_silu)))
    return qdit_fail(ctx, QDIT_ERR_ALIGN, "batched linear operands must be 16-byte aligned");
  if (R <= 0) return QDIT_OK;
  ProfScope prof(ctx, QDIT_PROF_OTHER, static_cast<double>(N) * K * 4.0);
  dim3 grid(static_cast<unsigned>((N + BL_BN - 1) / BL_BN), static_cast<unsigned>((R + BL_BM - 1) / BL_BM));
  batched_linear_kernel<<<grid, 256, 0, ctx->stream>>>(in, w, bias, table, y, out, out_silu, R, N, K, silu_input, silu_output,
                                                       y_period > 0 ? y_period : R);
  return qdit_after_launch(ctx, "batched_linear_kernel");
}

int32_t launch_timestep_features(qdit_ctx* ctx, const float* t, float* feat, int B, int F) {
  timestep_features_kernel<<<(B * F + 255) / 256, 256, 0, ctx->stream>>>(t, feat, B, F);
  return qdit_after_launch(ctx, "timestep_features_kernel");
}

// h[b,:] = SiLU(W1 . sinusoid(t_b) + b1); feat: scratch [B, F]
int32_t launch_cond1(qdit_ctx* ctx, const float* t, const float* w1, const float* b1, float* feat, float* h, int B, int D,
                     int F) {
  QDIT_TRY(launch_timestep_features(ctx, t, feat, B, F));
  return launch_small_linear(ctx, feat, w1, b1, nullptr, nullptr, h, nullptr, B, D, F, 0, 1, 0);
}

int32_t launch_final(qdit_ctx* ctx, const void* x, int64_t M, int D, int T, float eps, const float* modf,
                     const float* w, const float* bias, float* net, int grid, int patch, int OUT) {
  if (OUT != FIN_OUT) return qdit_fail(ctx, QDIT_ERR_SHAPE, "final layer width %d not supported (needs patch*patch*2*channels = %d)", OUT, FIN_OUT);
  const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
  if (D % FT_KC == 0 && D >= FT_DMIN && D <= FT_DMAX && T % FT_ROWS == 0 && reinterpret_cast<uintptr_t>(x) % 16 == 0) {   // the tensor-core form
    QDIT_TRY(qdit_allow_smem(ctx, final_tc_kernel, ft_smem_bytes(FT_DMAX)));
    ProfScope prof(ctx, QDIT_PROF_OTHER, static_cast<double>(M) * D * 2.0);
    final_tc_kernel<<<static_cast<unsigned>((M + FT_ROWS - 1) / FT_ROWS), FT_THREADS, ft_smem_bytes(D), ctx->stream>>>(
        xb, M, D, T, eps, modf, w, bias, net, grid, patch, ctx->d_status);
    return qdit_after_launch(ctx, "final_tc_kernel");
  }
  const int nv = (D / 8 + 31) / 32;
  const size_t smem = static_cast<size_t>(FIN_OUT) * nv * 2 * 32 * sizeof(float4);
  int64_t want = (M + 31) / 32;
  const unsigned g = static_cast<unsigned>(want < ctx->num_sms ? want : ctx->num_sms);
#define QDIT_FINAL_CASE(NV)                                                                                             \
  case NV: {                                                                                                            \
    QDIT_TRY(qdit_allow_smem(ctx, final_kernel<NV>, FIN_OUT * NV * 2 * 32 * static_cast<int>(sizeof(float4))));          \
    final_kernel<NV><<<g, 512, smem, ctx->stream>>>(xb, M, D, T, eps, modf, w, bias, net, grid, patch);                 \
  } break;
  ProfScope prof(ctx, QDIT_PROF_OTHER, static_cast<double>(M) * D * 2.0);
  switch (nv) {
    QDIT_FINAL_CASE(1) QDIT_FINAL_CASE(2) QDIT_FINAL_CASE(3) QDIT_FINAL_CASE(4) QDIT_FINAL_CASE(5) QDIT_FINAL_CASE(6)
    default: return qdit_fail(ctx, QDIT_ERR_SHAPE, "final layer supports hidden <= 1536");
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

int32_t launch_cfg_ddpm(qdit_ctx* ctx, float* latent, const float* net, const float* noise, int B, int C, int HW,
                        int use_cfg, float guidance, const DdpmCoef& k) {
  const int64_t n = static_cast<int64_t>(B) * C * HW;
  cfg_ddpm_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, ctx->stream>>>(latent, net, noise, B, C, HW, use_cfg,
                                                                                  guidance, k);
  return qdit_after_launch(ctx, "cfg_ddpm_kernel");
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
  ProfScope prof(ctx, QDIT_PROF_CACHE_REUSE, static_cast<double>(c->M) * c->D * 2.0 * (2.0 * c->blocks + 2.0));
  // rows per thread: 4 (else 2) when samples are made of whole groups of that many rows and there is work for every SM,
  // else 1: the gate vectors, as many bytes from L2 as the cache is from HBM with one row per thread, are then read
  // once per group of rows (0.71 / 0.81 / 0.95 of the measured copy bandwidth with 1 / 2 / 4 rows)
  constexpr int R = 2;
  const bool wide = c->M % R == 0 && T % R == 0 && c->M * (c->D / 8) >= static_cast<int64_t>(R) * 256 * 4 * ctx->num_sms;
  const bool wide4 = c->M % 4 == 0 && T % 4 == 0 && c->M * (c->D / 8) >= static_cast<int64_t>(4) * 256 * 4 * ctx->num_sms;
  if (wide4) {
    const int64_t n = (c->M / 4) * (c->D / 8);
    cache_reuse_all_kernel<4><<<static_cast<unsigned>((n + 255) / 256), 256, 0, ctx->stream>>>(
        static_cast<__nv_bfloat16*>(x), c->data, mod_all, ld_mod, c->M, static_cast<int>(c->D), T, c->blocks);
  } else if (wide) {
    const int64_t n = (c->M / R) * (c->D / 8);
    cache_reuse_all_kernel<R><<<static_cast<unsigned>((n + 255) / 256), 256, 0, ctx->stream>>>(
        static_cast<__nv_bfloat16*>(x), c->data, mod_all, ld_mod, c->M, static_cast<int>(c->D), T, c->blocks);
  } else {
    const int64_t n = c->M * (c->D / 8);
    cache_reuse_all_kernel<1><<<static_cast<unsigned>((n + 255) / 256), 256, 0, ctx->stream>>>(
        static_cast<__nv_bfloat16*>(x), c->data, mod_all, ld_mod, c->M, static_cast<int>(c->D), T, c->blocks);
  }
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

int32_t qdit_tap_laplacian(qdit_ctx* ctx, const float* x, const float* t, int n, int d, float alpha, float exponent,
                           float* workspace, float* L) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (n <= 0 || d <= 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "n and d must be positive");
  if (n % 4 != 0 || d % 16 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "n must be a multiple of 4 and d a multiple of 16");
  if (!x || !t || !workspace || !L) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  if (!(alpha >= 0.0f && alpha <= 1.0f)) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "alpha must lie in [0, 1]");
  if (!aligned16(x) || !aligned16(workspace) || !aligned16(L)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "x, workspace and L must be 16-byte aligned");
  float* xn = workspace;                               // [n, d]
  float* zero = workspace + static_cast<int64_t>(n) * d;  // [n] zeros (bias of the product)
  float* deg = zero + n;                               // [n]
  QDIT_CUDA_CHECK(ctx, cudaMemsetAsync(zero, 0, static_cast<size_t>(n) * sizeof(float), ctx->stream));
  tap_normalize_kernel<<<static_cast<unsigned>(n), 256, 0, ctx->stream>>>(x, d, xn);
  QDIT_TRY(qdit_after_launch(ctx, "tap_normalize_kernel"));
  QDIT_TRY(launch_batched_linear(ctx, xn, xn, zero, nullptr, nullptr, L, nullptr, n, n, d, 0, 0, 0));
  tap_combine_kernel<<<static_cast<unsigned>(n), 256, 0, ctx->stream>>>(L, t, n, alpha, deg);
  QDIT_TRY(qdit_after_launch(ctx, "tap_combine_kernel"));
  tap_scale_kernel<<<static_cast<unsigned>(n), 256, 0, ctx->stream>>>(L, deg, n, exponent);
  return qdit_after_launch(ctx, "tap_scale_kernel");
}

int32_t qdit_vc_fit(qdit_ctx* ctx, const float* x_hat, const float* x_target, int N, int C, int HW, float eps, int form,
                    double* workspace, float* K) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (N <= 0 || C <= 0 || HW <= 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "N, C and HW must be positive");
  if (form != QDIT_VC_FIT_DERIVED && form != QDIT_VC_FIT_PRINTED) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "unknown fit form %d", form);
  if (!x_hat || !x_target || !workspace || !K) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  if (reinterpret_cast<uintptr_t>(workspace) & 7u) return qdit_fail(ctx, QDIT_ERR_ALIGN, "workspace must be 8-byte aligned");
  if (static_cast<int64_t>(N) * C > 0x7fffffff) return qdit_fail(ctx, QDIT_ERR_SHAPE, "N * C too large");
  vc_fit_partial_kernel<<<static_cast<unsigned>(N) * C, 256, 0, ctx->stream>>>(x_hat, x_target, HW, static_cast<double>(eps),
                                                                              form == QDIT_VC_FIT_PRINTED ? 1 : 0, workspace);
  QDIT_TRY(qdit_after_launch(ctx, "vc_fit_partial_kernel"));
  vc_fit_finish_kernel<<<(C + 63) / 64, 64, 0, ctx->stream>>>(workspace, N, C, K);
  return qdit_after_launch(ctx, "vc_fit_finish_kernel");
}

}  // extern "C"
