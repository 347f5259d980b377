// HBM-bound quantizer kernels: activation quantizer (Eq. 1), abs-max reduction for dynamic ranges,
// channel-wise weight quantizer, and LayerNorm + adaLN modulation with the fused activation quantizer.
#include "common.cuh"
#include "internal.h"

namespace {

using namespace qd;

// ----------------------------------------------------------------------------- activation quantizer
// One thread per 16 consecutive elements of a row (two 8-element halves); K % 8 == 0.
template <typename T>
__global__ void __launch_bounds__(256) act_quant_kernel(const T* __restrict__ x, int64_t M, int64_t K, int64_t ldx,
                                                        QuantArgs qa, uint8_t* __restrict__ q, int64_t ldq) {
  const int64_t chunks_per_row = (K + 15) / 16;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= M * chunks_per_row) return;
  const int64_t row = idx / chunks_per_row;
  const int64_t col = (idx - row * chunks_per_row) * 16;
  const float scale = qa.scale_dev ? __ldg(qa.scale_dev) : qa.scale;
  const float inv = __fdiv_rn(1.0f, scale);
  const T* src = x + row * ldx + col;
  uint8_t* dst = q + row * ldq + col;
  const bool second = col + 8 < K;
  float a[8], b[8];
  Load8<T>::load(src, a);
  if (second) Load8<T>::load(src + 8, b);
  const uint2 lo = quantize_pack8(a, inv, qa.zp, qa.qmin, qa.qmax);
  if (second) {
    const uint2 hi = quantize_pack8(b, inv, qa.zp, qa.qmin, qa.qmax);
    if ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
      *reinterpret_cast<uint4*>(dst) = make_uint4(lo.x, lo.y, hi.x, hi.y);
    } else {
      *reinterpret_cast<uint2*>(dst) = lo;
      *reinterpret_cast<uint2*>(dst + 8) = hi;
    }
  } else {
    *reinterpret_cast<uint2*>(dst) = lo;
  }
}

// Per-token dynamic quantizer: one warp per row finds max|x| of its row, s[m] = max / 127 (1 for a zero row),
// and writes the symmetric codes; the row is read twice (the second time from L1 / L2).
template <typename T>
__global__ void __launch_bounds__(256) act_quant_token_kernel(const T* __restrict__ x, int64_t M, int64_t K, int64_t ldx,
                                                              float* __restrict__ scales, uint8_t* __restrict__ q,
                                                              int64_t ldq) {
  const int lane = threadIdx.x & 31;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= M) return;
  const T* src = x + row * ldx;
  float m = 0.0f;
  for (int64_t k = lane * 8; k < K; k += 256) {
    float v[8];
    Load8<T>::load(src + k, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(v[i]));
  }
  m = warp_max(m);
  float s = __fdiv_rn(m, 127.0f);
  if (!(s > 0.0f)) s = 1.0f;
  const float inv = __fdiv_rn(1.0f, s);
  if (lane == 0) scales[row] = s;
  uint8_t* dst = q + row * ldq;
  for (int64_t k = lane * 8; k < K; k += 256) {
    float v[8];
    Load8<T>::load(src + k, v);
    *reinterpret_cast<uint2*>(dst + k) = quantize_pack8(v, inv, 0.0f, -127.0f, 127.0f);
  }
}

// ----------------------------------------------------------------------------- abs-max reduction
// Non-negative floats order like their bit patterns, so the global maximum is an atomicMax on uint32.
template <typename T>
__global__ void __launch_bounds__(256) absmax_kernel(const T* __restrict__ x, int64_t M, int64_t K, int64_t ldx,
                                                     float* __restrict__ absmax) {
  const int64_t vec_per_row = K / 8;
  const int64_t total = M * vec_per_row;
  float m = 0.0f;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total;
       idx += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t row = idx / vec_per_row;
    const int64_t col = (idx - row * vec_per_row) * 8;
    float v[8];
    Load8<T>::load(x + row * ldx + col, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(v[i]));
  }
  m = warp_max(m);
  __shared__ float smax[8];
  if ((threadIdx.x & 31) == 0) smax[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < (blockDim.x >> 5) ? smax[threadIdx.x] : 0.0f;
    m = warp_max(m);
    if (threadIdx.x == 0) atomicMax(reinterpret_cast<unsigned int*>(absmax), __float_as_uint(m));
  }
}

// scale[i] = absmax[i] / 127 (1 if the range is empty); optionally widens a running maximum.
__global__ void absmax_to_scale_kernel(const float* __restrict__ absmax, float* __restrict__ scale,
                                       float* __restrict__ running, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float a = absmax[i];
  if (running) running[i] = fmaxf(running[i], a);
  if (scale) {
    const float s = __fdiv_rn(a, 127.0f);
    scale[i] = s > 0.0f ? s : 1.0f;
  }
}

// ----------------------------------------------------------------------------- channel-wise weight quantizer
// One CTA per output row: abs-max over K, then codes and their sum.
__global__ void __launch_bounds__(256) weight_quant_kernel(const float* __restrict__ w, int64_t K,
                                                           int8_t* __restrict__ q, float* __restrict__ w_scale,
                                                           int32_t* __restrict__ w_colsum, float top) {
  const int64_t n = blockIdx.x;
  const float* row = w + n * K;
  __shared__ float sm[8];
  __shared__ int si[8];
  float m = 0.0f;
  for (int64_t k = threadIdx.x * 4; k < K; k += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(row + k);
    m = fmaxf(fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
  }
  m = warp_max(m);
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = m;
  __syncthreads();
  m = 0.0f;
  for (int i = 0; i < (blockDim.x >> 5); ++i) m = fmaxf(m, sm[i]);
  float s = __fdiv_rn(m, top);
  if (!(s > 0.0f)) s = 1.0f;
  const float inv = __fdiv_rn(1.0f, s);
  int sum = 0;
  for (int64_t k = threadIdx.x * 4; k < K; k += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(row + k);
    const int c0 = __float2int_rn(quantize_code(v.x, inv, 0.0f, -top, top));
    const int c1 = __float2int_rn(quantize_code(v.y, inv, 0.0f, -top, top));
    const int c2 = __float2int_rn(quantize_code(v.z, inv, 0.0f, -top, top));
    const int c3 = __float2int_rn(quantize_code(v.w, inv, 0.0f, -top, top));
    sum += c0 + c1 + c2 + c3;
    const uint32_t packed = (c0 & 0xFF) | ((c1 & 0xFF) << 8) | ((c2 & 0xFF) << 16) | (static_cast<uint32_t>(c3 & 0xFF) << 24);
    *reinterpret_cast<uint32_t*>(q + n * K + k) = packed;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if ((threadIdx.x & 31) == 0) si[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    int t = 0;
    for (int i = 0; i < (blockDim.x >> 5); ++i) t += si[i];
    w_scale[n] = s;
    w_colsum[n] = t;
  }
}

// ----------------------------------------------------------------------------- LayerNorm + modulate (+ quantize)
// A CTA owns a contiguous range of rows; its 8 warps take the rows in turn, one warp per row, the row in
// registers (NV vectors of 8 per lane), statistics two-pass in f32.  While a warp works on one row the next
// row's loads are already in flight.  The kernel is bound by instruction issue, so everything that does not
// depend on the row is done once per CTA: for the (at most two) samples its range touches, the per-column
// factors  mul = (1 + scale) / s_out  and  add = shift / s_out  (s_out = 1 unless the output is quantized) are
// staged in shared memory, laid out so that a lane's 16-byte reads are conflict-free.  Per element that leaves
// y / s_out = (x - mean) * (rstd * mul) + add: one multiply and one fused multiply-add.  A row of a third
// sample (only when a sample has fewer rows than a CTA's minimum range) computes its factors from global memory.
template <int NV>
__device__ __forceinline__ void ln_load_row(const __nv_bfloat16* __restrict__ xr, int nvec, int lane, uint4 (&raw)[NV]) {
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int vi = lane + 32 * j;
    if (vi < nvec) raw[j] = *reinterpret_cast<const uint4*>(xr + vi * 8);
  }
}

template <int NV>
__global__ void __launch_bounds__(256) ln_modulate_kernel(const __nv_bfloat16* __restrict__ x, int M, int D, int T,
                                                          float eps, const float* __restrict__ shift,
                                                          const float* __restrict__ scale, int64_t ld_mod,
                                                          void* __restrict__ out, int out_dtype, QuantArgs qa,
                                                          int rows_per_cta) {
  extern __shared__ float4 s_par[];  // [2 samples][mul, add][NV][2 halves][32 lanes]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int row_begin = blockIdx.x * rows_per_cta;
  const int row_end = row_begin + rows_per_cta < M ? row_begin + rows_per_cta : M;
  if (row_begin >= M) return;
  grid_dependency_wait();  // x and the modulation come from earlier kernels of the stream
  grid_dependency_release();
  const int nvec = D >> 3;
  int row = row_begin + warp;
  uint4 raw[NV], raw_next[NV];
  if (row < row_end) ln_load_row<NV>(x + static_cast<int64_t>(row) * D, nvec, lane, raw);
  float inv = 1.0f;
  if (out_dtype == QDIT_I8) inv = __fdiv_rn(1.0f, qa.scale_dev ? __ldg(qa.scale_dev) : qa.scale);
  const int b0 = row_begin / T;
  for (int s = 0; s < 2; ++s) {
    if (static_cast<int64_t>(b0 + s) * T >= row_end) break;
    const float* gs = shift + (b0 + s) * ld_mod;
    const float* gc = scale + (b0 + s) * ld_mod;
    for (int i = threadIdx.x; i < NV * 64; i += blockDim.x) {
      const int l = i & 31, h = (i >> 5) & 1, j = i >> 6;
      const int vi = l + 32 * j;
      if (vi < nvec) {
        const float4 c4 = *reinterpret_cast<const float4*>(gc + vi * 8 + 4 * h);
        const float4 h4 = *reinterpret_cast<const float4*>(gs + vi * 8 + 4 * h);
        s_par[(s * 2 + 0) * NV * 64 + i] = make_float4((1.0f + c4.x) * inv, (1.0f + c4.y) * inv, (1.0f + c4.z) * inv, (1.0f + c4.w) * inv);
        s_par[(s * 2 + 1) * NV * 64 + i] = make_float4(h4.x * inv, h4.y * inv, h4.z * inv, h4.w * inv);
      }
    }
  }
  __syncthreads();
  const float inv_d = 1.0f / static_cast<float>(D);
  const int64_t second = static_cast<int64_t>(b0 + 1) * T;  // first row of the second staged sample
  for (; row < row_end; row += nwarps) {
    const int next = row + nwarps;
    if (next < row_end) ln_load_row<NV>(x + static_cast<int64_t>(next) * D, nvec, lane, raw_next);
    float v[NV][8];
    float sum = 0.0f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      if (lane + 32 * j < nvec) {
        unpack_bf16x2(raw[j].x, v[j][0], v[j][1]);
        unpack_bf16x2(raw[j].y, v[j][2], v[j][3]);
        unpack_bf16x2(raw[j].z, v[j][4], v[j][5]);
        unpack_bf16x2(raw[j].w, v[j][6], v[j][7]);
#pragma unroll
        for (int i = 0; i < 8; ++i) sum += v[j][i];
      }
    }
    const float mean = warp_sum(sum) * inv_d;
    float ssq = 0.0f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      if (lane + 32 * j < nvec) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          v[j][i] -= mean;
          ssq = fmaf(v[j][i], v[j][i], ssq);
        }
      }
    }
    const float rstd = rsqrtf(warp_sum(ssq) * inv_d + eps);
    const int sidx = row < second ? 0 : (row - second < T ? 1 : 2);
    const float4* pm = s_par + (sidx * 2 + 0) * NV * 64 + lane;
    const float4* pa = s_par + (sidx * 2 + 1) * NV * 64 + lane;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      const int vi = lane + 32 * j;
      if (vi < nvec) {
        float mul[8], add[8], y[8];
        if (sidx < 2) {
          const float4 m0 = pm[j * 64], m1 = pm[j * 64 + 32], a0 = pa[j * 64], a1 = pa[j * 64 + 32];
          mul[0] = m0.x; mul[1] = m0.y; mul[2] = m0.z; mul[3] = m0.w; mul[4] = m1.x; mul[5] = m1.y; mul[6] = m1.z; mul[7] = m1.w;
          add[0] = a0.x; add[1] = a0.y; add[2] = a0.z; add[3] = a0.w; add[4] = a1.x; add[5] = a1.y; add[6] = a1.z; add[7] = a1.w;
        } else {
          const int b = row / T;
          Load8<float>::load(scale + b * ld_mod + vi * 8, mul);
          Load8<float>::load(shift + b * ld_mod + vi * 8, add);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            mul[i] = (1.0f + mul[i]) * inv;
            add[i] *= inv;
          }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) y[i] = fmaf(v[j][i], rstd * mul[i], add[i]);
        const int64_t o = static_cast<int64_t>(row) * D + vi * 8;
        if (out_dtype == QDIT_I8) {
          *reinterpret_cast<uint2*>(static_cast<uint8_t*>(out) + o) = quantize_pack8_scaled(y, qa.zp, qa.qmin, qa.qmax);
        } else if (out_dtype == QDIT_BF16) {
          *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(out) + o) = pack_bf16x8(y);
        } else {
          float* of = static_cast<float*>(out) + o;
          *reinterpret_cast<float4*>(of) = make_float4(y[0], y[1], y[2], y[3]);
          *reinterpret_cast<float4*>(of + 4) = make_float4(y[4], y[5], y[6], y[7]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < NV; ++j) raw[j] = raw_next[j];
  }
}

// The same operation for the shape the network's blocks use: 8-bit output and D = 128 * NV4.  A lane owns NV4
// groups of 4 consecutive columns (group lane + 32 j), so all 32 lanes are busy for every group (D = 1152 has 4.5
// groups of 8 per lane, which leaves half a warp idle for a fifth of the work), and the f32 arithmetic runs on
// the two-wide instructions (add / mul / fma on a pair of floats: same rounding per element as the scalar forms).
// Together that is less than half of the general kernel's instructions per row.  Values are identical to the
// general kernel's except for the summation order of the two statistics.  A CTA's row range must lie within two
// samples (rows_per_cta <= T).
__device__ __forceinline__ float2 f2(float a, float b) { return make_float2(a, b); }

template <int NV4>
__global__ void __launch_bounds__(256, 3) ln_modulate_q8_kernel(const __nv_bfloat16* __restrict__ x, int M, int T, float eps,
                                                                const float* __restrict__ shift,
                                                                const float* __restrict__ scale, int64_t ld_mod,
                                                                uint8_t* __restrict__ out, QuantArgs qa, int rows_per_cta) {
  constexpr int D = NV4 * 128, D4 = D / 4;
  extern __shared__ float4 s_par[];  // [2 samples][mul, add][D / 4]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row_begin = blockIdx.x * rows_per_cta;
  const int row_end = row_begin + rows_per_cta < M ? row_begin + rows_per_cta : M;
  if (row_begin >= M) return;
  grid_dependency_wait();  // x and the modulation come from earlier kernels of the stream
  grid_dependency_release();
  int row = row_begin + warp;
  uint2 raw[NV4], raw_next[NV4];
  if (row < row_end) {
    const uint2* xr = reinterpret_cast<const uint2*>(x + static_cast<int64_t>(row) * D) + lane;
#pragma unroll
    for (int j = 0; j < NV4; ++j) raw[j] = xr[32 * j];
  }
  const float inv = __fdiv_rn(1.0f, qa.scale_dev ? __ldg(qa.scale_dev) : qa.scale);
  const int b0 = row_begin / T;
  for (int s = 0; s < 2; ++s) {
    if (static_cast<int64_t>(b0 + s) * T >= row_end) break;
    const float4* gs = reinterpret_cast<const float4*>(shift + (b0 + s) * ld_mod);
    const float4* gc = reinterpret_cast<const float4*>(scale + (b0 + s) * ld_mod);
    for (int i = threadIdx.x; i < D4; i += 256) {
      const float4 c4 = gc[i], h4 = gs[i];
      s_par[(s * 2 + 0) * D4 + i] = make_float4((1.0f + c4.x) * inv, (1.0f + c4.y) * inv, (1.0f + c4.z) * inv, (1.0f + c4.w) * inv);
      s_par[(s * 2 + 1) * D4 + i] = make_float4(h4.x * inv, h4.y * inv, h4.z * inv, h4.w * inv);
    }
  }
  __syncthreads();
  constexpr float inv_d = 1.0f / static_cast<float>(D);
  const int second = (b0 + 1) * T;  // first row of the second staged sample
  const float lo_f = qa.qmin - qa.zp, hi_f = qa.qmax - qa.zp;
  const uint32_t z4 = (static_cast<uint32_t>(static_cast<int>(qa.zp)) & 0xFFu) * 0x01010101u;
  const float2 magic = f2(12582912.0f, 12582912.0f);
  for (; row < row_end; row += 8) {
    const int next = row + 8;
    if (next < row_end) {
      const uint2* xr = reinterpret_cast<const uint2*>(x + static_cast<int64_t>(next) * D) + lane;
#pragma unroll
      for (int j = 0; j < NV4; ++j) raw_next[j] = xr[32 * j];
    }
    float2 v[NV4][2];
    float2 s0 = f2(0.0f, 0.0f), s1 = f2(0.0f, 0.0f);
#pragma unroll
    for (int j = 0; j < NV4; ++j) {
      v[j][0] = f2(__uint_as_float(raw[j].x << 16), __uint_as_float(raw[j].x & 0xFFFF0000u));
      v[j][1] = f2(__uint_as_float(raw[j].y << 16), __uint_as_float(raw[j].y & 0xFFFF0000u));
      s0 = __fadd2_rn(s0, v[j][0]);
      s1 = __fadd2_rn(s1, v[j][1]);
    }
    const float mean = warp_sum((s0.x + s0.y) + (s1.x + s1.y)) * inv_d;
    const float2 nmean = f2(-mean, -mean);
    float2 q0 = f2(0.0f, 0.0f), q1 = f2(0.0f, 0.0f);
#pragma unroll
    for (int j = 0; j < NV4; ++j) {
      v[j][0] = __fadd2_rn(v[j][0], nmean);
      v[j][1] = __fadd2_rn(v[j][1], nmean);
      q0 = __ffma2_rn(v[j][0], v[j][0], q0);
      q1 = __ffma2_rn(v[j][1], v[j][1], q1);
    }
    const float rstd = rsqrtf(warp_sum((q0.x + q0.y) + (q1.x + q1.y)) * inv_d + eps);
    const float2 r2 = f2(rstd, rstd);
    const float4* pm = s_par + (row < second ? 0 : 2) * D4 + lane;
    const float4* pa = pm + D4;
    uint32_t* orow = reinterpret_cast<uint32_t*>(out + static_cast<int64_t>(row) * D) + lane;
#pragma unroll
    for (int j = 0; j < NV4; ++j) {
      const float4 m4 = pm[32 * j], a4 = pa[32 * j];
      // y / s_out = (x - mean) * (rstd * mul) + add, then Eq. 1's clip and round on the scaled value
      float2 y0 = __ffma2_rn(v[j][0], __fmul2_rn(r2, f2(m4.x, m4.y)), f2(a4.x, a4.y));
      float2 y1 = __ffma2_rn(v[j][1], __fmul2_rn(r2, f2(m4.z, m4.w)), f2(a4.z, a4.w));
      y0 = __fadd2_rn(f2(fminf(fmaxf(y0.x, lo_f), hi_f), fminf(fmaxf(y0.y, lo_f), hi_f)), magic);
      y1 = __fadd2_rn(f2(fminf(fmaxf(y1.x, lo_f), hi_f), fminf(fmaxf(y1.y, lo_f), hi_f)), magic);
      uint32_t w = __byte_perm(__byte_perm(__float_as_uint(y0.x), __float_as_uint(y0.y), 0x0040),
                               __byte_perm(__float_as_uint(y1.x), __float_as_uint(y1.y), 0x0040), 0x5410);
      if (z4 != 0u) w = __vadd4(w, z4);  // code + z stays inside a byte
      orow[32 * j] = w;
    }
#pragma unroll
    for (int j = 0; j < NV4; ++j) raw[j] = raw_next[j];
  }
}

template <int NV4>
void launch_ln_q8(qdit_ctx* ctx, const void* x, int64_t M, const float* shift, const float* scale, int64_t ld_mod,
                  int64_t T, float eps, void* out, QuantArgs qa, int64_t rows) {
  const unsigned grid = static_cast<unsigned>((M + rows - 1) / rows);
  qdit_launch_overlapped(ctx, ln_modulate_q8_kernel<NV4>, dim3(grid), dim3(256), static_cast<size_t>(NV4) * 128 * 16,
                         static_cast<const __nv_bfloat16*>(x), static_cast<int>(M), static_cast<int>(T), eps, shift, scale,
                         ld_mod, static_cast<uint8_t*>(out), qa, static_cast<int>(rows));
}

// Row range per CTA: `per_sm` CTAs per SM, at least one row per warp, at most what keeps a range within two samples.
int64_t ln_rows_per_cta(const qdit_ctx* ctx, int64_t M, int64_t T, int per_sm) {
  const int64_t ctas = per_sm * static_cast<int64_t>(ctx->num_sms);
  int64_t rows = (M + ctas - 1) / ctas;
  if (rows < 8) rows = 8;
  if (rows > T) rows = T;
  return rows;
}

template <int NV>
void launch_ln(qdit_ctx* ctx, const void* x, int64_t M, int D, int64_t T, float eps, const float* shift,
               const float* scale, int64_t ld_mod, void* out, int out_dtype, QuantArgs qa) {
  const int64_t rows = ln_rows_per_cta(ctx, M, T, 2);
  const unsigned grid = static_cast<unsigned>((M + rows - 1) / rows);
  qdit_launch_overlapped(ctx, ln_modulate_kernel<NV>, dim3(grid), dim3(256), static_cast<size_t>(NV) * 4096,
                         static_cast<const __nv_bfloat16*>(x), static_cast<int>(M), D, static_cast<int>(T), eps, shift, scale,
                         ld_mod, out, out_dtype, qa, static_cast<int>(rows));
}

}  // namespace

int32_t launch_absmax(qdit_ctx* ctx, const void* x, int x_dtype, int64_t M, int64_t K, int64_t ldx, float* absmax_dev) {
  const int64_t total = M * (K / 8);
  if (total == 0) return QDIT_OK;
  const int64_t want = (total + 255) / 256;
  const unsigned grid = static_cast<unsigned>(want < ctx->num_sms * 16 ? want : ctx->num_sms * 16);
  if (x_dtype == QDIT_BF16)
    absmax_kernel<__nv_bfloat16><<<grid, 256, 0, ctx->stream>>>(static_cast<const __nv_bfloat16*>(x), M, K, ldx, absmax_dev);
  else
    absmax_kernel<float><<<grid, 256, 0, ctx->stream>>>(static_cast<const float*>(x), M, K, ldx, absmax_dev);
  return qdit_after_launch(ctx, "absmax_kernel");
}

int32_t launch_absmax_to_scale(qdit_ctx* ctx, const float* absmax_dev, float* scale_dev, float* running_absmax, int n) {
  if (n <= 0) return QDIT_OK;
  absmax_to_scale_kernel<<<(n + 127) / 128, 128, 0, ctx->stream>>>(absmax_dev, scale_dev, running_absmax, n);
  return qdit_after_launch(ctx, "absmax_to_scale_kernel");
}

int32_t qdit_quantize_act_dev(qdit_ctx* ctx, const float* x, int64_t M, int64_t K, qdit_qparams qp,
                              const float* scale_dev, uint8_t* q) {
  if (M == 0 || K == 0) return QDIT_OK;
  const QuantArgs qa = make_quant_args(qp, scale_dev);
  const int64_t threads = M * ((K + 15) / 16);
  act_quant_kernel<float><<<static_cast<unsigned>((threads + 255) / 256), 256, 0, ctx->stream>>>(x, M, K, K, qa, q, K);
  return qdit_after_launch(ctx, "act_quant_kernel");
}

extern "C" {

int32_t qdit_quantize_act(qdit_ctx* ctx, const void* x, int x_dtype, int64_t M, int64_t K, int64_t ldx, int mode,
                          const qdit_qparams* qp, float* dyn_scale, void* q, int64_t ldq) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (M < 0 || K < 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "negative size");
  if (M == 0 || K == 0) return QDIT_OK;
  if (!x || !q) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "x or q is NULL");
  if (x_dtype != QDIT_BF16 && x_dtype != QDIT_F32) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "x_dtype must be bf16 or f32");
  if (K % 8 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "K = %lld must be a multiple of 8", static_cast<long long>(K));
  if (ldx < K || ldq < K) return qdit_fail(ctx, QDIT_ERR_SHAPE, "leading dimension smaller than K");
  const int64_t esz = x_dtype == QDIT_BF16 ? 2 : 4;
  if (!aligned16(x) || (ldx * esz) % 16 != 0) return qdit_fail(ctx, QDIT_ERR_ALIGN, "x must be 16-byte aligned (base and row pitch)");
  if ((reinterpret_cast<uintptr_t>(q) & 7u) || ldq % 8 != 0) return qdit_fail(ctx, QDIT_ERR_ALIGN, "q must be 8-byte aligned (base and row pitch)");
  QuantArgs qa;
  if (mode == QDIT_QUANT_STATIC) {
    QDIT_TRY(qdit_check_qparams(ctx, qp, false));
    qa = make_quant_args(*qp, nullptr);
  } else if (mode == QDIT_QUANT_DYNAMIC_TOKEN) {
    if (!dyn_scale) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "per-token mode needs dyn_scale [M]");
    const unsigned grid = static_cast<unsigned>((M + 7) / 8);
    if (x_dtype == QDIT_BF16)
      act_quant_token_kernel<__nv_bfloat16><<<grid, 256, 0, ctx->stream>>>(static_cast<const __nv_bfloat16*>(x), M, K, ldx, dyn_scale,
                                                                        static_cast<uint8_t*>(q), ldq);
    else
      act_quant_token_kernel<float><<<grid, 256, 0, ctx->stream>>>(static_cast<const float*>(x), M, K, ldx, dyn_scale,
                                                                   static_cast<uint8_t*>(q), ldq);
    return qdit_after_launch(ctx, "act_quant_token_kernel");
  } else if (mode == QDIT_QUANT_DYNAMIC) {
    if (!dyn_scale) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "dynamic mode needs dyn_scale");
    // dyn_scale doubles as the abs-max accumulator before it is turned into the scale in place
    QDIT_CUDA_CHECK(ctx, cudaMemsetAsync(dyn_scale, 0, sizeof(float), ctx->stream));
    QDIT_TRY(launch_absmax(ctx, x, x_dtype, M, K, ldx, dyn_scale));
    QDIT_TRY(launch_absmax_to_scale(ctx, dyn_scale, dyn_scale, nullptr, 1));
    qdit_qparams sym{1.0f, 0, -127, 127};
    qa = make_quant_args(sym, dyn_scale);
  } else {
    return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "unknown quantizer mode %d", mode);
  }
  const int64_t threads = M * ((K + 15) / 16);
  const unsigned grid = static_cast<unsigned>((threads + 255) / 256);
  ProfScope prof(ctx, QDIT_PROF_ACT_QUANT, static_cast<double>(M) * K * (esz + 1.0));
  if (x_dtype == QDIT_BF16)
    act_quant_kernel<__nv_bfloat16><<<grid, 256, 0, ctx->stream>>>(static_cast<const __nv_bfloat16*>(x), M, K, ldx, qa,
                                                                   static_cast<uint8_t*>(q), ldq);
  else
    act_quant_kernel<float><<<grid, 256, 0, ctx->stream>>>(static_cast<const float*>(x), M, K, ldx, qa,
                                                           static_cast<uint8_t*>(q), ldq);
  return qdit_after_launch(ctx, "act_quant_kernel");
}

int32_t qdit_quantize_weight_bits(qdit_ctx* ctx, const float* w, int64_t N, int64_t K, int bits, void* q, float* w_scale,
                             int32_t* w_colsum) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (bits < 2 || bits > 8) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "bits = %d outside 2..8", bits);
  if (N < 0 || K < 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "negative size");
  if (N == 0 || K == 0) return QDIT_OK;
  if (!w || !q || !w_scale || !w_colsum) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  if (K % 4 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "K must be a multiple of 4");
  if (!aligned16(w) || (reinterpret_cast<uintptr_t>(q) & 3u)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "w must be 16-byte, q 4-byte aligned");
  weight_quant_kernel<<<static_cast<unsigned>(N), 256, 0, ctx->stream>>>(w, K, static_cast<int8_t*>(q), w_scale, w_colsum,
                                                                         static_cast<float>((1 << (bits - 1)) - 1));
  return qdit_after_launch(ctx, "weight_quant_kernel");
}

int32_t qdit_quantize_weight(qdit_ctx* ctx, const float* w, int64_t N, int64_t K, void* q, float* w_scale,
                             int32_t* w_colsum) {
  return qdit_quantize_weight_bits(ctx, w, N, K, 8, q, w_scale, w_colsum);
}

int32_t qdit_adaln_modulate(qdit_ctx* ctx, const void* x, int64_t M, int64_t D, int64_t T, float eps,
                            const float* shift, const float* scale, int64_t ld_mod, void* out, int out_dtype,
                            const qdit_qparams* out_qp, const float* out_scale_dev) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (M < 0 || D <= 0 || T <= 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "bad sizes");
  if (M > (int64_t(1) << 30) || T > (int64_t(1) << 30)) return qdit_fail(ctx, QDIT_ERR_SHAPE, "M and T must be at most 2^30");
  if (M == 0) return QDIT_OK;
  if (!x || !shift || !scale || !out) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  if (D % 8 != 0 || D > 2048) return qdit_fail(ctx, QDIT_ERR_SHAPE, "D must be a multiple of 8 and <= 2048");
  if (ld_mod % 4 != 0 || !aligned16(shift) || !aligned16(scale) || !aligned16(x) || !aligned16(out))
    return qdit_fail(ctx, QDIT_ERR_ALIGN, "pointers must be 16-byte aligned and ld_mod a multiple of 4");
  if (out_dtype != QDIT_I8 && out_dtype != QDIT_BF16 && out_dtype != QDIT_F32)
    return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "bad out_dtype");
  QuantArgs qa{};
  if (out_dtype == QDIT_I8) {
    QDIT_TRY(qdit_check_qparams(ctx, out_qp, out_scale_dev != nullptr));
    qa = make_quant_args(*out_qp, out_scale_dev);
  }
  const int nv = static_cast<int>((D / 8 + 31) / 32);
  const int d = static_cast<int>(D);
  const double out_bytes = out_dtype == QDIT_I8 ? 1.0 : out_dtype == QDIT_BF16 ? 2.0 : 4.0;
  ProfScope prof(ctx, QDIT_PROF_LN_MODULATE, static_cast<double>(M) * D * (2.0 + out_bytes));
  if (out_dtype == QDIT_I8 && D % 128 == 0) {
    // the widths of the DiT family (S 384, B 768, L 1024, XL 1152) with 8-bit output: the two-wide kernel
    const int64_t rows = ln_rows_per_cta(ctx, M, T, 3);  // 80 registers: three CTAs of 8 warps per SM
    bool done = true;
    switch (D / 128) {
      case 3: launch_ln_q8<3>(ctx, x, M, shift, scale, ld_mod, T, eps, out, qa, rows); break;
      case 6: launch_ln_q8<6>(ctx, x, M, shift, scale, ld_mod, T, eps, out, qa, rows); break;
      case 8: launch_ln_q8<8>(ctx, x, M, shift, scale, ld_mod, T, eps, out, qa, rows); break;
      case 9: launch_ln_q8<9>(ctx, x, M, shift, scale, ld_mod, T, eps, out, qa, rows); break;
      default: done = false; break;
    }
    if (done) return qdit_after_launch(ctx, "ln_modulate_q8_kernel");
  }
  switch (nv) {
    case 1: launch_ln<1>(ctx, x, M, d, T, eps, shift, scale, ld_mod, out, out_dtype, qa); break;
    case 2: launch_ln<2>(ctx, x, M, d, T, eps, shift, scale, ld_mod, out, out_dtype, qa); break;
    case 3: launch_ln<3>(ctx, x, M, d, T, eps, shift, scale, ld_mod, out, out_dtype, qa); break;
    case 4: launch_ln<4>(ctx, x, M, d, T, eps, shift, scale, ld_mod, out, out_dtype, qa); break;
    case 5: launch_ln<5>(ctx, x, M, d, T, eps, shift, scale, ld_mod, out, out_dtype, qa); break;
    case 6: launch_ln<6>(ctx, x, M, d, T, eps, shift, scale, ld_mod, out, out_dtype, qa); break;
    case 7: launch_ln<7>(ctx, x, M, d, T, eps, shift, scale, ld_mod, out, out_dtype, qa); break;
    default: launch_ln<8>(ctx, x, M, d, T, eps, shift, scale, ld_mod, out, out_dtype, qa); break;
  }
  return qdit_after_launch(ctx, "ln_modulate_kernel");
}

}  // extern "C"
