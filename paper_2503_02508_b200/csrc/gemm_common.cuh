// Shared pieces of the int8 GEMM kernels: tile constants, launch parameters and the fused epilogue.
#pragma once

#include "common.cuh"
#include "internal.h"

namespace qgemm {

using namespace qd;


constexpr int BM = 128;        // tile rows = TMEM lanes
constexpr int BK = 128;        // K bytes per stage = one swizzle row
constexpr int UMMA_K = 32;     // K per kind::i8 instruction
#ifndef QDIT_EPI_WARPS
#define QDIT_EPI_WARPS 12
#endif
constexpr int NUM_EPI_WARPS = QDIT_EPI_WARPS;  // a multiple of 4: EPI_SPLIT warps share each TMEM lane quadrant
constexpr int EPI_SPLIT = NUM_EPI_WARPS / 4;
constexpr int NUM_THREADS = 64 + NUM_EPI_WARPS * 32;
constexpr int STAGING_BYTES = NUM_EPI_WARPS * 32 * 128;  // one 32 x 32 x int32 patch per epilogue warp

struct GemmParams {
  int M, N, K;
  uint32_t flags;
  float a_scale;
  const float* a_scale_dev;
  const float* a_scale_rows;  // per-row activation scales (QDIT_EPI_ROW_SCALE, generic epilogue class only)
  int a_zp;
  const float* w_scale;
  const int32_t* w_colsum;
  const float* bias;
  const float* gate;
  int64_t ld_gate;
  int tokens;
  const __nv_bfloat16* residual;
  __nv_bfloat16* cache_out;
  float o_scale;
  const float* o_scale_dev;
  float o_zp, o_qmin, o_qmax;
  void* out;
  int64_t ldo;
  int* status;
  int num_m_tiles, num_n_tiles;
};

// Epilogue classes.  The three block-level layers get kernels whose epilogue flags are compile-time
// constants (no flag branches, no dead registers, a smaller instruction footprint: instruction-fetch stalls
// were a top stall reason of the all-in-one kernel); class 0 keeps the flags as run-time values.
constexpr uint32_t EPI_FLAGS_QKV = QDIT_EPI_BIAS | QDIT_EPI_OUT_BF16;
constexpr uint32_t EPI_FLAGS_FC1 = QDIT_EPI_BIAS | QDIT_EPI_GELU | QDIT_EPI_QUANT_OUT;
constexpr uint32_t EPI_FLAGS_GATED = QDIT_EPI_BIAS | QDIT_EPI_GATE | QDIT_EPI_RESIDUAL | QDIT_EPI_CACHE_STORE | QDIT_EPI_OUT_BF16;
template <int EPI>
__device__ __forceinline__ uint32_t epi_flags(const GemmParams& p) {
  return EPI == 1 ? EPI_FLAGS_QKV : EPI == 2 ? EPI_FLAGS_FC1 : (EPI == 3 || EPI == 4) ? EPI_FLAGS_GATED : p.flags;
}
inline int epi_class(uint32_t flags) {
  return flags == EPI_FLAGS_QKV ? 1 : flags == EPI_FLAGS_FC1 ? 2 : flags == EPI_FLAGS_GATED ? 3 : 0;
}

// Per-column parameters of the 8 columns a lane owns within a chunk.
struct ColParams {
  float sc[8];  // s_a * s_w[n]
  float bi[8];
  float gt[8];
};

template <int EPI>
__device__ __forceinline__ void load_col_params(const GemmParams& p, int n, int b, float a_scale, ColParams& cp) {
  const uint32_t flags = epi_flags<EPI>(p);
  float t[8];
  Load8<float>::load(p.w_scale + n, t);
#pragma unroll
  for (int i = 0; i < 8; ++i) cp.sc[i] = __fmul_rn(a_scale, t[i]);
  if (flags & QDIT_EPI_BIAS) Load8<float>::load(p.bias + n, cp.bi);
  if (flags & QDIT_EPI_GATE) Load8<float>::load(p.gate + static_cast<int64_t>(b) * p.ld_gate + n, cp.gt);
}

// Epilogue for 8 consecutive columns of one row; `res` holds the residual's 8 bf16 values (if used).
template <int EPI>
__device__ __forceinline__ void epilogue8(const GemmParams& p, const uint4 lo, const uint4 hi, const ColParams& cp,
                                          const uint4 res, int row, int n, float o_inv) {
  const uint32_t flags = epi_flags<EPI>(p);
  const int64_t o = static_cast<int64_t>(row) * p.ldo + n;
  if (flags & QDIT_EPI_OUT_I32) {
    int32_t* op = static_cast<int32_t*>(p.out) + o;
    *reinterpret_cast<uint4*>(op) = lo;
    *reinterpret_cast<uint4*>(op + 4) = hi;
    return;
  }
  int acc[8] = {static_cast<int>(lo.x), static_cast<int>(lo.y), static_cast<int>(lo.z), static_cast<int>(lo.w),
                static_cast<int>(hi.x), static_cast<int>(hi.y), static_cast<int>(hi.z), static_cast<int>(hi.w)};
  if (p.a_zp != 0) {  // asymmetric activations (Eq. 1's unsigned range): remove z_a * sum_k W[n,k]
    const int4 c0 = *reinterpret_cast<const int4*>(p.w_colsum + n);
    const int4 c1 = *reinterpret_cast<const int4*>(p.w_colsum + n + 4);
    acc[0] -= p.a_zp * c0.x; acc[1] -= p.a_zp * c0.y; acc[2] -= p.a_zp * c0.z; acc[3] -= p.a_zp * c0.w;
    acc[4] -= p.a_zp * c1.x; acc[5] -= p.a_zp * c1.y; acc[6] -= p.a_zp * c1.z; acc[7] -= p.a_zp * c1.w;
  }
  // de-quantisation: one fused multiply-add acc * (s_a s_w) + bias in every kernel and epilogue class (explicit,
  // so that the result does not depend on what the compiler contracts)
  float f[8];
  float rs = 1.0f;  // per-token activation scale (cp.sc then holds s_w alone)
  if (flags & QDIT_EPI_ROW_SCALE) rs = p.a_scale_rows[row];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float sc = (flags & QDIT_EPI_ROW_SCALE) ? __fmul_rn(rs, cp.sc[i]) : cp.sc[i];
    f[i] = (flags & QDIT_EPI_BIAS) ? __fmaf_rn(static_cast<float>(acc[i]), sc, cp.bi[i]) : __fmul_rn(static_cast<float>(acc[i]), sc);
  }
  if (flags & QDIT_EPI_GELU) {
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = gelu_tanh_f(f[i]);
  }
  if (flags & QDIT_EPI_CACHE_STORE)
    *reinterpret_cast<uint4*>(p.cache_out + static_cast<int64_t>(row) * p.N + n) = pack_bf16x8(f);
  // gate and residual: one rounded multiply and one rounded add, never a fused multiply-add, so that the
  // token-major and the channel-major kernels (which add the residual after a transpose) give the same bits
  if (flags & QDIT_EPI_GATE) {
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = __fmul_rn(f[i], cp.gt[i]);
  }
  if (flags & QDIT_EPI_RESIDUAL) {
    float r[8];
    unpack_bf16x2(res.x, r[0], r[1]);
    unpack_bf16x2(res.y, r[2], r[3]);
    unpack_bf16x2(res.z, r[4], r[5]);
    unpack_bf16x2(res.w, r[6], r[7]);
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = __fadd_rn(f[i], r[i]);
  }
  if (flags & QDIT_EPI_QUANT_OUT) {
    // clip(rne(t) + z, qmin, qmax) == rne(clamp(t, qmin - z, qmax - z)) + z because the bounds are integers;
    // adding 1.5 * 2^23 performs the rne and leaves the integer in the low mantissa bits (magic & 0xFF == 0)
    const float lo_f = p.o_qmin - p.o_zp, hi_f = p.o_qmax - p.o_zp;
    const int zp = static_cast<int>(p.o_zp);
    uint32_t m[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float t = fminf(fmaxf(__fmul_rn(f[i], o_inv), lo_f), hi_f);
      m[i] = static_cast<uint32_t>(__float_as_int(__fadd_rn(t, 12582912.0f)) + zp);
    }
    uint2 packed;
    packed.x = __byte_perm(__byte_perm(m[0], m[1], 0x0040), __byte_perm(m[2], m[3], 0x0040), 0x5410);
    packed.y = __byte_perm(__byte_perm(m[4], m[5], 0x0040), __byte_perm(m[6], m[7], 0x0040), 0x5410);
    *reinterpret_cast<uint2*>(static_cast<uint8_t*>(p.out) + o) = packed;
  } else if (flags & QDIT_EPI_OUT_BF16) {
    *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + o) = pack_bf16x8(f);
  } else {
    float* of = static_cast<float*>(p.out) + o;
    *reinterpret_cast<float4*>(of) = make_float4(f[0], f[1], f[2], f[3]);
    *reinterpret_cast<float4*>(of + 4) = make_float4(f[4], f[5], f[6], f[7]);
  }
}


// Global loads a lane needs for one chunk: parameters of its 8 columns and the residual of its 4 rows.
struct ChunkInputs {
  ColParams cp;
  uint4 res[4];
};

template <int EPI>
__device__ __forceinline__ void prefetch_chunk(const GemmParams& p, int n, int row_base, int rsub, float a_scale,
                                               ChunkInputs& in) {
  const uint32_t flags = epi_flags<EPI>(p);
  // a warp whose 32 rows lie wholly past M (ragged last tile) has no sample: it loads nothing
  if (n < p.N && row_base < p.M && !(flags & QDIT_EPI_OUT_I32)) {
    load_col_params<EPI>(p, n, row_base / p.tokens, a_scale, in.cp);
    if (flags & QDIT_EPI_RESIDUAL) {
#pragma unroll
      for (int sidx = 0; sidx < 4; ++sidx) {
        const int row = row_base + sidx * 8 + rsub;
        if (row < p.M) in.res[sidx] = *reinterpret_cast<const uint4*>(p.residual + static_cast<int64_t>(row) * p.ldo + n);
      }
    }
  }
}

// Epilogue of one 128 x BN accumulator tile for one epilogue warp (see the data-flow note in gemm_i8.cu).
// `tacc` = TMEM address of the accumulator stage (lane 0 of the CTA, first column); `release()` hands the
// stage back to the MMA issuer once this warp has read its share.  `stg` = this warp's 4 KB staging patch.
// The epilogue is bound by the latency chain of one chunk (global loads, TMEM load, transpose, stores), so
// the tile's chunks are spread over as many warps as the register file allows.
template <int BN, int EPI, int SPLIT = EPI_SPLIT, typename Release>
__device__ __forceinline__ void epilogue_tile(const GemmParams& p, uint32_t tacc, int m0, int n0, int quad, int half,
                                              uint32_t stg, int lane, float a_scale, float o_inv, Release release) {
  const int cg = lane & 3;     // after the transpose: column group (8 columns) ...
  const int rsub = lane >> 2;  // ... of rows rsub, rsub + 8, rsub + 16, rsub + 24
  const uint32_t flags = epi_flags<EPI>(p);
  const bool gate_uniform = (p.tokens % 32) == 0;  // the warp's 32 rows then belong to one sample
  constexpr int CHUNKS = BN / 32;
  // this warp takes chunks half, half + SPLIT, ... (SPLIT = epilogue warps per lane quadrant); c_last = the last of them (-1: none)
  const int c_last = half < CHUNKS ? half + ((CHUNKS - 1 - half) / SPLIT) * SPLIT : -1;
  if (c_last < 0) {  // nothing to read: hand the accumulator stage back untouched
    tc_fence_before();
    __syncwarp();
    if (lane == 0) release();
    return;
  }
  const int row_base = m0 + quad * 32;
  const uint32_t taddr = tacc + (static_cast<uint32_t>(quad * 32) << 16);

  // plain order per chunk: global loads -> TMEM load -> transpose -> math and stores
#pragma unroll 1
  for (int c = half; c < CHUNKS; c += SPLIT) {
    const int n = n0 + c * 32 + cg * 8;
    const bool col_ok = n < p.N;
    const uint32_t patch = stg;
    ChunkInputs cur;
    prefetch_chunk<EPI>(p, n, row_base, rsub, a_scale, cur);
    uint32_t v[32];
    __syncwarp();
    tmem_ld_32x32(taddr + static_cast<uint32_t>(c * 32), v);
    tmem_ld_wait();
    if (c == c_last) {
      tc_fence_before();
      __syncwarp();
      if (lane == 0) release();
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint32_t addr = patch + static_cast<uint32_t>(lane * 128 + ((j ^ (lane & 7)) << 4));
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v[4 * j]), "r"(v[4 * j + 1]),
                   "r"(v[4 * j + 2]), "r"(v[4 * j + 3])
                   : "memory");
    }
    __syncwarp();
    uint4 lo[4], hi[4];  // all eight shared-memory reads are issued before the first is consumed
#pragma unroll
    for (int sidx = 0; sidx < 4; ++sidx) {
      const int r = sidx * 8 + rsub;
      const uint32_t a_lo = patch + static_cast<uint32_t>(r * 128 + (((2 * cg) ^ (r & 7)) << 4));
      const uint32_t a_hi = patch + static_cast<uint32_t>(r * 128 + (((2 * cg + 1) ^ (r & 7)) << 4));
      asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(lo[sidx].x), "=r"(lo[sidx].y), "=r"(lo[sidx].z), "=r"(lo[sidx].w) : "r"(a_lo));
      asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(hi[sidx].x), "=r"(hi[sidx].y), "=r"(hi[sidx].z), "=r"(hi[sidx].w) : "r"(a_hi));
    }
#pragma unroll
    for (int sidx = 0; sidx < 4; ++sidx) {
      const int row = row_base + sidx * 8 + rsub;
      if (row < p.M && col_ok) {
        if (!gate_uniform && (flags & QDIT_EPI_GATE))
          Load8<float>::load(p.gate + static_cast<int64_t>(row / p.tokens) * p.ld_gate + n, cur.cp.gt);
        epilogue8<EPI>(p, lo[sidx], hi[sidx], cur.cp, cur.res[sidx], row, n, o_inv);
      }
    }
  }
}

}  // namespace qgemm

// Channel-major accumulator kernel (gemm_i8_t.cu): tiles of 128 channels x bt tokens, bt in {128, 256}.
int32_t qdit_launch_gemm_t(qdit_ctx* ctx, const void* A, const void* W, qgemm::GemmParams& p, bool a_unsigned, int bt);

// Packed 4-bit weights widened inside the kernel (gemm_w4.cu): token-major tiles of 128 x 128.
int32_t qdit_launch_gemm_w4(qdit_ctx* ctx, const void* A, const void* W_packed, qgemm::GemmParams& p, bool a_unsigned);
