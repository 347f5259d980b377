// W8A8 linear layer: persistent tcgen05 kind::i8 GEMM with TMEM int32 accumulators and a fused
// de-quantising epilogue (bias / GELU / cache store / adaLN gate / residual / re-quantisation).
//
// CTA = 10 warps: warp 0 lane 0  TMA producer  (A and W tiles -> 128B-swizzled smem ring, mbarrier tx)
//                 warp 1 lane 0  MMA issuer    (tcgen05.mma into one of two TMEM accumulator stages)
//                 warps 2..9     epilogue      (two warps per TMEM lane quadrant, alternating 32-column chunks)
// The two accumulator stages let the epilogue of tile i overlap the main loop of tile i+1.
// Tiles are 128 x BN, K is consumed in blocks of 128 bytes (4 MMAs of K = 32 each).
//
// Epilogue data flow per 32x32 chunk: tcgen05.ld gives each thread one ROW of the chunk, which is the
// wrong shape for global memory (32 lanes -> 32 different lines).  The raw accumulators are therefore
// transposed through a 4 KB XOR-swizzled shared-memory patch per warp; afterwards lane (r, g) owns 8
// consecutive columns g of rows r, r+8, r+16, r+24, so that every global load/store instruction of the
// warp covers 8 rows x 64..128 contiguous bytes, and the per-column parameters (scales, bias, gate) sit
// in registers for the whole chunk.
#include "common.cuh"
#include "internal.h"

namespace {

using namespace qd;

constexpr int BM = 128;        // tile rows = TMEM lanes
constexpr int BK = 128;        // K bytes per stage = one swizzle row
constexpr int UMMA_K = 32;     // K per kind::i8 instruction
constexpr int NUM_EPI_WARPS = 8;
constexpr int NUM_THREADS = 64 + NUM_EPI_WARPS * 32;
constexpr int STAGING_BYTES = NUM_EPI_WARPS * 32 * 128;  // one 32 x 32 x int32 patch per epilogue warp

struct GemmParams {
  int M, N, K;
  uint32_t flags;
  float a_scale;
  const float* a_scale_dev;
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

template <int BN>
struct Cfg {
  static constexpr int A_BYTES = BM * BK;
  static constexpr int B_BYTES = BN * BK;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_BYTES = 256;
  static constexpr int SMEM_LIMIT = 232448;  // 227 KB per CTA
  static constexpr int STAGES_FIT = (SMEM_LIMIT - 1024 - BAR_BYTES - STAGING_BYTES) / STAGE_BYTES;
  static constexpr int STAGES = STAGES_FIT > 8 ? 8 : STAGES_FIT;
  static constexpr int TMEM_COLS = 2 * BN <= 128 ? 128 : (2 * BN <= 256 ? 256 : 512);
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + BAR_BYTES + 1024;  // + alignment slack
};

// Per-column parameters of the 8 columns a lane owns within a chunk.
struct ColParams {
  float sc[8];  // s_a * s_w[n]
  float bi[8];
  float gt[8];
  int cs[8];    // z_a * colsum[n]
};

__device__ __forceinline__ void load_col_params(const GemmParams& p, int n, int b, float a_scale, ColParams& cp) {
  float t[8];
  Load8<float>::load(p.w_scale + n, t);
#pragma unroll
  for (int i = 0; i < 8; ++i) cp.sc[i] = __fmul_rn(a_scale, t[i]);
  if (p.a_zp != 0) {
    const int4 c0 = *reinterpret_cast<const int4*>(p.w_colsum + n);
    const int4 c1 = *reinterpret_cast<const int4*>(p.w_colsum + n + 4);
    cp.cs[0] = p.a_zp * c0.x; cp.cs[1] = p.a_zp * c0.y; cp.cs[2] = p.a_zp * c0.z; cp.cs[3] = p.a_zp * c0.w;
    cp.cs[4] = p.a_zp * c1.x; cp.cs[5] = p.a_zp * c1.y; cp.cs[6] = p.a_zp * c1.z; cp.cs[7] = p.a_zp * c1.w;
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) cp.cs[i] = 0;
  }
  if (p.flags & QDIT_EPI_BIAS) Load8<float>::load(p.bias + n, cp.bi);
  if (p.flags & QDIT_EPI_GATE) Load8<float>::load(p.gate + static_cast<int64_t>(b) * p.ld_gate + n, cp.gt);
}

// Epilogue for 8 consecutive columns of one row; `res` holds the residual's 8 bf16 values (if used).
__device__ __forceinline__ void epilogue8(const GemmParams& p, const uint4 lo, const uint4 hi, const ColParams& cp,
                                          const uint4 res, int row, int n, float o_inv) {
  const int acc[8] = {static_cast<int>(lo.x), static_cast<int>(lo.y), static_cast<int>(lo.z), static_cast<int>(lo.w),
                      static_cast<int>(hi.x), static_cast<int>(hi.y), static_cast<int>(hi.z), static_cast<int>(hi.w)};
  const int64_t o = static_cast<int64_t>(row) * p.ldo + n;
  if (p.flags & QDIT_EPI_OUT_I32) {
    int32_t* op = static_cast<int32_t*>(p.out) + o;
    *reinterpret_cast<uint4*>(op) = lo;
    *reinterpret_cast<uint4*>(op + 4) = hi;
    return;
  }
  float f[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) f[i] = int_to_float_rn(acc[i] - cp.cs[i]) * cp.sc[i];
  if (p.flags & QDIT_EPI_BIAS) {
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] += cp.bi[i];
  }
  if (p.flags & QDIT_EPI_GELU) {
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = gelu_tanh_f(f[i]);
  }
  if (p.flags & QDIT_EPI_CACHE_STORE)
    *reinterpret_cast<uint4*>(p.cache_out + static_cast<int64_t>(row) * p.N + n) = pack_bf16x8(f);
  if (p.flags & QDIT_EPI_GATE) {
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] *= cp.gt[i];
  }
  if (p.flags & QDIT_EPI_RESIDUAL) {
    float r[8];
    unpack_bf16x2(res.x, r[0], r[1]);
    unpack_bf16x2(res.y, r[2], r[3]);
    unpack_bf16x2(res.z, r[4], r[5]);
    unpack_bf16x2(res.w, r[6], r[7]);
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] += r[i];
  }
  if (p.flags & QDIT_EPI_QUANT_OUT) {
    int code[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
      code[i] = quantize_code_i(f[i], o_inv, static_cast<int>(p.o_zp), static_cast<int>(p.o_qmin), static_cast<int>(p.o_qmax));
    *reinterpret_cast<uint2*>(static_cast<uint8_t*>(p.out) + o) = pack_codes8_i(code);
  } else if (p.flags & QDIT_EPI_OUT_BF16) {
    *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + o) = pack_bf16x8(f);
  } else {
    float* of = static_cast<float*>(p.out) + o;
    *reinterpret_cast<float4*>(of) = make_float4(f[0], f[1], f[2], f[3]);
    *reinterpret_cast<float4*>(of + 4) = make_float4(f[4], f[5], f[6], f[7]);
  }
}

template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
               const GemmParams p, const uint32_t idesc) {
  using C = Cfg<BN>;
  constexpr int STAGES = C::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = smem + STAGES * C::A_BYTES;
  uint8_t* staging = smem + STAGES * C::STAGE_BYTES;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(staging + STAGING_BYTES);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* tfull_bar = empty_bar + STAGES;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&tfull_bar[s], 1);
      mbar_init(&tempty_bar[s], NUM_EPI_WARPS);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_holder, C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  const int num_kb = (p.K + BK - 1) / BK;
  const int total_tiles = p.num_m_tiles * p.num_n_tiles;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer
      tma_prefetch_desc(&tmap_a);
      tma_prefetch_desc(&tmap_w);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile / p.num_n_tiles) * BM;
        const int n0 = (tile % p.num_n_tiles) * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
          mbar_expect_tx(&full_bar[stage], C::STAGE_BYTES);
          tma_load_2d(sA + stage * C::A_BYTES, &tmap_a, kb * BK, m0, &full_bar[stage]);
          tma_load_2d(sB + stage * C::B_BYTES, &tmap_w, kb * BK, n0, &full_bar[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // give copies already in flight time to land before the CTA's shared memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------------------------ MMA issuer
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
        const int as = it & 1;
        const uint32_t aphase = static_cast<uint32_t>(it >> 1) & 1u;
        if (!mbar_wait(&tempty_bar[as], aphase ^ 1u, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(as * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(&full_bar[stage], phase, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t a_desc = umma_desc_k_sw128(smem_u32(sA + stage * C::A_BYTES));
          const uint64_t b_desc = umma_desc_k_sw128(smem_u32(sB + stage * C::B_BYTES));
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing K by 32 bytes inside the swizzle row = +2 in the (address >> 4) field
            umma_i8(d_tmem, a_desc + static_cast<uint64_t>(k * (UMMA_K >> 4)),
                    b_desc + static_cast<uint64_t>(k * (UMMA_K >> 4)), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&empty_bar[stage]);  // frees the smem stage once these MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(&tfull_bar[as]);  // accumulator complete
      }
    }
  } else {
    // -------------------------------------------------------------------- epilogue warps
    const int e = warp - 2;
    const int quad = warp & 3;   // TMEM lane quadrant this warp may access
    const int half = e >> 2;     // this warp takes chunks half, half + 2, ...
    const uint32_t stg = smem_u32(staging + e * (32 * 128));  // [32 rows][8 x 16 B], 16-byte index XOR (row & 7)
    const int cg = lane & 3;     // after the transpose: column group (8 columns) ...
    const int rsub = lane >> 2;  // ... of rows rsub, rsub + 8, rsub + 16, rsub + 24
    const float a_scale = p.a_scale_dev ? __ldg(p.a_scale_dev) : p.a_scale;
    float o_inv = 0.0f;
    if (p.flags & QDIT_EPI_QUANT_OUT) o_inv = __fdiv_rn(1.0f, p.o_scale_dev ? __ldg(p.o_scale_dev) : p.o_scale);
    const bool gate_uniform = (p.tokens % 32) == 0;  // the warp's 32 rows then belong to one sample
    constexpr int CHUNKS = BN / 32;
    constexpr int LAST_EVEN = ((CHUNKS - 1) / 2) * 2, LAST_ODD = ((CHUNKS - 2) / 2) * 2 + 1;
    const int c_last = half ? LAST_ODD : LAST_EVEN;
    int it = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
      const int as = it & 1;
      const uint32_t aphase = static_cast<uint32_t>(it >> 1) & 1u;
      const int m0 = (tile / p.num_n_tiles) * BM;
      const int n0 = (tile % p.num_n_tiles) * BN;
      if (!mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status)) break;
      __syncwarp();
      tc_fence_after();
      const int row_base = m0 + quad * 32;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(as * BN);
#pragma unroll 1
      for (int c = half; c < CHUNKS; c += 2) {
        const int n = n0 + c * 32 + cg * 8;
        const bool col_ok = n < p.N;
        // ---- global loads first: column parameters and the residual rows, in flight during the transpose
        ColParams cp;
        uint4 res[4];
        if (col_ok && !(p.flags & QDIT_EPI_OUT_I32)) {
          load_col_params(p, n, row_base / p.tokens, a_scale, cp);
          if (p.flags & QDIT_EPI_RESIDUAL) {
#pragma unroll
            for (int sidx = 0; sidx < 4; ++sidx) {
              const int row = row_base + sidx * 8 + rsub;
              if (row < p.M) res[sidx] = *reinterpret_cast<const uint4*>(p.residual + static_cast<int64_t>(row) * p.ldo + n);
            }
          }
        }
        // ---- TMEM -> registers (one row per thread) -> swizzled staging patch
        uint32_t v[32];
        __syncwarp();  // the previous chunk's reads of the patch are complete
        tmem_ld_32x32(taddr + static_cast<uint32_t>(c * 32), v);
        tmem_ld_wait();
        if (c == c_last) {
          // this warp has read all of its share of the accumulator stage: hand it back to the MMA warp
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty_bar[as]);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t addr = stg + static_cast<uint32_t>(lane * 128 + ((j ^ (lane & 7)) << 4));
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v[4 * j]), "r"(v[4 * j + 1]),
                       "r"(v[4 * j + 2]), "r"(v[4 * j + 3])
                       : "memory");
        }
        __syncwarp();
        // ---- transposed ownership: 8 columns of 4 rows per lane
#pragma unroll
        for (int sidx = 0; sidx < 4; ++sidx) {
          const int r = sidx * 8 + rsub;
          const int row = row_base + r;
          uint4 lo, hi;
          const uint32_t a_lo = stg + static_cast<uint32_t>(r * 128 + (((2 * cg) ^ (r & 7)) << 4));
          const uint32_t a_hi = stg + static_cast<uint32_t>(r * 128 + (((2 * cg + 1) ^ (r & 7)) << 4));
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w) : "r"(a_lo));
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w) : "r"(a_hi));
          if (row < p.M && col_ok) {
            if (!gate_uniform && (p.flags & QDIT_EPI_GATE))
              Load8<float>::load(p.gate + static_cast<int64_t>(row / p.tokens) * p.ld_gate + n, cp.gt);
            epilogue8(p, lo, hi, cp, res[sidx], row, n, o_inv);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

template <int BN>
int32_t launch_gemm(qdit_ctx* ctx, const void* A, const void* W, GemmParams& p, bool a_unsigned) {
  using C = Cfg<BN>;
  static bool attr_set[64] = {};
  if (!attr_set[ctx->device & 63]) {
    QDIT_CUDA_CHECK(ctx, cudaFuncSetAttribute(gemm_i8_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_set[ctx->device & 63] = true;
  }
  CUtensorMap ta, tw;
  QDIT_TRY(qdit_get_tmap(ctx, A, p.M, p.K, p.K, BM, BK, 1, 1, &ta));
  QDIT_TRY(qdit_get_tmap(ctx, W, p.N, p.K, p.K, BN, BK, 1, 1, &tw));
  p.num_m_tiles = (p.M + BM - 1) / BM;
  p.num_n_tiles = (p.N + BN - 1) / BN;
  const int total = p.num_m_tiles * p.num_n_tiles;
  const int grid = total < ctx->num_sms ? total : ctx->num_sms;
  const uint32_t idesc = umma_idesc_i8(BM, BN, a_unsigned);
  ProfScope prof(ctx, QDIT_PROF_GEMM, 2.0 * p.M * static_cast<double>(p.N) * p.K);
  gemm_i8_kernel<BN><<<grid, NUM_THREADS, C::SMEM_BYTES, ctx->stream>>>(ta, tw, p, idesc);
  return qdit_after_launch(ctx, "gemm_i8_kernel");
}

// Tile width: prefer 192 (divides every DiT-XL/2 layer width); fall back to narrower tiles when that
// fills the SMs better.  Cost model: waves * (BN + fixed per-tile overhead).
int pick_bn(int M, int N, int num_sms) {
  const char* env = getenv("QDIT_GEMM_BN");
  if (env) {
    const int v = atoi(env);
    if (v == 64 || v == 128 || v == 192) return v;
  }
  const int mt = (M + BM - 1) / BM;
  int best = 192;
  double best_cost = 1e30;
  const int cands[3] = {192, 128, 64};
  for (int bn : cands) {
    const int tiles = mt * ((N + bn - 1) / bn);
    const int waves = (tiles + num_sms - 1) / num_sms;
    const double cost = static_cast<double>(waves) * (bn + 24);
    if (cost < best_cost * 0.97) {  // keep the wider tile unless the narrower one wins clearly
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

}  // namespace

extern "C" int32_t qdit_w8a8_linear(qdit_ctx* ctx, const void* A, const void* W, int64_t M, int64_t N, int64_t K,
                                    qdit_qparams a_qp, const float* a_scale_dev, uint32_t flags,
                                    const qdit_epilogue* epi, void* out, int64_t ldo) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (M < 0 || N < 0 || K < 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "negative size");
  if (M == 0 || N == 0) return QDIT_OK;
  if (!A || !W || !out) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "A, W or out is NULL");
  if (K == 0 || K % 16 != 0 || K > 32768) return qdit_fail(ctx, QDIT_ERR_SHAPE, "K = %lld must be a positive multiple of 16, at most 32768", static_cast<long long>(K));
  if (N % 8 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "N = %lld must be a multiple of 8", static_cast<long long>(N));
  if (M > (1 << 30) || N > (1 << 30)) return qdit_fail(ctx, QDIT_ERR_SHAPE, "M or N too large");
  const uint32_t out_modes = flags & (QDIT_EPI_OUT_BF16 | QDIT_EPI_OUT_F32 | QDIT_EPI_OUT_I32 | QDIT_EPI_QUANT_OUT);
  if (out_modes == 0 || (out_modes & (out_modes - 1)) != 0)
    return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "exactly one of OUT_BF16, OUT_F32, OUT_I32, QUANT_OUT must be set");
  if ((flags & QDIT_EPI_OUT_I32) && (flags & ~QDIT_EPI_OUT_I32))
    return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "OUT_I32 returns raw accumulators and takes no other flag");
  if (ldo < N) return qdit_fail(ctx, QDIT_ERR_SHAPE, "ldo smaller than N");
  if (!aligned16(A) || !aligned16(W) || !aligned16(out)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "A, W and out must be 16-byte aligned");
  const int64_t osz = (flags & QDIT_EPI_QUANT_OUT) ? 1 : (flags & QDIT_EPI_OUT_BF16) ? 2 : 4;
  if ((ldo * osz) % 8 != 0 || ((flags & QDIT_EPI_QUANT_OUT) == 0 && (ldo * osz) % 16 != 0))
    return qdit_fail(ctx, QDIT_ERR_ALIGN, "row pitch of out must be a multiple of 16 bytes (8 for byte output)");
  QDIT_TRY(qdit_check_qparams(ctx, &a_qp, a_scale_dev != nullptr));
  const bool a_unsigned = a_qp.qmin >= 0 && a_qp.qmax > 127;

  GemmParams p{};
  p.M = static_cast<int>(M);
  p.N = static_cast<int>(N);
  p.K = static_cast<int>(K);
  p.flags = flags;
  p.a_scale = a_qp.scale;
  p.a_scale_dev = a_scale_dev;
  p.a_zp = a_qp.zero_point;
  p.out = out;
  p.ldo = ldo;
  p.status = ctx->d_status;
  p.tokens = 1;
  if (!(flags & QDIT_EPI_OUT_I32)) {
    if (!epi || !epi->w_scale) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "epilogue with w_scale is required");
    if (!aligned16(epi->w_scale)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "w_scale must be 16-byte aligned");
    p.w_scale = epi->w_scale;
    if (a_qp.zero_point != 0) {
      if (!epi->w_colsum) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "w_colsum is required with a non-zero activation zero point");
      if (!aligned16(epi->w_colsum)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "w_colsum must be 16-byte aligned");
      p.w_colsum = epi->w_colsum;
    }
    if (flags & QDIT_EPI_BIAS) {
      if (!epi->bias) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "BIAS set but bias is NULL");
      if (!aligned16(epi->bias)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "bias must be 16-byte aligned");
      p.bias = epi->bias;
    }
    if (flags & QDIT_EPI_GATE) {
      if (!epi->gate || epi->tokens_per_sample <= 0) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "GATE needs gate and tokens_per_sample > 0");
      if (!aligned16(epi->gate) || epi->ld_gate % 4 != 0) return qdit_fail(ctx, QDIT_ERR_ALIGN, "gate must be 16-byte aligned with ld_gate a multiple of 4");
      p.gate = epi->gate;
      p.ld_gate = epi->ld_gate;
      p.tokens = static_cast<int>(epi->tokens_per_sample);
    }
    if (flags & QDIT_EPI_RESIDUAL) {
      if (!epi->residual) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "RESIDUAL set but residual is NULL");
      if (!aligned16(epi->residual) || ldo % 8 != 0) return qdit_fail(ctx, QDIT_ERR_ALIGN, "residual must be 16-byte aligned (base and row pitch ldo)");
      p.residual = static_cast<const __nv_bfloat16*>(epi->residual);
    }
    if (flags & QDIT_EPI_CACHE_STORE) {
      if (!epi->cache_out) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "CACHE_STORE set but cache_out is NULL");
      if (!aligned16(epi->cache_out)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "cache_out must be 16-byte aligned");
      p.cache_out = static_cast<__nv_bfloat16*>(epi->cache_out);
    }
    if (flags & QDIT_EPI_QUANT_OUT) {
      QDIT_TRY(qdit_check_qparams(ctx, &epi->out_qp, epi->out_scale_dev != nullptr));
      p.o_scale = epi->out_qp.scale;
      p.o_scale_dev = epi->out_scale_dev;
      p.o_zp = static_cast<float>(epi->out_qp.zero_point);
      p.o_qmin = static_cast<float>(epi->out_qp.qmin);
      p.o_qmax = static_cast<float>(epi->out_qp.qmax);
    }
  }
  switch (pick_bn(p.M, p.N, ctx->num_sms)) {
    case 64: return launch_gemm<64>(ctx, A, W, p, a_unsigned);
    case 128: return launch_gemm<128>(ctx, A, W, p, a_unsigned);
    default: return launch_gemm<192>(ctx, A, W, p, a_unsigned);
  }
}
