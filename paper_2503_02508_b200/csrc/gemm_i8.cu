// W8A8 linear layer: persistent tcgen05 kind::i8 GEMM with TMEM int32 accumulators and a fused
// de-quantising epilogue (bias / GELU / cache store / adaLN gate / residual / re-quantisation).
//
// CTA = 2 + NUM_EPI_WARPS warps: warp 0 lane 0  TMA producer  (A and W tiles -> 128B-swizzled smem ring, mbarrier tx)
//                 warp 1 lane 0  MMA issuer    (tcgen05.mma into one of two TMEM accumulator stages)
//                 warps 2..      epilogue      (EPI_SPLIT warps per TMEM lane quadrant, taking 32-column chunks in turn)
// The two accumulator stages let the epilogue of tile i overlap the main loop of tile i+1.
// Tiles are 128 x BN, K is consumed in blocks of 128 bytes (4 MMAs of K = 32 each).
//
// Epilogue data flow per 32x32 chunk: tcgen05.ld gives each thread one ROW of the chunk, which is the
// wrong shape for global memory (32 lanes -> 32 different lines).  The raw accumulators are therefore
// transposed through a 4 KB XOR-swizzled shared-memory patch per warp; afterwards lane (r, g) owns 8
// consecutive columns g of rows r, r+8, r+16, r+24, so that every global load/store instruction of the
// warp covers 8 rows x 64..128 contiguous bytes, and the per-column parameters (scales, bias, gate) sit
// in registers for the whole chunk.
#include "gemm_common.cuh"

namespace {

using namespace qgemm;

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

template <int BN, int EPI>
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
  // everything above touched only this CTA's shared and tensor memory; from here on the kernel reads what
  // the previous kernel of the stream wrote
  grid_dependency_wait();
  grid_dependency_release();

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
    const int half = e >> 2;     // this warp takes chunks half, half + EPI_SPLIT, ...
    const uint32_t stg = smem_u32(staging + e * (32 * 128));  // [32 rows][8 x 16 B], 16-byte index XOR (row & 7)
    const float a_scale = p.a_scale_dev ? __ldg(p.a_scale_dev) : p.a_scale;
    float o_inv = 0.0f;
    if (epi_flags<EPI>(p) & QDIT_EPI_QUANT_OUT) o_inv = __fdiv_rn(1.0f, p.o_scale_dev ? __ldg(p.o_scale_dev) : p.o_scale);
    int it = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
      const int as = it & 1;
      const uint32_t aphase = static_cast<uint32_t>(it >> 1) & 1u;
      const int m0 = (tile / p.num_n_tiles) * BM;
      const int n0 = (tile % p.num_n_tiles) * BN;
      if (!mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status)) break;
      __syncwarp();
      tc_fence_after();
      uint64_t* release_bar = &tempty_bar[as];
      epilogue_tile<BN, EPI>(p, tmem_base + static_cast<uint32_t>(as * BN), m0, n0, quad, half, stg, lane, a_scale, o_inv,
                        [release_bar]() { mbar_arrive_relaxed(release_bar); });
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

template <int BN, int EPI>
int32_t launch_gemm_epi(qdit_ctx* ctx, const void* A, const void* W, GemmParams& p, bool a_unsigned) {
  using C = Cfg<BN>;
  QDIT_TRY(qdit_allow_smem(ctx, gemm_i8_kernel<BN, EPI>, C::SMEM_BYTES));
  CUtensorMap ta, tw;
  QDIT_TRY(qdit_get_tmap(ctx, A, p.M, p.K, p.K, BM, BK, 1, 1, &ta));
  QDIT_TRY(qdit_get_tmap(ctx, W, p.N, p.K, p.K, BN, BK, 1, 1, &tw));
  p.num_m_tiles = (p.M + BM - 1) / BM;
  p.num_n_tiles = (p.N + BN - 1) / BN;
  const int total = p.num_m_tiles * p.num_n_tiles;
  const int grid = total < ctx->num_sms ? total : ctx->num_sms;
  const uint32_t idesc = umma_idesc_i8(BM, BN, a_unsigned);
  ProfScope prof(ctx, QDIT_PROF_GEMM, 2.0 * p.M * static_cast<double>(p.N) * p.K);
  QDIT_CUDA_CHECK(ctx, qdit_launch_overlapped(ctx, gemm_i8_kernel<BN, EPI>, dim3(grid), dim3(NUM_THREADS), C::SMEM_BYTES, ta, tw, p, idesc));
  return qdit_after_launch(ctx, "gemm_i8_kernel");
}

template <int BN>
int32_t launch_gemm(qdit_ctx* ctx, const void* A, const void* W, GemmParams& p, bool a_unsigned) {
  const int cls = ctx->opt[QDIT_OPT_GEMM_GENERIC_EPILOGUE] ? 0 : epi_class(p.flags);
  switch (cls) {
    case 1: return launch_gemm_epi<BN, 1>(ctx, A, W, p, a_unsigned);
    case 2: return launch_gemm_epi<BN, 2>(ctx, A, W, p, a_unsigned);
    case 3: return launch_gemm_epi<BN, 3>(ctx, A, W, p, a_unsigned);
    default: return launch_gemm_epi<BN, 0>(ctx, A, W, p, a_unsigned);
  }
}

// Tile width: prefer 192 (divides every DiT-XL/2 layer width); fall back to narrower tiles when that
// fills the SMs better.  Cost model: waves * (BN + fixed per-tile overhead).
int pick_bn(int M, int N, int num_sms, int forced) {
  if (forced == 64 || forced == 128 || forced == 192) return forced;
  const int mt = (M + BM - 1) / BM;
  int best = 192;
  double best_cost = 1e30;
  const int cands[3] = {192, 128, 64};
  for (int bn : cands) {
    const int tiles = mt * ((N + bn - 1) / bn);
    const int waves = (tiles + num_sms - 1) / num_sms;
    const double cost = static_cast<double>(waves) * (bn + 24);
    if (cost < best_cost * 0.85) {  // measured: the wider tile wins unless the narrower one saves a whole wave or more
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

}  // namespace

// Both linear layers: `packed4` = W holds 4-bit codes two per byte ([N, K/2]); `w8_scratch` = optional [N, K] int8
// matrix the packed weights of a many-row layer are widened into first.
static int32_t linear_impl(qdit_ctx* ctx, const void* A, const void* W, int64_t M, int64_t N, int64_t K, qdit_qparams a_qp,
                           const float* a_scale_dev, uint32_t flags, const qdit_epilogue* epi, void* out, int64_t ldo,
                           bool packed4, void* w8_scratch) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (M < 0 || N < 0 || K < 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "negative size");
  if (M == 0 || N == 0) return QDIT_OK;
  if (!A || !W || !out) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "A, W or out is NULL");
  if (K == 0 || K % 16 != 0 || K > 32768) return qdit_fail(ctx, QDIT_ERR_SHAPE, "K = %lld must be a positive multiple of 16, at most 32768", static_cast<long long>(K));
  if (packed4 && K % 32 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "K = %lld must be a multiple of 32 for packed 4-bit weights", static_cast<long long>(K));
  if (packed4 && (flags & QDIT_EPI_ROW_SCALE)) return qdit_fail(ctx, QDIT_ERR_UNSUPPORTED, "per-token scales are not available with packed 4-bit weights");
  if (w8_scratch && !aligned16(w8_scratch)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "the weight scratch must be 16-byte aligned");
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
    if (flags & QDIT_EPI_ROW_SCALE) {
      if (!epi->a_scale_rows) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "ROW_SCALE set but a_scale_rows is NULL");
      if (a_qp.zero_point != 0) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "ROW_SCALE needs a symmetric activation quantizer (zero_point 0)");
      p.a_scale_rows = epi->a_scale_rows;
      p.a_scale = 1.0f;
      p.a_scale_dev = nullptr;
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
  if (packed4) {
    // many rows: the layer is bound by the tensor core and its epilogue, so the weights are widened once into the
    // scratch matrix and the W8A8 kernels run on it; few rows (or no scratch): the weight bytes bound the layer and
    // the kernel that widens them in front of the tensor core reads half of them
    if (w8_scratch && M >= 1024) {
      QDIT_TRY(qdit_unpack_weight_int4(ctx, W, N, K, w8_scratch));
      W = w8_scratch;
    } else {
      return qdit_launch_gemm_w4(ctx, A, W, p, a_unsigned);
    }
  }
  // QDIT_OPT_GEMM_T forces the channel-major kernel with 128 x bt tiles (per-token scales exist only in the
  // token-major kernel's generic epilogue)
  const bool row_scale = (flags & QDIT_EPI_ROW_SCALE) != 0;
  if (!row_scale && ctx->opt[QDIT_OPT_GEMM_T] != 0) return qdit_launch_gemm_t(ctx, A, W, p, a_unsigned, ctx->opt[QDIT_OPT_GEMM_T]);
  // Kernel choice (measured at M = 8192 on the DiT-XL/2 layers, see profiles/): the block's four layers run
  // channel-major with 128 x 256 tiles (QKV: bias -> bf16 and the gated proj / fc2 through shared-memory tiles and
  // TMA stores; fc1: bias + GELU -> 8-bit through shuffle transposes); everything else (small M, narrow N, f32 or
  // raw outputs, per-token scales) runs token-major.
  if (ctx->opt[QDIT_OPT_GEMM_BN] == 0 && !row_scale && p.M >= 1024) {
    const int cls = epi_class(p.flags);
    if ((cls == 1 || cls == 2) && p.N >= 2304) return qdit_launch_gemm_t(ctx, A, W, p, a_unsigned, 256);
    if (cls == 3 && p.N >= 1024 && p.tokens % 32 == 0) return qdit_launch_gemm_t(ctx, A, W, p, a_unsigned, 256);
  }
  switch (pick_bn(p.M, p.N, ctx->num_sms, ctx->opt[QDIT_OPT_GEMM_BN])) {
    case 64: return launch_gemm<64>(ctx, A, W, p, a_unsigned);
    case 128: return launch_gemm<128>(ctx, A, W, p, a_unsigned);
    default: return launch_gemm<192>(ctx, A, W, p, a_unsigned);
  }
}

extern "C" int32_t qdit_w8a8_linear(qdit_ctx* ctx, const void* A, const void* W, int64_t M, int64_t N, int64_t K,
                                    qdit_qparams a_qp, const float* a_scale_dev, uint32_t flags,
                                    const qdit_epilogue* epi, void* out, int64_t ldo) {
  return linear_impl(ctx, A, W, M, N, K, a_qp, a_scale_dev, flags, epi, out, ldo, false, nullptr);
}

extern "C" int32_t qdit_w4a8_linear(qdit_ctx* ctx, const void* A, const void* W_packed, int64_t M, int64_t N, int64_t K,
                                    qdit_qparams a_qp, const float* a_scale_dev, uint32_t flags,
                                    const qdit_epilogue* epi, void* out, int64_t ldo, void* w8_scratch) {
  return linear_impl(ctx, A, W_packed, M, N, K, a_qp, a_scale_dev, flags, epi, out, ldo, true, w8_scratch);
}
