// W4A8 linear layer (the 512 x 512 setting of Table 2): 8-bit activations, 4-bit channel-wise weights stored two
// codes per byte (byte j of a row = code 2j in the low nibble, code 2j + 1 in the high nibble, two's complement).
//
// The weights cross HBM and L2 at half the bytes of the W8A8 layer and are widened to int8 inside the kernel,
// right in front of the tensor core: the same tcgen05 kind::i8 main loop, TMEM accumulators and fused epilogue as
// gemm_i8.cu (token-major, 128 x 128 tiles), with one more role.
//   warp 0 lane 0   TMA producer: activation tile (128 x 128 B, 128B swizzle) and PACKED weight tile (128 x 64 B)
//   warps 2..5      unpackers: nibbles -> sign-extended bytes, written into the weight stage in the 128B-swizzled
//                   K-major layout the MMA descriptor expects; fence.proxy.async; arrive on ready[stage]
//   warp 1 lane 0   MMA issuer: waits for ready[stage] instead of the TMA barrier
//   warps 6..13     epilogue (the fused epilogue of gemm_i8.cu, two warps per lane quadrant)
// This is the form for weight-streaming shapes (few rows: the stacked modulation GEMM, small batches), where the
// weight bytes are what bounds the layer.  Layers with thousands of rows are bound by the tensor core and their
// epilogue instead; for them qdit_w4a8_linear widens the weights into a caller-provided scratch matrix first
// (unpack_w4_kernel) and runs the W8A8 kernels on it.
#include "gemm_common.cuh"

namespace {

using namespace qgemm;

constexpr int W4_BN = 128;
constexpr int W4_UNPACK_WARPS = 4;   // measured: two warps take 0.36 us per 128 x 128 weight stage, more than the loads and the MMAs
constexpr int W4_EPI_WARPS = 8;
constexpr int W4_THREADS = 64 + W4_UNPACK_WARPS * 32 + W4_EPI_WARPS * 32;
constexpr int W4_STAGING_BYTES = W4_EPI_WARPS * 32 * 128;

struct W4Cfg {
  static constexpr int A_BYTES = BM * BK;
  static constexpr int B_BYTES = W4_BN * BK;
  static constexpr int P_BYTES = W4_BN * BK / 2;   // packed weight tile
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + P_BYTES;
  static constexpr int BAR_BYTES = 512;
  static constexpr int SMEM_LIMIT = 232448;
  static constexpr int STAGES_FIT = (SMEM_LIMIT - 1024 - BAR_BYTES - W4_STAGING_BYTES) / STAGE_BYTES;
  static constexpr int STAGES = STAGES_FIT > 6 ? 6 : STAGES_FIT;
  static constexpr int TMEM_COLS = 256;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + W4_STAGING_BYTES + BAR_BYTES + 1024;
};

// 8 packed bytes (16 codes) -> 16 sign-extended bytes.
__device__ __forceinline__ uint4 widen16(uint2 pk) {
  auto widen = [](uint32_t w, uint32_t& lo4, uint32_t& hi4) {
    // even codes sit in the low nibbles, odd codes in the high nibbles.  Sign extension of a nibble x inside its byte:
    // x + 0x1E * (x & 8) sets bits 4..7 exactly when bit 3 is set (8 * 0x1E = 0xF0, no carry into the next byte)
    uint32_t e = w & 0x0F0F0F0Fu, o = (w >> 4) & 0x0F0F0F0Fu;
    e = (e & 0x08080808u) * 0x1Eu + e;
    o = (o & 0x08080808u) * 0x1Eu + o;
    lo4 = __byte_perm(e, o, 0x5140);  // codes 0, 1, 2, 3 of the word
    hi4 = __byte_perm(e, o, 0x7362);  // codes 4, 5, 6, 7
  };
  uint4 r;
  widen(pk.x, r.x, r.y);
  widen(pk.y, r.z, r.w);
  return r;
}

template <int EPI>
__global__ void __launch_bounds__(W4_THREADS, 1)
gemm_w4_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_wp,
               const GemmParams p, const uint32_t idesc) {
  using C = W4Cfg;
  constexpr int STAGES = C::STAGES;
  constexpr int BN = W4_BN;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = sA + STAGES * C::A_BYTES;
  uint8_t* sP = sB + STAGES * C::B_BYTES;
  uint8_t* staging = sP + STAGES * C::P_BYTES;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(staging + W4_STAGING_BYTES);   // activation + packed weight tiles landed (tx)
  uint64_t* ready_bar = full_bar + STAGES;                                      // weight tile widened (one arrival per unpack warp)
  uint64_t* empty_bar = ready_bar + STAGES;                                     // the MMAs have read the stage (commit)
  uint64_t* tfull_bar = empty_bar + STAGES;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&ready_bar[s], W4_UNPACK_WARPS);
      mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&tfull_bar[s], 1);
      mbar_init(&tempty_bar[s], W4_EPI_WARPS);
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
  grid_dependency_wait();
  grid_dependency_release();

  const int num_kb = (p.K + BK - 1) / BK;
  const int total_tiles = p.num_m_tiles * p.num_n_tiles;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer
      tma_prefetch_desc(&tmap_a);
      tma_prefetch_desc(&tmap_wp);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        // tiles of one weight block are neighbours in time across the CTAs: m fastest
        const int m0 = (tile % p.num_m_tiles) * BM;
        const int n0 = (tile / p.num_m_tiles) * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
          mbar_expect_tx(&full_bar[stage], C::A_BYTES + C::P_BYTES);
          tma_load_2d(sA + stage * C::A_BYTES, &tmap_a, kb * BK, m0, &full_bar[stage]);
          tma_load_2d(sP + stage * C::P_BYTES, &tmap_wp, kb * (BK / 2), n0, &full_bar[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies in flight land before shared memory goes away
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
          if (!mbar_wait(&ready_bar[stage], phase, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t a_desc = umma_desc_k_sw128(smem_u32(sA + stage * C::A_BYTES));
          const uint64_t b_desc = umma_desc_k_sw128(smem_u32(sB + stage * C::B_BYTES));
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            umma_i8(d_tmem, a_desc + static_cast<uint64_t>(k * (UMMA_K >> 4)),
                    b_desc + static_cast<uint64_t>(k * (UMMA_K >> 4)), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&empty_bar[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(&tfull_bar[as]);
      }
    }
  } else if (warp < 2 + W4_UNPACK_WARPS) {
    // -------------------------------------------------------------------- unpackers
    // A weight stage is 128 rows x 128 bytes; its 16-byte piece c of row n sits at n * 128 + ((c ^ (n & 7)) << 4)
    // (the 128B swizzle the MMA descriptor assumes) and comes from bytes 8 c .. 8 c + 7 of packed row n.
    const int ut = (warp - 2) * 32 + lane;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      for (int kb = 0; kb < num_kb; ++kb) {
        if (!mbar_wait(&full_bar[stage], phase, abort_flag, p.status)) { ok = false; break; }
        const uint8_t* src = sP + stage * C::P_BYTES;
        uint8_t* dst = sB + stage * C::B_BYTES;
        // a thread's pieces: i = ut + 64 j, j = 0..15: row (ut >> 3) + 8 j, piece ut & 7 (the row's low three bits, and
        // with them the swizzle term, do not depend on j).  All loads are issued before the first store.
        constexpr int PER_THREAD = BN * 8 / (W4_UNPACK_WARPS * 32);
        const int n_first = ut >> 3, c = ut & 7;
        const uint8_t* s0 = src + n_first * 64 + c * 8;
        uint8_t* d0 = dst + n_first * 128 + ((c ^ (n_first & 7)) << 4);
        constexpr int ROW_STEP = W4_UNPACK_WARPS * 32 / 8;   // rows between a thread's consecutive pieces (a multiple of 8)
        uint2 pk[PER_THREAD];
#pragma unroll
        for (int j = 0; j < PER_THREAD; ++j) pk[j] = *reinterpret_cast<const uint2*>(s0 + j * ROW_STEP * 64);
#pragma unroll
        for (int j = 0; j < PER_THREAD; ++j) *reinterpret_cast<uint4*>(d0 + j * ROW_STEP * 128) = widen16(pk[j]);
        fence_async_smem();   // the tensor core reads the stage through the async proxy
        __syncwarp();
        if (lane == 0) mbar_arrive(&ready_bar[stage]);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else {
    // -------------------------------------------------------------------- epilogue warps
    const int e = warp - 2 - W4_UNPACK_WARPS;
    const int quad = warp & 3;   // TMEM lane quadrant this warp may access
    const int half = e >> 2;
    const uint32_t stg = smem_u32(staging + e * (32 * 128));
    const float a_scale = p.a_scale_dev ? __ldg(p.a_scale_dev) : p.a_scale;
    float o_inv = 0.0f;
    if (epi_flags<EPI>(p) & QDIT_EPI_QUANT_OUT) o_inv = __fdiv_rn(1.0f, p.o_scale_dev ? __ldg(p.o_scale_dev) : p.o_scale);
    int it = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
      const int as = it & 1;
      const uint32_t aphase = static_cast<uint32_t>(it >> 1) & 1u;
      const int m0 = (tile % p.num_m_tiles) * BM;
      const int n0 = (tile / p.num_m_tiles) * BN;
      if (!mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status)) break;
      __syncwarp();
      tc_fence_after();
      uint64_t* release_bar = &tempty_bar[as];
      epilogue_tile<BN, EPI, W4_EPI_WARPS / 4>(p, tmem_base + static_cast<uint32_t>(as * BN), m0, n0, quad, half, stg, lane, a_scale, o_inv,
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

// Pre-pass for the many-row layers: widens packed rows into an int8 matrix [N, K].
__global__ void __launch_bounds__(256) unpack_w4_kernel(const uint8_t* __restrict__ wp, int64_t n_chunks, uint8_t* __restrict__ w8) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;   // one 16-code piece per thread
  if (i >= n_chunks) return;
  const uint2 pk = *reinterpret_cast<const uint2*>(wp + i * 8);
  *reinterpret_cast<uint4*>(w8 + i * 16) = widen16(pk);
}

// The other direction (offline): int8 codes in [-8, 7] -> two per byte.
__global__ void __launch_bounds__(256) pack_w4_kernel(const int8_t* __restrict__ w8, int64_t n_chunks, uint8_t* __restrict__ wp,
                                                      int* __restrict__ out_of_range) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n_chunks) return;
  const uint4 v = *reinterpret_cast<const uint4*>(w8 + i * 16);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  uint32_t o[2] = {0u, 0u};
  bool bad = false;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int code = static_cast<int8_t>((w[j] >> (8 * b)) & 0xFFu);
      bad |= code < -8 || code > 7;
      const int idx = 4 * j + b;   // code index inside the piece
      o[idx >> 3] |= static_cast<uint32_t>(code & 0xF) << (4 * (idx & 7));
    }
  }
  *reinterpret_cast<uint2*>(wp + i * 8) = make_uint2(o[0], o[1]);
  if (bad) atomicExch(out_of_range, 1);
}

template <int EPI>
int32_t launch_w4_epi(qdit_ctx* ctx, const void* A, const void* Wp, GemmParams& p, bool a_unsigned) {
  using C = W4Cfg;
  QDIT_TRY(qdit_allow_smem(ctx, gemm_w4_kernel<EPI>, C::SMEM_BYTES));
  CUtensorMap ta, tw;
  QDIT_TRY(qdit_get_tmap(ctx, A, p.M, p.K, p.K, BM, BK, 1, 1, &ta));
  QDIT_TRY(qdit_get_tmap(ctx, Wp, p.N, p.K / 2, p.K / 2, W4_BN, BK / 2, 0, 1, &tw));
  p.num_m_tiles = (p.M + BM - 1) / BM;
  p.num_n_tiles = (p.N + W4_BN - 1) / W4_BN;
  const int total = p.num_m_tiles * p.num_n_tiles;
  const int grid = total < ctx->num_sms ? total : ctx->num_sms;
  const uint32_t idesc = umma_idesc_i8(BM, W4_BN, a_unsigned);
  ProfScope prof(ctx, QDIT_PROF_GEMM, 2.0 * p.M * static_cast<double>(p.N) * p.K);
  QDIT_CUDA_CHECK(ctx, qdit_launch_overlapped(ctx, gemm_w4_kernel<EPI>, dim3(grid), dim3(W4_THREADS), C::SMEM_BYTES, ta, tw, p, idesc));
  return qdit_after_launch(ctx, "gemm_w4_kernel");
}

}  // namespace

int32_t qdit_launch_gemm_w4(qdit_ctx* ctx, const void* A, const void* Wp, qgemm::GemmParams& p, bool a_unsigned) {
  switch (ctx->opt[QDIT_OPT_GEMM_GENERIC_EPILOGUE] ? 0 : epi_class(p.flags)) {
    case 1: return launch_w4_epi<1>(ctx, A, Wp, p, a_unsigned);
    case 2: return launch_w4_epi<2>(ctx, A, Wp, p, a_unsigned);
    case 3: return launch_w4_epi<3>(ctx, A, Wp, p, a_unsigned);
    default: return launch_w4_epi<0>(ctx, A, Wp, p, a_unsigned);
  }
}

extern "C" int32_t qdit_unpack_weight_int4(qdit_ctx* ctx, const void* packed, int64_t N, int64_t K, void* w8) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (N < 0 || K < 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "negative size");
  if (N == 0 || K == 0) return QDIT_OK;
  if (!packed || !w8) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "packed or w8 is NULL");
  if (K % 16 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "K = %lld must be a multiple of 16", static_cast<long long>(K));
  if (N > (1ll << 31) || K > (1ll << 31)) return qdit_fail(ctx, QDIT_ERR_SHAPE, "N or K too large");
  if ((reinterpret_cast<uintptr_t>(packed) & 7u) || !aligned16(w8)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "packed must be 8-byte and w8 16-byte aligned");
  const int64_t chunks = N * (K / 16);
  unpack_w4_kernel<<<static_cast<unsigned>((chunks + 255) / 256), 256, 0, ctx->stream>>>(static_cast<const uint8_t*>(packed), chunks,
                                                                                       static_cast<uint8_t*>(w8));
  return qdit_after_launch(ctx, "unpack_w4_kernel");
}

extern "C" int32_t qdit_pack_weight_int4(qdit_ctx* ctx, const void* w8, int64_t N, int64_t K, void* packed) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (N < 0 || K < 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "negative size");
  if (N == 0 || K == 0) return QDIT_OK;
  if (!packed || !w8) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "packed or w8 is NULL");
  if (K % 16 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "K = %lld must be a multiple of 16", static_cast<long long>(K));
  if (N > (1ll << 31) || K > (1ll << 31)) return qdit_fail(ctx, QDIT_ERR_SHAPE, "N or K too large");
  if ((reinterpret_cast<uintptr_t>(packed) & 7u) || !aligned16(w8)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "packed must be 8-byte and w8 16-byte aligned");
  // codes outside [-8, 7] cannot be stored: the kernel raises a flag that this call reads back (the one synchronous step)
  int* flag = nullptr;
  QDIT_CUDA_CHECK(ctx, cudaMalloc(&flag, sizeof(int)));
  cudaMemsetAsync(flag, 0, sizeof(int), ctx->stream);
  const int64_t chunks = N * (K / 16);
  pack_w4_kernel<<<static_cast<unsigned>((chunks + 255) / 256), 256, 0, ctx->stream>>>(static_cast<const int8_t*>(w8), chunks,
                                                                                     static_cast<uint8_t*>(packed), flag);
  int32_t st = qdit_after_launch(ctx, "pack_w4_kernel");
  int h = 0;
  cudaError_t e = cudaMemcpyAsync(&h, flag, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  cudaFree(flag);
  if (st != QDIT_OK) return st;
  if (e != cudaSuccess) return qdit_fail(ctx, QDIT_ERR_CUDA, "pack: %s", cudaGetErrorString(e));
  if (h) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "a weight code lies outside the 4-bit range [-8, 7]");
  return QDIT_OK;
}
