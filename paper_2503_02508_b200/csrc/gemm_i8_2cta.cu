// W8A8 linear layer, CTA-pair variant: two CTAs of a cluster share one 256 x BN output tile.
//
// Each CTA stages its own 128 rows of A and only HALF of the weight tile (BN/2 rows); one thread of the
// leader CTA issues tcgen05.mma.cta_group::2 (M = 256), which reads both CTAs' shared memory and writes
// each CTA's 128 accumulator rows into that CTA's tensor memory.  Per CTA and k-block this moves
// 128 + BN/2 operand rows through the L2 -> SM path instead of 128 + BN, which is what bounds the
// single-CTA kernel.  No multicast loads are used: every CTA loads exactly the slices it keeps.
//
// Synchronisation (all waits bounded):
//   full[s]    leader CTA only; the leader's producer expects the bytes of BOTH CTAs' loads, the peer's
//              TMA loads complete on the leader's barrier (cta_group::2 loads may signal the peer CTA)
//   empty[s]   one per CTA; the leader's tcgen05.commit arrives on both (commit multicast)
//   tfull[a]   one per CTA; commit multicast when an accumulator stage is complete
//   tempty[a]  leader CTA only, 2 x 8 arrivals: every epilogue warp of both CTAs arrives (the peer's remotely)
// A cluster barrier after set-up and before exit keeps each CTA's shared memory, barriers and tensor
// memory alive while the peer can still touch them.
#include "gemm_common.cuh"

namespace {

using namespace qgemm;

template <int BN>
struct PairCfg {
  static constexpr int A_BYTES = BM * BK;
  static constexpr int B_BYTES = (BN / 2) * BK;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int BAR_BYTES = 256;
  static constexpr int SMEM_LIMIT = 232448;
  static constexpr int STAGES_FIT = (SMEM_LIMIT - 1024 - BAR_BYTES - STAGING_BYTES) / STAGE_BYTES;
  static constexpr int STAGES = STAGES_FIT > 8 ? 8 : STAGES_FIT;
  static constexpr int TMEM_COLS = 2 * BN <= 128 ? 128 : (2 * BN <= 256 ? 256 : 512);
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + BAR_BYTES + 1024;
};

template <int BN, int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_i8_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                    const GemmParams p, const uint32_t idesc) {
  using C = PairCfg<BN>;
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
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&tfull_bar[s], 1);
      mbar_init(&tempty_bar[s], 2 * NUM_EPI_WARPS);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_holder, C::TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers exist before anything arrives on them remotely
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  const int num_kb = (p.K + BK - 1) / BK;
  const int total_tiles = p.num_m_tiles * p.num_n_tiles;  // tiles of 256 x BN
  const int pair_id = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer (both CTAs)
      tma_prefetch_desc(&tmap_a);
      tma_prefetch_desc(&tmap_w);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair_id; tile < total_tiles && ok; tile += num_pairs) {
        const int m0 = (tile / p.num_n_tiles) * (2 * BM) + static_cast<int>(rank) * BM;
        const int n0 = (tile % p.num_n_tiles) * BN + static_cast<int>(rank) * (BN / 2);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
          if (leader) mbar_expect_tx(&full_bar[stage], 2 * C::STAGE_BYTES);
          const uint32_t leader_full = mapa_shared(smem_u32(&full_bar[stage]), 0);
          tma_load_2d_pair(sA + stage * C::A_BYTES, &tmap_a, kb * BK, m0, leader_full);
          tma_load_2d_pair(sB + stage * C::B_BYTES, &tmap_w, kb * BK, n0, leader_full);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies in flight land before shared memory goes away
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      // ------------------------------------------------------------------ MMA issuer (leader CTA only)
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = pair_id; tile < total_tiles && ok; tile += num_pairs, ++it) {
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
            umma_i8_pair(d_tmem, a_desc + static_cast<uint64_t>(k * (UMMA_K >> 4)),
                         b_desc + static_cast<uint64_t>(k * (UMMA_K >> 4)), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit_pair(&empty_bar[stage], 3);  // frees this stage in both CTAs
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit_pair(&tfull_bar[as], 3);  // accumulator complete, in both CTAs
      }
    }
  } else {
    // -------------------------------------------------------------------- epilogue warps (both CTAs)
    const int e = warp - 2;
    const int quad = warp & 3;
    const int half = e >> 2;
    const uint32_t stg = smem_u32(staging + e * (32 * 128));
    const float a_scale = p.a_scale_dev ? __ldg(p.a_scale_dev) : p.a_scale;
    float o_inv = 0.0f;
    if (epi_flags<EPI>(p) & QDIT_EPI_QUANT_OUT) o_inv = __fdiv_rn(1.0f, p.o_scale_dev ? __ldg(p.o_scale_dev) : p.o_scale);
    int it = 0;
    for (int tile = pair_id; tile < total_tiles; tile += num_pairs, ++it) {
      const int as = it & 1;
      const uint32_t aphase = static_cast<uint32_t>(it >> 1) & 1u;
      const int m0 = (tile / p.num_n_tiles) * (2 * BM) + static_cast<int>(rank) * BM;
      const int n0 = (tile % p.num_n_tiles) * BN;
      if (!mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status)) break;
      __syncwarp();
      tc_fence_after();
      const uint32_t leader_tempty = mapa_shared(smem_u32(&tempty_bar[as]), 0);
      epilogue_tile<BN, EPI>(p, tmem_base + static_cast<uint32_t>(as * BN), m0, n0, quad, half, stg, lane, a_scale, o_inv,
                        [leader_tempty]() { mbar_arrive_cluster_relaxed(leader_tempty); });
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // neither CTA leaves while its peer may still read its smem or signal its barriers
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
  }
}

template <int BN, int EPI>
int32_t launch_pair_epi(qdit_ctx* ctx, const void* A, const void* W, GemmParams& p, bool a_unsigned) {
  using C = PairCfg<BN>;
  static bool attr_set[64] = {};
  if (!attr_set[ctx->device & 63]) {
    QDIT_CUDA_CHECK(ctx, cudaFuncSetAttribute(gemm_i8_pair_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_set[ctx->device & 63] = true;
  }
  CUtensorMap ta, tw;
  QDIT_TRY(qdit_get_tmap(ctx, A, p.M, p.K, p.K, BM, BK, 1, 1, &ta));
  QDIT_TRY(qdit_get_tmap(ctx, W, p.N, p.K, p.K, BN / 2, BK, 1, 1, &tw));
  p.num_m_tiles = (p.M + 2 * BM - 1) / (2 * BM);
  p.num_n_tiles = (p.N + BN - 1) / BN;
  const int total = p.num_m_tiles * p.num_n_tiles;
  const int max_pairs = ctx->num_sms / 2;
  const int pairs = total < max_pairs ? total : max_pairs;
  const uint32_t idesc = umma_idesc_i8(2 * BM, BN, a_unsigned);
  ProfScope prof(ctx, QDIT_PROF_GEMM, 2.0 * p.M * static_cast<double>(p.N) * p.K);
  gemm_i8_pair_kernel<BN, EPI><<<2 * pairs, NUM_THREADS, C::SMEM_BYTES, ctx->stream>>>(ta, tw, p, idesc);
  return qdit_after_launch(ctx, "gemm_i8_pair_kernel");
}

template <int BN>
int32_t launch_pair(qdit_ctx* ctx, const void* A, const void* W, GemmParams& p, bool a_unsigned) {
  switch (getenv("QDIT_GEMM_GENERIC_EPILOGUE") ? 0 : epi_class(p.flags)) {
    case 1: return launch_pair_epi<BN, 1>(ctx, A, W, p, a_unsigned);
    case 2: return launch_pair_epi<BN, 2>(ctx, A, W, p, a_unsigned);
    case 3: return launch_pair_epi<BN, 3>(ctx, A, W, p, a_unsigned);
    default: return launch_pair_epi<BN, 0>(ctx, A, W, p, a_unsigned);
  }
}

}  // namespace

int32_t qdit_launch_gemm_pair(qdit_ctx* ctx, const void* A, const void* W, qgemm::GemmParams& p, bool a_unsigned, int bn) {
  switch (bn) {
    case 128: return launch_pair<128>(ctx, A, W, p, a_unsigned);
    case 192: return launch_pair<192>(ctx, A, W, p, a_unsigned);
    default: return launch_pair<256>(ctx, A, W, p, a_unsigned);
  }
}
