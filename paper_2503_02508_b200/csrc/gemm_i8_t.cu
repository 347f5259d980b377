// W8A8 linear layer with the accumulator held CHANNEL-major: the tensor core computes D^T = W . A^T, so a
// TMEM lane (and with it an epilogue thread) is an output channel and the TMEM columns are tokens.
//
// Why: tcgen05.ld hands each thread one TMEM lane.  With tokens on the lanes (the usual orientation) a thread
// holds one token's row and needs the per-channel parameters of every column, and its stores are 32 lanes ->
// 32 rows: the epilogue then has to transpose through shared memory, and that traffic competes with the
// operand fill and the operand reads for the SM's 128 B/clk shared-memory port, which is what bounds these
// short-K GEMMs.  With channels on the lanes the per-channel scale / bias / gate are per-thread scalars, a
// warp's 32 lanes are 32 consecutive channels of one token, so every global access of the warp is one
// contiguous 32..128-byte segment, and the epilogue uses no shared memory at all.  It also lets the token
// tile be 256 wide (one MMA of N = 256) and makes every DiT-XL/2 layer width (multiples of 128 channels)
// tile without remainder.
//
// CTA = 2 + 8 or 12 warps (see TWarps), roles and barriers as in gemm_i8.cu: warp 0 lane 0 TMA producer (weight
// tile 128 x 128 B as operand A, activation tile BT x 128 B as operand B, both K-major, 128B swizzle), warp 1
// lane 0 MMA issuer (two TMEM accumulator stages of BT columns), epilogue warps: 2 or 3 per lane quadrant,
// taking 32-token chunks in turn.
//
// Epilogues that write 16-bit outputs (bias -> bf16; the gated one: bias, cache copy, x gate, + residual -> bf16)
// read the accumulator in the matrix-fragment layout (tcgen05.ld 16x256b: a thread holds pairs of adjacent tokens
// of 4 channels), so that the finished bf16 pairs are exactly the operands of stmatrix.trans: four of them lay a
// chunk of 32 tokens x 32 channels into a 2 KB shared-memory tile in token-major order (64-byte rows, 64B
// swizzle, conflict-free), and one thread hands the tile to a TMA store.  No shuffles, no per-thread global
// stores (warp-level stores of 64-byte row pieces reach 4.2 TB/s on this chip, TMA stores of the same tiles
// 6.7 TB/s, and they do not hold the issuing warp), and the residual of the gated epilogue arrives the same way
// in reverse (TMA load one chunk ahead, ldmatrix.trans).
// The epilogue that writes 8-bit codes (bias + GELU -> codes, class 2) keeps a channel per thread (per-channel
// scalars, tcgen05.ld 32x32b) and writes each code with a one-byte shared-memory store into a tile of 32 tokens x 128
// channels that the four quadrant warps of a token chunk fill together; one thread hands it to a TMA store (full
// 128-byte rows; per-thread global stores of this layout are 32-byte pieces of 8 rows, which held that layer at the
// speed of its stores).
#include "gemm_common.cuh"


namespace {

using namespace qgemm;

constexpr int BC = 128;  // channels per tile = TMEM lanes
// Epilogue warps per epilogue class (a multiple of 4: each TMEM lane quadrant is read by warps with warp % 4 =
// quadrant).  The staged epilogues (classes 1 and 3) are light and asynchronous: 2 warps per quadrant, which split
// the 8 chunks of a 256-token tile evenly; the others use 3 (measured: 16 warps are slower than 12 for them).
#ifndef QDIT_T_STAGED_WARPS
#define QDIT_T_STAGED_WARPS 8
#endif
template <int EPI>
struct TWarps {
  static constexpr bool GATED = EPI == 3 || EPI == 4;   // 4: the gated class for short reductions (see launch_t)
  static constexpr bool STAGED = EPI == 1 || GATED;
  static constexpr int EPI_WARPS = EPI == 4 ? 12 : (STAGED ? QDIT_T_STAGED_WARPS : 12);
  static constexpr int SPLIT = EPI_WARPS / 4;
  static constexpr int THREADS = 64 + EPI_WARPS * 32;
#ifndef QDIT_T_GATED_TILES
#define QDIT_T_GATED_TILES 2
#endif
  // 2 KB tiles of 32 tokens x 32 channels bf16 per warp: class 1 two output tiles used in turn; class 3 the residual
  // tile plus one tile shared by the cache copy and the output (2) or one tile each (3)
  static constexpr int TILES = GATED ? QDIT_T_GATED_TILES : 2;
  static constexpr int STAGING_PER_WARP = STAGED ? TILES * 2048 : 0;
  // class 2 (8-bit codes): the four quadrant warps that work on the same token chunk share a tile of 32 tokens x 128
  // channels (4 KB), two tiles used in turn per group of four
  static constexpr bool GROUPED = EPI == 2;
  static constexpr int GROUP_TILE_BYTES = 32 * BC;
  static constexpr int STAGING_BYTES = STAGED ? EPI_WARPS * STAGING_PER_WARP : GROUPED ? SPLIT * 2 * GROUP_TILE_BYTES : 0;
};

template <int BT, int EPI>
struct TCfg {
  static constexpr int W_BYTES = BC * BK;
  static constexpr int X_BYTES = BT * BK;
  static constexpr int STAGE_BYTES = W_BYTES + X_BYTES;
  static constexpr int BAR_BYTES = 512;
  static constexpr int SMEM_LIMIT = 232448;
  static constexpr int STAGES_FIT = (SMEM_LIMIT - 1024 - BAR_BYTES - TWarps<EPI>::STAGING_BYTES) / STAGE_BYTES;
  static constexpr int STAGES = STAGES_FIT > 8 ? 8 : STAGES_FIT;
  static constexpr int TMEM_COLS = 2 * BT <= 128 ? 128 : (2 * BT <= 256 ? 256 : 512);
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + TWarps<EPI>::STAGING_BYTES + BAR_BYTES + 1024;
};

// One 32-token chunk of one channel (this thread): v[j] = accumulator of token m_base + j.
template <int EPI>
__device__ __forceinline__ void epilogue_chunk_t(const GemmParams& p, const uint32_t (&v)[32], int n, int m_base,
                                                 float sc, float bias, int zcs, float o_inv) {
  const uint32_t flags = epi_flags<EPI>(p);
  const int m_end = p.M - m_base < 32 ? p.M - m_base : 32;  // tokens of this chunk inside the matrix
  if (flags & QDIT_EPI_OUT_I32) {
    int32_t* o = static_cast<int32_t*>(p.out) + static_cast<int64_t>(m_base) * p.ldo + n;
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (j < m_end) o[static_cast<int64_t>(j) * p.ldo] = static_cast<int32_t>(v[j]);
    return;
  }
  const bool gate_uniform = (p.tokens % 32) == 0;  // a 32-token chunk then lies inside one sample
  float gate = 1.0f;
  if ((flags & QDIT_EPI_GATE) && gate_uniform) gate = p.gate[static_cast<int64_t>(m_base / p.tokens) * p.ld_gate + n];
#pragma unroll
  for (int j0 = 0; j0 < 32; j0 += 8) {
    float res[8];
    if (flags & QDIT_EPI_RESIDUAL) {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        res[i] = j0 + i < m_end ? __bfloat162float(p.residual[static_cast<int64_t>(m_base + j0 + i) * p.ldo + n]) : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int j = j0 + i;
      const int acc = static_cast<int>(v[j]) - zcs;
      float f = (flags & QDIT_EPI_BIAS) ? __fmaf_rn(static_cast<float>(acc), sc, bias) : __fmul_rn(static_cast<float>(acc), sc);
      if (flags & QDIT_EPI_GELU) f = gelu_tanh_f(f);
      if (j < m_end) {
        const int64_t m = m_base + j;
        if (flags & QDIT_EPI_CACHE_STORE) p.cache_out[m * p.N + n] = __float2bfloat16_rn(f);
        if (flags & QDIT_EPI_GATE) {
          if (!gate_uniform) gate = p.gate[(m / p.tokens) * p.ld_gate + n];
          f = __fmul_rn(f, gate);
        }
        if (flags & QDIT_EPI_RESIDUAL) f = __fadd_rn(f, res[i]);
        const int64_t o = m * p.ldo + n;
        if (flags & QDIT_EPI_QUANT_OUT) {
          // clip(rne(t) + z, qmin, qmax) == rne(clamp(t, qmin - z, qmax - z)) + z; adding 1.5 * 2^23 rounds to
          // nearest-even and leaves the integer in the low mantissa bits
          const float t = fminf(fmaxf(__fmul_rn(f, o_inv), p.o_qmin - p.o_zp), p.o_qmax - p.o_zp);
          static_cast<uint8_t*>(p.out)[o] =
              static_cast<uint8_t>(__float_as_int(__fadd_rn(t, 12582912.0f)) + static_cast<int>(p.o_zp));
        } else if (flags & QDIT_EPI_OUT_BF16) {
          static_cast<__nv_bfloat16*>(p.out)[o] = __float2bfloat16_rn(f);
        } else {
          static_cast<float*>(p.out)[o] = f;
        }
      }
    }
  }
}

// GELU layer (bias + GELU -> 8-bit codes): the math runs channel-major with scalar parameters; the code of token j
// goes to byte (j, col) of the group's tile with a one-byte store (a warp instruction writes 32 consecutive bytes).
template <int EPI>
__device__ __forceinline__ void epilogue_chunk_t_codes(const GemmParams& p, const uint32_t (&v)[32], float sc, float bias, int zcs,
                                                       float o_inv, uint32_t tile_col_addr) {
  const uint32_t flags = epi_flags<EPI>(p);
  // The epilogue of the GELU layer has the most arithmetic per element, so work that a symmetric quantizer does not
  // need (zero-point terms) is skipped through branches that are uniform over the whole grid.
  float f[32];
  if (p.a_zp == 0) {
#pragma unroll
    for (int j = 0; j < 32; ++j) f[j] = static_cast<float>(static_cast<int>(v[j]));
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j) f[j] = static_cast<float>(static_cast<int>(v[j]) - zcs);
  }
  const float lo_f = p.o_qmin - p.o_zp, hi_f = p.o_qmax - p.o_zp;
  const uint32_t zp = static_cast<uint32_t>(static_cast<int>(p.o_zp));
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    float x = (flags & QDIT_EPI_BIAS) ? __fmaf_rn(f[j], sc, bias) : __fmul_rn(f[j], sc);
    if (flags & QDIT_EPI_GELU) x = gelu_tanh_f(x);
    // clip(rne(t) + z, qmin, qmax) == rne(clamp(t, qmin - z, qmax - z)) + z; adding 1.5 * 2^23 rounds to nearest-even and
    // leaves the integer in the low mantissa bits; the low byte is the stored code
    const float q = fminf(fmaxf(__fmul_rn(x, o_inv), lo_f), hi_f);
    uint32_t m = static_cast<uint32_t>(__float_as_int(__fadd_rn(q, 12582912.0f)));
    if (zp != 0u) m += zp;
    asm volatile("st.shared.u8 [%0], %1;" ::"r"(tile_col_addr + static_cast<uint32_t>(j * BC)), "r"(m) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------------------
// Staged epilogues (classes 1 and 3).  A chunk = 32 tokens x the warp's 32 channels.  The accumulator is read as
// two fragment loads (TMEM lanes 0..15 and 16..31 of the warp's quadrant); thread t then holds, for channel
// k = 0..3 (channel offset t/4 + 8k) and token group i = 0..3, the token pair 8i + 2(t%4), + 1:
//   k = 0: a[4i], a[4i+1]   k = 1: a[4i+2], a[4i+3]   k = 2: b[4i], b[4i+1]   k = 3: b[4i+2], b[4i+3]
// stmatrix.trans of the four packed pairs of a token group writes rows 8i..8i+7 of the tile (64 bytes = 32 channels
// per row; the 16-byte piece of channel group k sits at index k ^ ((row >> 1) & 3): the 64B swizzle of the tensor maps).
struct FragChannels {
  float sc[4], bias[4];
  int zcs[4];
};

// Shared-memory offset of the row this thread addresses in stmatrix / ldmatrix for token group 0 (group i: + 512 i).
__device__ __forceinline__ uint32_t frag_row_offset(int lane) {
  const uint32_t row = static_cast<uint32_t>(lane & 7), piece = static_cast<uint32_t>(lane >> 3);
  return row * 64u + ((piece ^ ((row >> 1) & 3u)) << 4);
}

// f[k][2i + e] = de-quantised value of channel k, token 8i + 2(t%4) + e:  (acc - z_a colsum) * (s_a s_w) + bias.
__device__ __forceinline__ void frag_dequant(const uint32_t (&a)[16], const uint32_t (&b)[16], const FragChannels& fc,
                                             float (&f)[4][8]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      f[0][2 * i + e] = __fmaf_rn(static_cast<float>(static_cast<int>(a[4 * i + e]) - fc.zcs[0]), fc.sc[0], fc.bias[0]);
      f[1][2 * i + e] = __fmaf_rn(static_cast<float>(static_cast<int>(a[4 * i + 2 + e]) - fc.zcs[1]), fc.sc[1], fc.bias[1]);
      f[2][2 * i + e] = __fmaf_rn(static_cast<float>(static_cast<int>(b[4 * i + e]) - fc.zcs[2]), fc.sc[2], fc.bias[2]);
      f[3][2 * i + e] = __fmaf_rn(static_cast<float>(static_cast<int>(b[4 * i + 2 + e]) - fc.zcs[3]), fc.sc[3], fc.bias[3]);
    }
  }
}

// The chunk as bf16 into a staging tile (token-major, swizzled).
__device__ __forceinline__ void frag_store_tile(uint32_t tile_row_addr, const float (&f)[4][8]) {
#pragma unroll
  for (int i = 0; i < 4; ++i)
    stmatrix_x4_trans(tile_row_addr + 512u * i, pack_bf16x2(f[0][2 * i], f[0][2 * i + 1]), pack_bf16x2(f[1][2 * i], f[1][2 * i + 1]),
                      pack_bf16x2(f[2][2 * i], f[2][2 * i + 1]), pack_bf16x2(f[3][2 * i], f[3][2 * i + 1]));
}

template <int BT, int EPI>
__global__ void __launch_bounds__(TWarps<EPI>::THREADS, 1)
gemm_i8_t_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                 const __grid_constant__ CUtensorMap tmap_out, const __grid_constant__ CUtensorMap tmap_cache,
                 const __grid_constant__ CUtensorMap tmap_res, const GemmParams p, const uint32_t idesc) {
  using C = TCfg<BT, EPI>;
  using TW = TWarps<EPI>;
  constexpr int STAGES = C::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sW = smem;
  uint8_t* sX = smem + STAGES * C::W_BYTES;
  uint8_t* staging = smem + STAGES * C::STAGE_BYTES;  // classes 1, 3: [EPI_WARPS][tiles][2 KB]; class 2: [SPLIT][2][4 KB]; 1024-byte aligned
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(staging + TW::STAGING_BYTES);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* tfull_bar = empty_bar + STAGES;
  uint64_t* tempty_bar = tfull_bar + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tempty_bar + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  uint64_t* res_bar = full_bar + 32;  // [EPI_WARPS] residual tile of a warp landed (tx)

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&tfull_bar[s], 1);
      mbar_init(&tempty_bar[s], TW::EPI_WARPS);
    }
    for (int s = 0; s < TW::EPI_WARPS; ++s) mbar_init(&res_bar[s], 1);
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
  // the preamble above used only this CTA's shared and tensor memory; global memory is read from here on
  grid_dependency_wait();
  grid_dependency_release();

  const int num_kb = (p.K + BK - 1) / BK;
  // tiles: channel block fastest, so CTAs running together share the activation tile
  const int num_c_tiles = p.num_n_tiles, total_tiles = p.num_m_tiles * p.num_n_tiles;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ TMA producer
      tma_prefetch_desc(&tmap_w);
      tma_prefetch_desc(&tmap_x);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int t0 = (tile / num_c_tiles) * BT;
        const int c0 = (tile % num_c_tiles) * BC;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
          mbar_expect_tx(&full_bar[stage], C::STAGE_BYTES);
          tma_load_2d(sW + stage * C::W_BYTES, &tmap_w, kb * BK, c0, &full_bar[stage]);
          tma_load_2d(sX + stage * C::X_BYTES, &tmap_x, kb * BK, t0, &full_bar[stage]);
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
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(as * BT);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(&full_bar[stage], phase, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t w_desc = umma_desc_k_sw128(smem_u32(sW + stage * C::W_BYTES));
          const uint64_t x_desc = umma_desc_k_sw128(smem_u32(sX + stage * C::X_BYTES));
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            umma_i8(d_tmem, w_desc + static_cast<uint64_t>(k * (UMMA_K >> 4)),
                    x_desc + static_cast<uint64_t>(k * (UMMA_K >> 4)), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&empty_bar[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(&tfull_bar[as]);
      }
    }
  } else {
    // -------------------------------------------------------------------- epilogue warps
    const int e = warp - 2;
    const int quad = warp & 3;   // TMEM lane quadrant = 32 channels
    constexpr int T_EPI_SPLIT = TW::SPLIT;
    const int part = e >> 2;     // this warp takes token chunks part, part + T_EPI_SPLIT, ...
    const uint32_t flags = epi_flags<EPI>(p);
    const float a_scale = p.a_scale_dev ? __ldg(p.a_scale_dev) : p.a_scale;
    float o_inv = 0.0f;
    if (flags & QDIT_EPI_QUANT_OUT) o_inv = __fdiv_rn(1.0f, p.o_scale_dev ? __ldg(p.o_scale_dev) : p.o_scale);
    constexpr int CHUNKS = BT / 32;
    const int c_last = part < CHUNKS ? part + ((CHUNKS - 1 - part) / T_EPI_SPLIT) * T_EPI_SPLIT : -1;
    // the staged form of the gated epilogue needs a chunk to lie inside one sample (one gate row per chunk)
    const bool staged = TW::STAGED && (EPI == 1 || (p.tokens % 32) == 0);
    if (staged) {
      // ------------------------------------------------------------ classes 1 and 3 through shared-memory tiles and TMA
      uint8_t* stg = staging + e * TW::STAGING_PER_WARP;
      // class 1: two output tiles used in turn; class 3: tile 0 receives the residual, tile 1 carries the cache copy and then the output
      const uint32_t tile0 = smem_u32(stg), tile1 = tile0 + 2048u;
      constexpr bool SEPARATE = TW::TILES == 3;                       // class 3: the output has a tile of its own
      const uint32_t tile_o = SEPARATE ? tile0 + 4096u : tile1;
      uint8_t* const stg_o = stg + (SEPARATE ? 4096 : 2048);
      const uint32_t row_off = frag_row_offset(lane);
      uint64_t* rbar = &res_bar[e];
      uint32_t r_phase = 0;
      bool r_inflight = false;
      int out_turn = 0;
      auto chunk_live = [&](int tile, int c) {
        return tile < total_tiles && c < CHUNKS && (tile / num_c_tiles) * BT + 32 * c < p.M && (tile % num_c_tiles) * BC + quad * 32 < p.N;
      };
      auto issue_residual = [&](int tile, int c) {  // one lane
        mbar_expect_tx(rbar, 2048u);
        tma_load_2d(stg, &tmap_res, (tile % num_c_tiles) * BC + quad * 32, (tile / num_c_tiles) * BT + 32 * c, rbar);
      };
      if (lane == 0) {
        tma_prefetch_desc(&tmap_out);
        if (TW::GATED) {
          tma_prefetch_desc(&tmap_cache);
          tma_prefetch_desc(&tmap_res);
        }
      }
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
        // the residual of the tile's first chunk, unless the previous tile's last chunk has already asked for it
        if (TW::GATED && !r_inflight && chunk_live(tile, part)) {
          if (lane == 0) issue_residual(tile, part);
          r_inflight = true;
        }
        const int as = it & 1;
        const uint32_t aphase = static_cast<uint32_t>(it >> 1) & 1u;
        const int t0 = (tile / num_c_tiles) * BT;
        const int c0q = (tile % num_c_tiles) * BC + quad * 32;   // first channel of this warp's quadrant
        // parameters of this thread's 4 channels (channel c0q + lane / 4 + 8 k), fetched before the accumulator is waited for
        FragChannels fc;
        int nk[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          nk[k] = c0q + (lane >> 2) + 8 * k;
          const bool n_ok = nk[k] < p.N;
          fc.sc[k] = n_ok ? __fmul_rn(a_scale, p.w_scale[nk[k]]) : 0.0f;
          fc.bias[k] = n_ok ? p.bias[nk[k]] : 0.0f;
          fc.zcs[k] = (n_ok && p.a_zp != 0) ? p.a_zp * p.w_colsum[nk[k]] : 0;
        }
        if (!mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status)) { ok = false; break; }
        __syncwarp();
        tc_fence_after();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(as * BT);
        if (c_last < 0) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_relaxed(&tempty_bar[as]);
          continue;
        }
#pragma unroll 1
        for (int c = part; c < CHUNKS; c += T_EPI_SPLIT) {
          const int m_base = t0 + c * 32;
          const bool live = m_base < p.M && c0q < p.N;   // uniform over the warp
          uint32_t a[16], b[16];
          float gate[4] = {0.0f, 0.0f, 0.0f, 0.0f};
          if (TW::GATED && live) {
            const float* grow = p.gate + static_cast<int64_t>(m_base / p.tokens) * p.ld_gate;
#pragma unroll
            for (int k = 0; k < 4; ++k)
              if (nk[k] < p.N) gate[k] = grow[nk[k]];
          }
          __syncwarp();
          if (live) {
            tmem_ld_16x256b_x4(taddr + static_cast<uint32_t>(c * 32), a);
            tmem_ld_16x256b_x4(taddr + (16u << 16) + static_cast<uint32_t>(c * 32), b);
            tmem_ld_wait();
          }
          if (c == c_last) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_relaxed(&tempty_bar[as]);
          }
          if (!live) continue;
          float f[4][8];
          frag_dequant(a, b, fc, f);
          if (EPI == 1) {
            const uint32_t tile = out_turn ? tile1 : tile0;
            if (lane == 0) tma_store_wait_read<1>();  // the store that used this tile two chunks ago has read it
            __syncwarp();
            frag_store_tile(tile + row_off, f);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&tmap_out, stg + (out_turn ? 2048 : 0), c0q, m_base);
              tma_store_commit();
            }
            out_turn ^= 1;
          } else {
            // cache copy (the branch output before the gate)
            // tile 1 is free once the store that last used it has read it: the previous chunk's output store, or
            // (separate tiles) the previous chunk's cache store, one group further back
            if (lane == 0) {
              if (SEPARATE) tma_store_wait_read<1>(); else tma_store_wait_read<0>();
            }
            __syncwarp();
            frag_store_tile(tile1 + row_off, f);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&tmap_cache, stg + 2048, c0q, m_base);
              tma_store_commit();
            }
            // residual of this chunk (requested one chunk ahead)
            if (!mbar_wait(rbar, r_phase, abort_flag, p.status)) { ok = false; break; }
            r_phase ^= 1u;
            r_inflight = false;
            uint32_t rw[4][4];  // [token group][channel]: bf16 pair (token 8i + 2(t%4), + 1)
#pragma unroll
            for (int i = 0; i < 4; ++i) ldmatrix_x4_trans(tile0 + row_off + 512u * i, rw[i][0], rw[i][1], rw[i][2], rw[i][3]);
            // x gate, + residual: one rounded multiply and one rounded add, as in every other kernel of this layer
#pragma unroll
            for (int k = 0; k < 4; ++k) {
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                float r0, r1;
                unpack_bf16x2(rw[i][k], r0, r1);
                f[k][2 * i] = __fadd_rn(__fmul_rn(f[k][2 * i], gate[k]), r0);
                f[k][2 * i + 1] = __fadd_rn(__fmul_rn(f[k][2 * i + 1], gate[k]), r1);
              }
            }
            __syncwarp();  // every lane has consumed the residual tile: the next one may land
            {
              int nt = tile, nc = c + T_EPI_SPLIT;
              if (!(nc < CHUNKS && t0 + 32 * nc < p.M)) {
                nt = tile + static_cast<int>(gridDim.x);
                nc = part;
              }
              if (chunk_live(nt, nc)) {
                if (lane == 0) issue_residual(nt, nc);
                r_inflight = true;
              }
            }
            if (lane == 0) {  // the output tile is free: this chunk's cache store has read it, or (separate tiles) the previous chunk's output store
              if (SEPARATE) tma_store_wait_read<1>(); else tma_store_wait_read<0>();
            }
            __syncwarp();
            frag_store_tile(tile_o + row_off, f);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&tmap_out, stg_o, c0q, m_base);
              tma_store_commit();
            }
          }
        }
      }
      // a residual tile still in flight must land before the CTA's shared memory is released
      if (r_inflight) mbar_wait(rbar, r_phase, abort_flag, p.status);
      if (lane == 0) tma_store_wait_all();
    } else {
      // class 2: the tile pair of this warp's group (the four quadrant warps with the same `part`), used in turn
      uint8_t* const gtile = staging + part * (2 * TW::GROUP_TILE_BYTES);
      const bool issuer = quad == 0 && lane == 0;   // one thread per group hands the tiles to TMA
      int turn = 0;
      if (TW::GROUPED && issuer) tma_prefetch_desc(&tmap_out);
      int it = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
        const int as = it & 1;
        const uint32_t aphase = static_cast<uint32_t>(it >> 1) & 1u;
        const int t0 = (tile / num_c_tiles) * BT;
        const int n = (tile % num_c_tiles) * BC + quad * 32 + lane;
        const bool n_ok = n < p.N;
        // this channel's parameters: scalars, fetched before the accumulator is waited for
        float sc = 0.0f, bias = 0.0f;
        int zcs = 0;
        if (n_ok && !(flags & QDIT_EPI_OUT_I32)) {
          sc = __fmul_rn(a_scale, p.w_scale[n]);
          if (flags & QDIT_EPI_BIAS) bias = p.bias[n];
          if (p.a_zp != 0) zcs = p.a_zp * p.w_colsum[n];
        }
        if (!mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status)) break;
        __syncwarp();
        tc_fence_after();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + static_cast<uint32_t>(as * BT);
        if (c_last < 0) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_relaxed(&tempty_bar[as]);
          continue;
        }
#pragma unroll 1
        for (int c = part; c < CHUNKS; c += T_EPI_SPLIT) {
          uint32_t v[32];
          __syncwarp();
          tmem_ld_32x32(taddr + static_cast<uint32_t>(c * 32), v);
          tmem_ld_wait();
          if (c == c_last) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_relaxed(&tempty_bar[as]);
          }
          const int m_base = t0 + c * 32;
          if (m_base < p.M) {   // uniform over the four warps of a group: they work on the same token chunk
            if (TW::GROUPED) {
              uint8_t* const buf = gtile + turn * TW::GROUP_TILE_BYTES;
              epilogue_chunk_t_codes<EPI>(p, v, sc, bias, zcs, o_inv, smem_u32(buf) + static_cast<uint32_t>(quad * 32 + lane));
              fence_async_smem();
              // the store that used the other tile (issued one chunk ago) has read it before anybody passes the barrier,
              // so the next chunk may overwrite it
              if (issuer) tma_store_wait_read<0>();
              asm volatile("bar.sync %0, %1;" ::"r"(1 + part), "r"(128) : "memory");
              if (issuer) {
                tma_store_2d(&tmap_out, buf, (tile % num_c_tiles) * BC, m_base);
                tma_store_commit();
              }
              turn ^= 1;
            } else if (n_ok) {
              epilogue_chunk_t<EPI>(p, v, n, m_base, sc, bias, zcs, o_inv);
            }
          }
        }
      }
      if (TW::GROUPED && issuer) tma_store_wait_all();
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

template <int BT, int EPI>
int32_t launch_t_epi(qdit_ctx* ctx, const void* A, const void* W, GemmParams& p, bool a_unsigned) {
  using C = TCfg<BT, EPI>;
  QDIT_TRY(qdit_allow_smem(ctx, gemm_i8_t_kernel<BT, EPI>, C::SMEM_BYTES));
  CUtensorMap tw, tx;
  QDIT_TRY(qdit_get_tmap(ctx, W, p.N, p.K, p.K, BC, BK, 1, 1, &tw));
  QDIT_TRY(qdit_get_tmap(ctx, A, p.M, p.K, p.K, BT, BK, 1, 1, &tx));
  // staged epilogues: 32 tokens x 32 channels bf16 tiles (64-byte rows, 64B swizzle) of the output, the cache slot and the residual
  CUtensorMap to = tx, tc = tx, tr = tx;
  if (TWarps<EPI>::GROUPED) QDIT_TRY(qdit_get_tmap(ctx, p.out, p.M, p.N, p.ldo, 32, BC, 0, 1, &to));   // 32 tokens x 128 channels of bytes
  if (TWarps<EPI>::STAGED) {
    QDIT_TRY(qdit_get_tmap(ctx, p.out, p.M, p.N, p.ldo, 32, 32, 2, 2, &to));
    tc = tr = to;
    if (TWarps<EPI>::GATED) {
      QDIT_TRY(qdit_get_tmap(ctx, p.cache_out, p.M, p.N, p.N, 32, 32, 2, 2, &tc));
      QDIT_TRY(qdit_get_tmap(ctx, p.residual, p.M, p.N, p.ldo, 32, 32, 2, 2, &tr));
    }
  }
  p.num_m_tiles = (p.M + BT - 1) / BT;   // token tiles
  p.num_n_tiles = (p.N + BC - 1) / BC;   // channel tiles
  const int total = p.num_m_tiles * p.num_n_tiles;
  const int grid = total < ctx->num_sms ? total : ctx->num_sms;
  // operand A = weights (signed), operand B = activations (signed or unsigned)
  const uint32_t idesc = (2u << 4) | (1u << 7) | ((a_unsigned ? 0u : 1u) << 10) | ((static_cast<uint32_t>(BT) >> 3) << 17) |
                         ((static_cast<uint32_t>(BC) >> 4) << 24);
  ProfScope prof(ctx, QDIT_PROF_GEMM, 2.0 * p.M * static_cast<double>(p.N) * p.K);
  QDIT_CUDA_CHECK(ctx, qdit_launch_overlapped(ctx, gemm_i8_t_kernel<BT, EPI>, dim3(grid), dim3(TWarps<EPI>::THREADS), C::SMEM_BYTES, tw, tx, to, tc, tr, p, idesc));
  return qdit_after_launch(ctx, "gemm_i8_t_kernel");
}

template <int BT>
int32_t launch_t(qdit_ctx* ctx, const void* A, const void* W, GemmParams& p, bool a_unsigned) {
  switch (ctx->opt[QDIT_OPT_GEMM_GENERIC_EPILOGUE] ? 0 : epi_class(p.flags)) {
    case 1: return launch_t_epi<BT, 1>(ctx, A, W, p, a_unsigned);
    case 2: return launch_t_epi<BT, 2>(ctx, A, W, p, a_unsigned);
    case 3:
      // A short reduction leaves the gated epilogue (residual in, two tiles out per chunk) as the longer part of a tile,
      // and with few tiles per CTA the last one is exposed: three warps per lane quadrant instead of two shorten it,
      // at the price of one pipeline stage (48 KB of staging instead of 32), which only a long reduction would miss
      // (K = 1152: 17.5 -> 16.6 us at 8192 rows, 129 -> 120 us at 65536; K = 4608: 37.0 -> 41.3 us).
      if (p.K < 2048) return launch_t_epi<BT, 4>(ctx, A, W, p, a_unsigned);
      return launch_t_epi<BT, 3>(ctx, A, W, p, a_unsigned);
    default: return launch_t_epi<BT, 0>(ctx, A, W, p, a_unsigned);
  }
}

}  // namespace

int32_t qdit_launch_gemm_t(qdit_ctx* ctx, const void* A, const void* W, qgemm::GemmParams& p, bool a_unsigned, int bt) {
  if (bt == 128) return launch_t<128>(ctx, A, W, p, a_unsigned);
  return launch_t<256>(ctx, A, W, p, a_unsigned);
}
