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
// CTA = 2 + 12 (or more, see TWarps) warps, roles and barriers as in gemm_i8.cu: warp 0 lane 0 TMA producer (weight
// tile 128 x 128 B as operand A, activation tile BT x 128 B as operand B, both K-major, 128B swizzle), warp 1
// lane 0 MMA issuer (two TMEM accumulator stages of BT columns), epilogue warps: 3 (or more) per lane quadrant,
// taking 32-token chunks in turn.
#include "gemm_common.cuh"


namespace {

using namespace qgemm;

constexpr int BC = 128;  // channels per tile = TMEM lanes
// This kernel has no per-warp staging buffer, so its epilogue could be wider than the token-major kernel's;
// measured, 16 warps (4 per lane quadrant) are slower than 12 for every epilogue class, so 12 it is.
#ifndef QDIT_T_GATED_WARPS
#define QDIT_T_GATED_WARPS 12
#endif
// Epilogue warps per epilogue class (a multiple of 4: each TMEM lane quadrant is read by warps with warp % 4 = quadrant).
template <int EPI>
struct TWarps {
  static constexpr int EPI_WARPS = EPI == 3 ? QDIT_T_GATED_WARPS : 12;
  static constexpr int SPLIT = EPI_WARPS / 4;
  static constexpr int THREADS = 64 + EPI_WARPS * 32;
};

template <int BT>
struct TCfg {
  static constexpr int W_BYTES = BC * BK;
  static constexpr int X_BYTES = BT * BK;
  static constexpr int STAGE_BYTES = W_BYTES + X_BYTES;
  static constexpr int BAR_BYTES = 256;
  static constexpr int SMEM_LIMIT = 232448;
  static constexpr int STAGES_FIT = (SMEM_LIMIT - 1024 - BAR_BYTES) / STAGE_BYTES;
  static constexpr int STAGES = STAGES_FIT > 8 ? 8 : STAGES_FIT;
  static constexpr int TMEM_COLS = 2 * BT <= 128 ? 128 : (2 * BT <= 256 ? 256 : 512);
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + BAR_BYTES + 1024;
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

// 8 x 8 transpose of 32-bit words across the 8 lanes of a lane group (xor 4, 2, 1): afterwards x[c] on lane i
// is what lane c held in x[i].
__device__ __forceinline__ void transpose8(uint32_t (&x)[8], int lane) {
#pragma unroll
  for (int d = 4; d >= 1; d >>= 1) {
    const bool up = (lane & d) != 0;
#pragma unroll
    for (int a = 0; a < 8; ++a) {
      if ((a & d) == 0) {
        const int b = a | d;
        const uint32_t send = up ? x[a] : x[b];
        const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, d);
        if (up) x[a] = recv; else x[b] = recv;
      }
    }
  }
}

// Light epilogues (bias -> bf16, bias + GELU -> 8-bit codes): the math runs channel-major with scalar
// parameters; the finished 16-bit / 8-bit results are then transposed inside each group of 8 lanes with
// shuffles, so that a lane stores 8 consecutive channels of a token at once (16 or 8 bytes) and a warp
// instruction covers 8 tokens x 32 channels, without touching shared memory.
// Lane (g, i) = (lane >> 3, lane & 7) ends up with channels 8g..8g+7 of tokens i, 8 + i, 16 + i, 24 + i.
template <int EPI>
__device__ __forceinline__ void epilogue_chunk_t_packed(const GemmParams& p, const uint32_t (&v)[32], int n, int lane,
                                                        int m_base, float sc, float bias, int zcs, float o_inv) {
  const uint32_t flags = epi_flags<EPI>(p);
  const int i8 = lane & 7;
  const int n8 = n - i8;  // first channel of this lane group
  // The epilogue of the GELU layer is bound by instruction issue, so work that a symmetric quantizer does not
  // need (zero-point terms) is skipped through branches that are uniform over the whole grid.
  float f[32];
  if (p.a_zp == 0) {
#pragma unroll
    for (int j = 0; j < 32; ++j) f[j] = static_cast<float>(static_cast<int>(v[j]));
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j) f[j] = static_cast<float>(static_cast<int>(v[j]) - zcs);
  }
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    f[j] = (flags & QDIT_EPI_BIAS) ? __fmaf_rn(f[j], sc, bias) : __fmul_rn(f[j], sc);
    if (flags & QDIT_EPI_GELU) f[j] = gelu_tanh_f(f[j]);
  }
  if (flags & QDIT_EPI_QUANT_OUT) {
    // one byte per token: word t = codes of tokens t, 8 + t, 16 + t, 24 + t
    const float lo_f = p.o_qmin - p.o_zp, hi_f = p.o_qmax - p.o_zp;
    const int zp = static_cast<int>(p.o_zp);
    uint32_t w[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      uint32_t m4[4];
#pragma unroll
      for (int s4 = 0; s4 < 4; ++s4) {
        const float q = fminf(fmaxf(__fmul_rn(f[8 * s4 + t], o_inv), lo_f), hi_f);
        m4[s4] = static_cast<uint32_t>(__float_as_int(__fadd_rn(q, 12582912.0f)));
      }
      w[t] = __byte_perm(__byte_perm(m4[0], m4[1], 0x0040), __byte_perm(m4[2], m4[3], 0x0040), 0x5410);
      if (zp != 0) w[t] = __vadd4(w[t], static_cast<uint32_t>(zp & 0xFF) * 0x01010101u);  // code + z stays inside a byte
    }
    transpose8(w, lane);  // w[c] = codes of channel n8 + c for tokens i8, 8 + i8, 16 + i8, 24 + i8
    if (n8 < p.N) {
#pragma unroll
      for (int s4 = 0; s4 < 4; ++s4) {
        const int64_t m = m_base + 8 * s4 + i8;
        if (m < p.M) {
          // byte s4 of each of the 8 words
          const uint32_t sel = 0x0000 | (s4) | ((4 + s4) << 4);  // (w_a byte s4, w_b byte s4) -> low two bytes
          const uint32_t lo = __byte_perm(__byte_perm(w[0], w[1], sel), __byte_perm(w[2], w[3], sel), 0x5410);
          const uint32_t hi = __byte_perm(__byte_perm(w[4], w[5], sel), __byte_perm(w[6], w[7], sel), 0x5410);
          *reinterpret_cast<uint2*>(static_cast<uint8_t*>(p.out) + m * p.ldo + n8) = make_uint2(lo, hi);
        }
      }
    }
  } else {
    // bf16: word t of pair (s, s + 1) = (token 8 s + t, token 8 (s + 1) + t)
#pragma unroll
    for (int s2 = 0; s2 < 4; s2 += 2) {
      uint32_t w[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) w[t] = pack_bf16x2(f[8 * s2 + t], f[8 * (s2 + 1) + t]);
      transpose8(w, lane);  // w[c] = channel n8 + c: (token 8 s2 + i8 in the low half, token 8 (s2 + 1) + i8 in the high half)
      if (n8 < p.N) {
        const int64_t m_lo = m_base + 8 * s2 + i8, m_hi = m_lo + 8;
        if (m_lo < p.M) {
          const uint4 o = make_uint4(__byte_perm(w[0], w[1], 0x5410), __byte_perm(w[2], w[3], 0x5410),
                                     __byte_perm(w[4], w[5], 0x5410), __byte_perm(w[6], w[7], 0x5410));
          *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + m_lo * p.ldo + n8) = o;
        }
        if (m_hi < p.M) {
          const uint4 o = make_uint4(__byte_perm(w[0], w[1], 0x7632), __byte_perm(w[2], w[3], 0x7632),
                                     __byte_perm(w[4], w[5], 0x7632), __byte_perm(w[6], w[7], 0x7632));
          *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + m_hi * p.ldo + n8) = o;
        }
      }
    }
  }
}

// Gated epilogue (bias, cache store, x gate, + residual -> bf16) in the same style: the branch value and its
// gated copy are computed channel-major with scalar parameters; the bf16 cache copy travels through two word
// transposes, the gated f32 value through four, and the residual is then added token-major, where a lane loads
// and stores 8 consecutive channels of a token (16 bytes).  Needs the chunk inside one sample (tokens % 32 == 0).
// The residual words `rv` (token 8 s + i8, channels n8..n8+7) and the gate were fetched by the caller one chunk
// ahead, so that their latency is not part of the chunk's dependency chain.
__device__ __forceinline__ void epilogue_chunk_t_gated(const GemmParams& p, const uint32_t (&v)[32], int n, int lane,
                                                       int m_base, float sc, float bias, int zcs, const uint4 (&rv)[4],
                                                       float gate) {
  const int i8 = lane & 7;
  const int n8 = n - i8;
  const bool n8_ok = n8 < p.N;
  float f[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) f[j] = __fmaf_rn(static_cast<float>(static_cast<int>(v[j]) - zcs), sc, bias);
  // cache copy (pre-gate), bf16
#pragma unroll
  for (int s2 = 0; s2 < 4; s2 += 2) {
    uint32_t w[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) w[t] = pack_bf16x2(f[8 * s2 + t], f[8 * (s2 + 1) + t]);
    transpose8(w, lane);
    if (n8_ok) {
      const int64_t m_lo = m_base + 8 * s2 + i8, m_hi = m_lo + 8;
      if (m_lo < p.M)
        *reinterpret_cast<uint4*>(p.cache_out + m_lo * p.N + n8) =
            make_uint4(__byte_perm(w[0], w[1], 0x5410), __byte_perm(w[2], w[3], 0x5410), __byte_perm(w[4], w[5], 0x5410),
                       __byte_perm(w[6], w[7], 0x5410));
      if (m_hi < p.M)
        *reinterpret_cast<uint4*>(p.cache_out + m_hi * p.N + n8) =
            make_uint4(__byte_perm(w[0], w[1], 0x7632), __byte_perm(w[2], w[3], 0x7632), __byte_perm(w[4], w[5], 0x7632),
                       __byte_perm(w[6], w[7], 0x7632));
    }
  }
#pragma unroll
  for (int s4 = 0; s4 < 4; ++s4) {
    const int64_t m = m_base + 8 * s4 + i8;
    const bool live = n8_ok && m < p.M;
    uint32_t w[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) w[t] = __float_as_uint(__fmul_rn(f[8 * s4 + t], gate));
    transpose8(w, lane);  // w[c] = gated value of channel n8 + c, token m
    if (live) {
      float r[8];
      unpack_bf16x2(rv[s4].x, r[0], r[1]);
      unpack_bf16x2(rv[s4].y, r[2], r[3]);
      unpack_bf16x2(rv[s4].z, r[4], r[5]);
      unpack_bf16x2(rv[s4].w, r[6], r[7]);
#pragma unroll
      for (int c = 0; c < 8; ++c) r[c] = __fadd_rn(__uint_as_float(w[c]), r[c]);
      *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + m * p.ldo + n8) = pack_bf16x8(r);
    }
  }
}

template <int BT, int EPI>
__global__ void __launch_bounds__(TWarps<EPI>::THREADS, 1)
gemm_i8_t_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                 const GemmParams p, const uint32_t idesc) {
  using C = TCfg<BT>;
  constexpr int STAGES = C::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sW = smem;
  uint8_t* sX = smem + STAGES * C::W_BYTES;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + STAGES * C::STAGE_BYTES);
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
      mbar_init(&tempty_bar[s], TWarps<EPI>::EPI_WARPS);
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
    constexpr int T_EPI_SPLIT = TWarps<EPI>::SPLIT;
    const int part = e >> 2;     // this warp takes token chunks part, part + T_EPI_SPLIT, ...
    const uint32_t flags = epi_flags<EPI>(p);
    const float a_scale = p.a_scale_dev ? __ldg(p.a_scale_dev) : p.a_scale;
    float o_inv = 0.0f;
    if (flags & QDIT_EPI_QUANT_OUT) o_inv = __fdiv_rn(1.0f, p.o_scale_dev ? __ldg(p.o_scale_dev) : p.o_scale);
    constexpr int CHUNKS = BT / 32;
    const int c_last = part < CHUNKS ? part + ((CHUNKS - 1 - part) / T_EPI_SPLIT) * T_EPI_SPLIT : -1;
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
      // gated layers: residual and gate of a chunk are fetched one chunk ahead (the first before the accumulator is waited for)
      const bool gated_fast = EPI == 3 && (p.tokens % 32) == 0;
      uint4 rv_next[4] = {};
      float gate_next = 0.0f;
      auto prefetch_gated = [&](int c) {
        const int mb = t0 + c * 32, i8 = lane & 7, n8 = n - i8;
#pragma unroll
        for (int s4 = 0; s4 < 4; ++s4) {
          const int64_t m = mb + 8 * s4 + i8;
          rv_next[s4] = (n8 < p.N && m < p.M) ? *reinterpret_cast<const uint4*>(p.residual + m * p.ldo + n8) : make_uint4(0u, 0u, 0u, 0u);
        }
        gate_next = (n_ok && mb < p.M) ? p.gate[static_cast<int64_t>(mb / p.tokens) * p.ld_gate + n] : 0.0f;
      };
      if (gated_fast && c_last >= 0) prefetch_gated(part);
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
        uint4 rv[4];
        float gate = gate_next;
#pragma unroll
        for (int s4 = 0; s4 < 4; ++s4) rv[s4] = rv_next[s4];
        if (gated_fast && c + T_EPI_SPLIT < CHUNKS) prefetch_gated(c + T_EPI_SPLIT);
        __syncwarp();
        tmem_ld_32x32(taddr + static_cast<uint32_t>(c * 32), v);
        tmem_ld_wait();
        if (c == c_last) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_relaxed(&tempty_bar[as]);
        }
        const int m_base = t0 + c * 32;
        if (m_base < p.M) {
          if (EPI == 1 || EPI == 2) epilogue_chunk_t_packed<EPI>(p, v, n, lane, m_base, sc, bias, zcs, o_inv);
          else if (gated_fast) epilogue_chunk_t_gated(p, v, n, lane, m_base, sc, bias, zcs, rv, gate);
          else if (n_ok) epilogue_chunk_t<EPI>(p, v, n, m_base, sc, bias, zcs, o_inv);
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

template <int BT, int EPI>
int32_t launch_t_epi(qdit_ctx* ctx, const void* A, const void* W, GemmParams& p, bool a_unsigned) {
  using C = TCfg<BT>;
  static bool attr_set[64] = {};
  if (!attr_set[ctx->device & 63]) {
    QDIT_CUDA_CHECK(ctx, cudaFuncSetAttribute(gemm_i8_t_kernel<BT, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_set[ctx->device & 63] = true;
  }
  CUtensorMap tw, tx;
  QDIT_TRY(qdit_get_tmap(ctx, W, p.N, p.K, p.K, BC, BK, 1, 1, &tw));
  QDIT_TRY(qdit_get_tmap(ctx, A, p.M, p.K, p.K, BT, BK, 1, 1, &tx));
  p.num_m_tiles = (p.M + BT - 1) / BT;   // token tiles
  p.num_n_tiles = (p.N + BC - 1) / BC;   // channel tiles
  const int total = p.num_m_tiles * p.num_n_tiles;
  const int grid = total < ctx->num_sms ? total : ctx->num_sms;
  // operand A = weights (signed), operand B = activations (signed or unsigned)
  const uint32_t idesc = (2u << 4) | (1u << 7) | ((a_unsigned ? 0u : 1u) << 10) | ((static_cast<uint32_t>(BT) >> 3) << 17) |
                         ((static_cast<uint32_t>(BC) >> 4) << 24);
  ProfScope prof(ctx, QDIT_PROF_GEMM, 2.0 * p.M * static_cast<double>(p.N) * p.K);
  QDIT_CUDA_CHECK(ctx, qdit_launch_overlapped(ctx, gemm_i8_t_kernel<BT, EPI>, dim3(grid), dim3(TWarps<EPI>::THREADS), C::SMEM_BYTES, tw, tx, p, idesc));
  return qdit_after_launch(ctx, "gemm_i8_t_kernel");
}

template <int BT>
int32_t launch_t(qdit_ctx* ctx, const void* A, const void* W, GemmParams& p, bool a_unsigned) {
  switch (getenv("QDIT_GEMM_GENERIC_EPILOGUE") ? 0 : epi_class(p.flags)) {
    case 1: return launch_t_epi<BT, 1>(ctx, A, W, p, a_unsigned);
    case 2: return launch_t_epi<BT, 2>(ctx, A, W, p, a_unsigned);
    case 3: return launch_t_epi<BT, 3>(ctx, A, W, p, a_unsigned);
    default: return launch_t_epi<BT, 0>(ctx, A, W, p, a_unsigned);
  }
}

}  // namespace

int32_t qdit_launch_gemm_t(qdit_ctx* ctx, const void* A, const void* W, qgemm::GemmParams& p, bool a_unsigned, int bt) {
  if (bt == 128) return launch_t<128>(ctx, A, W, p, a_unsigned);
  return launch_t<256>(ctx, A, W, p, a_unsigned);
}
