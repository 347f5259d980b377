// Non-causal softmax attention on the 5th-generation tensor cores (tcgen05 kind::f16, bf16 operands).
//
// One CTA = 128 queries of one (sample, head).  Keys are consumed in blocks of 128:
//   S = Q K^T     tcgen05.mma, A = Q and B = K tiles (K-major, TMA-staged), accumulator in tensor memory
//   softmax       two threads per query row: tcgen05.ld S, running max / sum in f32 (no shuffles needed),
//                 P = exp2(..) written as bf16 into a 128B-swizzled shared-memory tile
//   O_blk = P V   tcgen05.mma, A = P (K-major), B = V tile used MN-major (its head-dim index is contiguous),
//                 accumulator re-uses the S columns; the row's threads fold it into their f32 registers
// Head dim 72 does not fill a 128-byte swizzle row: every operand is staged as a 64-column tile (128B
// swizzle) plus a 16-column tail tile (32B swizzle, columns 64..79).  The tail's columns 72..79 belong to the
// next head; they are zeroed in the Q tail, so they add nothing to S, and in V they only produce output
// columns 72..79, which are dropped.
// Warps 0-7: softmax, two threads per query row: each reads its 64 columns of S, the two exchange their maxima
// through shared memory, then each exponentiates, stores and accumulates its half.  Warp 8 lane 0: TMA producer;
// warp 9 lane 0: MMA issuer (warp 9 owns the TMEM allocation).
// S is double-buffered in tensor memory (2 x 128 columns): S of the next key block is issued as soon as its K
// tile has landed, so it is computed while the softmax of the current block runs; O_blk of block j re-uses the
// columns of S_j, is folded into the registers during the next block (after that block's row maximum is known),
// and only then is the buffer handed back for S of block j + 2.
// Two CTAs fit per SM (97 KB shared memory, 256 TMEM columns each) and overlap each other's phases.
#include "common.cuh"
#include "internal.h"

namespace {

using namespace qd;

constexpr int TQ = 128;   // queries per CTA
constexpr int TK = 128;   // keys per block
constexpr int SM_WARPS = 8;                    // softmax warps: two threads share a query row
constexpr int TC_THREADS = (SM_WARPS + 2) * 32;

struct AttnTcParams {
  int T, H;
  float scale_log2;  // softmax_scale * log2(e)
  void* out;
  int out_dtype;
  QuantArgs qa;
  int* status;
  int stagger_ns;      // 256-token kernel: start delay of an SM's second CTA in the first wave
  unsigned num_sms;
};

template <int DH>
struct TCfg {
  static constexpr bool TAIL = DH > 64;                 // 64 < DH <= 80: a 16-column tail tile
  static constexpr int MAIN_BYTES = 128 * 128;          // 128 rows x 64 bf16
  static constexpr int TAIL_BYTES = TAIL ? 128 * 32 : 0;
  static constexpr int OP_BYTES = MAIN_BYTES + TAIL_BYTES;
  static constexpr int P_BYTES = 2 * MAIN_BYTES;        // 128 rows x 128 keys bf16 = two 64-key tiles
  static constexpr int SMEM_BYTES = 3 * OP_BYTES + P_BYTES + 4096 + 1024;
  static constexpr int O_COLS = TAIL ? 80 : 64;
  static constexpr int O_HALF = O_COLS / 2;             // accumulator columns per thread of a row pair (40 or 32)
};

template <int DH>
__global__ void __launch_bounds__(TC_THREADS, 2)
attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_qt,
                    const __grid_constant__ CUtensorMap tm_kt, const __grid_constant__ CUtensorMap tm_vt,
                    const AttnTcParams p) {
  using C = TCfg<DH>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + C::MAIN_BYTES;
  uint8_t* sV = sK + C::MAIN_BYTES;
  uint8_t* sP = sV + C::MAIN_BYTES;             // two 64-key tiles
  uint8_t* sQt = sP + C::P_BYTES;               // tails (256-byte aligned: 32B-swizzle atoms)
  uint8_t* sKt = sQt + C::TAIL_BYTES;
  uint8_t* sVt = sKt + C::TAIL_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sVt + C::TAIL_BYTES);
  uint64_t* bar_q = bars + 0;      // Q tiles landed (tx)
  uint64_t* bar_qz = bars + 1;     // Q tail padding zeroed (256 arrivals)
  uint64_t* bar_kfull = bars + 2;  // K block landed (tx)
  uint64_t* bar_vfull = bars + 3;  // V block landed (tx)
  uint64_t* bar_kfree = bars + 4;  // S MMAs done reading K (commit)
  uint64_t* bar_vfree = bars + 5;  // PV MMAs done reading V and P (commit)
  uint64_t* bar_s = bars + 6;      // [2] S complete in buffer 0 / 1 (commit)
  uint64_t* bar_p = bars + 8;      // P written (256 arrivals)
  uint64_t* bar_o = bars + 9;      // O_blk complete (commit)
  uint64_t* bar_sfree = bars + 10; // O_blk folded: its buffer may take the S of two blocks later (256 arrivals)
  uint64_t* bar_l = bars + 11;     // row sums exchanged (256 arrivals)
  uint64_t* bar_mx = bars + 12;    // [4] row maxima exchanged between the two warps of a lane quadrant (64 arrivals)
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  float* s_l = reinterpret_cast<float*>(tmem_holder + 4);  // [2][128] partial row sums
  float* s_m = s_l + 256;                                  // [2 (block parity)][2][128] partial row maxima

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * TQ, h = blockIdx.y, b = blockIdx.z;
  const int row0 = b * p.T, col0 = h * DH;
  const int n_blk = p.T / TK;

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_qz, SM_WARPS * 32);
    mbar_init(bar_kfull, 1);
    mbar_init(bar_vfull, 1);
    mbar_init(bar_kfree, 1);
    mbar_init(bar_vfree, 1);
    mbar_init(&bar_s[0], 1);
    mbar_init(&bar_s[1], 1);
    mbar_init(bar_p, SM_WARPS * 32);
    mbar_init(bar_o, 1);
    mbar_init(bar_sfree, SM_WARPS * 32);
    mbar_init(bar_l, SM_WARPS * 32);
    for (int i = 0; i < 4; ++i) mbar_init(&bar_mx[i], 64);
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == SM_WARPS + 1) {
    tmem_alloc(tmem_holder, 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_holder;
  // shared and tensor memory only so far; Q, K and V come from the previous kernel of the stream
  grid_dependency_wait();
  grid_dependency_release();

  if (warp == SM_WARPS) {
    if (lane == 0) {
      // ---------------------------------------------------------------- TMA producer
      mbar_expect_tx(bar_q, C::OP_BYTES);
      tma_load_2d(sQ, &tm_q, col0, row0 + q0, bar_q);
      if (C::TAIL) tma_load_2d(sQt, &tm_qt, col0 + 64, row0 + q0, bar_q);
      for (int j = 0; j < n_blk; ++j) {
        if (j > 0 && !mbar_wait(bar_kfree, (j - 1) & 1, abort_flag, p.status)) break;
        mbar_expect_tx(bar_kfull, C::OP_BYTES);
        tma_load_2d(sK, &tm_k, col0, row0 + j * TK, bar_kfull);
        if (C::TAIL) tma_load_2d(sKt, &tm_kt, col0 + 64, row0 + j * TK, bar_kfull);
        if (j > 0 && !mbar_wait(bar_vfree, (j - 1) & 1, abort_flag, p.status)) break;
        mbar_expect_tx(bar_vfull, C::OP_BYTES);
        tma_load_2d(sV, &tm_v, col0, row0 + j * TK, bar_vfull);
        if (C::TAIL) tma_load_2d(sVt, &tm_vt, col0 + 64, row0 + j * TK, bar_vfull);
      }
    }
  } else if (warp == SM_WARPS + 1) {
    if (lane == 0) {
      // ---------------------------------------------------------------- MMA issuer
      const uint32_t id_s = umma_idesc_bf16(128, TK, false);
      const uint32_t id_o = umma_idesc_bf16(128, 64, true);
      const uint32_t id_ot = umma_idesc_bf16(128, 16, true);
      // S_j = Q K_j^T into buffer j & 1: 4 k-steps of 16 out of the 64-column tiles, one out of the tails
      auto issue_s = [&](int j) {
        const uint32_t d = tmem + static_cast<uint32_t>((j & 1) * 128);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(d, umma_desc(smem_u32(sQ) + k * 32, 1024, 2), umma_desc(smem_u32(sK) + k * 32, 1024, 2), id_s, k ? 1u : 0u);
        if (C::TAIL) umma_bf16(d, umma_desc(smem_u32(sQt), 256, 6), umma_desc(smem_u32(sKt), 256, 6), id_s, 1u);
        umma_commit(&bar_s[j & 1]);
        umma_commit(bar_kfree);
      };
      bool ok = mbar_wait(bar_qz, 0, abort_flag, p.status) && mbar_wait(bar_kfull, 0, abort_flag, p.status);
      if (ok) {
        tc_fence_after();
        issue_s(0);
      }
      for (int j = 0; j < n_blk && ok; ++j) {
        const uint32_t ph = j & 1;
        if (j + 1 < n_blk) {
          // the next block's S goes into the other buffer, which held O_blk of block j - 1
          if (!mbar_wait(bar_kfull, (j + 1) & 1, abort_flag, p.status)) break;
          if (j >= 1 && !mbar_wait(bar_sfree, (j - 1) & 1, abort_flag, p.status)) break;
          tc_fence_after();
          issue_s(j + 1);
        }
        if (!mbar_wait(bar_p, ph, abort_flag, p.status)) break;
        if (!mbar_wait(bar_vfull, ph, abort_flag, p.status)) break;
        tc_fence_after();
        // O_blk = P V over the columns of S_j: 8 k-steps of 16 keys; V's 8-key groups are 1024 (main) / 256 (tail) bytes apart
        const uint32_t d = tmem + static_cast<uint32_t>((j & 1) * 128);
#pragma unroll
        for (int k = 0; k < TK / 16; ++k) {
          const uint64_t a = umma_desc(smem_u32(sP) + (k >> 2) * C::MAIN_BYTES + (k & 3) * 32, 1024, 2);
          umma_bf16(d, a, umma_desc(smem_u32(sV) + k * 2048, 1024, 2), id_o, k ? 1u : 0u);
          if (C::TAIL) umma_bf16(d + 64, a, umma_desc(smem_u32(sVt) + k * 512, 256, 6), id_ot, k ? 1u : 0u);
        }
        umma_commit(bar_o);
        umma_commit(bar_vfree);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax (two threads per query row)
    const int quad = warp & 3, half = warp >> 2;
    const int r = quad * 32 + lane;
    const uint32_t trow = tmem + (static_cast<uint32_t>(quad * 32) << 16);
    bool ok = mbar_wait(bar_q, 0, abort_flag, p.status);
    if (ok) {
      if (C::TAIL && half == 0) {  // zero columns 72..79 of this row of the Q tail (second 16-byte slot, 32B swizzle)
        const uint32_t addr = smem_u32(sQt) + static_cast<uint32_t>(r * 32) + ((1u ^ ((static_cast<uint32_t>(r) >> 2) & 1u)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
        fence_async_smem();
      }
      mbar_arrive(bar_qz);
    }
    float o[C::O_HALF];
#pragma unroll
    for (int i = 0; i < C::O_HALF; ++i) o[i] = 0.0f;
    // o = o * alpha + O_blk for this thread's half of the output columns (O_blk sits in buffer `buf`)
    auto fold = [&](int buf, float alpha) {
      const uint32_t src = trow + static_cast<uint32_t>(buf * 128 + half * C::O_HALF);
      uint32_t v[32];
      tmem_ld_32x32(src, v);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; ++i) o[i] = fmaf(o[i], alpha, __uint_as_float(v[i]));
      if (C::TAIL) {
        uint32_t w[8];
        tmem_ld_32x8(src + 32, w);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 8; ++i) o[32 + i] = fmaf(o[32 + i], alpha, __uint_as_float(w[i]));
      }
    };
    float m_run = -INFINITY, l_run = 0.0f, alpha_prev = 0.0f;
    ok = ok && mbar_wait(&bar_s[0], 0, abort_flag, p.status);
    for (int j = 0; j < n_blk && ok; ++j) {
      const uint32_t sbuf = trow + static_cast<uint32_t>((j & 1) * 128 + half * 64);
      __syncwarp();
      tc_fence_after();
      // pass 1: maximum over this thread's 64 keys, then over the row with the other thread's value
      float mx;
      {
        uint32_t v0[32], v1[32];  // both loads in flight, one wait
        tmem_ld_32x32(sbuf, v0);
        tmem_ld_32x32(sbuf + 32, v1);
        tmem_ld_wait();
        float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          m0 = fmaxf(m0, __uint_as_float(v0[i]));
          m1 = fmaxf(m1, __uint_as_float(v1[i]));
        }
        mx = fmaxf(m0, m1);
      }
      s_m[((j & 1) * 2 + half) * 128 + r] = mx;
      mbar_arrive(&bar_mx[quad]);
      if (!mbar_wait(&bar_mx[quad], j & 1, abort_flag, p.status)) { ok = false; break; }
      mx = fmaxf(mx, s_m[((j & 1) * 2 + (half ^ 1)) * 128 + r]);
      const float m_new = fmaxf(m_run, mx * p.scale_log2);
      const float alpha = ex2_approx(m_run - m_new);
      m_run = m_new;
      if (j > 0) {
        // O_blk of the previous block: fold it, then its buffer is free for S of block j + 1; its completion
        // also means that the tensor core has finished reading P, which pass 2 is about to overwrite
        if (!mbar_wait(bar_o, (j - 1) & 1, abort_flag, p.status)) { ok = false; break; }
        __syncwarp();
        tc_fence_after();
        fold((j - 1) & 1, alpha_prev);
        tc_fence_before();
        mbar_arrive(bar_sfree);
      }
      alpha_prev = alpha;
      // pass 2 (this thread's 64 keys): P = exp2(s * scale - m), row sum, bf16 into the swizzled tile
      float rs = 0.0f;
      const uint32_t tile = smem_u32(sP) + static_cast<uint32_t>(half * C::MAIN_BYTES + r * 128);
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {  // 32 keys = four 16-byte slots
        uint32_t v[32];
        tmem_ld_32x32(sbuf + c * 32, v);
        tmem_ld_wait();
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float p0 = ex2_approx(fmaf(__uint_as_float(v[2 * i]), p.scale_log2, -m_new));
          const float p1 = ex2_approx(fmaf(__uint_as_float(v[2 * i + 1]), p.scale_log2, -m_new));
          rs += p0 + p1;
          pk[i] = pack_bf16x2(p0, p1);
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const uint32_t slot = static_cast<uint32_t>(c * 4 + g);
          const uint32_t addr = tile + ((slot ^ (static_cast<uint32_t>(r) & 7u)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pk[4 * g]), "r"(pk[4 * g + 1]),
                       "r"(pk[4 * g + 2]), "r"(pk[4 * g + 3])
                       : "memory");
        }
      }
      l_run = l_run * alpha + rs;
      fence_async_smem();   // P is read by the tensor core through the async proxy
      tc_fence_before();    // and the S columns are about to be overwritten by O_blk
      mbar_arrive(bar_p);
      if (j + 1 < n_blk && !mbar_wait(&bar_s[(j + 1) & 1], ((j + 1) >> 1) & 1, abort_flag, p.status)) { ok = false; break; }
    }
    if (ok && mbar_wait(bar_o, (n_blk - 1) & 1, abort_flag, p.status)) {
      __syncwarp();
      tc_fence_after();
      fold((n_blk - 1) & 1, alpha_prev);
    } else {
      ok = false;
    }
    // the two threads of a row exchange their partial sums
    if (ok) {
      s_l[half * 128 + r] = l_run;
      mbar_arrive(bar_l);
      ok = mbar_wait(bar_l, 0, abort_flag, p.status);
    }
    if (ok) {
      const float inv_l = 1.0f / (s_l[r] + s_l[128 + r]);
      const int64_t row = static_cast<int64_t>(row0) + q0 + r;
      const int64_t base = row * (static_cast<int64_t>(p.H) * DH) + col0 + half * C::O_HALF;
      const int ngroups = half == 0 ? C::O_HALF / 8 : (DH - C::O_HALF) / 8;  // output columns beyond DH are padding
      float q_inv = 0.0f;
      if (p.out_dtype == QDIT_I8) q_inv = __fdiv_rn(1.0f, p.qa.scale_dev ? __ldg(p.qa.scale_dev) : p.qa.scale);
#pragma unroll
      for (int g = 0; g < C::O_HALF / 8; ++g) {
        if (g < ngroups) {
          float y[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) y[i] = o[8 * g + i] * inv_l;
          if (p.out_dtype == QDIT_I8) {
            *reinterpret_cast<uint2*>(static_cast<uint8_t*>(p.out) + base + 8 * g) = quantize_pack8(y, q_inv, p.qa.zp, p.qa.qmin, p.qa.qmax);
          } else if (p.out_dtype == QDIT_BF16) {
            *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + base + 8 * g) = pack_bf16x8(y);
          } else {
            float* of = static_cast<float*>(p.out) + base + 8 * g;
            *reinterpret_cast<float4*>(of) = make_float4(y[0], y[1], y[2], y[3]);
            *reinterpret_cast<float4*>(of + 4) = make_float4(y[4], y[5], y[6], y[7]);
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == SM_WARPS + 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

// ---------------------------------------------------------------------------------------------------------
// T = 256 (two key blocks): the whole score row fits the CTA's 256 tensor-memory columns, so the softmax is
// taken in one piece instead of online, and the probabilities never leave tensor memory.
//   * Q, both K blocks and V_0 are requested at once; S_0 and S_1 are issued back to back; V_1 is requested into
//     Q's place as soon as the S products have finished reading Q.
//   * One row maximum (one exchange between the two threads of a row), no rescaling.
//   * P = exp2(..) is written back as bf16 pairs over the score columns the same thread has already read
//     (tcgen05.st), and P.V takes its A operand from tensor memory: no shared-memory tile for P, no proxy fence,
//     and P_1 does not wait for the first P.V product.
// Tensor-memory columns of the CTA:  0..63 P_0 | 64..127 O (head dims 0..63) | 128..191 P_1 | 192..207 O (dims 64..79).
// The two threads of a row split a key block into 32-key chunks 0, 2 (first thread) and 1, 3 (second): chunk c of
// block j is read from columns 128 j + 32 c and its 16 packed columns go to 128 j + 32 (c & 1) + 16 (c >> 1), inside
// columns that thread has read before.  P's key order along the columns is therefore chunk 0, 2, 1, 3, and the
// k-steps of P.V pick their V rows in that order.  O's columns are free once both threads of every row have written
// P_0 (main part) and P_1 (tail part): the barriers the MMA issuer waits for anyway.
//   * Head dim 72: the row sum comes out of the tensor core.  Columns 72..79 of a V tail tile are padding (whatever
//     follows the head in memory); the loader warp sets column 72 of every key row to one once the tile has landed, so
//     accumulator column 200 is sum_k P[q,k] over the same bf16 probabilities that multiply V, and the softmax threads
//     neither add the probabilities up nor exchange partial sums.
//   * 8-bit output: the codes of a CTA (128 rows x 72 bytes) are staged in shared memory (K_0's place) and leave with
//     row-contiguous 8-byte stores, 9 per row, instead of every thread writing pieces of its own row.
// 85 KB shared memory and 256 tensor-memory columns: two CTAs per SM.  Every barrier completes exactly once (phase 0).
template <int DH>
struct T256Cfg {
  using B = TCfg<DH>;
  static constexpr int SMEM_BYTES = 4 * B::OP_BYTES + 4096 + 1024;  // Q, K_0, K_1, V_0 (+ tails), barriers and row statistics, alignment
};

template <int DH>
__global__ void __launch_bounds__(TC_THREADS, 2)
attention_tc256_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_qt,
                       const __grid_constant__ CUtensorMap tm_kt, const __grid_constant__ CUtensorMap tm_vt,
                       const AttnTcParams p) {
  using C = TCfg<DH>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                           // Q, later V_1
  uint8_t* sK0 = sQ + C::MAIN_BYTES;
  uint8_t* sK1 = sK0 + C::MAIN_BYTES;
  uint8_t* sV0 = sK1 + C::MAIN_BYTES;
  uint8_t* sQt = sV0 + C::MAIN_BYTES;           // tails (256-byte aligned: 32B-swizzle atoms); Q's, later V_1's
  uint8_t* sK0t = sQt + C::TAIL_BYTES;
  uint8_t* sK1t = sK0t + C::TAIL_BYTES;
  uint8_t* sV0t = sK1t + C::TAIL_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sV0t + C::TAIL_BYTES);
  uint64_t* bar_q = bars + 0;      // Q tiles landed (tx)
  uint64_t* bar_qz = bars + 1;     // Q tail padding zeroed (256 arrivals)
  uint64_t* bar_k = bars + 2;      // [2] K block landed (tx)
  uint64_t* bar_v = bars + 4;      // [2] V block landed (tx)
  uint64_t* bar_s = bars + 6;      // [2] S block complete (commit); [1] also: Q and both K blocks have been read
  uint64_t* bar_p = bars + 8;      // [2] P block written to tensor memory (256 arrivals)
  uint64_t* bar_o = bars + 10;     // both P.V products complete (commit)
  uint64_t* bar_l = bars + 11;     // row sums exchanged (256 arrivals)
  uint64_t* bar_mx = bars + 12;    // [4] row maxima exchanged between the two warps of a lane quadrant (64 arrivals)
  uint64_t* bar_vp = bars + 16;    // [2] V tail block patched: column 72 set to one (32 arrivals)
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 18);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  float* s_l = reinterpret_cast<float*>(tmem_holder + 4);  // [2][128] partial row sums
  float* s_m = s_l + 256;                                  // [2][128] partial row maxima

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * TQ, h = blockIdx.y, b = blockIdx.z;
  const int row0 = b * p.T, col0 = h * DH;
  constexpr uint32_t COL_O = 64, COL_OT = 192;   // accumulator columns: head dims 0..63, head dims 64..79

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_qz, SM_WARPS * 32);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bar_k[i], 1);
      mbar_init(&bar_v[i], 1);
      mbar_init(&bar_s[i], 1);
      mbar_init(&bar_p[i], SM_WARPS * 32);
    }
    mbar_init(bar_o, 1);
    mbar_init(bar_l, SM_WARPS * 32);
    for (int i = 0; i < 4; ++i) mbar_init(&bar_mx[i], 64);
    for (int i = 0; i < 2; ++i) mbar_init(&bar_vp[i], 32);
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == SM_WARPS) {
    if (lane == 0) {
      tma_prefetch_desc(&tm_q);
      tma_prefetch_desc(&tm_k);
      tma_prefetch_desc(&tm_v);
    }
  } else if (warp == SM_WARPS + 1) {
    tmem_alloc(tmem_holder, 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_holder;
  // shared and tensor memory only so far; Q, K and V come from the previous kernel of the stream
  grid_dependency_wait();
  grid_dependency_release();
  // The CTAs of the first wave that share an SM would run their phases (loads, products, exponentials, output) in
  // lockstep, each phase's unit busy in bursts and idle in between.  The second CTA of every SM starts `stagger_ns`
  // late, once: after that the CTAs of an SM stay out of phase, since every later CTA starts when another one ends.
  if (p.stagger_ns > 0) {
    const unsigned linear = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
    if (linear >= p.num_sms && linear < 2u * p.num_sms) {
      const long long t0 = clock64();
      const long long span = static_cast<long long>(p.stagger_ns) * 2;   // clocks at <= 2 GHz: an upper bound, not a timer
      for (int i = 0; i < 4096 && clock64() - t0 < span; ++i) __nanosleep(200);
    }
  }

  if (warp == SM_WARPS) {
    if (lane == 0) {
      // ---------------------------------------------------------------- TMA producer
      mbar_expect_tx(bar_q, C::OP_BYTES);
      tma_load_2d(sQ, &tm_q, col0, row0 + q0, bar_q);
      if (C::TAIL) tma_load_2d(sQt, &tm_qt, col0 + 64, row0 + q0, bar_q);
      mbar_expect_tx(&bar_k[0], C::OP_BYTES);
      tma_load_2d(sK0, &tm_k, col0, row0, &bar_k[0]);
      if (C::TAIL) tma_load_2d(sK0t, &tm_kt, col0 + 64, row0, &bar_k[0]);
      mbar_expect_tx(&bar_k[1], C::OP_BYTES);
      tma_load_2d(sK1, &tm_k, col0, row0 + TK, &bar_k[1]);
      if (C::TAIL) tma_load_2d(sK1t, &tm_kt, col0 + 64, row0 + TK, &bar_k[1]);
      mbar_expect_tx(&bar_v[0], C::OP_BYTES);
      tma_load_2d(sV0, &tm_v, col0, row0, &bar_v[0]);
      if (C::TAIL) tma_load_2d(sV0t, &tm_vt, col0 + 64, row0, &bar_v[0]);
      // V_1 takes Q's place once both S products have read Q
      if (mbar_wait(&bar_s[1], 0, abort_flag, p.status)) {
        mbar_expect_tx(&bar_v[1], C::OP_BYTES);
        tma_load_2d(sQ, &tm_v, col0, row0 + TK, &bar_v[1]);
        if (C::TAIL) tma_load_2d(sQt, &tm_vt, col0 + 64, row0 + TK, &bar_v[1]);
      }
    }
    if (C::TAIL) {
      // the whole warp: column 72 of the landed V tail tiles := 1 (second 16-byte slot of the 32-byte row, 32B swizzle)
#pragma unroll 1
      for (int j = 0; j < 2; ++j) {
        if (!mbar_wait(&bar_v[j], 0, abort_flag, p.status)) break;
        const uint32_t tile = smem_u32(j == 0 ? sV0t : sQt);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t kr = static_cast<uint32_t>(lane + 32 * i);
          asm volatile("st.shared.u16 [%0], %1;" ::"r"(tile + kr * 32u + ((1u ^ ((kr >> 2) & 1u)) << 4)), "h"(static_cast<uint16_t>(0x3F80)) : "memory");
        }
        fence_async_smem();
        mbar_arrive(&bar_vp[j]);
      }
    }
  } else if (warp == SM_WARPS + 1) {
    if (lane == 0) {
      // ---------------------------------------------------------------- MMA issuer
      const uint32_t id_s = umma_idesc_bf16(128, TK, false);
      const uint32_t id_o = umma_idesc_bf16(128, 64, true);
      const uint32_t id_ot = umma_idesc_bf16(128, 16, true);
      // S_j = Q K_j^T into columns 128 j: 4 k-steps of 16 out of the 64-column tiles, one out of the tails
      auto issue_s = [&](int j, const uint8_t* k_main, const uint8_t* k_tail) {
        const uint32_t d = tmem + static_cast<uint32_t>(j * 128);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(d, umma_desc(smem_u32(sQ) + k * 32, 1024, 2), umma_desc(smem_u32(k_main) + k * 32, 1024, 2), id_s, k ? 1u : 0u);
        if (C::TAIL) umma_bf16(d, umma_desc(smem_u32(sQt), 256, 6), umma_desc(smem_u32(k_tail), 256, 6), id_s, 1u);
        umma_commit(&bar_s[j]);
      };
      // k-step s of a P.V product reads P columns 8 s .. 8 s + 7 of its block = 16 keys starting at key_of(s)
      // (chunk order 0, 2, 1, 3); V's 8-key groups are 1024 (main tile) / 256 (tail tile) bytes apart
      auto key16_of = [](int s) { return ((s & 4) ? 2 : 0) + ((s & 2) ? 4 : 0) + (s & 1); };  // in units of 16 keys
      auto issue_pv_main = [&](int j, const uint8_t* v_main) {
#pragma unroll
        for (int s = 0; s < 8; ++s)
          umma_bf16_ta(tmem + COL_O, tmem + static_cast<uint32_t>(j * 128 + 8 * s),
                       umma_desc(smem_u32(v_main) + key16_of(s) * 2048, 1024, 2), id_o, (j | s) ? 1u : 0u);
      };
      auto issue_pv_tail = [&](int j, const uint8_t* v_tail) {
#pragma unroll
        for (int s = 0; s < 8; ++s)
          umma_bf16_ta(tmem + COL_OT, tmem + static_cast<uint32_t>(j * 128 + 8 * s),
                       umma_desc(smem_u32(v_tail) + key16_of(s) * 512, 256, 6), id_ot, (j | s) ? 1u : 0u);
      };
      bool ok = mbar_wait(bar_qz, 0, abort_flag, p.status) && mbar_wait(&bar_k[0], 0, abort_flag, p.status);
      if (ok) {
        tc_fence_after();
        issue_s(0, sK0, sK0t);
      }
      ok = ok && mbar_wait(&bar_k[1], 0, abort_flag, p.status);
      if (ok) {
        tc_fence_after();
        issue_s(1, sK1, sK1t);
      }
      // P_0 written: every thread has finished with the columns of S_0, which now hold P_0 and will hold O
      ok = ok && mbar_wait(&bar_p[0], 0, abort_flag, p.status) && mbar_wait(&bar_v[0], 0, abort_flag, p.status);
      if (ok) {
        tc_fence_after();
        issue_pv_main(0, sV0);
      }
      ok = ok && mbar_wait(&bar_p[1], 0, abort_flag, p.status) && mbar_wait(&bar_v[1], 0, abort_flag, p.status);
      if (C::TAIL) ok = ok && mbar_wait(&bar_vp[0], 0, abort_flag, p.status) && mbar_wait(&bar_vp[1], 0, abort_flag, p.status);
      if (ok) {
        tc_fence_after();
        issue_pv_main(1, sQ);
        if (C::TAIL) {
          issue_pv_tail(0, sV0t);
          issue_pv_tail(1, sQt);
        }
        umma_commit(bar_o);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax (two threads per query row)
    const int quad = warp & 3, half = warp >> 2;
    const int r = quad * 32 + lane;
    const uint32_t trow = tmem + (static_cast<uint32_t>(quad * 32) << 16);
    // the output quantizer's scale is fetched now, long before it is needed (a load from global memory at the end
    // of the chain would add its whole latency to the CTA's life)
    float q_inv = 0.0f;
    if (p.out_dtype == QDIT_I8) q_inv = __fdiv_rn(1.0f, p.qa.scale_dev ? __ldg(p.qa.scale_dev) : p.qa.scale);
    bool ok = mbar_wait(bar_q, 0, abort_flag, p.status);
    if (ok) {
      if (C::TAIL && half == 0) {  // zero columns 72..79 of this row of the Q tail (second 16-byte slot, 32B swizzle)
        const uint32_t addr = smem_u32(sQt) + static_cast<uint32_t>(r * 32) + ((1u ^ ((static_cast<uint32_t>(r) >> 2) & 1u)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
        fence_async_smem();
      }
      mbar_arrive(bar_qz);
    }
    // row maximum over this thread's 64 keys of each block (chunks half and half + 2), then over the row with the
    // other thread's value
    float mx = -INFINITY;
#pragma unroll 1
    for (int j = 0; j < 2 && ok; ++j) {
      if (!mbar_wait(&bar_s[j], 0, abort_flag, p.status)) { ok = false; break; }
      __syncwarp();
      tc_fence_after();
      uint32_t v0[32], v1[32];  // both loads in flight, one wait
      const uint32_t sbuf = trow + static_cast<uint32_t>(j * 128 + half * 32);
      tmem_ld_32x32(sbuf, v0);
      tmem_ld_32x32(sbuf + 64, v1);
      tmem_ld_wait();
      float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        m0 = fmaxf(m0, __uint_as_float(v0[i]));
        m1 = fmaxf(m1, __uint_as_float(v1[i]));
      }
      mx = fmaxf(mx, fmaxf(m0, m1));
    }
    if (ok) {
      s_m[half * 128 + r] = mx;
      mbar_arrive(&bar_mx[quad]);
      ok = mbar_wait(&bar_mx[quad], 0, abort_flag, p.status);
    }
    float rs = 0.0f;
    bool staged = false;
    if (ok) {
      const float m_row = fmaxf(mx, s_m[(half ^ 1) * 128 + r]) * p.scale_log2;
      const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nm2 = make_float2(-m_row, -m_row);
#pragma unroll 1
      for (int j = 0; j < 2; ++j) {
        // P_j = exp2(s * scale - m) for this thread's two chunks of block j: bf16 pairs back into tensor memory,
        // over columns this thread has already read; row sum in f32
        uint32_t va[32], vb[32];   // both chunks in flight, one wait
        tmem_ld_32x32(trow + static_cast<uint32_t>(j * 128 + half * 32), va);
        tmem_ld_32x32(trow + static_cast<uint32_t>(j * 128 + half * 32 + 64), vb);
        tmem_ld_wait();
#pragma unroll
        for (int w = 0; w < 2; ++w) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float2 a = __ffma2_rn(make_float2(__uint_as_float(w ? vb[2 * i] : va[2 * i]), __uint_as_float(w ? vb[2 * i + 1] : va[2 * i + 1])), sc2, nm2);
            const float p0 = ex2_approx(a.x), p1 = ex2_approx(a.y);
            if (!C::TAIL) rs += p0 + p1;
            pk[i] = pack_bf16x2(p0, p1);
          }
          tmem_st_32x16(trow + static_cast<uint32_t>(j * 128 + half * 32 + w * 16), pk);
        }
        tmem_st_wait();
        tc_fence_before();   // P_j is read, and the rest of S_j overwritten, by the tensor core
        mbar_arrive(&bar_p[j]);
      }
    }
    // the two threads of a row exchange their partial sums (with a tail, the sum is accumulator column 200)
    if (ok && !C::TAIL) {
      s_l[half * 128 + r] = rs;
      mbar_arrive(bar_l);
      ok = mbar_wait(bar_l, 0, abort_flag, p.status);
    }
    if (ok && mbar_wait(bar_o, 0, abort_flag, p.status)) {
      __syncwarp();
      tc_fence_after();
      // first thread of a row: head dims 0..31; second: head dims 32..63 and the tail 64..71
      float o[40];
      float l_row = 0.0f;
      {
        uint32_t v[32];
        tmem_ld_32x32(trow + COL_O + static_cast<uint32_t>(half * 32), v);
        if (C::TAIL) {
          uint32_t w[8], wl[8];
          if (half == 1) tmem_ld_32x8(trow + COL_OT, w);
          tmem_ld_32x8(trow + COL_OT + 8, wl);   // column 200: the row sum
          tmem_ld_wait();
          if (half == 1) {
#pragma unroll
            for (int i = 0; i < 8; ++i) o[32 + i] = __uint_as_float(w[i]);
          }
          l_row = __uint_as_float(wl[0]);
        } else {
          tmem_ld_wait();
          l_row = s_l[r] + s_l[128 + r];
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = __uint_as_float(v[i]);
      }
      const float inv_l = 1.0f / l_row;
      const int64_t row = static_cast<int64_t>(row0) + q0 + r;
      const int64_t base = row * (static_cast<int64_t>(p.H) * DH) + col0 + half * 32;
      const int ngroups = (C::TAIL && half == 1) ? 5 : 4;
      if (p.out_dtype == QDIT_I8) {
        // codes into the staging tile (K_0's place: both S products are long done): rows of DH bytes, pitch DH + 8
        uint8_t* srow = sK0 + r * (DH + 8) + half * 32;
#pragma unroll
        for (int g = 0; g < 5; ++g) {
          if (g < ngroups) {
            float y[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) y[i] = o[8 * g + i] * inv_l;
            *reinterpret_cast<uint2*>(srow + 8 * g) = quantize_pack8(y, q_inv, p.qa.zp, p.qa.qmin, p.qa.qmax);
          }
        }
        staged = true;
      } else {
#pragma unroll
        for (int g = 0; g < 5; ++g) {
          if (g < ngroups) {
            float y[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) y[i] = o[8 * g + i] * inv_l;
            if (p.out_dtype == QDIT_BF16) {
              *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + base + 8 * g) = pack_bf16x8(y);
            } else {
              float* of = static_cast<float*>(p.out) + base + 8 * g;
              *reinterpret_cast<float4*>(of) = make_float4(y[0], y[1], y[2], y[3]);
              *reinterpret_cast<float4*>(of + 4) = make_float4(y[4], y[5], y[6], y[7]);
            }
          }
        }
      }
    }
    // 8-bit output: the staged codes leave row by row, 8 bytes per thread and piece.  Every softmax thread comes here
    // (also after a failed wait), so the named barrier is complete.
    if (p.out_dtype == QDIT_I8) {
      asm volatile("bar.sync 1, %0;" ::"n"(SM_WARPS * 32) : "memory");
      if (staged && !*abort_flag) {
        constexpr int PIECES = DH / 8;
        uint8_t* gout = static_cast<uint8_t*>(p.out) + (static_cast<int64_t>(row0) + q0) * (static_cast<int64_t>(p.H) * DH) + col0;
        for (int i = threadIdx.x; i < 128 * PIECES; i += SM_WARPS * 32) {
          const int rr = i / PIECES, pc = i % PIECES;
          *reinterpret_cast<uint2*>(gout + static_cast<int64_t>(rr) * (static_cast<int64_t>(p.H) * DH) + 8 * pc) =
              *reinterpret_cast<const uint2*>(sK0 + rr * (DH + 8) + 8 * pc);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == SM_WARPS + 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

template <int DH>
int32_t launch_tc(qdit_ctx* ctx, const void* q, const void* k, const void* v, int64_t ld, int B, int H, int T,
                  const AttnTcParams& p) {
  using C = TCfg<DH>;
  QDIT_TRY(qdit_allow_smem(ctx, attention_tc_kernel<DH>, C::SMEM_BYTES));
  QDIT_TRY(qdit_allow_smem(ctx, attention_tc256_kernel<DH>, T256Cfg<DH>::SMEM_BYTES));
  const uint64_t rows = static_cast<uint64_t>(B) * T, cols = static_cast<uint64_t>(H) * DH;
  CUtensorMap tq, tk, tv, tqt, tkt, tvt;
  QDIT_TRY(qdit_get_tmap(ctx, q, rows, cols, ld, 128, 64, 1, 2, &tq));
  QDIT_TRY(qdit_get_tmap(ctx, k, rows, cols, ld, 128, 64, 1, 2, &tk));
  QDIT_TRY(qdit_get_tmap(ctx, v, rows, cols, ld, 128, 64, 1, 2, &tv));
  tqt = tq;
  tkt = tk;
  tvt = tv;
  if (C::TAIL) {
    QDIT_TRY(qdit_get_tmap(ctx, q, rows, cols, ld, 128, 16, 3, 2, &tqt));
    QDIT_TRY(qdit_get_tmap(ctx, k, rows, cols, ld, 128, 16, 3, 2, &tkt));
    QDIT_TRY(qdit_get_tmap(ctx, v, rows, cols, ld, 128, 16, 3, 2, &tvt));
  }
  dim3 grid(T / TQ, H, B);
  ProfScope prof(ctx, QDIT_PROF_ATTENTION, 4.0 * B * H * static_cast<double>(T) * T * DH);
  if (T == 2 * TK && ctx->opt[QDIT_OPT_ATTN] != 2) {  // the whole score row in tensor memory (option 2 forces the general kernel)
    QDIT_CUDA_CHECK(ctx, qdit_launch_overlapped(ctx, attention_tc256_kernel<DH>, grid, dim3(TC_THREADS), T256Cfg<DH>::SMEM_BYTES, tq, tk, tv, tqt, tkt, tvt, p));
    return qdit_after_launch(ctx, "attention_tc256_kernel");
  }
  QDIT_CUDA_CHECK(ctx, qdit_launch_overlapped(ctx, attention_tc_kernel<DH>, grid, dim3(TC_THREADS), C::SMEM_BYTES, tq, tk, tv, tqt, tkt, tvt, p));
  return qdit_after_launch(ctx, "attention_tc_kernel");
}

}  // namespace

// Tensor-core attention for T % 128 == 0 and head dim 64 or 72 (arguments already validated by qdit_attention).
int32_t qdit_launch_attention_tc(qdit_ctx* ctx, const void* q, const void* k, const void* v, int64_t ld, int B, int H,
                                 int T, int dh, float softmax_scale, void* out, int out_dtype, QuantArgs qa) {
  AttnTcParams p{};
  p.T = T;
  p.H = H;
  p.scale_log2 = softmax_scale * 1.4426950408889634f;
  p.out = out;
  p.out_dtype = out_dtype;
  p.qa = qa;
  p.status = ctx->d_status;
  p.stagger_ns = ctx->opt[QDIT_OPT_ATTN_STAGGER_NS];
  p.num_sms = static_cast<unsigned>(ctx->num_sms);
  if (dh == 64) return launch_tc<64>(ctx, q, k, v, ld, B, H, T, p);
  return launch_tc<72>(ctx, q, k, v, ld, B, H, T, p);
}
