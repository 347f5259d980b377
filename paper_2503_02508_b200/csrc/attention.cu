// Non-causal softmax attention in bf16 between the quantized linears: the entry point qdit_attention and the
// mma.sync kernel that serves token counts that are not a multiple of 128 (the tcgen05 kernel in attention_tc.cu
// takes all others, among them both image sizes of the paper's experiments).
//
// One CTA = 128 (or 64) queries of one (sample, head); one warp per 16 query rows.  Q and 64-key K/V tiles
// are staged by TMA (a 4-deep ring with mbarrier completion: at 256 tokens the whole K and V of the head are
// requested up front and the loop never synchronises) straight out of the token-major QKV matrix:
// head_dim 64 uses 128-byte-swizzled rows, head_dim 72 keeps its natural 144-byte rows (which are
// already bank-conflict-free for ldmatrix).  S = Q K^T and O = P V run on bf16 mma.sync with f32
// accumulation; softmax is the online (running max / running sum) form in f32, exponentials in base 2.
// The output can be written as f32, bf16, or directly as the projection's 8-bit activation codes.
#include <cstdlib>

#include "common.cuh"
#include "internal.h"

namespace {

using namespace qd;

constexpr int BKV = 64;     // keys per staged tile
constexpr int KV_STAGES = 4;  // ring depth

struct AttnParams {
  int T, H, dh;
  float scale_log2;  // softmax_scale * log2(e)
  void* out;
  int out_dtype;
  QuantArgs qa;
  int* status;
};

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t& r0, uint32_t& r1, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2_t(uint32_t& r0, uint32_t& r1, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int DH>
struct ACfg {
  static constexpr int ROW_BYTES = DH * 2;
  static constexpr bool SWZ = (DH == 64);
  static constexpr int TILE_BYTES = 64 * ROW_BYTES;  // 8192 or 9216: both multiples of 1024
  static constexpr int KSTEPS = (DH + 15) / 16;      // k16 steps of Q K^T; the last one is half for DH = 72
  static constexpr bool HALF_TAIL = (DH % 16) == 8;
  static constexpr int NT_O = DH / 8;                // 8-wide column tiles of O
  static constexpr int smem_bytes(int qw) { return (qw / 4 + 2 * KV_STAGES) * TILE_BYTES + 128 + 1024; }
};

template <int DH>
__device__ __forceinline__ uint32_t tile_addr(uint32_t base, int row, int col_elem) {
  uint32_t c = static_cast<uint32_t>(col_elem) * 2u;
  if (ACfg<DH>::SWZ) c ^= static_cast<uint32_t>(row & 7) << 4;
  return base + static_cast<uint32_t>(row) * ACfg<DH>::ROW_BYTES + c;
}

template <int DH, int QW>  // QW query warps (4 or 8) -> 16 * QW queries per CTA
__global__ void __launch_bounds__(QW * 32, QW == 8 ? 2 : 4)
attention_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
  using C = ACfg<DH>;
  constexpr int BQ = QW * 16, QTILES = QW / 4;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                                      // QTILES tiles of 64 rows
  uint8_t* sK = smem + QTILES * C::TILE_BYTES;             // KV_STAGES tiles
  uint8_t* sV = sK + KV_STAGES * C::TILE_BYTES;            // KV_STAGES tiles
  uint64_t* bar_q = reinterpret_cast<uint64_t*>(sV + KV_STAGES * C::TILE_BYTES);
  uint64_t* bar_kv = bar_q + 1;                            // one per stage
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_kv + KV_STAGES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * BQ, h = blockIdx.y, b = blockIdx.z;
  const int row0 = b * p.T;       // first token row of this sample
  const int col0 = h * DH;        // first column of this head
  const int n_kv = p.T / BKV;

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    for (int s = 0; s < KV_STAGES; ++s) mbar_init(&bar_kv[s], 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    mbar_expect_tx(bar_q, QTILES * C::TILE_BYTES);
    for (int t = 0; t < QTILES; ++t) tma_load_2d(sQ + t * C::TILE_BYTES, &tm_q, col0, row0 + q0 + t * 64, bar_q);
    for (int j = 0; j < KV_STAGES && j < n_kv; ++j) {
      mbar_expect_tx(&bar_kv[j], 2 * C::TILE_BYTES);
      tma_load_2d(sK + j * C::TILE_BYTES, &tm_k, col0, row0 + j * BKV, &bar_kv[j]);
      tma_load_2d(sV + j * C::TILE_BYTES, &tm_v, col0, row0 + j * BKV, &bar_kv[j]);
    }
  }

  const uint32_t aQ = smem_u32(sQ);
  uint32_t qf[C::KSTEPS][4];
  bool ok = mbar_wait(bar_q, 0, abort_flag, p.status);
  if (ok) {
    const uint32_t aQw = aQ + static_cast<uint32_t>((warp >> 2) * C::TILE_BYTES);  // 64-row tile of this warp
    const int r = (warp & 3) * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
    for (int ks = 0; ks < C::KSTEPS; ++ks) {
      if (C::HALF_TAIL && ks == C::KSTEPS - 1) {
        ldsm_x2(qf[ks][0], qf[ks][1], tile_addr<DH>(aQw, r, ks * 16));
        qf[ks][2] = 0u;
        qf[ks][3] = 0u;
      } else {
        ldsm_x4(qf[ks], tile_addr<DH>(aQw, r, ks * 16 + (lane >> 4) * 8));
      }
    }
  }

  float o[C::NT_O][4];
#pragma unroll
  for (int i = 0; i < C::NT_O; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.0f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.0f, 0.0f};

  for (int j = 0; j < n_kv && ok; ++j) {
    const int st = j % KV_STAGES;
    if (!mbar_wait(&bar_kv[st], static_cast<uint32_t>(j / KV_STAGES) & 1u, abort_flag, p.status)) {
      ok = false;
      break;
    }
    __syncwarp();
    const uint32_t aK = smem_u32(sK + st * C::TILE_BYTES);
    const uint32_t aV = smem_u32(sV + st * C::TILE_BYTES);

    // ---- S = Q K^T for 64 keys: 8 column tiles of 8 keys
    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.0f;
#pragma unroll
    for (int np = 0; np < 4; ++np) {
#pragma unroll
      for (int ks = 0; ks < C::KSTEPS; ++ks) {
        if (C::HALF_TAIL && ks == C::KSTEPS - 1) {
          uint32_t b0, b1;
          ldsm_x2(b0, b1, tile_addr<DH>(aK, np * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, ks * 16));
          mma_bf16(s[2 * np], qf[ks][0], qf[ks][1], 0u, 0u, b0, 0u);
          mma_bf16(s[2 * np + 1], qf[ks][0], qf[ks][1], 0u, 0u, b1, 0u);
        } else {
          uint32_t bb[4];
          ldsm_x4(bb, tile_addr<DH>(aK, np * 16 + (lane & 7) + (lane >> 4) * 8, ks * 16 + ((lane >> 3) & 1) * 8));
          mma_bf16(s[2 * np], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], bb[0], bb[1]);
          mma_bf16(s[2 * np + 1], qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], bb[2], bb[3]);
        }
      }
    }

    // ---- online softmax; this thread holds rows g (regs 0,1) and g+8 (regs 2,3)
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      s[i][0] *= p.scale_log2; s[i][1] *= p.scale_log2; s[i][2] *= p.scale_log2; s[i][3] *= p.scale_log2;
      mx[0] = fmaxf(mx[0], fmaxf(s[i][0], s[i][1]));
      mx[1] = fmaxf(mx[1], fmaxf(s[i][2], s[i][3]));
    }
    float alpha[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float m_new = fmaxf(m_run[r], mx[r]);
      alpha[r] = exp2f(m_run[r] - m_new);
      m_run[r] = m_new;
    }
    float rs[2] = {0.0f, 0.0f};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      s[i][0] = exp2f(s[i][0] - m_run[0]);
      s[i][1] = exp2f(s[i][1] - m_run[0]);
      s[i][2] = exp2f(s[i][2] - m_run[1]);
      s[i][3] = exp2f(s[i][3] - m_run[1]);
      rs[0] += s[i][0] + s[i][1];
      rs[1] += s[i][2] + s[i][3];
    }
    l_run[0] = l_run[0] * alpha[0] + rs[0];
    l_run[1] = l_run[1] * alpha[1] + rs[1];
#pragma unroll
    for (int i = 0; i < C::NT_O; ++i) {
      o[i][0] *= alpha[0]; o[i][1] *= alpha[0]; o[i][2] *= alpha[1]; o[i][3] *= alpha[1];
    }

    // ---- O += P V; P fragments come from the S accumulators
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      const uint32_t a0 = pack_bf16x2(s[2 * kk][0], s[2 * kk][1]);
      const uint32_t a1 = pack_bf16x2(s[2 * kk][2], s[2 * kk][3]);
      const uint32_t a2 = pack_bf16x2(s[2 * kk + 1][0], s[2 * kk + 1][1]);
      const uint32_t a3 = pack_bf16x2(s[2 * kk + 1][2], s[2 * kk + 1][3]);
      const int vr = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int dp = 0; dp < DH / 16; ++dp) {
        uint32_t bb[4];
        ldsm_x4_t(bb, tile_addr<DH>(aV, vr, dp * 16 + (lane >> 4) * 8));
        mma_bf16(o[2 * dp], a0, a1, a2, a3, bb[0], bb[1]);
        mma_bf16(o[2 * dp + 1], a0, a1, a2, a3, bb[2], bb[3]);
      }
      if (C::HALF_TAIL) {
        uint32_t b0, b1;
        ldsm_x2_t(b0, b1, tile_addr<DH>(aV, vr, DH - 8));
        mma_bf16(o[C::NT_O - 1], a0, a1, a2, a3, b0, b1);
      }
    }
    if (j + KV_STAGES < n_kv) {
      __syncthreads();  // everyone is done with stage st before it is refilled
      if (threadIdx.x == 0) {
        mbar_expect_tx(&bar_kv[st], 2 * C::TILE_BYTES);
        tma_load_2d(sK + st * C::TILE_BYTES, &tm_k, col0, row0 + (j + KV_STAGES) * BKV, &bar_kv[st]);
        tma_load_2d(sV + st * C::TILE_BYTES, &tm_v, col0, row0 + (j + KV_STAGES) * BKV, &bar_kv[st]);
      }
    }
  }
  if (!ok) return;

  // ---- finish: divide by the row sums and store
  float inv_l[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    float l = l_run[r];
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    inv_l[r] = 1.0f / l;
  }
  const int g = lane >> 2, t = lane & 3;
  const int64_t ldo = static_cast<int64_t>(p.H) * DH;
  float q_inv = 0.0f;
  if (p.out_dtype == QDIT_I8) q_inv = __fdiv_rn(1.0f, p.qa.scale_dev ? __ldg(p.qa.scale_dev) : p.qa.scale);
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int64_t row = static_cast<int64_t>(row0) + q0 + warp * 16 + g + r * 8;
    const int64_t base = row * ldo + col0 + 2 * t;
#pragma unroll
    for (int i = 0; i < C::NT_O; ++i) {
      const float v0 = o[i][2 * r] * inv_l[r], v1 = o[i][2 * r + 1] * inv_l[r];
      const int64_t off = base + i * 8;
      if (p.out_dtype == QDIT_I8) {
        const int c0 = __float2int_rn(quantize_code(v0, q_inv, p.qa.zp, p.qa.qmin, p.qa.qmax));
        const int c1 = __float2int_rn(quantize_code(v1, q_inv, p.qa.zp, p.qa.qmin, p.qa.qmax));
        // the 4 lanes of a quad hold 8 consecutive columns of this row: gather them into one 8-byte store
        uint32_t w = static_cast<uint32_t>((c0 & 0xFF) | ((c1 & 0xFF) << 8));
        w |= __shfl_down_sync(0xffffffffu, w, 1) << 16;            // lanes t = 0, 2: columns 2t .. 2t + 3
        const uint32_t w_hi = __shfl_down_sync(0xffffffffu, w, 2);  // lane t = 0 receives lane 2's word
        if (t == 0) *reinterpret_cast<uint2*>(static_cast<uint8_t*>(p.out) + off) = make_uint2(w, w_hi);
      } else if (p.out_dtype == QDIT_BF16) {
        *reinterpret_cast<uint32_t*>(static_cast<__nv_bfloat16*>(p.out) + off) = pack_bf16x2(v0, v1);
      } else {
        *reinterpret_cast<float2*>(static_cast<float*>(p.out) + off) = make_float2(v0, v1);
      }
    }
  }
}

template <int DH, int QW>
int32_t launch_attention(qdit_ctx* ctx, const void* q, const void* k, const void* v, int64_t ld, int B, int H, int T,
                         const AttnParams& p) {
  using C = ACfg<DH>;
  QDIT_TRY(qdit_allow_smem(ctx, attention_kernel<DH, QW>, C::smem_bytes(QW)));
  const uint64_t rows = static_cast<uint64_t>(B) * T, cols = static_cast<uint64_t>(H) * DH;
  CUtensorMap tq, tk, tv;
  QDIT_TRY(qdit_get_tmap(ctx, q, rows, cols, ld, 64, DH, C::SWZ ? 1 : 0, 2, &tq));
  QDIT_TRY(qdit_get_tmap(ctx, k, rows, cols, ld, 64, DH, C::SWZ ? 1 : 0, 2, &tk));
  QDIT_TRY(qdit_get_tmap(ctx, v, rows, cols, ld, 64, DH, C::SWZ ? 1 : 0, 2, &tv));
  dim3 grid(T / (QW * 16), H, B);
  ProfScope prof(ctx, QDIT_PROF_ATTENTION, 4.0 * B * H * static_cast<double>(T) * T * DH);
  attention_kernel<DH, QW><<<grid, QW * 32, C::smem_bytes(QW), ctx->stream>>>(tq, tk, tv, p);
  return qdit_after_launch(ctx, "attention_kernel");
}

}  // namespace

int32_t qdit_launch_attention_tc(qdit_ctx* ctx, const void* q, const void* k, const void* v, int64_t ld, int B, int H,
                                 int T, int dh, float softmax_scale, void* out, int out_dtype, QuantArgs qa);

extern "C" int32_t qdit_attention(qdit_ctx* ctx, const void* q, const void* k, const void* v, int64_t ld, int B, int H,
                                  int T, int dh, float softmax_scale, void* out, int out_dtype,
                                  const qdit_qparams* out_qp, const float* out_scale_dev) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (B < 0 || H <= 0 || T < 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "bad sizes");
  if (B == 0 || T == 0) return QDIT_OK;
  if (!q || !k || !v || !out) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  if (dh != 64 && dh != 72) return qdit_fail(ctx, QDIT_ERR_SHAPE, "head_dim %d not supported (64 or 72)", dh);
  if (T % 64 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "T = %d must be a multiple of 64", T);
  if (H > 65535 || B > 65535) return qdit_fail(ctx, QDIT_ERR_SHAPE, "H or B too large");
  if (ld < static_cast<int64_t>(H) * dh || ld % 8 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "ld must be >= H*dh and a multiple of 8");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "pointers must be 16-byte aligned");
  if (out_dtype != QDIT_I8 && out_dtype != QDIT_BF16 && out_dtype != QDIT_F32) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "bad out_dtype");
  AttnParams p{};
  p.T = T;
  p.H = H;
  p.dh = dh;
  p.scale_log2 = softmax_scale * 1.4426950408889634f;
  p.out = out;
  p.out_dtype = out_dtype;
  p.status = ctx->d_status;
  if (out_dtype == QDIT_I8) {
    QDIT_TRY(qdit_check_qparams(ctx, out_qp, out_scale_dev != nullptr));
    p.qa = make_quant_args(*out_qp, out_scale_dev);
  }
  // token counts that fill 128-query tiles run on the tcgen05 kernel; the mma.sync kernel covers the rest
  if (T % 128 == 0 && ctx->opt[QDIT_OPT_ATTN] != 1)
    return qdit_launch_attention_tc(ctx, q, k, v, ld, B, H, T, dh, softmax_scale, out, out_dtype, p.qa);
  const bool wide = T % 128 == 0;  // 128 queries per CTA when the token count allows
  if (dh == 64) return wide ? launch_attention<64, 8>(ctx, q, k, v, ld, B, H, T, p) : launch_attention<64, 4>(ctx, q, k, v, ld, B, H, T, p);
  return wide ? launch_attention<72, 8>(ctx, q, k, v, ld, B, H, T, p) : launch_attention<72, 4>(ctx, q, k, v, ld, B, H, T, p);
}
