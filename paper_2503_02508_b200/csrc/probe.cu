// Tensor-pipe probes: what the int8 GEMM kernels' main loop can reach at most on this device, measured rather than
// quoted.  Not part of the denoising path (the paper has no counterpart); bench.py --workload mma_probe prints them.
//   mode 0: one thread per SM issues tcgen05.mma kind::i8 (M 128, N = n, K 32) on operands that stay in shared memory:
//           the instruction path's own rate.
//   mode 1: the same instruction stream fed the way the GEMM kernels feed it: a TMA producer refills a ring of
//           128B-swizzled stages (128 weight rows + n activation rows of 128 bytes) from an L2-resident matrix, the
//           issuer waits for each stage and frees it with a commit: the main loop of the channel-major kernel with
//           no epilogue.
// Every wait is bounded; the accumulator is never read (the products are discarded).
#include "common.cuh"
#include "internal.h"

namespace {

using namespace qd;

constexpr int PROBE_STAGES = 4;
constexpr int PROBE_THREADS = 96;   // warp 0: TMA producer, warp 1: MMA issuer, warp 2: tensor-memory owner

struct ProbeParams {
  int n, iters, mode, rows_w, rows_a;
  int* status;
};

__global__ void __launch_bounds__(PROBE_THREADS, 1) mma_probe_kernel(const __grid_constant__ CUtensorMap tm_w,
                                                                     const __grid_constant__ CUtensorMap tm_a, const ProbeParams p) {
  extern __shared__ uint8_t probe_smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(probe_smem_raw) + 1023) & ~uintptr_t(1023));
  const int a_bytes = 128 * 128, b_bytes = p.n * 128, stage_bytes = a_bytes + b_bytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + PROBE_STAGES * stage_bytes);
  uint64_t* empty_bar = full_bar + PROBE_STAGES;
  uint64_t* done_bar = empty_bar + PROBE_STAGES;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(done_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < PROBE_STAGES; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&empty_bar[i], 1);
    }
    mbar_init(done_bar, 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  // operands of mode 0 (and the first contents of every stage): zeros, a valid int8 tile in any layout
  for (int i = threadIdx.x; i < PROBE_STAGES * stage_bytes / 16; i += PROBE_THREADS) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
  fence_async_smem();
  if (warp == 2) {
    tmem_alloc(tmem_holder, 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_holder;
  if (warp == 0 && lane == 0 && p.mode == 1) {
    int stage = 0;
    uint32_t phase = 0;
    for (int it = 0; it < p.iters; ++it) {
      if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, p.status)) break;
      uint8_t* sW = smem + stage * stage_bytes;
      mbar_expect_tx(&full_bar[stage], static_cast<uint32_t>(stage_bytes));
      // walk the small matrices so that consecutive stages come from different lines of L2
      const int kc = (it & 7) * 128;
      tma_load_2d(sW, &tm_w, kc, ((it >> 3) * 128) % p.rows_w, &full_bar[stage]);
      tma_load_2d(sW + a_bytes, &tm_a, kc, ((it >> 3) * p.n) % p.rows_a, &full_bar[stage]);
      if (++stage == PROBE_STAGES) { stage = 0; phase ^= 1u; }
    }
    if (*abort_flag) {
      // a wait ran out somewhere: let this thread's copies in flight land (bounded) before the CTA's memory goes away
      volatile int never = 0;
      for (int i = 0; i < PROBE_STAGES; ++i) {
        if (--stage < 0) { stage = PROBE_STAGES - 1; phase ^= 1u; }
        mbar_wait_limited(&full_bar[stage], phase, &never, p.status, 1u << 16);
      }
    }
  } else if (warp == 1 && lane == 0) {
    const uint32_t idesc = umma_idesc_i8(128, static_cast<uint32_t>(p.n), false);
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int it = 0; it < p.iters && ok; ++it) {
      if (p.mode == 1) {
        if (!mbar_wait(&full_bar[stage], phase, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
      }
      const uint64_t a_desc = umma_desc_k_sw128(smem_u32(smem + stage * stage_bytes));
      const uint64_t b_desc = umma_desc_k_sw128(smem_u32(smem + stage * stage_bytes + a_bytes));
#pragma unroll
      for (int k = 0; k < 4; ++k) umma_i8(tmem, a_desc + static_cast<uint64_t>(2 * k), b_desc + static_cast<uint64_t>(2 * k), idesc, (it | k) ? 1u : 0u);
      if (p.mode == 1) umma_commit(&empty_bar[stage]);
      if (++stage == PROBE_STAGES) { stage = 0; phase ^= 1u; }
    }
    umma_commit(done_bar);
    mbar_wait(done_bar, 0, abort_flag, p.status);   // all products (and with them all stage reads) have completed
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

}  // namespace

extern "C" int32_t qdit_probe_mma_rate(qdit_ctx* ctx, int mode, int n, int iters, const void* operands, int64_t rows, float* ms_host) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (!ms_host) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "ms_host is NULL");
  if (mode != 0 && mode != 1) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "mode must be 0 or 1");
  if (n < 64 || n > 256 || n % 64) return qdit_fail(ctx, QDIT_ERR_SHAPE, "n must be 64, 128, 192 or 256");
  if (iters < 1 || iters > (1 << 16)) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "iters must be in 1..65536");
  if (!operands || rows < 256 || rows % 256 || !aligned16(operands)) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "operands: int8 [rows][1024], rows a multiple of 256, 16-byte aligned");
  CUtensorMap tw, ta;
  QDIT_TRY(qdit_get_tmap(ctx, operands, static_cast<uint64_t>(rows), 1024, 1024, 128, 128, 1, 1, &tw));
  QDIT_TRY(qdit_get_tmap(ctx, operands, static_cast<uint64_t>(rows), 1024, 1024, static_cast<uint32_t>(n), 128, 1, 1, &ta));
  ProbeParams p{};
  p.n = n;
  p.iters = iters;
  p.mode = mode;
  p.rows_w = static_cast<int>(rows);
  p.rows_a = static_cast<int>(rows - rows % n);
  p.status = ctx->d_status;
  const int smem = PROBE_STAGES * (128 * 128 + n * 128) + 256 + 1024;
  QDIT_TRY(qdit_allow_smem(ctx, mma_probe_kernel, PROBE_STAGES * (128 * 128 + 256 * 128) + 256 + 1024));
  cudaEvent_t e0, e1;
  QDIT_CUDA_CHECK(ctx, cudaEventCreate(&e0));
  if (cudaEventCreate(&e1) != cudaSuccess) {
    cudaEventDestroy(e0);
    return qdit_fail(ctx, QDIT_ERR_CUDA, "probe timing: event creation failed");
  }
  cudaEventRecord(e0, ctx->stream);
  mma_probe_kernel<<<ctx->num_sms, PROBE_THREADS, smem, ctx->stream>>>(tw, ta, p);
  int32_t st = qdit_after_launch(ctx, "mma_probe_kernel");
  cudaEventRecord(e1, ctx->stream);
  cudaError_t err = cudaEventSynchronize(e1);
  float ms = 0.0f;
  if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (st != QDIT_OK) return st;
  if (err != cudaSuccess) return qdit_fail(ctx, QDIT_ERR_CUDA, "probe timing: %s", cudaGetErrorString(err));
  *ms_host = ms;
  return QDIT_OK;
}
