// Dynamic activation quantizer that brings its own scratch memory.
//
// The dynamic quantizer needs a place to reduce max|x| before it can quantize.  The regular entry point
// borrows that place from the caller (dyn_scale) or, inside the sampler, from a workspace the library
// allocated.  Some callers can do neither: code that runs where the CUDA allocator must not be touched
// (inside a region that is being stream-captured, in a plug-in that was handed only its input and output
// tensors, in a process whose memory budget is fixed up front).  For them the partial maxima live in a
// fixed array in the library's own device image.  Nothing here calls cudaMalloc, cudaFree or any routine
// that allocates.
#include <mutex>

#include "common.cuh"
#include "internal.h"

namespace {

using namespace qd;

constexpr int kElemsPerCta = 256 * 8;          // one 16-byte-aligned group of 8 per thread
constexpr int kMaxPartials = 65536;            // => at most 65536 * 2048 = 134,217,728 elements per call
// Per-CTA partial maxima.  256 KB on every device that loads the library, for the life of the process.
// Shared by all calls: it keeps the last call's values (each call overwrites exactly the slots it reads,
// so nothing has to be cleared), and two calls running at the same time on one device would race.
static __device__ __align__(256) float g_partial_absmax[kMaxPartials];

// In host code `g_partial_absmax` is only a handle; the device address comes from cudaGetSymbolAddress,
// looked up once per device (under a lock: first calls from two threads may coincide) and kept here.
float* g_scratch_ptr[64] = {};
std::mutex g_scratch_lock;

// Device address of the array on `device`.  The lookup needs that device to be current; the caller's current
// device is put back afterwards.
cudaError_t scratch_address(int device, float** out) {
  std::lock_guard<std::mutex> guard(g_scratch_lock);
  if (!g_scratch_ptr[device]) {
    int prev = -1;
    cudaError_t e = cudaGetDevice(&prev);
    if (e != cudaSuccess) return e;
    if (prev != device && (e = cudaSetDevice(device)) != cudaSuccess) return e;
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_partial_absmax);
    if (prev != device) cudaSetDevice(prev);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[device] = static_cast<float*>(p);
  }
  *out = g_scratch_ptr[device];
  return cudaSuccess;
}

template <typename T>
__global__ void __launch_bounds__(256) partial_absmax_kernel(const T* __restrict__ x, int64_t M, int64_t K, int64_t ldx,
                                                             float* __restrict__ partial) {
  const int64_t vec_per_row = K / 8;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  float m = 0.0f;
  if (idx < M * vec_per_row) {
    const int64_t row = idx / vec_per_row;
    const int64_t col = (idx - row * vec_per_row) * 8;
    float v[8];
    Load8<T>::load(x + row * ldx + col, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(v[i]));
  }
  m = warp_max(m);
  __shared__ float sm[8];
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < 8; ++i) m = fmaxf(m, sm[i]);
    partial[blockIdx.x] = m;   // every slot in [0, gridDim.x) is written: no stale value is ever read
  }
}

__global__ void __launch_bounds__(256) finish_scale_kernel(const float* __restrict__ partial, int n, float* __restrict__ scale) {
  float m = 0.0f;
  for (int i = threadIdx.x; i < n; i += blockDim.x) m = fmaxf(m, partial[i]);
  m = warp_max(m);
  __shared__ float sm[8];
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < 8; ++i) m = fmaxf(m, sm[i]);
    const float s = __fdiv_rn(m, 127.0f);
    *scale = s > 0.0f ? s : 1.0f;
  }
}

template <typename T>
__global__ void __launch_bounds__(256) quantize_with_device_scale_kernel(const T* __restrict__ x, int64_t M, int64_t K,
                                                                         int64_t ldx, const float* __restrict__ scale,
                                                                         uint8_t* __restrict__ q, int64_t ldq) {
  const int64_t vec_per_row = K / 8;
  const int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= M * vec_per_row) return;
  const int64_t row = idx / vec_per_row;
  const int64_t col = (idx - row * vec_per_row) * 8;
  const float inv = __fdiv_rn(1.0f, __ldg(scale));
  float v[8];
  Load8<T>::load(x + row * ldx + col, v);
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = quantize_code(v[i], inv, 0.0f, -127.0f, 127.0f);
  *reinterpret_cast<uint2*>(q + row * ldq + col) = pack_codes8(v);
}

}  // namespace

extern "C" int32_t qdit_quantize_act_dynamic_static(qdit_ctx* ctx, const void* x, int x_dtype, int64_t M, int64_t K,
                                                    int64_t ldx, float* dyn_scale, void* q, int64_t ldq) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (M < 0 || K < 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "negative size");
  if (M == 0 || K == 0) return QDIT_OK;
  if (!x || !q || !dyn_scale) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "x, q or dyn_scale is NULL");
  if (x_dtype != QDIT_BF16 && x_dtype != QDIT_F32) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "x_dtype must be bf16 or f32");
  if (K % 8 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "K = %lld must be a multiple of 8", static_cast<long long>(K));
  if (ldx < K || ldq < K) return qdit_fail(ctx, QDIT_ERR_SHAPE, "leading dimension smaller than K");
  const int64_t esz = x_dtype == QDIT_BF16 ? 2 : 4;
  if (!aligned16(x) || (ldx * esz) % 16 != 0) return qdit_fail(ctx, QDIT_ERR_ALIGN, "x must be 16-byte aligned (base and row pitch)");
  if ((reinterpret_cast<uintptr_t>(q) & 7u) || ldq % 8 != 0) return qdit_fail(ctx, QDIT_ERR_ALIGN, "q must be 8-byte aligned (base and row pitch)");
  constexpr int64_t kMaxElems = static_cast<int64_t>(kMaxPartials) * kElemsPerCta;
  // each factor is bounded before the product is formed, so M * K cannot overflow
  if (M > kMaxElems || K > kMaxElems || M * K > kMaxElems)
    return qdit_fail(ctx, QDIT_ERR_SHAPE, "M = %lld, K = %lld exceed the built-in scratch (at most %lld elements per call)",
                     static_cast<long long>(M), static_cast<long long>(K), static_cast<long long>(kMaxElems));
  const int64_t ctas = (M * K + kElemsPerCta - 1) / kElemsPerCta;
  if (ctx->device < 0 || ctx->device >= 64) return qdit_fail(ctx, QDIT_ERR_UNSUPPORTED, "device index out of range");
  float* scratch = nullptr;
  QDIT_CUDA_CHECK(ctx, scratch_address(ctx->device, &scratch));  // first call on a device: the one-time lookup
  const unsigned grid = static_cast<unsigned>(ctas);
  if (x_dtype == QDIT_BF16)
    partial_absmax_kernel<__nv_bfloat16><<<grid, 256, 0, ctx->stream>>>(static_cast<const __nv_bfloat16*>(x), M, K, ldx, scratch);
  else
    partial_absmax_kernel<float><<<grid, 256, 0, ctx->stream>>>(static_cast<const float*>(x), M, K, ldx, scratch);
  QDIT_TRY(qdit_after_launch(ctx, "partial_absmax_kernel"));
  finish_scale_kernel<<<1, 256, 0, ctx->stream>>>(scratch, static_cast<int>(ctas), dyn_scale);
  QDIT_TRY(qdit_after_launch(ctx, "finish_scale_kernel"));
  if (x_dtype == QDIT_BF16)
    quantize_with_device_scale_kernel<__nv_bfloat16><<<grid, 256, 0, ctx->stream>>>(
        static_cast<const __nv_bfloat16*>(x), M, K, ldx, dyn_scale, static_cast<uint8_t*>(q), ldq);
  else
    quantize_with_device_scale_kernel<float><<<grid, 256, 0, ctx->stream>>>(static_cast<const float*>(x), M, K, ldx,
                                                                            dyn_scale, static_cast<uint8_t*>(q), ldq);
  return qdit_after_launch(ctx, "quantize_with_device_scale_kernel");
}
