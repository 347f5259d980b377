// Context, status reporting and tensor-map creation.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <new>

#include "common.cuh"
#include "internal.h"

int32_t qdit_fail(qdit_ctx* ctx, int32_t code, const char* fmt, ...) {
  if (ctx) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    ctx->last_error = buf;
  }
  return code;
}

int32_t qdit_after_launch(qdit_ctx* ctx, const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return qdit_fail(ctx, QDIT_ERR_CUDA, "launch of %s failed: %s", what, cudaGetErrorString(e));
  ctx->launches += 1;
  return QDIT_OK;
}

int32_t qdit_check_qparams(qdit_ctx* ctx, const qdit_qparams* qp, bool scale_from_device) {
  if (!qp) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "quantizer parameters are NULL");
  if (!scale_from_device && !(qp->scale > 0.0f)) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "scale must be > 0");
  const bool is_signed = qp->qmin >= -128 && qp->qmax <= 127;
  const bool is_unsigned = qp->qmin >= 0 && qp->qmax <= 255;
  if (qp->qmin > qp->qmax || !(is_signed || is_unsigned))
    return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "clip range [%d,%d] fits neither int8 nor uint8", qp->qmin, qp->qmax);
  if (qp->zero_point < -255 || qp->zero_point > 255)
    return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "zero point %d out of range", qp->zero_point);
  return QDIT_OK;
}

static cudaEvent_t take_event(qdit_ctx* ctx) {
  cudaEvent_t e = nullptr;
  if (!ctx->event_pool.empty()) {
    e = ctx->event_pool.back();
    ctx->event_pool.pop_back();
  } else if (cudaEventCreate(&e) != cudaSuccess) {
    cudaGetLastError();
    e = nullptr;
  }
  return e;
}

ProfScope::ProfScope(qdit_ctx* c, int kind, double work) : ctx(c), on(false), stop(nullptr) {
  if (!c || !c->profiling) return;
  cudaEvent_t start = take_event(c);
  stop = take_event(c);
  if (!start || !stop) return;
  cudaEventRecord(start, c->stream);
  c->prof.push_back(qdit_ctx::ProfRec{kind, work, start, stop});
  on = true;
}
ProfScope::~ProfScope() {
  if (on) cudaEventRecord(stop, ctx->stream);
}

// Self-test of the bounded wait that every pipelined kernel uses: warp 1 waits (with a small poll limit) on a
// barrier that nobody arrives at, so the wait runs out, raises the CTA's abort flag and the device status word;
// warp 0 waits on a second such barrier with the full limit and leaves as soon as it sees the abort flag.  The
// kernel then exits normally: the context stays usable and the next qdit_sync reports the time-out.
__global__ void wait_timeout_selftest_kernel(uint32_t polls, int* status, int* observed) {
  __shared__ uint64_t bars[2];
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    qd::mbar_init(&bars[0], 1);
    qd::mbar_init(&bars[1], 1);
    abort_flag = 0;
    qd::mbar_fence_init();
  }
  __syncthreads();
  volatile int* af = &abort_flag;
  if (threadIdx.x == 32) {
    const bool ok = qd::mbar_wait_limited(&bars[0], 0, af, status, polls);
    observed[0] = ok ? 0 : 1;  // 1: the limited wait ran out
  } else if (threadIdx.x == 0) {
    const bool ok = qd::mbar_wait(&bars[1], 0, af, status);
    observed[1] = ok ? 0 : 1;  // 1: left through the abort flag
  }
}

extern "C" {

int32_t qdit_selftest_wait_timeout(qdit_ctx* ctx, uint32_t polls, int* observed_dev) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (!observed_dev) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "observed_dev is NULL");
  if (polls == 0 || polls > (1u << 20)) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "polls must be in 1..2^20");
  wait_timeout_selftest_kernel<<<1, 64, 0, ctx->stream>>>(polls, ctx->d_status, observed_dev);
  return qdit_after_launch(ctx, "wait_timeout_selftest_kernel");
}

int32_t qdit_profile_enable(qdit_ctx* ctx, int enable) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  QDIT_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
  for (auto& r : ctx->prof) {
    ctx->event_pool.push_back(r.start);
    ctx->event_pool.push_back(r.stop);
  }
  ctx->prof.clear();
  ctx->profiling = enable != 0;
  return QDIT_OK;
}

int32_t qdit_profile_read(qdit_ctx* ctx, int kind, int64_t* launches, double* ms, double* work) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (kind < 0 || kind >= QDIT_PROF_KINDS) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "unknown kernel kind %d", kind);
  QDIT_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
  int64_t n = 0;
  double t = 0.0, w = 0.0;
  for (auto& r : ctx->prof) {
    if (r.kind != kind) continue;
    float e = 0.0f;
    if (cudaEventElapsedTime(&e, r.start, r.stop) != cudaSuccess) {
      cudaGetLastError();
      continue;
    }
    n += 1;
    t += e;
    w += r.work;
  }
  if (launches) *launches = n;
  if (ms) *ms = t;
  if (work) *work = w;
  return QDIT_OK;
}

int32_t qdit_create(qdit_ctx** out, int device, void* cuda_stream) {
  if (!out) return QDIT_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
    cudaGetLastError();
    return QDIT_ERR_CUDA;
  }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return QDIT_ERR_CUDA;
  if (prop.major != 10) return QDIT_ERR_CUDA;  // kernels are built for sm_100a only
  if (cudaSetDevice(device) != cudaSuccess) return QDIT_ERR_CUDA;
  qdit_ctx* ctx = new (std::nothrow) qdit_ctx();
  if (!ctx) return QDIT_ERR_NOMEM;
  ctx->device = device;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  ctx->num_sms = prop.multiProcessorCount;
  ctx->opt[QDIT_OPT_PDL] = 1;
  ctx->opt[QDIT_OPT_ATTN_STAGGER_NS] = 2000;
  {  // initial option values from the environment, read here once and nowhere else
    static const struct { const char* name; int opt; } kEnv[] = {
        {"QDIT_PDL", QDIT_OPT_PDL}, {"QDIT_GEMM_BN", QDIT_OPT_GEMM_BN}, {"QDIT_GEMM_T", QDIT_OPT_GEMM_T},
        {"QDIT_GEMM_GENERIC_EPILOGUE", QDIT_OPT_GEMM_GENERIC_EPILOGUE}, {"QDIT_ATTN", QDIT_OPT_ATTN},
        {"QDIT_CONDITIONING_CHUNK", QDIT_OPT_CONDITIONING_CHUNK}, {"QDIT_ATTN_STAGGER_NS", QDIT_OPT_ATTN_STAGGER_NS}};
    for (const auto& e : kEnv)
      if (const char* v = getenv(e.name)) qdit_set_option(ctx, e.opt, atoi(v));
  }
  if (cudaMalloc(&ctx->d_status, sizeof(int)) != cudaSuccess ||
      cudaMemset(ctx->d_status, 0, sizeof(int)) != cudaSuccess ||
      cudaMallocHost(&ctx->h_status, sizeof(int)) != cudaSuccess) {
    if (ctx->d_status) cudaFree(ctx->d_status);
    delete ctx;
    return QDIT_ERR_CUDA;
  }
  *ctx->h_status = 0;
  cudaDriverEntryPointQueryResult qres;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    cudaFree(ctx->d_status);
    cudaFreeHost(ctx->h_status);
    delete ctx;
    return QDIT_ERR_CUDA;
  }
  ctx->encode_fn = fn;
  *out = ctx;
  return QDIT_OK;
}

int32_t qdit_set_option(qdit_ctx* ctx, int option, int value) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  bool ok = false;
  switch (option) {
    case QDIT_OPT_PDL: ok = value == 0 || value == 1; break;
    case QDIT_OPT_GEMM_BN: ok = value == 0 || value == 64 || value == 128 || value == 192; break;
    case QDIT_OPT_GEMM_T: ok = value == 0 || value == 128 || value == 256; break;
    case QDIT_OPT_GEMM_GENERIC_EPILOGUE: ok = value == 0 || value == 1; break;
    case QDIT_OPT_ATTN: ok = value >= 0 && value <= 2; break;
    case QDIT_OPT_CONDITIONING_CHUNK: ok = value >= -1; break;
    case QDIT_OPT_ATTN_STAGGER_NS: ok = value >= 0 && value <= 20000; break;
    default: return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "unknown option %d", option);
  }
  if (!ok) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "value %d not valid for option %d", value, option);
  ctx->opt[option] = value;
  if (option == QDIT_OPT_PDL) ctx->overlap_launches = value != 0;
  return QDIT_OK;
}

int32_t qdit_get_option(const qdit_ctx* ctx, int option, int* value) {
  if (!ctx || !value || option < 0 || option >= QDIT_OPT_COUNT) return QDIT_ERR_INVALID_ARG;
  *value = ctx->opt[option];
  return QDIT_OK;
}

int32_t qdit_destroy(qdit_ctx* ctx) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  if (ctx->d_status) cudaFree(ctx->d_status);
  if (ctx->h_status) cudaFreeHost(ctx->h_status);
  for (auto& r : ctx->prof) {
    cudaEventDestroy(r.start);
    cudaEventDestroy(r.stop);
  }
  for (cudaEvent_t e : ctx->event_pool) cudaEventDestroy(e);
  delete ctx;
  return QDIT_OK;
}

int32_t qdit_sync(qdit_ctx* ctx) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
  QDIT_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
  if (*ctx->h_status != QDIT_DEV_OK) {
    *ctx->h_status = 0;
    cudaMemsetAsync(ctx->d_status, 0, sizeof(int), ctx->stream);
    cudaStreamSynchronize(ctx->stream);
    return qdit_fail(ctx, QDIT_ERR_TIMEOUT, "a bounded device-side wait ran out since the last sync");
  }
  return QDIT_OK;
}

const char* qdit_status_string(int32_t s) {
  switch (s) {
    case QDIT_OK: return "ok";
    case QDIT_ERR_INVALID_ARG: return "invalid argument";
    case QDIT_ERR_SHAPE: return "unsupported shape";
    case QDIT_ERR_ALIGN: return "misaligned pointer or leading dimension";
    case QDIT_ERR_UNSUPPORTED: return "unsupported";
    case QDIT_ERR_CUDA: return "CUDA error";
    case QDIT_ERR_STATE: return "invalid state";
    case QDIT_ERR_TIMEOUT: return "device-side wait timed out";
    case QDIT_ERR_NOMEM: return "out of memory";
    default: return "unknown status";
  }
}

const char* qdit_last_error(const qdit_ctx* ctx) { return ctx ? ctx->last_error.c_str() : "no context"; }
int64_t qdit_launch_count(const qdit_ctx* ctx) { return ctx ? ctx->launches : 0; }

}  // extern "C"

int32_t qdit_get_tmap(qdit_ctx* ctx, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows,
                      uint32_t box_cols, uint32_t swizzle, uint32_t esize, CUtensorMap* out) {
  TmapKey key{ptr, rows, cols, ld, box_rows, box_cols, swizzle, esize};
  auto it = ctx->tmaps.find(key);
  if (it != ctx->tmaps.end()) {
    *out = it->second;
    return QDIT_OK;
  }
  if (!aligned16(ptr) || (ld * esize) % 16 != 0 || (static_cast<uint64_t>(box_cols) * esize) % 16 != 0)
    return qdit_fail(ctx, QDIT_ERR_ALIGN, "tensor map needs a 16-byte aligned base, row pitch and box width");
  if (box_rows > 256 || box_cols > 256) return qdit_fail(ctx, QDIT_ERR_SHAPE, "tensor map box too large");
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  EncodeFn encode = reinterpret_cast<EncodeFn>(ctx->encode_fn);
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstride[1] = {ld * esize};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMapDataType dt = esize == 1   ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                           : esize == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                        : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  CUtensorMap tm;
  CUresult r = encode(&tm, dt, 2, const_cast<void*>(ptr), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                      swizzle == 1 ? CU_TENSOR_MAP_SWIZZLE_128B : swizzle == 2 ? CU_TENSOR_MAP_SWIZZLE_64B : swizzle == 3 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return qdit_fail(ctx, QDIT_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", static_cast<int>(r));
  if (ctx->tmaps.size() > 4096) ctx->tmaps.clear();
  ctx->tmaps.emplace(key, tm);
  *out = tm;
  return QDIT_OK;
}
