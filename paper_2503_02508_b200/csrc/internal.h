// Internal declarations shared by the translation units of libqdit (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <unordered_map>
#include <unordered_set>
#include <vector>

#include "qdit.h"

// Device status word values (written by kernels, read by qdit_sync).
enum : int { QDIT_DEV_OK = 0, QDIT_DEV_TIMEOUT = 1 };

struct TmapKey {
  const void* ptr;
  uint64_t rows, cols, ld;
  uint32_t box_rows, box_cols, swizzle, esize;
  bool operator==(const TmapKey& o) const {
    return ptr == o.ptr && rows == o.rows && cols == o.cols && ld == o.ld && box_rows == o.box_rows &&
           box_cols == o.box_cols && swizzle == o.swizzle && esize == o.esize;
  }
};
struct TmapKeyHash {
  size_t operator()(const TmapKey& k) const {
    uint64_t h = reinterpret_cast<uint64_t>(k.ptr);
    auto mix = [&](uint64_t v) { h ^= v + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2); };
    mix(k.rows); mix(k.cols); mix(k.ld); mix(k.box_rows); mix(k.box_cols); mix(k.swizzle); mix(k.esize);
    return static_cast<size_t>(h);
  }
};

struct qdit_ctx {
  int device = 0;
  cudaStream_t stream = nullptr;
  int* d_status = nullptr;  // device status word
  int* h_status = nullptr;  // pinned host mirror
  int num_sms = 0;
  int64_t launches = 0;
  // Kernel-selection options (qdit_set_option).  Set once at creation from the QDIT_* environment variables of the
  // same names, afterwards only through the call; no kernel launch reads the environment.
  int opt[QDIT_OPT_COUNT] = {};
  bool overlap_launches = true;  // = opt[QDIT_OPT_PDL]: programmatic dependent launch for the kernels that support it
  std::unordered_set<const void*> attr_done;  // kernels whose dynamic shared-memory limit has been raised for this context
  std::string last_error;
  void* encode_fn = nullptr;  // cuTensorMapEncodeTiled
  std::unordered_map<TmapKey, CUtensorMap, TmapKeyHash> tmaps;
  // per-kernel event timing (qdit_profile_*)
  bool profiling = false;
  struct ProfRec { int kind; double work; cudaEvent_t start, stop; };
  std::vector<ProfRec> prof;
  std::vector<cudaEvent_t> event_pool;
};

// Records a formatted message on the context and returns `code`.
int32_t qdit_fail(qdit_ctx* ctx, int32_t code, const char* fmt, ...);

// Brackets one kernel launch with events while profiling is enabled.
struct ProfScope {
  qdit_ctx* ctx;
  bool on;
  cudaEvent_t stop;
  ProfScope(qdit_ctx* c, int kind, double work);
  ~ProfScope();
};

// Launches `kernel` on the context's stream.  With ctx->overlap_launches the launch carries the
// programmatic-stream-serialization attribute: the kernel may start its preamble before the previous kernel
// of the stream has finished, and MUST call grid_dependency_wait() before its first global-memory access.
template <typename... KArgs, typename... Args>
cudaError_t qdit_launch_overlapped(qdit_ctx* ctx, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                   Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = ctx->stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = ctx->overlap_launches ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Raises a kernel's dynamic shared-memory limit once per context (the attribute is per device and function; a context
// belongs to one device and is used by one thread at a time, so no process-wide state is involved).
template <typename K>
int32_t qdit_allow_smem(qdit_ctx* ctx, K kernel, int bytes) {
  const void* key = reinterpret_cast<const void*>(kernel);
  if (ctx->attr_done.count(key)) return QDIT_OK;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return qdit_fail(ctx, QDIT_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  ctx->attr_done.insert(key);
  return QDIT_OK;
}

// Checks the last launch; counts it.
int32_t qdit_after_launch(qdit_ctx* ctx, const char* what);

#define QDIT_CUDA_CHECK(ctx, expr)                                                                             \
  do {                                                                                                         \
    cudaError_t e__ = (expr);                                                                                  \
    if (e__ != cudaSuccess) return qdit_fail((ctx), QDIT_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)
#define QDIT_TRY(expr)                 \
  do {                                 \
    int32_t st__ = (expr);             \
    if (st__ != QDIT_OK) return st__;  \
  } while (0)

// 2-D tensor map over a row-major matrix [rows, cols] of `esize`-byte elements with row pitch `ld`
// elements; box = box_rows x box_cols elements; swizzle: 0 none, 1 = 128-byte, 2 = 64-byte, 3 = 32-byte.
// Cached per context.
int32_t qdit_get_tmap(qdit_ctx* ctx, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows,
                      uint32_t box_cols, uint32_t swizzle, uint32_t esize, CUtensorMap* out);

// Quantizer parameters as the kernels take them.
struct QuantArgs {
  float scale;             // s (by value)
  const float* scale_dev;  // if non-null, overrides `scale`
  float zp, qmin, qmax;    // as floats (exact small integers)
};
inline QuantArgs make_quant_args(const qdit_qparams& qp, const float* scale_dev) {
  QuantArgs a;
  a.scale = qp.scale;
  a.scale_dev = scale_dev;
  a.zp = static_cast<float>(qp.zero_point);
  a.qmin = static_cast<float>(qp.qmin);
  a.qmax = static_cast<float>(qp.qmax);
  return a;
}
int32_t qdit_check_qparams(qdit_ctx* ctx, const qdit_qparams* qp, bool scale_from_device);

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- internal launchers used by the model/sampler orchestration (all enqueue on ctx->stream) ----
int32_t launch_absmax(qdit_ctx* ctx, const void* x, int x_dtype, int64_t M, int64_t K, int64_t ldx, float* absmax_dev);
int32_t launch_absmax_to_scale(qdit_ctx* ctx, const float* absmax_dev, float* scale_dev, float* running_absmax, int n);
// Quantizes an f32 tensor [M,K] (contiguous) with the scale held in device memory.
int32_t qdit_quantize_act_dev(qdit_ctx* ctx, const float* x, int64_t M, int64_t K, qdit_qparams qp,
                              const float* scale_dev, uint8_t* q);
