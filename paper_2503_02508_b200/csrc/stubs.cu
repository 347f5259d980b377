// Entry points not implemented yet: they report QDIT_ERR_UNSUPPORTED.
#include "internal.h"
extern "C" {
int32_t qdit_attention(qdit_ctx* ctx, const void*, const void*, const void*, int64_t, int, int, int, int, float, void*, int, const qdit_qparams*, const float*) { return qdit_fail(ctx, QDIT_ERR_UNSUPPORTED, "not implemented"); }
int32_t qdit_cache_create(qdit_ctx* ctx, int, int64_t, int64_t, qdit_cache**) { return qdit_fail(ctx, QDIT_ERR_UNSUPPORTED, "not implemented"); }
int32_t qdit_cache_destroy(qdit_cache*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_cache_should_refresh(int, int) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_cache_invalidate(qdit_cache*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_cache_store(qdit_ctx*, qdit_cache*, int, int, const void*) { return QDIT_ERR_UNSUPPORTED; }
void* qdit_cache_slot(qdit_cache*, int, int, int) { return nullptr; }
int32_t qdit_cache_reuse(qdit_ctx*, qdit_cache*, int, int, const float*, int64_t, int64_t, void*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_cache_reuse_all(qdit_ctx*, qdit_cache*, const float*, int64_t, int64_t, void*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_vc_correct(qdit_ctx*, float*, int, int, int, int, int, const float*, float) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_model_create(qdit_ctx*, const qdit_model_desc*, qdit_model**) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_model_destroy(qdit_model*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_model_set_act_scales(qdit_ctx*, qdit_model*, const float*, const float*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_model_get_act_scales(qdit_ctx*, qdit_model*, float*, float*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_model_linear(qdit_model*, int, int, const void**, const float**, const int32_t**, const float**, int64_t*, int64_t*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_sampler_create(qdit_ctx*, qdit_model*, const qdit_sampler_desc*, qdit_sampler**) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_sampler_destroy(qdit_sampler*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_sampler_reset(qdit_ctx*, qdit_sampler*, const float*, const int32_t*) { return QDIT_ERR_UNSUPPORTED; }
float* qdit_sampler_latent(qdit_sampler*) { return nullptr; }
int32_t qdit_sample_step(qdit_ctx*, qdit_sampler*, int) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_sample(qdit_ctx*, qdit_sampler*, const float*, const int32_t*, float*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_forward(qdit_ctx*, qdit_sampler*, const float*, const float*, const int32_t*, int, float*, uint32_t) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_model_begin_calibration(qdit_ctx*, qdit_model*) { return QDIT_ERR_UNSUPPORTED; }
int32_t qdit_model_finish_calibration(qdit_ctx*, qdit_model*) { return QDIT_ERR_UNSUPPORTED; }
void* qdit_sampler_buffer(qdit_sampler*, const char*) { return nullptr; }
qdit_cache* qdit_sampler_cache(qdit_sampler*) { return nullptr; }
}
