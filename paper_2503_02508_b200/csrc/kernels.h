// Launchers of the glue kernels (embedders, final layer, sampler update), used by the model/sampler code.
#pragma once
#include "internal.h"

struct DdimCoef {
  float sqrt_ab_t, sqrt_1mab_t, sqrt_ab_prev, sqrt_1mab_prev;
};

// Coefficients of one stochastic (DDPM) step: x0 = rs * x - rsm1 * eps, mean = c_x0 * x0 + c_xt * x,
// log variance = f * log_beta + (1 - f) * log_post with f = (v + 1) / 2, noise factor nz (0 at the last step).
struct DdpmCoef {
  float rs, rsm1, c_x0, c_xt, log_beta, log_post, nz;
};

// x[m,:] = bf16(W_patch . patch(m) + b + pos); sample b reads latent[b % latent_batch]; wT = W_patch transposed [pd][D].
// frag (optional, for pd = 16): the weights in tensor-core fragment order, (D / 8) * 512 bytes written by
// launch_embed_fragments; with it the product runs on the tensor cores.
int32_t launch_embed(qdit_ctx* ctx, const float* latent, int latent_batch, const float* wT, const void* frag, const float* bias,
                     const float* pos, void* x, int64_t M, int D, int grid, int patch, int C);
int32_t launch_embed_fragments(qdit_ctx* ctx, const float* wT, int D, void* frag);
// feat[b, :] = (cos(t_b w_j), sin(t_b w_j)), w_j = 10000^(-j / (F/2))
int32_t launch_timestep_features(qdit_ctx* ctx, const float* t, float* feat, int B, int F);
// h[b,:] = SiLU(W1 . sinusoid(t_b) + b1); feat is scratch [B, F]
int32_t launch_cond1(qdit_ctx* ctx, const float* t, const float* w1, const float* b1, float* feat, float* h, int B, int D,
                     int F);
// out[b,n] = g(W[n,:] . f(in[b,:]) + bias[n] (+ table[y[b % y_period],n])); f = SiLU if silu_input, g = SiLU if
// silu_output; out_silu (optional) = SiLU(out); y_period 0 means B (one label per row)
int32_t launch_small_linear(qdit_ctx* ctx, const float* in, const float* w, const float* bias, const float* table,
                            const int32_t* y, float* out, float* out_silu, int B, int N, int K, int silu_input,
                            int silu_output, int y_period);
// The same operation as launch_small_linear for many rows (register-tiled f32 GEMM; K % 16 == 0, N % 4 == 0).
int32_t launch_batched_linear(qdit_ctx* ctx, const float* in, const float* w, const float* bias, const float* table,
                              const int32_t* y, float* out, float* out_silu, int R, int N, int K, int silu_input,
                              int silu_output, int y_period);
// LayerNorm + modulate + linear D->OUT + un-patchify into net [B, OUT/p^2, side, side]
int32_t launch_final(qdit_ctx* ctx, const void* x, int64_t M, int D, int T, float eps, const float* modf,
                     const float* w, const float* bias, float* net, int grid, int patch, int OUT);
// guidance combine + DDIM (eta = 0) update of latent [B,C,HW] from net [Beff,2C,HW]
int32_t launch_cfg_ddim(qdit_ctx* ctx, float* latent, const float* net, int B, int C, int HW, int use_cfg,
                        float guidance, const DdimCoef& k);
// guidance combine + stochastic step with learned variance; noise: f32 [B,C,HW] standard normal for this step
int32_t launch_cfg_ddpm(qdit_ctx* ctx, float* latent, const float* net, const float* noise, int B, int C, int HW,
                        int use_cfg, float guidance, const DdpmCoef& k);
