// Spectral step of Temporal-Aware Parallel Clustering (Algorithm 1) for the m subsamples as one batch: top-k
// eigenvectors of each subsample's normalised similarity matrix L (qdit_tap_laplacian), k-means on the rows of the
// eigenvector matrix, and the aggregation of the subsamples' clusterings over the whole dataset.
//
// Eigenvectors: L is symmetric positive semi-definite (a congruence of the sum of a Gram matrix and a Laplacian
// kernel matrix), so its top eigenvectors are those of largest magnitude and orthogonal (subspace) iteration
// finds them: a block of p = k + 8 vectors is multiplied by L (the register-tiled f32 GEMM), re-orthonormalised
// (classical Gram-Schmidt, applied twice), and after the last multiplication a Rayleigh-Ritz step (cyclic Jacobi
// on the p x p projected matrix) separates the k leading pairs.  Vectors are kept as ROWS (V^T [p, n]): the GEMM
// computes out[r, c] = sum_h in[r, h] w[c, h], which with w = L (symmetric) is exactly (L V)^T.
// k-means: Lloyd's iterations from the farthest-point start (row 0, then the row farthest from the chosen centres,
// ties to the lowest index), nearest centre with ties to the lowest centre, an emptied cluster keeps its centre;
// sums are taken in ascending row order, so the result is reproducible.
#include <algorithm>
#include <cmath>
#include <vector>

#include "common.cuh"
#include "internal.h"
#include "kernels.h"

namespace {

using namespace qd;

constexpr int TAP_OVERSAMPLE = 8;
constexpr int TAP_MAX_P = 128;

__device__ __forceinline__ float block_sum256(float v, float* sm) {
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.0f;
  for (int i = 0; i < (blockDim.x >> 5); ++i) t += sm[i];
  return t;
}

// Start block: a fixed pseudo-random pattern (integer hash of the position), the same for every subsample.
__global__ void tap_init_kernel(float* __restrict__ vt, int64_t total, int pn) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= total) return;
  uint32_t h = static_cast<uint32_t>(i % pn) * 2654435761u + 0x9E3779B9u;
  h ^= h >> 16; h *= 0x85EBCA6Bu; h ^= h >> 13; h *= 0xC2B2AE35u; h ^= h >> 16;
  vt[i] = static_cast<float>(h >> 8) * (2.0f / 16777216.0f) - 1.0f;
}

// Orthonormalises the p rows (length n) of one subsample's block in place.  One CTA of 256 threads per subsample.
__global__ void __launch_bounds__(256) tap_orth_kernel(float* __restrict__ vt, int p, int n) {
  __shared__ float dots[TAP_MAX_P];
  __shared__ float red[8];
  float* base = vt + static_cast<int64_t>(blockIdx.x) * p * n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int j = 0; j < p; ++j) {
    float* wj = base + static_cast<int64_t>(j) * n;
    for (int pass = 0; pass < 2; ++pass) {
      for (int i = warp; i < j; i += 8) {
        const float* vi = base + static_cast<int64_t>(i) * n;
        float s = 0.0f;
        for (int e = lane; e < n; e += 32) s = fmaf(wj[e], vi[e], s);
        s = warp_sum(s);
        if (lane == 0) dots[i] = s;
      }
      __syncthreads();
      for (int e = threadIdx.x; e < n; e += 256) {
        float acc = wj[e];
        for (int i = 0; i < j; ++i) acc = fmaf(-dots[i], base[static_cast<int64_t>(i) * n + e], acc);
        wj[e] = acc;
      }
      __syncthreads();
    }
    float s = 0.0f;
    for (int e = threadIdx.x; e < n; e += 256) s = fmaf(wj[e], wj[e], s);
    s = block_sum256(s, red);
    const float inv = s > 1e-30f ? rsqrtf(s) : 0.0f;   // a vector inside the span of the earlier ones (rank-deficient L) becomes zero
    for (int e = threadIdx.x; e < n; e += 256) wj[e] *= inv;
    __syncthreads();
  }
}

// Rayleigh-Ritz on one subsample: eigen-decomposition of the symmetric p x p matrix H = V^T L V by cyclic Jacobi
// rotations, then the k leading eigenvalues (descending) and the matching columns of the rotation product Q.
// One CTA of 128 threads; shared memory: H and Q, p x (p + 1) floats each.
__global__ void __launch_bounds__(128) tap_ritz_kernel(const float* __restrict__ Hg, int p, int k, int sweeps, float* __restrict__ evals,
                                                       float* __restrict__ qsel) {
  extern __shared__ float sm_h[];
  const int ld = p + 1;
  float* H = sm_h;
  float* Q = sm_h + p * ld;
  __shared__ float cs[2];
  __shared__ int order[TAP_MAX_P];
  const float* Hb = Hg + static_cast<int64_t>(blockIdx.x) * p * p;
  for (int i = threadIdx.x; i < p * p; i += blockDim.x) {
    const int r = i / p, c = i % p;
    H[r * ld + c] = 0.5f * (Hb[r * p + c] + Hb[c * p + r]);   // symmetrised
    Q[r * ld + c] = r == c ? 1.0f : 0.0f;
  }
  __syncthreads();
  for (int sw = 0; sw < sweeps; ++sw) {
    for (int a = 0; a < p - 1; ++a) {
      for (int b = a + 1; b < p; ++b) {
        if (threadIdx.x == 0) {
          const float hab = H[a * ld + b];
          float c = 1.0f, s = 0.0f;
          if (fabsf(hab) > 1e-30f) {
            const float tau = (H[b * ld + b] - H[a * ld + a]) / (2.0f * hab);
            const float tt = (tau >= 0.0f ? 1.0f : -1.0f) / (fabsf(tau) + sqrtf(1.0f + tau * tau));
            c = rsqrtf(1.0f + tt * tt);
            s = tt * c;
          }
          cs[0] = c;
          cs[1] = s;
        }
        __syncthreads();
        const float c = cs[0], s = cs[1];
        const int kx = threadIdx.x;
        if (kx < p) {   // rows a and b:  H <- J^T H
          const float ha = H[a * ld + kx], hb = H[b * ld + kx];
          H[a * ld + kx] = c * ha - s * hb;
          H[b * ld + kx] = s * ha + c * hb;
        }
        __syncthreads();
        if (kx < p) {   // columns a and b:  H <- H J,  Q <- Q J
          const float ha = H[kx * ld + a], hb = H[kx * ld + b];
          H[kx * ld + a] = c * ha - s * hb;
          H[kx * ld + b] = s * ha + c * hb;
          const float qa = Q[kx * ld + a], qb = Q[kx * ld + b];
          Q[kx * ld + a] = c * qa - s * qb;
          Q[kx * ld + b] = s * qa + c * qb;
        }
        __syncthreads();
      }
    }
  }
  if (threadIdx.x == 0) {   // indices of the eigenvalues in descending order (ties to the lower index)
    for (int i = 0; i < p; ++i) order[i] = i;
    for (int i = 0; i < k; ++i) {
      int best = i;
      for (int j = i + 1; j < p; ++j)
        if (H[order[j] * ld + order[j]] > H[order[best] * ld + order[best]]) best = j;
      const int tmp = order[i];
      order[i] = order[best];
      order[best] = tmp;
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < k; i += blockDim.x) evals[static_cast<int64_t>(blockIdx.x) * k + i] = H[order[i] * ld + order[i]];
  for (int i = threadIdx.x; i < p * k; i += blockDim.x) {
    const int a = i / k, j = i % k;
    qsel[static_cast<int64_t>(blockIdx.x) * p * k + i] = Q[a * ld + order[j]];
  }
}

// Ritz vectors as rows of the samples: eigvecs[b, i, j] = sum_a qsel[b, a, j] V^T[b, a, i].
__global__ void __launch_bounds__(256) tap_ritz_vectors_kernel(const float* __restrict__ vt, const float* __restrict__ qsel, int p,
                                                               int n, int k, float* __restrict__ eigvecs) {
  const int b = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float* v = vt + static_cast<int64_t>(b) * p * n + i;
  const float* q = qsel + static_cast<int64_t>(b) * p * k;
  float* out = eigvecs + (static_cast<int64_t>(b) * n + i) * k;
  for (int j = 0; j < k; ++j) {
    float acc = 0.0f;
    for (int a = 0; a < p; ++a) acc = fmaf(q[a * k + j], v[static_cast<int64_t>(a) * n], acc);
    out[j] = acc;
  }
}

// k-means on the rows of Y [n, k] of one subsample (one CTA of 256 threads).  Shared memory: centres [k, k], the
// farthest-point distances [n], member counts [k].
__global__ void __launch_bounds__(256) tap_kmeans_kernel(const float* __restrict__ eigvecs, int n, int k, int iters,
                                                         int32_t* __restrict__ labels) {
  extern __shared__ float sm_k[];
  float* C = sm_k;                 // [k][k]
  float* dmin = sm_k + k * k;      // [n]
  int* count = reinterpret_cast<int*>(dmin + n);   // [k]
  __shared__ float red_v[8];
  __shared__ int red_i[8];
  __shared__ int flag;
  const float* Y = eigvecs + static_cast<int64_t>(blockIdx.x) * n * k;
  int32_t* lab = labels + static_cast<int64_t>(blockIdx.x) * n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // farthest-point start
  for (int j = threadIdx.x; j < k; j += 256) C[j] = Y[j];
  for (int i = threadIdx.x; i < n; i += 256) {
    dmin[i] = INFINITY;
    lab[i] = -1;
  }
  __syncthreads();
  for (int c = 0; c < k; ++c) {
    // distances to centre c, running minimum, and (for the next centre) the arg-max of the minimum, lowest index on ties
    float best_v = -1.0f;
    int best_i = 0x7fffffff;
    for (int i = threadIdx.x; i < n; i += 256) {
      float d2 = 0.0f;
      for (int j = 0; j < k; ++j) {
        const float df = Y[static_cast<int64_t>(i) * k + j] - C[c * k + j];
        d2 = fmaf(df, df, d2);
      }
      const float dm = fminf(dmin[i], d2);
      dmin[i] = dm;
      if (dm > best_v) {   // i ascends within a thread: the first maximum is kept
        best_v = dm;
        best_i = i;
      }
    }
    if (c + 1 == k) break;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, best_v, o);
      const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
      if (ov > best_v || (ov == best_v && oi < best_i)) {
        best_v = ov;
        best_i = oi;
      }
    }
    if (lane == 0) {
      red_v[warp] = best_v;
      red_i[warp] = best_i;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      float bv = red_v[0];
      int bi = red_i[0];
      for (int w = 1; w < 8; ++w)
        if (red_v[w] > bv || (red_v[w] == bv && red_i[w] < bi)) {
          bv = red_v[w];
          bi = red_i[w];
        }
      flag = bi;
    }
    __syncthreads();
    const int next = flag;
    for (int j = threadIdx.x; j < k; j += 256) C[(c + 1) * k + j] = Y[static_cast<int64_t>(next) * k + j];
    __syncthreads();
  }
  __syncthreads();
  // Lloyd's iterations
  for (int it = 0; it < iters; ++it) {
    if (threadIdx.x == 0) flag = 0;
    __syncthreads();
    bool changed = false;
    for (int i = threadIdx.x; i < n; i += 256) {
      float best = INFINITY;
      int bc = 0;
      for (int c = 0; c < k; ++c) {
        float d2 = 0.0f;
        for (int j = 0; j < k; ++j) {
          const float df = Y[static_cast<int64_t>(i) * k + j] - C[c * k + j];
          d2 = fmaf(df, df, d2);
        }
        if (d2 < best) {   // strict: ties stay with the lowest centre
          best = d2;
          bc = c;
        }
      }
      if (lab[i] != bc) {
        lab[i] = bc;
        changed = true;
      }
    }
    if (changed) flag = 1;
    __syncthreads();
    if (!flag) break;
    for (int c = threadIdx.x; c < k; c += 256) {
      int cnt = 0;
      for (int i = 0; i < n; ++i) cnt += lab[i] == c;
      count[c] = cnt;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < k * k; e += 256) {   // centre c, dimension j: mean of the members in ascending row order
      const int c = e / k, j = e % k;
      if (count[c] > 0) {
        float s = 0.0f;
        for (int i = 0; i < n; ++i)
          if (lab[i] == c) s += Y[static_cast<int64_t>(i) * k + j];
        C[e] = s / static_cast<float>(count[c]);
      }
    }
    __syncthreads();
  }
}

// Per (subsample, cluster): mean of the members' unit-length features, mean timestamp, size.
__global__ void __launch_bounds__(256) tap_summary_kernel(const float* __restrict__ xn, const float* __restrict__ t,
                                                          const int32_t* __restrict__ labels, int n, int d, int k,
                                                          float* __restrict__ F, float* __restrict__ tau, int32_t* __restrict__ size) {
  const int b = blockIdx.y, c = blockIdx.x;
  const int32_t* lab = labels + static_cast<int64_t>(b) * n;
  const float* X = xn + static_cast<int64_t>(b) * n * d;
  __shared__ int s_cnt;
  if (threadIdx.x == 0) {
    int cnt = 0;
    float ts = 0.0f;
    for (int i = 0; i < n; ++i)
      if (lab[i] == c) {
        ++cnt;
        ts += t[static_cast<int64_t>(b) * n + i];
      }
    s_cnt = cnt;
    size[b * k + c] = cnt;
    tau[b * k + c] = cnt > 0 ? ts / static_cast<float>(cnt) : 0.0f;
  }
  __syncthreads();
  const int cnt = s_cnt;
  float* out = F + (static_cast<int64_t>(b) * k + c) * d;
  for (int e = threadIdx.x; e < d; e += 256) {
    float s = 0.0f;
    for (int i = 0; i < n; ++i)
      if (lab[i] == c) s += X[static_cast<int64_t>(i) * d + e];
    out[e] = cnt > 0 ? s / static_cast<float>(cnt) : 0.0f;
  }
}

// labels_all[j] = argmax_a alpha S[j, a] + (1 - alpha) exp(-|t_j - tau_a|), ties to the lowest cluster.
__global__ void __launch_bounds__(256) tap_assign_kernel(const float* __restrict__ S, const float* __restrict__ t,
                                                         const float* __restrict__ tau, int64_t N, int k, float alpha,
                                                         int32_t* __restrict__ labels_all) {
  const int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (j >= N) return;
  float best = -INFINITY;
  int ba = 0;
  const float tj = t[j];
  for (int a = 0; a < k; ++a) {
    const float v = alpha * S[j * k + a] + (1.0f - alpha) * expf(-fabsf(tj - tau[a]));
    if (v > best) {
      best = v;
      ba = a;
    }
  }
  labels_all[j] = ba;
}

__global__ void __launch_bounds__(256) tap_normalize_rows_kernel(const float* __restrict__ x, int d, float* __restrict__ xn) {
  __shared__ float sm[8];
  const float* row = x + static_cast<int64_t>(blockIdx.x) * d;
  float* out = xn + static_cast<int64_t>(blockIdx.x) * d;
  float s = 0.0f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) s = fmaf(row[i], row[i], s);
  const float norm = sqrtf(block_sum256(s, sm));
  const float inv = norm > 0.0f ? 1.0f / norm : 0.0f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) out[i] = row[i] * inv;
}

int tap_block(int k) { return ((k + TAP_OVERSAMPLE + 3) / 4) * 4; }

}  // namespace

extern "C" {

int64_t qdit_tap_cluster_workspace(int m, int n, int d, int k) {
  if (m <= 0 || n <= 0 || d <= 0 || k <= 0) return 0;
  const int64_t p = tap_block(k);
  // L of every subsample, the Laplacian call's own workspace, two vector blocks, the projected matrices, the selected
  // rotation columns, a zero bias for the products
  return static_cast<int64_t>(m) * n * n + (static_cast<int64_t>(n) * d + 2 * n) + 2 * static_cast<int64_t>(m) * p * n +
         static_cast<int64_t>(m) * p * p + static_cast<int64_t>(m) * p * k + n + 64;
}

int32_t qdit_tap_cluster(qdit_ctx* ctx, const float* x, const float* t, int m, int n, int d, float alpha, float exponent, int k,
                         int power_iters, int kmeans_iters, float* workspace, float* eigvals, float* eigvecs, int32_t* labels) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (m <= 0 || n <= 0 || d <= 0 || k <= 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "m, n, d and k must be positive");
  if (n % 16 != 0 || d % 16 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "n and d must be multiples of 16");
  const int p = tap_block(k);
  if (p > TAP_MAX_P || p > n) return qdit_fail(ctx, QDIT_ERR_SHAPE, "k = %d needs a block of %d vectors: at most %d and at most n", k, p, TAP_MAX_P);
  if (n > 8192) return qdit_fail(ctx, QDIT_ERR_SHAPE, "n = %d exceeds 8192 samples per subsample", n);
  if (power_iters < 1 || power_iters > 10000 || kmeans_iters < 1) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "iteration counts must be positive");
  if (!x || !t || !workspace || !eigvals || !eigvecs || !labels) return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  if (!aligned16(x) || !aligned16(workspace) || !aligned16(eigvecs)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "x, workspace and eigvecs must be 16-byte aligned");
  const int64_t nn = static_cast<int64_t>(n) * n, pn = static_cast<int64_t>(p) * n;
  float* L = workspace;
  float* lws = L + m * nn;
  float* vt = lws + (static_cast<int64_t>(n) * d + 2 * n);
  float* wt = vt + m * pn;
  float* H = wt + m * pn;
  float* qsel = H + static_cast<int64_t>(m) * p * p;
  float* zero = qsel + static_cast<int64_t>(m) * p * k;
  zero = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(zero) + 15) & ~uintptr_t(15));
  QDIT_CUDA_CHECK(ctx, cudaMemsetAsync(zero, 0, static_cast<size_t>(n) * sizeof(float), ctx->stream));
  for (int b = 0; b < m; ++b)
    QDIT_TRY(qdit_tap_laplacian(ctx, x + static_cast<int64_t>(b) * n * d, t + static_cast<int64_t>(b) * n, n, d, alpha, exponent, lws, L + b * nn));
  const int64_t total = m * pn;
  tap_init_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, ctx->stream>>>(vt, total, static_cast<int>(pn));
  QDIT_TRY(qdit_after_launch(ctx, "tap_init_kernel"));
  tap_orth_kernel<<<m, 256, 0, ctx->stream>>>(vt, p, n);
  QDIT_TRY(qdit_after_launch(ctx, "tap_orth_kernel"));
  for (int it = 0; it < power_iters; ++it) {
    for (int b = 0; b < m; ++b)   // (L V)^T = V^T L (L symmetric)
      QDIT_TRY(launch_batched_linear(ctx, vt + b * pn, L + b * nn, zero, nullptr, nullptr, wt + b * pn, nullptr, p, n, n, 0, 0, 0));
    tap_orth_kernel<<<m, 256, 0, ctx->stream>>>(wt, p, n);
    QDIT_TRY(qdit_after_launch(ctx, "tap_orth_kernel"));
    float* tmp = vt;
    vt = wt;
    wt = tmp;
  }
  // Rayleigh-Ritz: H = V^T (L V)
  for (int b = 0; b < m; ++b) {
    QDIT_TRY(launch_batched_linear(ctx, vt + b * pn, L + b * nn, zero, nullptr, nullptr, wt + b * pn, nullptr, p, n, n, 0, 0, 0));
    QDIT_TRY(launch_batched_linear(ctx, vt + b * pn, wt + b * pn, zero, nullptr, nullptr, H + static_cast<int64_t>(b) * p * p, nullptr, p, p, n, 0, 0, 0));
  }
  const int ritz_smem = 2 * p * (p + 1) * static_cast<int>(sizeof(float));
  QDIT_TRY(qdit_allow_smem(ctx, tap_ritz_kernel, 2 * TAP_MAX_P * (TAP_MAX_P + 1) * static_cast<int>(sizeof(float))));  // the limit is raised once, to the largest block
  tap_ritz_kernel<<<m, 128, ritz_smem, ctx->stream>>>(H, p, k, 12, eigvals, qsel);
  QDIT_TRY(qdit_after_launch(ctx, "tap_ritz_kernel"));
  tap_ritz_vectors_kernel<<<dim3((n + 255) / 256, m), 256, 0, ctx->stream>>>(vt, qsel, p, n, k, eigvecs);
  QDIT_TRY(qdit_after_launch(ctx, "tap_ritz_vectors_kernel"));
  const int km_smem = (k * k + n + k) * static_cast<int>(sizeof(float));
  if (km_smem > 200 * 1024) return qdit_fail(ctx, QDIT_ERR_SHAPE, "k and n too large for the k-means kernel's shared memory");
  QDIT_TRY(qdit_allow_smem(ctx, tap_kmeans_kernel, 200 * 1024));
  tap_kmeans_kernel<<<m, 256, km_smem, ctx->stream>>>(eigvecs, n, k, kmeans_iters, labels);
  return qdit_after_launch(ctx, "tap_kmeans_kernel");
}

int64_t qdit_tap_aggregate_workspace(int m, int n, int d, int k, int64_t N) {
  if (m <= 0 || n <= 0 || d <= 0 || k <= 0 || N <= 0) return 0;
  // unit-length features of the subsamples and of the dataset, per-cluster summaries, similarities, small vectors
  return static_cast<int64_t>(m) * n * d + N * d + static_cast<int64_t>(m) * k * d + 3 * static_cast<int64_t>(m) * k + N * k +
         2 * static_cast<int64_t>(k) * d + 2 * k + 256;
}

int32_t qdit_tap_aggregate(qdit_ctx* ctx, const float* x, const float* t, const int32_t* labels, int m, int n, int d, int k,
                           float alpha, const float* x_all, const float* t_all, int64_t N, float* workspace,
                           int32_t* labels_all, float* centroids, float* tau_out) {
  if (!ctx) return QDIT_ERR_INVALID_ARG;
  if (m <= 0 || n <= 0 || d <= 0 || k <= 0 || N <= 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "sizes must be positive");
  if (d % 16 != 0 || k % 4 != 0) return qdit_fail(ctx, QDIT_ERR_SHAPE, "d must be a multiple of 16 and k of 4");
  if (N > 0x7fffffff) return qdit_fail(ctx, QDIT_ERR_SHAPE, "N too large");
  if (!x || !t || !labels || !x_all || !t_all || !workspace || !labels_all || !centroids || !tau_out)
    return qdit_fail(ctx, QDIT_ERR_INVALID_ARG, "NULL argument");
  if (!aligned16(x) || !aligned16(x_all) || !aligned16(workspace) || !aligned16(centroids)) return qdit_fail(ctx, QDIT_ERR_ALIGN, "x, x_all, workspace and centroids must be 16-byte aligned");
  float* xn = workspace;
  float* xa = xn + static_cast<int64_t>(m) * n * d;
  float* F = xa + N * d;
  float* tau = F + static_cast<int64_t>(m) * k * d;
  int32_t* size = reinterpret_cast<int32_t*>(tau + static_cast<int64_t>(m) * k);
  float* S = reinterpret_cast<float*>(size + static_cast<int64_t>(m) * k);
  S = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(S) + 15) & ~uintptr_t(15));
  float* Fn = S + N * k;
  float* zero = Fn + static_cast<int64_t>(k) * d;
  zero = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(zero) + 15) & ~uintptr_t(15));
  tap_normalize_rows_kernel<<<static_cast<unsigned>(m * n), 256, 0, ctx->stream>>>(x, d, xn);
  QDIT_TRY(qdit_after_launch(ctx, "tap_normalize_rows_kernel"));
  tap_summary_kernel<<<dim3(k, m), 256, 0, ctx->stream>>>(xn, t, labels, n, d, k, F, tau, size);
  QDIT_TRY(qdit_after_launch(ctx, "tap_summary_kernel"));
  // the matching of m * k cluster summaries is a few thousand small dot products: done on the host
  std::vector<float> hF(static_cast<size_t>(m) * k * d), htau(static_cast<size_t>(m) * k);
  std::vector<int32_t> hsize(static_cast<size_t>(m) * k);
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(hF.data(), F, hF.size() * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(htau.data(), tau, htau.size() * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(hsize.data(), size, hsize.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
  QDIT_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));
  auto unit = [&](const float* v, std::vector<double>& out) {
    double s = 0.0;
    for (int e = 0; e < d; ++e) s += static_cast<double>(v[e]) * v[e];
    const double inv = s > 0.0 ? 1.0 / std::sqrt(s) : 0.0;
    for (int e = 0; e < d; ++e) out[e] = v[e] * inv;
  };
  std::vector<double> accF(static_cast<size_t>(k) * d, 0.0), accT(k, 0.0), accN(k, 0.0);
  for (int a = 0; a < k; ++a) {
    for (int e = 0; e < d; ++e) accF[static_cast<size_t>(a) * d + e] = static_cast<double>(hF[static_cast<size_t>(a) * d + e]) * hsize[a];
    accT[a] = static_cast<double>(htau[a]) * hsize[a];
    accN[a] = hsize[a];
  }
  std::vector<double> u0(static_cast<size_t>(k) * d), ui(static_cast<size_t>(k) * d), tmp(d);
  for (int a = 0; a < k; ++a) {
    unit(&hF[static_cast<size_t>(a) * d], tmp);
    std::copy(tmp.begin(), tmp.end(), u0.begin() + static_cast<size_t>(a) * d);
  }
  for (int i = 1; i < m; ++i) {
    const float* Fi = &hF[static_cast<size_t>(i) * k * d];
    for (int b = 0; b < k; ++b) {
      unit(Fi + static_cast<size_t>(b) * d, tmp);
      std::copy(tmp.begin(), tmp.end(), ui.begin() + static_cast<size_t>(b) * d);
    }
    std::vector<double> sim(static_cast<size_t>(k) * k);
    for (int a = 0; a < k; ++a)
      for (int b = 0; b < k; ++b) {
        double dot = 0.0;
        for (int e = 0; e < d; ++e) dot += u0[static_cast<size_t>(a) * d + e] * ui[static_cast<size_t>(b) * d + e];
        sim[static_cast<size_t>(a) * k + b] = alpha * dot + (1.0 - alpha) * std::exp(-std::fabs(static_cast<double>(htau[a]) - htau[static_cast<size_t>(i) * k + b]));
      }
    std::vector<char> row_used(k, 0), col_used(k, 0);
    for (int round = 0; round < k; ++round) {   // greedy: the largest remaining entry, ties to the lowest row, then column
      double best = -1e300;
      int ba = -1, bb = -1;
      for (int a = 0; a < k; ++a) {
        if (row_used[a]) continue;
        for (int b = 0; b < k; ++b)
          if (!col_used[b] && sim[static_cast<size_t>(a) * k + b] > best) {
            best = sim[static_cast<size_t>(a) * k + b];
            ba = a;
            bb = b;
          }
      }
      row_used[ba] = col_used[bb] = 1;
      const double w = hsize[static_cast<size_t>(i) * k + bb];
      for (int e = 0; e < d; ++e) accF[static_cast<size_t>(ba) * d + e] += static_cast<double>(Fi[static_cast<size_t>(bb) * d + e]) * w;
      accT[ba] += static_cast<double>(htau[static_cast<size_t>(i) * k + bb]) * w;
      accN[ba] += w;
    }
  }
  std::vector<float> aggF(static_cast<size_t>(k) * d), aggT(k);
  for (int a = 0; a < k; ++a) {
    const double inv = accN[a] > 0.0 ? 1.0 / accN[a] : 0.0;
    for (int e = 0; e < d; ++e) aggF[static_cast<size_t>(a) * d + e] = static_cast<float>(accF[static_cast<size_t>(a) * d + e] * inv);
    aggT[a] = static_cast<float>(accT[a] * inv);
  }
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(centroids, aggF.data(), aggF.size() * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
  QDIT_CUDA_CHECK(ctx, cudaMemcpyAsync(tau_out, aggT.data(), aggT.size() * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
  QDIT_CUDA_CHECK(ctx, cudaStreamSynchronize(ctx->stream));   // the host vectors go out of scope below
  // every sample of the dataset goes to the aggregated cluster it is most similar to
  tap_normalize_rows_kernel<<<static_cast<unsigned>(k), 256, 0, ctx->stream>>>(centroids, d, Fn);
  QDIT_TRY(qdit_after_launch(ctx, "tap_normalize_rows_kernel"));
  tap_normalize_rows_kernel<<<static_cast<unsigned>(N), 256, 0, ctx->stream>>>(x_all, d, xa);
  QDIT_TRY(qdit_after_launch(ctx, "tap_normalize_rows_kernel"));
  QDIT_CUDA_CHECK(ctx, cudaMemsetAsync(zero, 0, static_cast<size_t>(k) * sizeof(float), ctx->stream));
  QDIT_TRY(launch_batched_linear(ctx, xa, Fn, zero, nullptr, nullptr, S, nullptr, static_cast<int>(N), k, d, 0, 0, 0));
  tap_assign_kernel<<<static_cast<unsigned>((N + 255) / 256), 256, 0, ctx->stream>>>(S, t_all, tau_out, N, k, alpha, labels_all);
  return qdit_after_launch(ctx, "tap_assign_kernel");
}

}  // extern "C"
