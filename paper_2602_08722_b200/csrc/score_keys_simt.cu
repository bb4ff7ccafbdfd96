// Scalar fp32 scoring kernel (Algorithm 1: S = Qbar K^T on normalised keys, max over queries).
// Serves the f32 dtype and is the on-device cross-check of the tensor-core kernel.
// One CTA = 128 cached keys of one (sequence, KV head); one thread = one key.  The key tile is
// staged in shared memory as fp32 (padded rows), Qbar streams through shared memory 32 queries at a
// time, each thread keeps 32 running dot products and folds them into its running maximum.
#include "common.cuh"

namespace quoka {

constexpr int kScoreTile = 128;
constexpr int kQChunk = 32;

template <typename E, int D>
__global__ void __launch_bounds__(kScoreTile) score_keys_simt_kernel(DevParams P, const E* __restrict__ qbar,
                                                                      const E* __restrict__ k,
                                                                      float* __restrict__ scores) {
  extern __shared__ __align__(16) float sm[];
  float* ksm = sm;                                   // [128][D+1]
  float* qsm = sm + kScoreTile * (D + 1);            // [32][D]
  const int s = blockIdx.z, kv = blockIdx.y;
  const int T = __ldg(P.ctx_len + s);
  const int t0 = blockIdx.x * kScoreTile;
  if (t0 >= T) return;
  const int tid = threadIdx.x;
  const int N = P.n_sel;

  // stage the key tile: D/8 lanes per row, coalesced
  constexpr int LG = D / 8;
  for (int e = tid; e < kScoreTile * LG; e += kScoreTile) {
    const int r = e / LG, c = e % LG;
    float x[8];
    if (t0 + r < T) {
      load_vec<E, 8>(k + kv_row_offset(P, s, kv, t0 + r) + c * 8, x);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) x[i] = 0.f;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) ksm[r * (D + 1) + c * 8 + i] = x[i];
  }
  __syncthreads();
  const float* krow = ksm + tid * (D + 1);
  float nn = 0.f;
  for (int x = 0; x < D; ++x) nn += krow[x] * krow[x];

  const E* qb = qbar + ((int64_t)s * P.n_kv + kv) * (int64_t)N * D;
  float best = -INFINITY, total = 0.f;
  for (int j0 = 0; j0 < N; j0 += kQChunk) {
    const int nq = min(kQChunk, N - j0);
    __syncthreads();
    for (int e = tid; e < kQChunk * D; e += kScoreTile) {
      const int j = e / D;
      qsm[e] = (j < nq) ? to_f32(qb[(int64_t)(j0 + j) * D + (e % D)]) : 0.f;
    }
    __syncthreads();
    float acc[kQChunk];
#pragma unroll
    for (int j = 0; j < kQChunk; ++j) acc[j] = 0.f;
    for (int x = 0; x < D; ++x) {
      const float kx = krow[x];
#pragma unroll
      for (int j = 0; j < kQChunk; ++j) acc[j] = fmaf(kx, qsm[j * D + x], acc[j]);
    }
#pragma unroll
    for (int j = 0; j < kQChunk; ++j)
      if (j < nq) { best = fmaxf(best, acc[j]); total += acc[j]; }
  }
  if (t0 + tid < T)
  {
    const float agg = P.agg_mean ? total / (float)N : best;
    float val;
    if (P.score_dot) val = agg;
    else if (P.k_inv_norm) val = agg * __ldg(P.k_inv_norm + kv_norm_index(P, s, kv, t0 + tid));
    else val = agg / fmaxf(sqrtf(nn), kNormEps);
    scores[((int64_t)s * P.n_kv + kv) * P.max_ctx + t0 + tid] = val;
  }
}

// Inverse norms of cache rows (one warp per row): rows [T_s, T_s + C) of every (sequence, KV head), or all of
// [0, T_s + C).  HBM-bound: one read of the rows.
template <typename E, int D>
__global__ void __launch_bounds__(256) key_norms_kernel(DevParams P, const E* __restrict__ k, float* __restrict__ out,
                                                         int all_rows, int rows_max) {
  constexpr int NE = D / 32;
  const int lane = threadIdx.x & 31;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int r = (int)(warp % rows_max);
  const int kv = (int)((warp / rows_max) % P.n_kv);
  const int s = (int)(warp / ((int64_t)rows_max * P.n_kv));
  if (s >= P.batch) return;
  const int T = __ldg(P.ctx_len + s);
  const int first = all_rows ? 0 : T, count = all_rows ? T + P.chunk : P.chunk;
  if (r >= count) return;
  const int t = first + r;
  float x[NE];
  load_vec<E, NE>(k + kv_row_offset(P, s, kv, t) + lane * NE, x);
  float nn = 0.f;
#pragma unroll
  for (int i = 0; i < NE; ++i) nn = fmaf(x[i], x[i], nn);
  nn = warp_sum(nn);
  if (lane == 0) out[kv_norm_index(P, s, kv, t)] = 1.f / fmaxf(sqrtf(nn), kNormEps);
}

cudaError_t launch_key_norms(const DevParams& P, int dtype, const void* k, float* k_inv_norm, int all_rows,
                             cudaStream_t st) {
  const int rows_max = all_rows ? P.max_ctx + P.chunk : P.chunk;
  const int64_t warps = (int64_t)P.batch * P.n_kv * rows_max;
  const int grid = (int)((warps * 32 + 255) / 256);
  if (grid <= 0) return cudaSuccess;
  log_launch("key_norms", dim3(grid), dim3(256), 0, 1, false);
  if (dtype == QUOKA_BF16) {
    if (P.d == 128) key_norms_kernel<__nv_bfloat16, 128><<<grid, 256, 0, st>>>(P, (const __nv_bfloat16*)k, k_inv_norm, all_rows, rows_max);
    else key_norms_kernel<__nv_bfloat16, 64><<<grid, 256, 0, st>>>(P, (const __nv_bfloat16*)k, k_inv_norm, all_rows, rows_max);
  } else {
    if (P.d == 128) key_norms_kernel<float, 128><<<grid, 256, 0, st>>>(P, (const float*)k, k_inv_norm, all_rows, rows_max);
    else key_norms_kernel<float, 64><<<grid, 256, 0, st>>>(P, (const float*)k, k_inv_norm, all_rows, rows_max);
  }
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_score_keys_simt(const DevParams& P, int dtype, const void* qbar, const void* k, float* scores,
                                   cudaStream_t st) {
  if (P.max_ctx <= 0) return cudaSuccess;
  dim3 grid((P.max_ctx + kScoreTile - 1) / kScoreTile, P.n_kv, P.batch);
  log_launch("score_keys_simt", grid, dim3(kScoreTile), (size_t)(kScoreTile * (P.d + 1) + kQChunk * P.d) * sizeof(float), 1, false);
#define QUOKA_SCORE(T_, D)                                                                                     \
  do {                                                                                                        \
    const size_t smem = (size_t)(kScoreTile * (D + 1) + kQChunk * D) * sizeof(float);                         \
    cudaError_t e = cudaFuncSetAttribute(score_keys_simt_kernel<T_, D>,                                        \
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);             \
    if (e != cudaSuccess) return e;                                                                           \
    score_keys_simt_kernel<T_, D><<<grid, kScoreTile, smem, st>>>(P, (const T_*)qbar, (const T_*)k, scores);      \
  } while (0)
  if (dtype == QUOKA_BF16) {
    if (P.d == 128) QUOKA_SCORE(__nv_bfloat16, 128); else QUOKA_SCORE(__nv_bfloat16, 64);
  } else {
    if (P.d == 128) QUOKA_SCORE(float, 128); else QUOKA_SCORE(float, 64);
  }
#undef QUOKA_SCORE
  count_launch();
  return cudaGetLastError();
}

}  // namespace quoka
