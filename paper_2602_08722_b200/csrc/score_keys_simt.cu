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
    scores[((int64_t)s * P.n_kv + kv) * P.max_ctx + t0 + tid] =
        (P.agg_mean ? total / (float)N : best) / (P.score_dot ? 1.f : fmaxf(sqrtf(nn), kNormEps));
}

cudaError_t launch_score_keys_simt(const DevParams& P, int dtype, const void* qbar, const void* k, float* scores,
                                   cudaStream_t st) {
  if (P.max_ctx <= 0) return cudaSuccess;
  dim3 grid((P.max_ctx + kScoreTile - 1) / kScoreTile, P.n_kv, P.batch);
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
