// Query sub-selection, normalisation and GQA pre-aggregation (Algorithm 1, first two blocks).
//
// rank_queries : one CTA per (sequence, query head).  Pass 1 sums the head's C query rows into the
//                mean query M; pass 2 computes CosSim(q_r, M) for every row (the second read of
//                the head's rows hits L2); a shared-memory bitonic sort of (cosine, position)
//                codes yields the N lowest cosines in ascending order, equal cosines by position.
// aggregate    : one warp per (sequence, KV head, rank j): mean over the G heads of the group of
//                their j-th retained query, each divided by its own norm; one rounding to dtype.
// Both are HBM/L2-bound passes over Q: rows are read with 16-byte vector loads, D/8 lanes per row.
#include "common.cuh"

namespace quoka {

constexpr int kRankThreads = 1024;

template <typename T, int D>
__global__ void __launch_bounds__(kRankThreads) rank_queries_kernel(DevParams P, const T* __restrict__ q,
                                                                     int32_t* __restrict__ q_idx) {
  constexpr int LG = D / 8;                 // lanes per row, 8 elements each
  constexpr int RPI = kRankThreads / LG;    // rows per iteration
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ float M[D];
  __shared__ float Mnorm;

  const int s = blockIdx.x / P.n_q;
  const int h = blockIdx.x % P.n_q;
  const int C = P.chunk;
  const int N = P.n_sel;
  int32_t* out = q_idx + ((int64_t)s * P.n_q + h) * N;
  const int tid = threadIdx.x;

  if (C <= P.n_retain) {                    // no sub-selection: every query, in position order
    for (int j = tid; j < C; j += kRankThreads) out[j] = j;
    return;
  }

  const T* qh = q + (int64_t)s * P.q_sb + (int64_t)h * P.q_sh;
  const int lane_in_row = tid % LG;
  const int row_slot = tid / LG;

  // ---- pass 1: column sums -> mean query
  float acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.f;
  for (int r = row_slot; r < C; r += RPI) {
    float x[8];
    load_vec<T, 8>(qh + (int64_t)r * P.q_st + lane_in_row * 8, x);
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] += x[i];
  }
  float* red = reinterpret_cast<float*>(smem_raw);        // [RPI][D]
#pragma unroll
  for (int i = 0; i < 8; ++i) red[row_slot * D + lane_in_row * 8 + i] = acc[i];
  __syncthreads();
  if (tid < D) {
    float sum = 0.f;
    for (int r = 0; r < RPI; ++r) sum += red[r * D + tid];
    M[tid] = sum / (float)C;
  }
  __syncthreads();
  if (tid < 32) {
    float p = 0.f;
    for (int x = tid; x < D; x += 32) p += M[x] * M[x];
    p = warp_sum(p);
    if (tid == 0) Mnorm = fmaxf(sqrtf(p), kNormEps);
  }
  __syncthreads();   // also: everyone is done reading `red` before the sort buffer overwrites it

  // ---- pass 2: cosine of every row to M, packed as (order code << 32 | position)
  int n_sort = 1;
  while (n_sort < C) n_sort <<= 1;
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);
  float m[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) m[i] = M[lane_in_row * 8 + i];
  const float mn = Mnorm;
  for (int r0 = 0; r0 < n_sort; r0 += RPI) {
    const int r = r0 + row_slot;
    float dot = 0.f, nn = 0.f;
    if (r < C) {
      float x[8];
      load_vec<T, 8>(qh + (int64_t)r * P.q_st + lane_in_row * 8, x);
#pragma unroll
      for (int i = 0; i < 8; ++i) { dot += x[i] * m[i]; nn += x[i] * x[i]; }
    }
#pragma unroll
    for (int o = LG / 2; o > 0; o >>= 1) {
      dot += __shfl_xor_sync(0xFFFFFFFFu, dot, o);
      nn += __shfl_xor_sync(0xFFFFFFFFu, nn, o);
    }
    if (lane_in_row == 0 && r < n_sort) {
      unsigned long long code = ~0ull;                    // padding sorts last
      if (r < C) {
        const float c = dot / (fmaxf(sqrtf(nn), kNormEps) * mn);
        code = ((unsigned long long)float_order_key(c) << 32) | (unsigned)r;
      }
      keys[r] = code;
    }
  }
  __syncthreads();

  // ---- bitonic sort, ascending
  for (int k = 2; k <= n_sort; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = tid; i < n_sort; i += kRankThreads) {
        const int ixj = i ^ j;
        if (ixj > i) {
          const unsigned long long a = keys[i], b = keys[ixj];
          const bool up = (i & k) == 0;
          if ((a > b) == up) { keys[i] = b; keys[ixj] = a; }
        }
      }
      __syncthreads();
    }
  }
  for (int j = tid; j < N; j += kRankThreads) out[j] = (int32_t)(keys[j] & 0xFFFFFFFFull);
}

template <typename T, int D>
__global__ void __launch_bounds__(256) aggregate_queries_kernel(DevParams P, const T* __restrict__ q,
                                                                 const int32_t* __restrict__ q_idx,
                                                                 T* __restrict__ qbar) {
  constexpr int NE = D / 32;
  const int N = P.n_sel;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int64_t total = (int64_t)P.batch * P.n_kv * N;
  if (warp >= total) return;
  const int j = (int)(warp % N);
  const int kv = (int)((warp / N) % P.n_kv);
  const int s = (int)(warp / ((int64_t)N * P.n_kv));
  float acc[NE];
#pragma unroll
  for (int i = 0; i < NE; ++i) acc[i] = 0.f;
  for (int g = 0; g < P.group; ++g) {
    const int h = kv * P.group + g;
    const int r = __ldg(q_idx + ((int64_t)s * P.n_q + h) * N + j);
    float x[NE];
    load_vec<T, NE>(q + (int64_t)s * P.q_sb + (int64_t)h * P.q_sh + (int64_t)r * P.q_st + lane * NE, x);
    float nn = 0.f;
#pragma unroll
    for (int i = 0; i < NE; ++i) nn += x[i] * x[i];
    nn = warp_sum(nn);
    const float norm = fmaxf(sqrtf(nn), kNormEps);
#pragma unroll
    for (int i = 0; i < NE; ++i) acc[i] += x[i] / norm;
  }
  const float inv_g = 1.f / (float)P.group;
#pragma unroll
  for (int i = 0; i < NE; ++i) acc[i] *= inv_g;
  store_vec<T, NE>(qbar + warp * D + lane * NE, acc);
}

cudaError_t launch_rank_queries(const DevParams& P, int dtype, const void* q, int32_t* q_idx, cudaStream_t st) {
  int n_sort = 1;
  while (n_sort < P.chunk) n_sort <<= 1;
  size_t smem = (size_t)n_sort * 8;
  if (smem < 32768) smem = 32768;           // the pass-1 reduction buffer [RPI][D] floats is 32 KiB
  const int grid = P.batch * P.n_q;
#define QUOKA_RANK(T, D)                                                                                       \
  do {                                                                                                         \
    cudaError_t e = cudaFuncSetAttribute(rank_queries_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                         (int)smem);                                                           \
    if (e != cudaSuccess) return e;                                                                            \
    rank_queries_kernel<T, D><<<grid, kRankThreads, smem, st>>>(P, (const T*)q, q_idx);                         \
  } while (0)
  if (dtype == QUOKA_BF16) {
    if (P.d == 128) QUOKA_RANK(__nv_bfloat16, 128); else QUOKA_RANK(__nv_bfloat16, 64);
  } else {
    if (P.d == 128) QUOKA_RANK(float, 128); else QUOKA_RANK(float, 64);
  }
#undef QUOKA_RANK
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_aggregate_queries(const DevParams& P, int dtype, const void* q, const int32_t* q_idx, void* qbar,
                                     cudaStream_t st) {
  const int64_t warps = (int64_t)P.batch * P.n_kv * P.n_sel;
  const int grid = (int)((warps * 32 + 255) / 256);
  if (dtype == QUOKA_BF16) {
    if (P.d == 128) aggregate_queries_kernel<__nv_bfloat16, 128><<<grid, 256, 0, st>>>(P, (const __nv_bfloat16*)q, q_idx, (__nv_bfloat16*)qbar);
    else aggregate_queries_kernel<__nv_bfloat16, 64><<<grid, 256, 0, st>>>(P, (const __nv_bfloat16*)q, q_idx, (__nv_bfloat16*)qbar);
  } else {
    if (P.d == 128) aggregate_queries_kernel<float, 128><<<grid, 256, 0, st>>>(P, (const float*)q, q_idx, (float*)qbar);
    else aggregate_queries_kernel<float, 64><<<grid, 256, 0, st>>>(P, (const float*)q, q_idx, (float*)qbar);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace quoka
