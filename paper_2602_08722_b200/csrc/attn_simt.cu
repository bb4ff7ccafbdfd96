// Scalar fp32 attention over [selected cached rows | the chunk's own causal rows] (Algorithm 2's
// attention line; Eq. 1 / Eq. 2).  Serves the f32 dtype and cross-checks the tensor-core kernel.
// One warp per (sequence, query head, chunk row); the 32 lanes split head_dim; keys are visited one
// by one with a running maximum, running denominator and running output (online softmax, fp32).
// The two running sums are compensated (Kahan): once a dominant key is in them, thousands of weights below half
// an ulp of the sum would otherwise vanish one by one, a bias of up to n * 2^-24 relative (5e-5 seen at 5000 keys).
// With k_idx == nullptr every cached row is visited (Eq. 2, dense chunk attention).
#include "common.cuh"

namespace quoka {

template <typename E, int D>
__global__ void __launch_bounds__(256) attn_simt_kernel(DevParams P, const E* __restrict__ q,
                                                         const E* __restrict__ k, const E* __restrict__ v,
                                                         const int32_t* __restrict__ k_idx,
                                                         const int32_t* __restrict__ k_cnt, E* __restrict__ out,
                                                         float* __restrict__ lse) {
  constexpr int NE = D / 32;
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int64_t total = (int64_t)P.batch * P.n_q * P.chunk;
  if (warp >= total) return;
  const int r = (int)(warp % P.chunk);
  const int h = (int)((warp / P.chunk) % P.n_q);
  const int s = (int)(warp / ((int64_t)P.chunk * P.n_q));
  const int kv = h / P.group;
  const int T = __ldg(P.ctx_len + s);
  const int n_cached = k_idx ? __ldg(k_cnt + s) : T;
  const int32_t* idx = k_idx ? k_idx + ((int64_t)s * P.n_kv + kv) * P.budget_cap : nullptr;

  float qv[NE];
  load_vec<E, NE>(q + (int64_t)s * P.q_sb + (int64_t)h * P.q_sh + (int64_t)r * P.q_st + lane * NE, qv);
#pragma unroll
  for (int i = 0; i < NE; ++i) qv[i] *= P.scale;

  float m = -INFINITY, l = 0.f, o[NE];
  float cl = 0.f, co[NE];                   // what the sums have lost so far
#pragma unroll
  for (int i = 0; i < NE; ++i) { o[i] = 0.f; co[i] = 0.f; }

  const int n_total = n_cached + r + 1;
  for (int u = 0; u < n_total; ++u) {
    const int t = (u < n_cached) ? (idx ? __ldg(idx + u) : u) : (T + (u - n_cached));
    const int64_t off = kv_row_offset(P, s, kv, t) + lane * NE;
    float kx[NE], vx[NE];
    load_vec<E, NE>(k + off, kx);
    load_vec<E, NE>(v + off, vx);
    float dot = 0.f;
#pragma unroll
    for (int i = 0; i < NE; ++i) dot = fmaf(qv[i], kx[i], dot);
    dot = warp_sum(dot);
    const float m_new = fmaxf(m, dot);
    const float alpha = expf(m - m_new);
    const float p = expf(dot - m_new);
    {
      l *= alpha; cl *= alpha;
      const float y = p - cl, t = l + y;
      cl = (t - l) - y;
      l = t;
    }
#pragma unroll
    for (int i = 0; i < NE; ++i) {
      o[i] *= alpha; co[i] *= alpha;
      const float y = p * vx[i] - co[i], t = o[i] + y;
      co[i] = (t - o[i]) - y;
      o[i] = t;
    }
    m = m_new;
  }
  const float inv = 1.f / l;
#pragma unroll
  for (int i = 0; i < NE; ++i) o[i] *= inv;
  store_vec<E, NE>(out + (int64_t)s * P.o_sb + (int64_t)h * P.o_sh + (int64_t)r * P.o_st + lane * NE, o);
  if (lse && lane == 0) lse[((int64_t)s * P.n_q + h) * P.chunk + r] = m + logf(l);
}

cudaError_t launch_attn_simt(const DevParams& P, int dtype, const void* q, const void* k, const void* v,
                             const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, cudaStream_t st) {
  const int64_t warps = (int64_t)P.batch * P.n_q * P.chunk;
  const int grid = (int)((warps * 32 + 255) / 256);
  log_launch("attn_simt", dim3(grid), dim3(256), 0, 1, false);
#define QUOKA_ATTN(T_, D) \
  attn_simt_kernel<T_, D><<<grid, 256, 0, st>>>(P, (const T_*)q, (const T_*)k, (const T_*)v, k_idx, k_cnt, (T_*)out, lse)
  if (dtype == QUOKA_BF16) {
    if (P.d == 128) QUOKA_ATTN(__nv_bfloat16, 128); else QUOKA_ATTN(__nv_bfloat16, 64);
  } else {
    if (P.d == 128) QUOKA_ATTN(float, 128); else QUOKA_ATTN(float, 64);
  }
#undef QUOKA_ATTN
  count_launch();
  return cudaGetLastError();
}

}  // namespace quoka
