// Generation phase (a chunk of ONE query per sequence; Section 4.4, Appendix B): Algorithm 1 skips the query
// sub-selection, Q-bar is one vector per KV head, and the two contraction steps lose their matrix shape:
//   scoring    S^_t = (Qbar . k_t) / |k_t|  is a matrix-vector product that reads every cached key once:
//              HBM-bound, 2 flops per 2 bytes.  score_keys_gemv_kernel streams the keys with 16-byte loads,
//              32 bytes of a row per lane, four rows in flight per lane.
//   attention  each query head attends B + 1 rows.  decode_attn_kernel gathers them once per head, keeps the
//              logits in shared memory, and accumulates P V per warp.
// The tensor-core kernels would spend a 128-row MMA tile on one query.  Everything is fp32 arithmetic on the
// stored values; the softmax weights are not rounded to bf16 here.
#include "common.cuh"

namespace quoka {

constexpr int kGemvThreads = 256;
constexpr int kGemvRowsPerCta = 512;
constexpr int kDecodeAttnThreads = 256;
constexpr int kDecodeMaxKeys = 8192;          // logits of one head kept in shared memory (32 KiB)

// 8 consecutive elements as floats from one 16-byte word (bf16) or two (f32 uses 4 per word: see LPR below).
template <typename T> struct VecOf;
template <> struct VecOf<__nv_bfloat16> { static constexpr int N = 8; };
template <> struct VecOf<float> { static constexpr int N = 4; };

template <typename T>
__device__ __forceinline__ void word_to_f32(const uint4& w, float* x) {
  if constexpr (sizeof(T) == 2) {
    const uint32_t v[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) { x[2 * j] = __uint_as_float(v[j] << 16); x[2 * j + 1] = __uint_as_float(v[j] & 0xFFFF0000u); }
  } else {
    x[0] = __uint_as_float(w.x); x[1] = __uint_as_float(w.y); x[2] = __uint_as_float(w.z); x[3] = __uint_as_float(w.w);
  }
}

// ------------------------------------------------------------------------------------------ scoring (N = 1)
// grid = (row slices, KV heads, sequences); a CTA scores kGemvRowsPerCta consecutive cached rows of one
// (sequence, KV head).  LPR lanes share a row, 32 bytes (two 16-byte words, one DRAM sector) each; a warp covers
// 32 / LPR rows per trip and keeps UNR trips (2 * UNR loads per lane) in flight.
template <typename T, int D>
__global__ void __launch_bounds__(kGemvThreads) score_keys_gemv_kernel(DevParams P, const T* __restrict__ qbar,
                                                                        const T* __restrict__ k,
                                                                        float* __restrict__ scores) {
  constexpr int NE = VecOf<T>::N;                    // elements per 16-byte word
  constexpr int LPR = D / (2 * NE);                  // lanes per row
  constexpr int RPW = 32 / LPR;                      // rows per warp trip
  constexpr int UNR = 4;
  grid_launch_dependents();
  const int s = blockIdx.z, kv = blockIdx.y;
  const int T_s = __ldg(P.ctx_len + s);
  const int row0 = blockIdx.x * kGemvRowsPerCta;
  if (row0 >= T_s) { grid_dependency_wait(); return; }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = lane % LPR, rsub = lane / LPR;
  grid_dependency_wait();                            // Q-bar comes from the kernel before
  float qv[2 * NE];
  {
    const uint4* qp = reinterpret_cast<const uint4*>(qbar + ((long long)s * P.n_kv + kv) * D) + 2 * c;
    word_to_f32<T>(__ldcg(qp), qv);
    word_to_f32<T>(__ldcg(qp + 1), qv + NE);
  }
  const bool cosine = !P.score_dot;
  const bool cached = cosine && P.k_inv_norm != nullptr;
  float* out = scores + ((long long)s * P.n_kv + kv) * P.max_ctx;
  const int row_end = min(T_s, row0 + kGemvRowsPerCta);
  constexpr int kWarps = kGemvThreads / 32;
  for (int r = row0 + warp * RPW * UNR; r < row_end; r += kWarps * RPW * UNR) {
    uint4 w[UNR][2];
    int t[UNR];
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      t[u] = r + u * RPW + rsub;
      const int tc = min(t[u], row_end - 1);         // clamped: no branch around the loads
      const uint4* kp = reinterpret_cast<const uint4*>(k + kv_row_offset(P, s, kv, tc)) + 2 * c;
      w[u][0] = __ldg(kp);
      w[u][1] = __ldg(kp + 1);
    }
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      float x[2 * NE];
      word_to_f32<T>(w[u][0], x);
      word_to_f32<T>(w[u][1], x + NE);
      float dot = 0.f, dot1 = 0.f, nn = 0.f, nn1 = 0.f;
#pragma unroll
      for (int i = 0; i < NE; ++i) {
        dot = fmaf(x[i], qv[i], dot); nn = fmaf(x[i], x[i], nn);
        dot1 = fmaf(x[NE + i], qv[NE + i], dot1); nn1 = fmaf(x[NE + i], x[NE + i], nn1);
      }
      dot += dot1; nn += nn1;
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) {
        dot += __shfl_xor_sync(0xFFFFFFFFu, dot, o);
        nn += __shfl_xor_sync(0xFFFFFFFFu, nn, o);
      }
      if (c == 0 && t[u] < row_end) {
        float val = dot;
        if (cached) val = dot * __ldg(P.k_inv_norm + kv_norm_index(P, s, kv, t[u]));
        else if (cosine) val = dot / fmaxf(sqrtf(nn), kNormEps);
        out[t[u]] = val;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------ attention (C = 1)
// grid = (query heads, sequences).  The head's single query attends the listed cached rows and its own row T_s.
template <typename T, int D>
__global__ void __launch_bounds__(kDecodeAttnThreads) decode_attn_kernel(DevParams P, const T* __restrict__ q,
                                                                          const T* __restrict__ k,
                                                                          const T* __restrict__ v,
                                                                          const int32_t* __restrict__ k_idx,
                                                                          const int32_t* __restrict__ k_cnt,
                                                                          T* __restrict__ out, float* __restrict__ lse) {
  constexpr int NE = VecOf<T>::N;
  constexpr int LPR = D / NE;
  constexpr int RPW = 32 / LPR;
  constexpr int kWarps = kDecodeAttnThreads / 32;
  extern __shared__ float logit[];                   // [n_keys], then the warps' partial outputs
  __shared__ float red[kWarps];
  __shared__ float red2[kWarps];
  const int h = blockIdx.x, s = blockIdx.y, kv = h / P.group;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = lane % LPR, rsub = lane / LPR;
  const int T_s = __ldg(P.ctx_len + s);
  float qv[NE];
  {
    const uint4 w = __ldg(reinterpret_cast<const uint4*>(q + (long long)s * P.q_sb + (long long)h * P.q_sh) + c);
    word_to_f32<T>(w, qv);
#pragma unroll
    for (int i = 0; i < NE; ++i) qv[i] *= P.scale;
  }
  grid_dependency_wait();                            // the list comes from the kernel before
  const int cnt = k_idx ? __ldcg(k_cnt + s) : T_s;   // without a list: every cached row (Eq. 2)
  const int32_t* idx = k_idx ? k_idx + ((long long)s * P.n_kv + kv) * P.budget_cap : nullptr;
  const int n_keys = cnt + 1;                        // the listed rows, then the query's own row T_s
  const auto row_of = [&](int u) { return u < cnt ? (idx ? __ldcg(idx + u) : u) : T_s; };
  // ---- logits.  A lane group takes UNR keys per trip: their list entries are fetched first, then their rows, so
  // a trip costs two memory round trips, not 2 * UNR.
  constexpr int UNR = 8;
  float m_loc = -INFINITY;
  for (int u0 = warp * RPW * UNR; u0 < n_keys; u0 += kWarps * RPW * UNR) {
    int t[UNR];
#pragma unroll
    for (int j = 0; j < UNR; ++j) t[j] = row_of(min(u0 + j * RPW + rsub, n_keys - 1));
    uint4 w[UNR];
#pragma unroll
    for (int j = 0; j < UNR; ++j) w[j] = __ldg(reinterpret_cast<const uint4*>(k + kv_row_offset(P, s, kv, t[j])) + c);
#pragma unroll
    for (int j = 0; j < UNR; ++j) {
      const int u = u0 + j * RPW + rsub;
      float x[NE];
      word_to_f32<T>(w[j], x);
      float dot = 0.f;
#pragma unroll
      for (int i = 0; i < NE; ++i) dot = fmaf(x[i], qv[i], dot);
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, o);
      if (u < n_keys) {
        if (c == 0) logit[u] = dot;
        m_loc = fmaxf(m_loc, dot);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m_loc = fmaxf(m_loc, __shfl_xor_sync(0xFFFFFFFFu, m_loc, o));
  if (lane == 0) red[warp] = m_loc;
  __syncthreads();
  float m = red[0];
#pragma unroll
  for (int i = 1; i < kWarps; ++i) m = fmaxf(m, red[i]);
  // ---- weights and P V: every warp takes the keys it scored; each lane accumulates its word of the row
  float acc[NE];
#pragma unroll
  for (int i = 0; i < NE; ++i) acc[i] = 0.f;
  float l_loc = 0.f;
  for (int u0 = warp * RPW * UNR; u0 < n_keys; u0 += kWarps * RPW * UNR) {
    int t[UNR];
#pragma unroll
    for (int j = 0; j < UNR; ++j) t[j] = row_of(min(u0 + j * RPW + rsub, n_keys - 1));
    uint4 w[UNR];
#pragma unroll
    for (int j = 0; j < UNR; ++j) w[j] = __ldg(reinterpret_cast<const uint4*>(v + kv_row_offset(P, s, kv, t[j])) + c);
#pragma unroll
    for (int j = 0; j < UNR; ++j) {
      const int u = u0 + j * RPW + rsub;
      float x[NE];
      word_to_f32<T>(w[j], x);
      const float p = u < n_keys ? __expf(logit[min(u, n_keys - 1)] - m) : 0.f;
      if (c == 0) l_loc += p;
#pragma unroll
      for (int i = 0; i < NE; ++i) acc[i] = fmaf(p, x[i], acc[i]);
    }
  }
  // lanes that hold the same word of different rows, then the warps
#pragma unroll
  for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
    for (int i = 0; i < NE; ++i) acc[i] += __shfl_xor_sync(0xFFFFFFFFu, acc[i], o);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l_loc += __shfl_xor_sync(0xFFFFFFFFu, l_loc, o);
  __syncthreads();                                   // the logits are done with: their memory takes the partial sums
  float* part = logit;                               // [kWarps][D]
  if (rsub == 0) {
#pragma unroll
    for (int i = 0; i < NE; ++i) part[warp * D + c * NE + i] = acc[i];
  }
  if (lane == 0) red2[warp] = l_loc;
  __syncthreads();
  float l = 0.f;
#pragma unroll
  for (int i = 0; i < kWarps; ++i) l += red2[i];
  for (int x = threadIdx.x; x < D; x += kDecodeAttnThreads) {
    float o = 0.f;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) o += part[i * D + x];
    out[(long long)s * P.o_sb + (long long)h * P.o_sh + x] = from_f32<T>(o / l);
  }
  if (lse && threadIdx.x == 0) lse[(long long)s * P.n_q + h] = m + logf(l);
}

// ---------------------------------------------------------------------------------------------- host
bool decode_path_applies(const DevParams& P) {
  return P.chunk == 1 && P.n_sel == 1;
}

cudaError_t launch_score_keys_gemv(const DevParams& P, int dtype, const void* qbar, const void* k, float* scores,
                                   cudaStream_t st, bool chained) {
  if (P.max_ctx <= 0) return cudaSuccess;
  const dim3 grid((P.max_ctx + kGemvRowsPerCta - 1) / kGemvRowsPerCta, P.n_kv, P.batch), block(kGemvThreads);
  cudaError_t e;
  if (dtype == QUOKA_BF16) {
    if (P.d == 128) e = launch_kernel("score_keys_gemv", score_keys_gemv_kernel<__nv_bfloat16, 128>, grid, block, 0, st, 1, chained, P, (const __nv_bfloat16*)qbar, (const __nv_bfloat16*)k, scores);
    else e = launch_kernel("score_keys_gemv", score_keys_gemv_kernel<__nv_bfloat16, 64>, grid, block, 0, st, 1, chained, P, (const __nv_bfloat16*)qbar, (const __nv_bfloat16*)k, scores);
  } else {
    if (P.d == 128) e = launch_kernel("score_keys_gemv", score_keys_gemv_kernel<float, 128>, grid, block, 0, st, 1, chained, P, (const float*)qbar, (const float*)k, scores);
    else e = launch_kernel("score_keys_gemv", score_keys_gemv_kernel<float, 64>, grid, block, 0, st, 1, chained, P, (const float*)qbar, (const float*)k, scores);
  }
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaGetLastError();
}

// Whether decode_attn_kernel can hold one head's logits (the listed rows and the query's own).
bool decode_attn_fits(const DevParams& P, bool with_list) {
  const long long keys = (with_list ? (long long)P.budget_cap : (long long)P.max_ctx) + 1;
  return keys <= kDecodeMaxKeys;
}

cudaError_t launch_decode_attn(const DevParams& P, int dtype, const void* q, const void* k, const void* v,
                               const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, cudaStream_t st,
                               bool chained) {
  const long long keys = (k_idx ? (long long)P.budget_cap : (long long)P.max_ctx) + 1;
  size_t smem = (size_t)keys * sizeof(float);
  const size_t part = (size_t)(kDecodeAttnThreads / 32) * P.d * sizeof(float);
  if (smem < part) smem = part;
  const dim3 grid(P.n_q, P.batch), block(kDecodeAttnThreads);
  cudaError_t e;
#define QUOKA_DECODE_ATTN(T_, D_)                                                                                  \
  e = launch_kernel("decode_attn", decode_attn_kernel<T_, D_>, grid, block, smem, st, 1, chained, P, (const T_*)q, \
                    (const T_*)k, (const T_*)v, k_idx, k_cnt, (T_*)out, lse)
  if (dtype == QUOKA_BF16) {
    if (P.d == 128) QUOKA_DECODE_ATTN(__nv_bfloat16, 128); else QUOKA_DECODE_ATTN(__nv_bfloat16, 64);
  } else {
    if (P.d == 128) QUOKA_DECODE_ATTN(float, 128); else QUOKA_DECODE_ATTN(float, 64);
  }
#undef QUOKA_DECODE_ATTN
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaGetLastError();
}

}  // namespace quoka
