// Query sub-selection, normalisation and GQA pre-aggregation (Algorithm 1, first two blocks).
//
// rank_queries : a thread-block cluster of 2 / 4 / 8 CTAs (by chunk length, about 256 rows per CTA) per
//                (sequence, query head); each CTA owns a contiguous slice of the head's C query rows.
//                Pass 1 brings the slice into shared memory with 16-byte cp.async in eight groups and sums
//                the columns group by group as they land (a slice beyond the staging limit is re-read
//                from L2 instead); the CTAs' shares of the mean query are added across the cluster
//                through distributed shared memory in a fixed order.  Pass 2 computes CosSim(q_r, M) for
//                every row of the slice (two lanes per row), packs (order code of the cosine, position)
//                into one 64-bit key, sorts 32-key runs in registers (bitonic network over shuffles) and
//                merges the runs by counting (branch-free binary searches, keys are unique).  Each CTA
//                then copies the first codes of its peers' sorted slices into local shared memory and
//                places each of its N smallest by global rank: own rank + number of smaller codes in
//                every peer.  The N lowest cosines come out in ascending order, equal cosines by position.
// aggregate    : one warp per (sequence, KV head, rank j): mean over the G heads of the group of
//                their j-th retained query, each divided by its own norm; one rounding to dtype.
#include <cooperative_groups.h>

#include <type_traits>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace quoka {

constexpr int kRankThreads = 512;
constexpr int kRankCluster = 8;
// A slice larger than this is not kept in shared memory but re-read from L2 in pass 2: two CTAs must still fit an
// SM (with 128 KB slices, chunk 4096, one CTA per SM meant two waves of the grid and a fifth more time).
constexpr size_t kRankStageLimit = 84 * 1024;

template <typename T> struct Raw8;                // 8 consecutive elements as 16-byte words
template <> struct Raw8<__nv_bfloat16> { uint4 w[1]; };
template <> struct Raw8<float> { uint4 w[2]; };

template <typename T>
__device__ __forceinline__ void raw_to_f32(const Raw8<T>& r, float (&x)[8]) {
  if constexpr (sizeof(T) == 2) {
    const uint32_t w[4] = {r.w[0].x, r.w[0].y, r.w[0].z, r.w[0].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      x[2 * j] = __uint_as_float(w[j] << 16);
      x[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
    }
  } else {
    x[0] = __uint_as_float(r.w[0].x); x[1] = __uint_as_float(r.w[0].y);
    x[2] = __uint_as_float(r.w[0].z); x[3] = __uint_as_float(r.w[0].w);
    x[4] = __uint_as_float(r.w[1].x); x[5] = __uint_as_float(r.w[1].y);
    x[6] = __uint_as_float(r.w[1].z); x[7] = __uint_as_float(r.w[1].w);
  }
}

template <typename T, int D, int CL>
__global__ void __launch_bounds__(kRankThreads, 2) rank_queries_kernel(DevParams P, const T* __restrict__ q,
                                                                     int32_t* __restrict__ q_idx, int rpc, int n_sort,
                                                                     int staged, int m_peer) {
  grid_launch_dependents();                 // the aggregation kernel may become resident; it waits for this grid itself
  constexpr int LG = D / 8;                 // lanes per row, 8 elements each
  constexpr int RPI = kRankThreads / LG;    // rows per iteration
  constexpr int NW = sizeof(T) * 8 / 16;    // 16-byte words per lane
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // dynamic shared memory: sort keys | reduction buffer | peer codes | staged rows
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);               // [n_sort] 32-key sorted runs
  unsigned long long* sorted = keys + n_sort;                                               // [n_sort] the sorted slice
  float* red = reinterpret_cast<float*>(smem_raw + (size_t)n_sort * 16);                    // [RPI][D]
  unsigned long long* peer_keys = reinterpret_cast<unsigned long long*>(red + RPI * D);     // [CL - 1][m_peer]
  uint4* rows = reinterpret_cast<uint4*>(peer_keys + (((size_t)(CL - 1) * m_peer + 1) & ~(size_t)1));   // [rpc][LG][NW]
  __shared__ float part[D];                 // this CTA's share of the column sums
  __shared__ __align__(16) float M[D];
  __shared__ float Mnorm;

  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int head = blockIdx.x / CL;
  const int s = head / P.n_q, h = head % P.n_q;
  const int C = P.chunk, N = P.n_sel;
  int32_t* out = q_idx + (long long)head * N;
  const int tid = threadIdx.x;

  // (C <= N_Q, where every query is kept, never reaches this kernel: the aggregation kernel writes those ranks)
  const T* qh = q + (long long)s * P.q_sb + (long long)h * P.q_sh;
  const int lane_in_row = tid % LG;
  const int row_slot = tid / LG;
  const int lo = min(C, rank * rpc), hi = min(C, lo + rpc);
  const int n_loc = hi - lo;

  // ---- pass 1: the slice goes to shared memory with every 16-byte copy in flight at once, committed in 8
  // groups of rows; the column sums are taken group by group as the copies land, so the arithmetic runs under
  // the HBM transfer
  const int n_iter = (n_loc + RPI - 1) / RPI;                // 32/64-row trips over the slice
  const int grp_rows = ((n_iter + 7) / 8) * RPI;             // rows per copy group
  if (staged) {
    constexpr int WPR = LG * NW;                             // 16-byte words per row
    constexpr int EPW = 16 / (int)sizeof(T);                 // elements per word
    const uint32_t rows_s = (uint32_t)__cvta_generic_to_shared(rows);
#pragma unroll 1
    for (int gi = 0; gi < 8; ++gi) {
      const int w_lo = min(n_loc, gi * grp_rows) * WPR, w_hi = min(n_loc, (gi + 1) * grp_rows) * WPR;
      for (int w = w_lo + tid; w < w_hi; w += kRankThreads) {
        const int r = w / WPR, c = w % WPR;
        const T* src = qh + (long long)(lo + r) * P.q_st + c * EPW;
        // word c of row r lives in slot c ^ (r & 7): both passes then read shared memory without bank conflicts
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(rows_s + (uint32_t)(r * WPR + (c ^ (r & 7))) * 16u), "l"(src) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
  }
  float acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
  for (int gi = 0; gi < 8; ++gi) {
    if (staged) {
      switch (gi) {                                          // all but the 7 - gi newest groups have landed
        case 0: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
      }
      __syncthreads();
    }
    const int g_lo = min(n_loc, gi * grp_rows), g_hi = min(n_loc, (gi + 1) * grp_rows);
    for (int r0 = g_lo; r0 < g_hi; r0 += RPI) {
      const int r = r0 + row_slot;
      Raw8<T> raw;
      const int rc = min(r, n_loc - 1);                      // clamped: no branch around the loads
      if (staged) {
#pragma unroll
        for (int w = 0; w < NW; ++w) raw.w[w] = rows[(size_t)rc * (LG * NW) + ((lane_in_row * NW + w) ^ (rc & 7))];
      } else {
        const uint4* src = reinterpret_cast<const uint4*>(qh + (long long)(lo + rc) * P.q_st + lane_in_row * 8);
#pragma unroll
        for (int w = 0; w < NW; ++w) raw.w[w] = __ldg(src + w);
      }
      float x[8];
      raw_to_f32<T>(raw, x);
      const float live = r < n_loc ? 1.f : 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = fmaf(x[i], live, acc[i]);
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) red[row_slot * D + lane_in_row * 8 + i] = acc[i];
  __syncthreads();
  if (tid < D) {
    float sum = 0.f;
    for (int r = 0; r < RPI; ++r) sum += red[r * D + tid];
    part[tid] = sum;
  }
  cluster.sync();
  if (tid < D) {
    float sum = 0.f;
#pragma unroll
    for (int r = 0; r < CL; ++r) sum += cluster.map_shared_rank(part, r)[tid];   // fixed order
    M[tid] = sum / (float)C;
  }
  __syncthreads();
  if (tid < 32) {
    float p = 0.f;
    for (int x = tid; x < D; x += 32) p += M[x] * M[x];
    p = warp_sum(p);
    if (tid == 0) Mnorm = fmaxf(sqrtf(p), kNormEps);
  }
  __syncthreads();

  // ---- pass 2: cosine of every row of the slice to M, packed as (order code << 32 | position).  Two adjacent
  // lanes take one row (half of its 16-byte words each, the row's norm and its dot product with M in the same
  // sweep, M read from shared memory as a broadcast); one shuffle joins the halves.
  {
    constexpr int WPR = LG * NW;                             // 16-byte words per row
    constexpr int EPW = 16 / (int)sizeof(T);                 // elements per word
    constexpr int HW = WPR / 2;                              // words per half row
    const int half = tid & 1;
    const float mn = Mnorm;
    auto sweep = [&](auto from_smem) {                       // the staged / re-read choice is made once, not per word
    for (int r0 = 0; r0 < n_sort; r0 += kRankThreads / 2) {
      const int r = r0 + (tid >> 1);
      const int rc = max(min(r, n_loc - 1), 0);              // clamped (an empty slice reads row 0 / the last row)
      const uint4* grow = reinterpret_cast<const uint4*>(qh + (long long)min(lo + rc, C - 1) * P.q_st);
      float dot = 0.f, nn = 0.f;
#pragma unroll 4      // all eight words at once made the compiler spill
      for (int i = 0; i < HW; ++i) {
        const int c = half * HW + i;
        uint4 wv;
        if constexpr (decltype(from_smem)::value) wv = rows[(size_t)rc * WPR + (c ^ (rc & 7))];
        else wv = __ldg(grow + c);
        float x[EPW];
        if constexpr (sizeof(T) == 2) {
          const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) { x[2 * j] = __uint_as_float(ww[j] << 16); x[2 * j + 1] = __uint_as_float(ww[j] & 0xFFFF0000u); }
        } else {
          x[0] = __uint_as_float(wv.x); x[1] = __uint_as_float(wv.y); x[2] = __uint_as_float(wv.z); x[3] = __uint_as_float(wv.w);
        }
#pragma unroll
        for (int j = 0; j < EPW; j += 4) {
          const float4 mv = *reinterpret_cast<const float4*>(&M[c * EPW + j]);
          dot = fmaf(x[j], mv.x, dot); dot = fmaf(x[j + 1], mv.y, dot);
          dot = fmaf(x[j + 2], mv.z, dot); dot = fmaf(x[j + 3], mv.w, dot);
          nn = fmaf(x[j], x[j], nn); nn = fmaf(x[j + 1], x[j + 1], nn);
          nn = fmaf(x[j + 2], x[j + 2], nn); nn = fmaf(x[j + 3], x[j + 3], nn);
        }
      }
      dot += __shfl_xor_sync(0xFFFFFFFFu, dot, 1);
      nn += __shfl_xor_sync(0xFFFFFFFFu, nn, 1);
      if (half == 0 && r < n_sort) {
        unsigned long long code = ~0ull;                    // padding sorts last
        if (r < n_loc) {
          const float c = dot / (fmaxf(sqrtf(nn), kNormEps) * mn);
          code = ((unsigned long long)float_order_key(c) << 32) | (unsigned)(lo + r);
        }
        keys[r] = code;
      }
    }
    };
    if (staged) sweep(std::true_type{}); else sweep(std::false_type{});
  }
  __syncthreads();

  // ---- sort of the slice, ascending.  Each warp sorts 32-key runs in registers (bitonic network over
  // shuffles, no block barriers); then every key finds its place by counting the smaller keys of the other
  // runs with branch-free binary searches (keys are unique) and is scattered to `sorted`.
  const int lane = tid & 31, wid = tid >> 5;
  const int n_runs = n_sort >> 5;
  for (int run = wid; run < n_runs; run += kRankThreads / 32) {
    unsigned long long v = keys[run * 32 + lane];
#pragma unroll
    for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
      for (int j = k >> 1; j > 0; j >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, v, j);
        const bool up = (lane & k) == 0, lower = (lane & j) == 0;
        const bool take_min = up == lower;
        v = take_min ? (v < o ? v : o) : (v < o ? o : v);
      }
    }
    keys[run * 32 + lane] = v;
  }
  for (int i = tid; i < n_sort; i += kRankThreads) sorted[i] = ~0ull;   // slots the padding keys do not reach
  __syncthreads();
  for (int i = tid; i < n_sort; i += kRankThreads) {
    const unsigned long long key = keys[i];
    const int my_run = i >> 5;
    int rk = i & 31;
#pragma unroll 1
    for (int run0 = 0; run0 < n_runs; run0 += 8) {        // eight searches side by side: their loads overlap
      int pos[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) pos[u] = 0;
#pragma unroll
      for (int step = 16; step > 0; step >>= 1) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int run = min(run0 + u, n_runs - 1);
          pos[u] += keys[run * 32 + pos[u] + step - 1] < key ? step : 0;
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int run = min(run0 + u, n_runs - 1);
        pos[u] += keys[run * 32 + pos[u]] < key ? 1 : 0;
        rk += (run0 + u < n_runs && run != my_run) ? pos[u] : 0;
      }
    }
    sorted[rk] = key;                                     // padding keys are equal: they may collide, all ~0
  }
  cluster.sync();                                         // every slice is sorted

  // ---- global rank of my N smallest: own rank + number of smaller codes in each peer's slice.  Only a
  // peer's first m_peer codes matter (m_peer = a power of two >= min(n_sort, N): more smaller ones than N
  // already push the rank past N); they are copied into local shared memory first, because a chain of
  // dependent remote reads is slow.
  for (int e = tid; e < (CL - 1) * m_peer; e += kRankThreads) {
    const int pr = e / m_peer, j = e % m_peer;
    const int r = pr + (pr >= rank ? 1 : 0);
    peer_keys[e] = cluster.map_shared_rank(sorted, r)[j];
  }
  __syncthreads();
  const int n_cand = min(N, n_loc);
  for (int li = tid; li < n_cand; li += kRankThreads) {
    const unsigned long long key = sorted[li];
    int rk = li;
    int pos[CL - 1];                            // number of each peer's codes below key; the
#pragma unroll                                            // branch-free searches run side by side
    for (int pr = 0; pr < CL - 1; ++pr) pos[pr] = 0;
    for (int step = m_peer >> 1; step > 0; step >>= 1) {
#pragma unroll
      for (int pr = 0; pr < CL - 1; ++pr)
        pos[pr] += peer_keys[(size_t)pr * m_peer + pos[pr] + step - 1] < key ? step : 0;
    }
#pragma unroll
    for (int pr = 0; pr < CL - 1; ++pr) {
      pos[pr] += peer_keys[(size_t)pr * m_peer + pos[pr]] < key ? 1 : 0;
      rk += pos[pr];
    }
    if (rk < N) out[rk] = (int32_t)(key & 0xFFFFFFFFull);
  }
  cluster.sync();                                         // my keys stay mapped until every peer is done
}

template <typename T, int D>
__global__ void __launch_bounds__(256) aggregate_queries_kernel(DevParams P, const T* __restrict__ q,
                                                                 int32_t* __restrict__ q_idx,
                                                                 T* __restrict__ qbar) {
  grid_launch_dependents();
  grid_dependency_wait();                   // the ranks come from the kernel before
  // a chunk no longer than the number of retained queries keeps every query, in position order (Alg. 1's `if`):
  // no ranking kernel runs then, and this kernel writes the identity ranks itself
  const bool identity = P.chunk <= P.n_retain;
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
  for (int g0 = 0; g0 < P.group; g0 += 32) {
    // the group's ranks in one load, then the rows four at a time so their loads overlap
    const int gl = g0 + lane;
    int r_lane = j;
    if (gl < P.group) {
      int32_t* slot = q_idx + ((int64_t)s * P.n_q + kv * P.group + gl) * N + j;
      if (identity) *slot = j; else r_lane = __ldcg(slot);
    }
    const int g_end = min(32, P.group - g0);
    for (int g4 = 0; g4 < g_end; g4 += 4) {
      float x[4][NE];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int g = g4 + u;
        const int r = __shfl_sync(0xFFFFFFFFu, r_lane, g & 31);
        if (g < g_end) {
          const int h = kv * P.group + g0 + g;
          load_vec<T, NE>(q + (int64_t)s * P.q_sb + (int64_t)h * P.q_sh + (int64_t)r * P.q_st + lane * NE, x[u]);
        } else {
#pragma unroll
          for (int i = 0; i < NE; ++i) x[u][i] = 0.f;
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float nn = 0.f;
#pragma unroll
        for (int i = 0; i < NE; ++i) nn += x[u][i] * x[u][i];
        nn = warp_sum(nn);
        const float norm = P.score_dot ? 1.f : fmaxf(sqrtf(nn), kNormEps);
        if (g4 + u < g_end) {
#pragma unroll
          for (int i = 0; i < NE; ++i) acc[i] += x[u][i] / norm;
        }
      }
    }
  }
  const float inv_g = 1.f / (float)P.group;
#pragma unroll
  for (int i = 0; i < NE; ++i) acc[i] *= inv_g;
  store_vec<T, NE>(qbar + warp * D + lane * NE, acc);
}

template <typename T, int D, int CL>
static cudaError_t launch_rank_t(const DevParams& P, const void* q, int32_t* q_idx, cudaStream_t st) {
  constexpr int LG = D / 8, RPI = kRankThreads / LG;
  int rpc = (P.chunk + CL - 1) / CL;
  int n_sort = 32;
  while (n_sort < rpc) n_sort <<= 1;
  const size_t row_bytes = (size_t)rpc * D * sizeof(T);
  int m_peer = 1;
  while (m_peer < P.n_sel && m_peer < n_sort) m_peer <<= 1;
  const size_t fixed = (size_t)n_sort * 16 + (size_t)RPI * D * 4 + (((size_t)(CL - 1) * m_peer + 1) & ~(size_t)1) * 8;
  const int staged = fixed + row_bytes <= kRankStageLimit + 48 * 1024 && row_bytes <= kRankStageLimit ? 1 : 0;
  const size_t smem = fixed + (staged ? row_bytes : 0);
  cudaError_t e = cudaFuncSetAttribute(rank_queries_kernel<T, D, CL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_kernel("rank_queries", rank_queries_kernel<T, D, CL>, dim3(P.batch * P.n_q * CL), dim3(kRankThreads), smem, st, CL, false, P,
                       (const T*)q, q_idx, rpc, n_sort, staged, m_peer);
}

// A cluster per (sequence, head), sized so that a CTA's slice is about 256 rows: shorter slices only multiply the
// per-CTA costs (four cluster barriers, the sort, the merge).
template <typename T, int D>
static cudaError_t launch_rank_d(const DevParams& P, const void* q, int32_t* q_idx, cudaStream_t st) {
  if (P.chunk <= 512) return launch_rank_t<T, D, 2>(P, q, q_idx, st);
  if (P.chunk <= 1024) return launch_rank_t<T, D, 4>(P, q, q_idx, st);
  return launch_rank_t<T, D, kRankCluster>(P, q, q_idx, st);
}

cudaError_t launch_rank_queries(const DevParams& P, int dtype, const void* q, int32_t* q_idx, cudaStream_t st) {
  if (P.chunk <= P.n_retain) return cudaSuccess;      // every query is kept: the aggregation kernel writes the ranks
  cudaError_t e;
  if (dtype == QUOKA_BF16) e = P.d == 128 ? launch_rank_d<__nv_bfloat16, 128>(P, q, q_idx, st) : launch_rank_d<__nv_bfloat16, 64>(P, q, q_idx, st);
  else e = P.d == 128 ? launch_rank_d<float, 128>(P, q, q_idx, st) : launch_rank_d<float, 64>(P, q, q_idx, st);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_aggregate_queries(const DevParams& P, int dtype, const void* q, int32_t* q_idx, void* qbar,
                                     cudaStream_t st, bool chained) {
  const int64_t warps = (int64_t)P.batch * P.n_kv * P.n_sel;
  const dim3 grid((unsigned)((warps * 32 + 255) / 256)), block(256);
  cudaError_t e;
  if (dtype == QUOKA_BF16) {
    if (P.d == 128) e = launch_kernel("aggregate_queries", aggregate_queries_kernel<__nv_bfloat16, 128>, grid, block, 0, st, 1, chained, P, (const __nv_bfloat16*)q, q_idx, (__nv_bfloat16*)qbar);
    else e = launch_kernel("aggregate_queries", aggregate_queries_kernel<__nv_bfloat16, 64>, grid, block, 0, st, 1, chained, P, (const __nv_bfloat16*)q, q_idx, (__nv_bfloat16*)qbar);
  } else {
    if (P.d == 128) e = launch_kernel("aggregate_queries", aggregate_queries_kernel<float, 128>, grid, block, 0, st, 1, chained, P, (const float*)q, q_idx, (float*)qbar);
    else e = launch_kernel("aggregate_queries", aggregate_queries_kernel<float, 64>, grid, block, 0, st, 1, chained, P, (const float*)q, q_idx, (float*)qbar);
  }
  if (e != cudaSuccess) return e;
  count_launch();
  return cudaGetLastError();
}

}  // namespace quoka
