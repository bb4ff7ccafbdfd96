// Top-B key selection (Algorithm 1: I = topk(S^, B_SA)) as a radix select.
//
// One CTA per (sequence, KV head).  The fp32 scores are mapped to order-preserving uint32 codes;
// four 8-bit passes, most significant digit first, narrow a (prefix, need) pair until `prefix` is the
// code of the B-th largest score and `need` is how many rows with exactly that code are still to be
// taken.  Digit histograms live in shared memory and are filled with warp-aggregated atomics
// (match + popc, one atomic per distinct digit per warp); the bin holding the B-th largest is found
// by one warp with a shuffle prefix sum.  The output pass walks the rows in position order and
// computes each selected row's slot with warp ballots and a block prefix sum, so the list comes out
// ascending and rows that tie at the threshold are taken lowest position first.
//
// Two kernels share that scheme.  select_keys_cluster_kernel (the default) gives each (sequence, KV
// head) a thread-block cluster of 8 CTAs: every CTA keeps its contiguous slice of the row in shared
// memory as order codes (one read of the scores from HBM, all later passes on chip), the per-CTA
// digit histograms are summed through distributed shared memory, and the per-CTA selected counts are
// prefix-summed the same way so the output stays ascending across the cluster.  select_keys_kernel
// (one CTA per head, scores re-read from L2 every pass) serves rows too long for the slices.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace quoka {

constexpr int kSelThreads = 1024;

__global__ void __launch_bounds__(kSelThreads) select_keys_kernel(DevParams P, const float* __restrict__ scores,
                                                                   int32_t* __restrict__ k_idx,
                                                                   int32_t* __restrict__ k_cnt) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_need;
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t warp_off[33];

  const int s = blockIdx.x / P.n_kv, kv = blockIdx.x % P.n_kv;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int T = __ldg(P.ctx_len + s);
  const int B = key_budget(T, P.kv_budget, P.budget_frac);
  const float* row = scores + ((int64_t)s * P.n_kv + kv) * P.max_ctx;
  int32_t* out = k_idx + ((int64_t)s * P.n_kv + kv) * P.budget_cap;
  if (kv == 0 && tid == 0) k_cnt[s] = B;
  for (int i = B + tid; i < P.budget_cap; i += kSelThreads) out[i] = -1;
  if (B <= 0) return;
  if (B >= T) {                              // budget covers the cache: identity
    for (int i = tid; i < T; i += kSelThreads) out[i] = i;
    return;
  }

  uint32_t prefix = 0, mask = 0, need = (uint32_t)B;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int t0 = 0; t0 < T; t0 += kSelThreads) {
      const int t = t0 + tid;
      const bool in = t < T;
      const uint32_t key = in ? float_order_key(__ldg(row + t)) : 0u;
      const bool live = in && ((key & mask) == prefix);
      const uint32_t digit = live ? ((key >> shift) & 255u) : 256u + (uint32_t)lane;   // dead lanes match nobody
      const uint32_t peers = __match_any_sync(0xFFFFFFFFu, digit);
      if (live && lane == (__ffs(peers) - 1)) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
    }
    __syncthreads();
    if (wid == 0) {
      // lane l owns bins 255-8l .. 248-8l (descending); find the bin where the running count reaches `need`
      uint32_t c[8], sum = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { c[i] = hist[255 - 8 * lane - i]; sum += c[i]; }
      uint32_t incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
      }
      const uint32_t excl = incl - sum;
      const uint32_t hit = __ballot_sync(0xFFFFFFFFu, incl >= need);
      if (lane == (__ffs(hit) - 1)) {
        uint32_t cum = excl;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (cum + c[i] >= need) {
            s_prefix = prefix | ((uint32_t)(255 - 8 * lane - i) << shift);
            s_need = need - cum;
            break;
          }
          cum += c[i];
        }
      }
    }
    __syncthreads();
    prefix = s_prefix;
    need = s_need;
    mask |= 255u << shift;
  }
  // prefix = code of the B-th largest score; take every row above it and the first `need` rows equal to it
  const uint32_t thr = prefix;
  uint32_t run_gt = 0, run_eq = 0;
  for (int t0 = 0; t0 < T; t0 += kSelThreads) {
    const int t = t0 + tid;
    const uint32_t key = (t < T) ? float_order_key(__ldg(row + t)) : 0u;
    const bool gt = (t < T) && key > thr;
    const bool eq = (t < T) && key == thr;
    const uint32_t b_gt = __ballot_sync(0xFFFFFFFFu, gt);
    const uint32_t b_eq = __ballot_sync(0xFFFFFFFFu, eq);
    if (lane == 0) warp_tot[wid] = (uint32_t)__popc(b_gt) | ((uint32_t)__popc(b_eq) << 16);
    __syncthreads();
    if (wid == 0) {
      const uint32_t v = warp_tot[lane];
      uint32_t incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += u;
      }
      warp_off[lane] = incl - v;
      if (lane == 31) warp_off[32] = incl;
    }
    __syncthreads();
    const uint32_t off = warp_off[wid], tot = warp_off[32];
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t gt_before = run_gt + (off & 0xFFFFu) + (uint32_t)__popc(b_gt & lt);
    const uint32_t eq_before = run_eq + (off >> 16) + (uint32_t)__popc(b_eq & lt);
    if (gt || (eq && eq_before < need)) out[gt_before + min(eq_before, need)] = t;
    run_gt += tot & 0xFFFFu;
    run_eq += tot >> 16;
  }
}

constexpr int kSelCluster = 8;
constexpr int kSelMaxSlice = 53248;       // order codes per CTA that fit in shared memory (208 KiB)

// Finds, among 256 bins summed over the cluster, the bin in which the running count (from bin 255
// down) reaches `need`.  Called by warp 0; lane l owns bins 255-8l .. 248-8l.
__device__ __forceinline__ void find_bin(const uint32_t* tot, uint32_t need, uint32_t prefix, int shift, int lane,
                                         uint32_t* s_prefix, uint32_t* s_need) {
  uint32_t c[8], sum = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) { c[i] = tot[255 - 8 * lane - i]; sum += c[i]; }
  uint32_t incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += v;
  }
  const uint32_t hit = __ballot_sync(0xFFFFFFFFu, incl >= need);
  if (lane == (__ffs(hit) - 1)) {
    uint32_t cum = incl - sum;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (cum + c[i] >= need) {
        *s_prefix = prefix | ((uint32_t)(255 - 8 * lane - i) << shift);
        *s_need = need - cum;
        break;
      }
      cum += c[i];
    }
  }
}

__global__ void __launch_bounds__(kSelThreads) select_keys_cluster_kernel(DevParams P, const float* __restrict__ scores,
                                                                           int32_t* __restrict__ k_idx,
                                                                           int32_t* __restrict__ k_cnt) {
  extern __shared__ uint32_t keys[];            // this CTA's slice as order codes
  __shared__ uint32_t hist[256];
  __shared__ uint32_t tot[256];
  __shared__ uint32_t s_prefix, s_need;
  __shared__ uint32_t my_cnt[2];                // rows of my slice above / equal to the threshold
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t warp_off[33];

  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int head = blockIdx.x / kSelCluster;
  const int s = head / P.n_kv, kv = head % P.n_kv;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int T = __ldg(P.ctx_len + s);
  const int B = key_budget(T, P.kv_budget, P.budget_frac);
  const float* row = scores + (long long)head * P.max_ctx;
  int32_t* out = k_idx + (long long)head * P.budget_cap;
  const int gtid = rank * kSelThreads + tid;
  constexpr int kAll = kSelCluster * kSelThreads;
  if (kv == 0 && gtid == 0) k_cnt[s] = B;
  for (int i = B + gtid; i < P.budget_cap; i += kAll) out[i] = -1;
  if (B <= 0) return;                           // uniform over the cluster
  if (B >= T) {
    for (int i = gtid; i < T; i += kAll) out[i] = i;
    return;
  }
  // slice [lo, hi) of the row, a multiple of the block size so the output pass sees whole chunks
  const int slice = ((T + kSelCluster - 1) / kSelCluster + kSelThreads - 1) / kSelThreads * kSelThreads;
  const int lo = min(T, rank * slice), hi = min(T, lo + slice);
  const int n = hi - lo;
  for (int i0 = 0; i0 < n; i0 += 4 * kSelThreads) {      // four independent loads in flight per thread
    float v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * kSelThreads + tid;
      v[u] = i < n ? __ldg(row + lo + i) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * kSelThreads + tid;
      if (i < n) keys[i] = float_order_key(v[u]);
    }
  }
  uint32_t prefix = 0, mask = 0, need = (uint32_t)B;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();                            // also orders the slice stores before the first pass
    for (int i0 = 0; i0 < n; i0 += kSelThreads) {
      const int i = i0 + tid;
      const bool in = i < n;
      const uint32_t key = in ? keys[i] : 0u;
      const bool live = in && ((key & mask) == prefix);
      const uint32_t digit = live ? ((key >> shift) & 255u) : 256u + (uint32_t)lane;
      const uint32_t peers = __match_any_sync(0xFFFFFFFFu, digit);
      if (live && lane == (__ffs(peers) - 1)) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
    }
    cluster.sync();                             // every CTA's histogram is complete
    if (tid < 256) {
      uint32_t sum = 0;
#pragma unroll
      for (int r = 0; r < kSelCluster; ++r) sum += cluster.map_shared_rank(hist, r)[tid];
      tot[tid] = sum;
    }
    __syncthreads();
    if (wid == 0) find_bin(tot, need, prefix, shift, lane, &s_prefix, &s_need);
    cluster.sync();                             // peers are done reading my histogram before it is zeroed
    prefix = s_prefix;
    need = s_need;
    mask |= 255u << shift;
  }
  const uint32_t thr = prefix;
  // rows of my slice above / equal to the threshold, then the offsets of my slice in the output
  uint32_t c_gt = 0, c_eq = 0;
  for (int i = tid; i < n; i += kSelThreads) {
    const uint32_t key = keys[i];
    c_gt += key > thr;
    c_eq += key == thr;
  }
  c_gt = __reduce_add_sync(0xFFFFFFFFu, c_gt);
  c_eq = __reduce_add_sync(0xFFFFFFFFu, c_eq);
  if (tid < 2) my_cnt[tid] = 0;
  __syncthreads();
  if (lane == 0) { atomicAdd(&my_cnt[0], c_gt); atomicAdd(&my_cnt[1], c_eq); }
  cluster.sync();
  uint32_t run_gt = 0, run_eq = 0;
  for (int r = 0; r < rank; ++r) {
    const uint32_t* pc = cluster.map_shared_rank(my_cnt, r);
    run_gt += pc[0];
    run_eq += pc[1];
  }
  for (int i0 = 0; i0 < n; i0 += kSelThreads) {
    const int i = i0 + tid;
    const uint32_t key = (i < n) ? keys[i] : 0u;
    const bool gt = (i < n) && key > thr;
    const bool eq = (i < n) && key == thr;
    const uint32_t b_gt = __ballot_sync(0xFFFFFFFFu, gt);
    const uint32_t b_eq = __ballot_sync(0xFFFFFFFFu, eq);
    if (lane == 0) warp_tot[wid] = (uint32_t)__popc(b_gt) | ((uint32_t)__popc(b_eq) << 16);
    __syncthreads();
    if (wid == 0) {
      const uint32_t v = warp_tot[lane];
      uint32_t incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += u;
      }
      warp_off[lane] = incl - v;
      if (lane == 31) warp_off[32] = incl;
    }
    __syncthreads();
    const uint32_t off = warp_off[wid], total = warp_off[32];
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t gt_before = run_gt + (off & 0xFFFFu) + (uint32_t)__popc(b_gt & lt);
    const uint32_t eq_before = run_eq + (off >> 16) + (uint32_t)__popc(b_eq & lt);
    if (gt || (eq && eq_before < need)) out[gt_before + min(eq_before, need)] = lo + i;
    run_gt += total & 0xFFFFu;
    run_eq += total >> 16;
  }
  cluster.sync();                               // my_cnt stays mapped until every peer has read it
}

cudaError_t launch_select_keys(const DevParams& P, const float* scores, int32_t* k_idx, int32_t* k_cnt,
                               cudaStream_t st) {
  const int slice = ((P.max_ctx + kSelCluster - 1) / kSelCluster + kSelThreads - 1) / kSelThreads * kSelThreads;
  if (slice <= kSelMaxSlice) {
    const size_t smem = (size_t)(slice > 0 ? slice : 1) * sizeof(uint32_t);
    cudaError_t e = cudaFuncSetAttribute(select_keys_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(P.batch * P.n_kv * kSelCluster);
    cfg.blockDim = dim3(kSelThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kSelCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, select_keys_cluster_kernel, P, scores, k_idx, k_cnt);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
  }
  select_keys_kernel<<<P.batch * P.n_kv, kSelThreads, 0, st>>>(P, scores, k_idx, k_cnt);
  count_launch();
  return cudaGetLastError();
}

}  // namespace quoka
