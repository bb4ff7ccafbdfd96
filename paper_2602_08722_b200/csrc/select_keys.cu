// Top-B key selection (Algorithm 1: I = topk(S^, B_SA)) as a radix select.
//
// One CTA per (sequence, KV head).  The fp32 scores are mapped to order-preserving uint32 codes;
// four 8-bit passes, most significant digit first, narrow a (prefix, need) pair until `prefix` is the
// code of the B-th largest score and `need` is how many rows with exactly that code are still to be
// taken.  Digit histograms live in shared memory and are filled with warp-aggregated atomics
// (match + popc, one atomic per distinct digit per warp); the bin holding the B-th largest is found
// by one warp with a shuffle prefix sum.  The output pass walks the rows in position order and
// computes each selected row's slot with warp ballots and a block prefix sum, so the list comes out
// ascending and rows that tie at the threshold are taken lowest position first.  After the first
// pass the scores are re-read from L2.
#include "common.cuh"

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

cudaError_t launch_select_keys(const DevParams& P, const float* scores, int32_t* k_idx, int32_t* k_cnt,
                               cudaStream_t st) {
  select_keys_kernel<<<P.batch * P.n_kv, kSelThreads, 0, st>>>(P, scores, k_idx, k_cnt);
  count_launch();
  return cudaGetLastError();
}

}  // namespace quoka
