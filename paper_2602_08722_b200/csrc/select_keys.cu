// Top-B key selection (Algorithm 1: I = topk(S^, B_SA)) as a radix select.
//
// The fp32 scores are mapped to order-preserving uint32 codes; digit passes, most significant first,
// narrow a (prefix, need) pair until `prefix` is the code of the B-th largest score and `need` is how
// many rows with exactly that code are still to be taken.  The output pass walks the rows in position
// order and computes each selected row's slot with warp ballots and prefix sums, so the list comes out
// ascending and rows that tie at the threshold are taken lowest position first.
//
// select_keys_reg_kernel (the default): one CTA of 1024 threads per (sequence, KV head), or a cluster
// of 2/4/8 CTAs for long rows, holds the whole row as order codes IN REGISTERS (up to 32 per thread:
// the scores are read from memory exactly once, coalesced).  A single CTA first histograms the row over
// bins linear in the score, finds the bin of the B-th largest with a block-wide suffix scan, and ranks
// that bin's few rows against each other.  Otherwise (clusters; many equal scores) three digit passes of
// 12 + 12 + 8 bits over (code - smallest code of the row) shifted up to the top bit: each pass histograms
// only the rows still matching the prefix, and with a cluster the per-CTA histograms and counts are
// summed through distributed shared memory.  The list is collected in shared memory and copied out with
// full-width stores (single CTA).
// select_keys_kernel (one CTA per head, scores re-read from L2 every pass, 8-bit digits) serves rows
// too long for that.
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

  grid_launch_dependents();     // the attention kernel may start now: it waits for this grid itself before it reads the list
  grid_dependency_wait();       // the scores come from the kernel before
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


constexpr int kRegBins = 4096;            // 12-bit digits
constexpr int kHistWords = 2 * kRegBins + 256;
constexpr int kCandMax = 256;              // rows of the threshold's bin that are listed instead of passed again

// Warp w of CTA r owns positions [r*1024*ITEMS + w*32*ITEMS, +32*ITEMS); lane l holds i*32 + l of them.
template <int ITEMS, int CL>
__global__ void __launch_bounds__(kSelThreads) select_keys_reg_kernel(DevParams P, const float* __restrict__ scores,
                                                                       int32_t* __restrict__ k_idx,
                                                                       int32_t* __restrict__ k_cnt) {
  __shared__ uint32_t hist_all[kHistWords];     // one histogram per pass, zeroed once: no barrier to re-use one
  __shared__ uint32_t s_bin, s_need, s_cand, s_n;
  __shared__ uint32_t warp_val[32];
  __shared__ uint32_t warp_off[33];
  __shared__ uint32_t cta_cnt[2];               // rows of this CTA above / equal to the threshold

  grid_launch_dependents();     // the attention kernel may start now: it waits for this grid itself before it reads the list
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = CL > 1 ? (int)cluster.block_rank() : 0;
  const int head = blockIdx.x / CL;
  const int s = head / P.n_kv, kv = head % P.n_kv;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int T = __ldg(P.ctx_len + s);
  const int B = key_budget(T, P.kv_budget, P.budget_frac);
  const float* row = scores + (long long)head * P.max_ctx;
  int32_t* out = k_idx + (long long)head * P.budget_cap;
  const int gtid = rank * kSelThreads + tid;
  constexpr int kAll = CL * kSelThreads;
  if (kv == 0 && gtid == 0) k_cnt[s] = B;
  for (int i = B + gtid; i < P.budget_cap; i += kAll) out[i] = -1;
  // Every exit path waits for the kernel before this one: the kernels of a fused call are ordered as a chain, and
  // "the last kernel has completed" implies "all of them have" only if no link finishes without having waited.
  if (B <= 0) { grid_dependency_wait(); return; }      // uniform over the cluster
  if (B >= T) {                                 // budget covers the cache: identity
    for (int i = gtid; i < T; i += kAll) out[i] = i;
    grid_dependency_wait();
    return;
  }
  const int base = (rank * kSelThreads + wid * 32) * ITEMS + lane;      // position of item i: base + 32 i
  for (int i = tid; i < kHistWords; i += kSelThreads) hist_all[i] = 0;
  if (tid == 0) s_n = 0;
  // Everything above needs nothing from the kernel before this one (launched early, it has run under that kernel's
  // tail); the scores do.
  grid_dependency_wait();
  uint32_t code[ITEMS];
  uint32_t cmin = 0xFFFFFFFFu, cmax = 0u;
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const int pos = base + 32 * i;
    const uint32_t c = float_order_key(__ldcg(row + min(pos, T - 1)));      // clamped load, no branch per item
    code[i] = c;                                                           // (a row past the end repeats the last one)
    cmin = min(cmin, c);
    cmax = max(cmax, c);
  }
  // smallest and largest code of the row
  cmin = __reduce_min_sync(0xFFFFFFFFu, cmin);
  cmax = __reduce_max_sync(0xFFFFFFFFu, cmax);
  if (lane == 0) { warp_val[wid] = cmin; warp_off[wid] = cmax; }
  __syncthreads();
  cmin = __reduce_min_sync(0xFFFFFFFFu, warp_val[lane]);
  cmax = __reduce_max_sync(0xFFFFFFFFu, warp_off[lane]);
  if (CL > 1) {
    if (tid == 0) { cta_cnt[0] = cmin; cta_cnt[1] = cmax; }
    cluster.sync();
#pragma unroll
    for (int r = 0; r < CL; ++r) {
      const uint32_t* pc = cluster.map_shared_rank(cta_cnt, r);
      cmin = min(cmin, pc[0]);
      cmax = max(cmax, pc[1]);
    }
    cluster.sync();                                // cta_cnt is used again below
  }
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t prefix = 0, need = (uint32_t)B;
  // Finds the bin (counted from the top) in which the running count reaches `need`: thread t owns the 4 bins
  // nb-1-4t .. nb-4-4t; leaves the bin in s_bin, what is still needed inside it in s_need, its size in s_cand.
  const auto find_bin = [&](uint32_t* hist, int nb) {
    uint32_t c[4] = {0, 0, 0, 0}, sum = 0;
    if (4 * tid < nb) {
      if (CL > 1) {
#pragma unroll
        for (int r = 0; r < CL; ++r) {              // independent remote loads, all in flight together
          const uint32_t* ph = cluster.map_shared_rank(hist, r);
#pragma unroll
          for (int k = 0; k < 4; ++k) c[k] += ph[nb - 1 - (4 * tid + k)];
        }
      } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) c[k] = hist[nb - 1 - (4 * tid + k)];
      }
      sum = (c[0] + c[1]) + (c[2] + c[3]);
    }
    uint32_t incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_val[wid] = incl;
    __syncthreads();
    if (wid == 0) {
      const uint32_t v = warp_val[lane];
      uint32_t w = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, w, o);
        if (lane >= o) w += u;
      }
      warp_off[lane] = w - v;
    }
    __syncthreads();
    const uint32_t excl = warp_off[wid] + incl - sum;
    if (excl < need && need <= excl + sum) {          // exactly one thread
      uint32_t cum = excl;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (cum + c[k] >= need) {
          s_bin = (uint32_t)(nb - 1 - (4 * tid + k));
          s_need = need - cum;
          s_cand = c[k];
          break;
        }
        cum += c[k];
      }
    }
    __syncthreads();
  };
  bool found = false;
  int up = 0;                                      // the codes are compared as (code - sub) << up: raw unless the digit
  uint32_t sub = 0;                                // passes ran
  if (CL == 1) {
    // ---- Single CTA, first try: ONE histogram over 4096 bins that are linear in the score between the row's
    // smallest and largest (a monotone map, so the bin of the B-th largest holds it).  A row of cosines then
    // leaves a few dozen rows in that bin; they are listed (over the second histogram's words) and every listed
    // row counts the listed rows above and equal to it, which gives the exact code of the B-th largest.
    const float fmin = order_key_to_float(cmin), fmax = order_key_to_float(cmax);
    const float scale = fmax > fmin ? (float)kRegBins / (fmax - fmin) : 0.f;
    const auto bin_of = [&](uint32_t c) { return min(kRegBins - 1, (int)((order_key_to_float(c) - fmin) * scale)); };
    __syncthreads();                               // the histograms are zero, warp_val / warp_off free again
#pragma unroll
    for (int i = 0; i < ITEMS; ++i)
      if (base + 32 * i < T) atomicAdd(&hist_all[bin_of(code[i])], 1u);
    __syncthreads();
    find_bin(hist_all, kRegBins);
    if (s_cand <= (uint32_t)kCandMax) {
      const uint32_t n_cand = s_cand, bin = s_bin;
      need = s_need;
      uint32_t* cand = hist_all + kRegBins;
#pragma unroll
      for (int i = 0; i < ITEMS; ++i)
        if (base + 32 * i < T && (uint32_t)bin_of(code[i]) == bin) cand[atomicAdd(&s_n, 1u)] = code[i];
      __syncthreads();
      if ((uint32_t)tid < n_cand) {
        const uint32_t my = cand[tid];
        uint32_t g = 0, e = 0;
        for (uint32_t j = 0; j < n_cand; ++j) {
          const uint32_t c2 = cand[j];
          g += c2 > my ? 1u : 0u;
          e += c2 == my ? 1u : 0u;
        }
        if (g < need && need <= g + e) { s_bin = my; s_need = need - g; }       // equal rows write the same values
      }
      __syncthreads();
      prefix = s_bin;
      need = s_need;
      found = true;
    } else {
      // many equal scores: start over with the digit passes below
      for (int i = tid; i < kRegBins; i += kSelThreads) hist_all[i] = 0;
      need = (uint32_t)B;
    }
  }
  if (!found) {
    // ---- Digit passes 12 + 12 + 8 bits, most significant first.  The codes of one row of scores share their leading
    // bits: the digits are taken from (code - smallest code) shifted up to the top bit, a map that keeps the order
    // and loses no bit.
    up = min(__clz((int)(cmax - cmin)), 31);
    sub = cmin;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) code[i] = (code[i] - sub) << up;
    __syncthreads();                               // the histograms are zero, warp_val / warp_off free again
    uint32_t mask = 0;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 20 : (pass == 1 ? 8 : 0);
      const int nb = pass == 2 ? 256 : kRegBins;
      uint32_t* hist = hist_all + pass * kRegBins;
#pragma unroll
      for (int i = 0; i < ITEMS; ++i) {
        const bool live = (base + 32 * i < T) && ((code[i] & mask) == prefix);
        if (live) atomicAdd(&hist[(code[i] >> shift) & (uint32_t)(nb - 1)], 1u);
      }
      if (CL > 1) cluster.sync(); else __syncthreads();
      find_bin(hist, nb);
      prefix |= s_bin << shift;
      need = s_need;
      mask |= (uint32_t)(nb - 1) << shift;
    }
  }
  // prefix = code of the B-th largest score (shifted, if the digit passes ran).  Rows at or above it, per warp and
  // before each warp:
  const uint32_t thr = prefix;
  uint32_t w_ge = 0;
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) w_ge += (base + 32 * i < T && code[i] >= thr) ? 1u : 0u;
  w_ge = __reduce_add_sync(0xFFFFFFFFu, w_ge);
  if (lane == 0) warp_val[wid] = w_ge;
  __syncthreads();
  if (wid == 0) {
    const uint32_t v = warp_val[lane];
    uint32_t vi = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, vi, o);
      if (lane >= o) vi += u;
    }
    warp_off[lane] = vi - v;                 // rows at or above the threshold in the warps before this one
    if (lane == 31) cta_cnt[0] = vi;
  }
  if (CL > 1) cluster.sync(); else __syncthreads();
  uint32_t run = warp_off[wid];
  uint32_t total_ge = cta_cnt[0];
  if (CL > 1) {
    uint32_t pg[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) pg[r] = cluster.map_shared_rank(cta_cnt, r)[0];      // independent remote loads
    total_ge = 0;
#pragma unroll
    for (int r = 0; r < CL; ++r) {
      total_ge += pg[r];
      if (r < rank) run += pg[r];
    }
  }
  if (total_ge == (uint32_t)B) {
    // No tie is cut (the usual case): the list is every row at or above the threshold, one ballot per item.
    // A single CTA collects the list in shared memory (over the histograms, which are done with) and copies
    // it out with full-width stores; a cluster writes straight to the list.
    const bool staged = CL == 1 && B <= kHistWords;
    uint32_t* dst = staged ? hist_all : reinterpret_cast<uint32_t*>(out);
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
      const int pos = base + 32 * i;
      const bool sel = pos < T && code[i] >= thr;
      const uint32_t bal = __ballot_sync(0xFFFFFFFFu, sel);
      if (sel) dst[run + (uint32_t)__popc(bal & lt)] = (uint32_t)pos;
      run += (uint32_t)__popc(bal);
    }
    if (staged) {
      __syncthreads();
      for (int i = tid; i < B; i += kSelThreads) out[i] = (int32_t)hist_all[i];
    }
  } else {
    // Rows that tie at the threshold and do not all fit: take the first `need` of them in position order.
    // Rare, so the codes are rebuilt from the scores one item at a time instead of keeping a second unrolled
    // loop over the registers (which made the compiler spill fifty of them).
    uint32_t w_gt = 0, w_eq = 0;
#pragma unroll 1
    for (int i = 0; i < ITEMS; ++i) {
      const int pos = base + 32 * i;
      const uint32_t c = (float_order_key(__ldcg(row + min(pos, T - 1))) - sub) << up;
      w_gt += (pos < T && c > thr) ? 1u : 0u;
      w_eq += (pos < T && c == thr) ? 1u : 0u;
    }
    w_gt = __reduce_add_sync(0xFFFFFFFFu, w_gt);
    w_eq = __reduce_add_sync(0xFFFFFFFFu, w_eq);
    if (CL > 1) cluster.sync(); else __syncthreads();        // warp_val / warp_off / cta_cnt were read above
    if (lane == 0) warp_val[wid] = w_gt | (w_eq << 16);      // at most 1024 each
    __syncthreads();
    if (wid == 0) {
      const uint32_t v = warp_val[lane];
      uint32_t g = v & 0xFFFFu, e = v >> 16, gi = g, ei = e;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t ug = __shfl_up_sync(0xFFFFFFFFu, gi, o), ue = __shfl_up_sync(0xFFFFFFFFu, ei, o);
        if (lane >= o) { gi += ug; ei += ue; }
      }
      warp_off[lane] = gi - g;                 // exclusive counts of rows above the threshold ...
      warp_val[lane] = ei - e;                 // ... and equal to it, over the warps before this one
      if (lane == 31) { cta_cnt[0] = gi; cta_cnt[1] = ei; }
    }
    if (CL > 1) cluster.sync(); else __syncthreads();
    uint32_t run_gt = warp_off[wid], run_eq = warp_val[wid];
    if (CL > 1) {
#pragma unroll
      for (int r = 0; r < CL; ++r) {
        const uint32_t* pc = cluster.map_shared_rank(cta_cnt, r);
        if (r < rank) { run_gt += pc[0]; run_eq += pc[1]; }
      }
    }
#pragma unroll 1
    for (int i = 0; i < ITEMS; ++i) {
      const int pos = base + 32 * i;
      const uint32_t c = (float_order_key(__ldcg(row + min(pos, T - 1))) - sub) << up;
      const bool gt = pos < T && c > thr, eq = pos < T && c == thr;
      const uint32_t b_gt = __ballot_sync(0xFFFFFFFFu, gt), b_eq = __ballot_sync(0xFFFFFFFFu, eq);
      const uint32_t gt_before = run_gt + (uint32_t)__popc(b_gt & lt);
      const uint32_t eq_before = run_eq + (uint32_t)__popc(b_eq & lt);
      if (gt || (eq && eq_before < need)) out[gt_before + min(eq_before, need)] = pos;
      run_gt += (uint32_t)__popc(b_gt);
      run_eq += (uint32_t)__popc(b_eq);
    }
  }
  if (CL > 1) cluster.sync();                   // histograms and counts stay mapped until every peer has read them
}

template <int ITEMS, int CL>
static cudaError_t launch_reg(const DevParams& P, const float* scores, int32_t* k_idx, int32_t* k_cnt, cudaStream_t st,
                              bool chained) {
  return launch_kernel("select_keys_reg", select_keys_reg_kernel<ITEMS, CL>, dim3(P.batch * P.n_kv * CL), dim3(kSelThreads), 0, st, CL, chained,
                       P, scores, k_idx, k_cnt);
}

cudaError_t launch_select_keys(const DevParams& P, const float* scores, int32_t* k_idx, int32_t* k_cnt,
                               cudaStream_t st, bool chained) {
  // One CTA per head while the row fits its registers (32 per thread); clusters only for longer rows: merging
  // the histograms through distributed shared memory costs more than it saves on a short row.
  const int per_thread = (P.max_ctx + kSelThreads - 1) / kSelThreads;    // items per thread with one CTA per head
  cudaError_t e;
  if (per_thread <= 4) e = launch_reg<4, 1>(P, scores, k_idx, k_cnt, st, chained);
  else if (per_thread <= 8) e = launch_reg<8, 1>(P, scores, k_idx, k_cnt, st, chained);
  else if (per_thread <= 16) e = launch_reg<16, 1>(P, scores, k_idx, k_cnt, st, chained);
  else if (per_thread <= 32) e = launch_reg<32, 1>(P, scores, k_idx, k_cnt, st, chained);
  else if (per_thread <= 64) e = launch_reg<32, 2>(P, scores, k_idx, k_cnt, st, chained);
  else if (per_thread <= 128) e = launch_reg<32, 4>(P, scores, k_idx, k_cnt, st, chained);
  else if (per_thread <= 256) e = launch_reg<32, 8>(P, scores, k_idx, k_cnt, st, chained);
  else e = launch_kernel("select_keys", select_keys_kernel, dim3(P.batch * P.n_kv), dim3(kSelThreads), 0, st, 1, chained, P, scores, k_idx, k_cnt);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace quoka
