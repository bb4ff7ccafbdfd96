// Key scoring on the 5th-generation tensor cores (Algorithm 1: S = Qbar K^T on normalised keys,
// S^ = max over the retained queries), bf16.
//
// Orientation: the 128 cached keys of a tile are the M rows of the MMA (A operand, fresh from TMA
// every tile), the retained queries are the N columns (B operand = Qbar of the current KV head,
// resident in shared memory).  The fp32 accumulator D[key][query] lives in tensor memory, so each
// epilogue thread owns one key's row of scores: the maximum over queries is a private register
// reduction and the N x T score matrix never exists outside TMEM.  The key's norm is computed from
// the same shared-memory tile the MMA reads (the swizzle only permutes 16-byte pieces inside a row,
// which a sum of squares does not care about) and applied in fp32: score = max_j(Qbar_j . k)/|k|.
//
// Persistent CTAs (one per SM), each taking a contiguous, equal share of the valid (sequence, KV
// head, key tile) list.  Warp 0 = TMA producer, warp 1 = MMA issuer, warps 2..5 = epilogue.  K tiles
// stream through a multi-stage ring (32 KiB per stage at d = 128); accumulators are double-buffered
// in TMEM when N <= 256 so the epilogue of tile i overlaps the MMAs of tile i+1.
// Arithmetic intensity is N flop per byte of K: HBM-bound below N ~ 200, tensor-bound above.
#include <cstdio>

#include "sm100_ptx.cuh"
#include "tensor_kernels.cuh"

namespace quoka {

using namespace ptx;

constexpr int kTileKeys = 128;
constexpr int kScoreThreads = 320;          // 10 warps: TMA, MMA, two epilogue groups of four
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxStages = 8;

struct ScoreSmemPlan {
  int n_pad;        // N rounded up to 16
  int n_parts;      // 1 or 2 MMA column groups of <= 256
  int box_rows;     // rows per Qbar TMA box
  int q_rows;       // Qbar rows held in shared memory (n_parts * box_rows)
  int stages;
  size_t q_bytes, stage_bytes, total;
};

static ScoreSmemPlan plan_score_smem(int N, int d) {
  ScoreSmemPlan pl{};
  pl.n_pad = (N + 15) / 16 * 16;
  pl.n_parts = pl.n_pad > 256 ? 2 : 1;
  pl.box_rows = pl.n_parts == 1 ? pl.n_pad : 256;
  pl.q_rows = pl.n_parts * pl.box_rows;
  pl.q_bytes = (size_t)pl.q_rows * d * 2;
  pl.stage_bytes = (size_t)kTileKeys * d * 2;
  const size_t budget = 227 * 1024 - 2048;    // alignment slack + barriers
  int st = (int)((budget - pl.q_bytes) / pl.stage_bytes);
  pl.stages = st > kMaxStages ? kMaxStages : st;
  pl.total = 1024 + pl.q_bytes + pl.stages * pl.stage_bytes + 1024;
  return pl;
}

struct ScoreArgs {
  int n, n_pad, n_parts, box_rows, q_rows, stages;
  int defer_q;   // launched early (chained): fetch the key tiles that fit the ring before the first Q-bar
};

// Walks the valid (sequence, KV head, tile) triples in linear order.
struct TileWalk {
  int s, kv, tile, tiles_s;
  long long idx, end;
  __device__ void seek(const DevParams& P, long long lo, long long hi) {
    idx = lo; end = hi; s = 0; kv = 0; tile = 0; tiles_s = 0;
    long long skip = lo;
    for (s = 0; s < P.batch; ++s) {
      tiles_s = (__ldg(P.ctx_len + s) + kTileKeys - 1) / kTileKeys;
      const long long here = (long long)tiles_s * P.n_kv;
      if (skip < here) { kv = (int)(skip / tiles_s); tile = (int)(skip % tiles_s); return; }
      skip -= here;
    }
    idx = end;   // nothing
  }
  __device__ bool valid() const { return idx < end; }
  __device__ void next(const DevParams& P) {
    ++idx;
    if (++tile < tiles_s) return;
    tile = 0;
    if (++kv < P.n_kv) return;
    kv = 0;
    for (++s; s < P.batch; ++s) {
      tiles_s = (__ldg(P.ctx_len + s) + kTileKeys - 1) / kTileKeys;
      if (tiles_s > 0) return;
    }
  }
};

__device__ __forceinline__ long long total_tiles(const DevParams& P) {
  long long t = 0;
  for (int s = 0; s < P.batch; ++s) t += (long long)((__ldg(P.ctx_len + s) + kTileKeys - 1) / kTileKeys) * P.n_kv;
  return t;
}

template <int HALVES>   // head_dim / 64
__global__ void __launch_bounds__(kScoreThreads, 1)
score_keys_tc_kernel(DevParams P, ScoreArgs A, const __grid_constant__ CUtensorMap tm_q,
                     const __grid_constant__ CUtensorMap tm_k, float* __restrict__ scores) {
  constexpr uint32_t kHalfBytes = kTileKeys * 128;             // one 64-column half of a K tile
  constexpr uint32_t kStageBytes = HALVES * kHalfBytes;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* q_smem = smem;                                 // [HALVES][q_rows][128 B]
  const uint32_t q_half_bytes = (uint32_t)A.q_rows * 128;
  unsigned char* k_smem = q_smem + (size_t)HALVES * q_half_bytes;   // [stages][HALVES][128][128 B]
  uint64_t* bars = reinterpret_cast<uint64_t*>(k_smem + (size_t)A.stages * kStageBytes);
  uint64_t* full = bars;                       // [stages]
  uint64_t* empty = bars + kMaxStages;         // [stages]
  uint64_t* acc_full = bars + 2 * kMaxStages;  // [2]
  uint64_t* acc_empty = acc_full + 2;          // [2]
  uint64_t* q_full = acc_empty + 2;
  uint64_t* q_empty = q_full + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(q_empty + 1);
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtx wc{&abort_flag, P.status};

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < A.stages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 5); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 4); }
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
  }
  if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Only now may the kernels after this one become resident (the selection kernel, and through it the attention
  // kernel, which also allocates tensor memory): every CTA of this grid holds its tensor memory by then, so a
  // later grid can never take the columns a CTA of this one still has to wait for.
  grid_launch_dependents();

  const long long total = total_tiles(P);
  const long long lo = total * blockIdx.x / gridDim.x, hi = total * (blockIdx.x + 1) / gridDim.x;
  const int slots = 2 / A.n_parts;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      TileWalk w; w.seek(P, lo, hi);
      int stage = 0; uint32_t phase = 0, qe_phase = 0; int head_cur = -1;
      // The key tiles do not depend on the kernel before this one, Q-bar does.  The first Q-bar of the CTA is
      // therefore fetched only after most of the ring has been filled with key tiles, and after the wait for the
      // grid that wrote it (which returns at once unless this kernel was launched early).
      bool waited = false;
      int q_deferred = -1, n_issued = 0;
      const auto load_q = [&](int head) {
        if (!waited) { grid_dependency_wait(); waited = true; }
        mbar_arrive_expect_tx(q_full, (uint32_t)(HALVES * A.n_parts * A.box_rows * 128));
        for (int h = 0; h < HALVES; ++h)
          for (int p = 0; p < A.n_parts; ++p)
            tma_load_3d(q_smem + (size_t)h * q_half_bytes + (size_t)p * A.box_rows * 128, &tm_q, q_full, h * 64,
                        p * A.box_rows, head);
      };
      for (; w.valid(); w.next(P)) {
        const int head = w.s * P.n_kv + w.kv;
        if (head != head_cur) {
          if (q_deferred >= 0) { load_q(q_deferred); q_deferred = -1; }
          if (head_cur >= 0) { if (!mbar_wait(q_empty, qe_phase, wc)) break; qe_phase ^= 1; }
          if (n_issued == 0 && A.defer_q) q_deferred = head; else load_q(head);
          head_cur = head;
        }
        if (!mbar_wait(&empty[stage], phase ^ 1, wc)) break;
        mbar_arrive_expect_tx(&full[stage], kStageBytes);
        unsigned char* dst = k_smem + (size_t)stage * kStageBytes;
        const int t0 = w.tile * kTileKeys;
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {           // two 64-row boxes per tile (one page each when paged)
          int c1, c3;
          if (P.page_size == 0) { c1 = t0 + sub * 64; c3 = w.s; }
          else {
            const int pi = (t0 >> 6) + sub;
            int page = pi < P.max_pages ? __ldg(P.block_table + (long long)w.s * P.max_pages + pi) : 0;
            c1 = 0; c3 = page < 0 ? 0 : page;
          }
#pragma unroll
          for (int h = 0; h < HALVES; ++h)
            tma_load_4d(dst + h * kHalfBytes + sub * 64 * 128, &tm_k, &full[stage], h * 64, c1, w.kv, c3);
        }
        if (++stage == A.stages) { stage = 0; phase ^= 1; }
        if (++n_issued >= A.stages - 1 && q_deferred >= 0) { load_q(q_deferred); q_deferred = -1; }
      }
      if (q_deferred >= 0) load_q(q_deferred);
      // a CTA without tiles still waits: the chain of a fused call is only transitive if every link has waited
      if (!waited) grid_dependency_wait();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      TileWalk w; w.seek(P, lo, hi);
      int stage = 0; uint32_t phase = 0, q_phase = 0; int head_cur = -1;
      int slot = 0; uint32_t acc_phase = 0;
      const uint32_t q_base = smem_u32(q_smem), k_base = smem_u32(k_smem);
      for (; w.valid(); w.next(P)) {
        const int head = w.s * P.n_kv + w.kv;
        if (head != head_cur) {
          if (head_cur >= 0) mma_commit(q_empty);     // arrives when every MMA on the old Qbar is done
          if (!mbar_wait(q_full, q_phase, wc)) break;
          q_phase ^= 1;
          head_cur = head;
        }
        if (!mbar_wait(&full[stage], phase, wc)) break;
        if (!mbar_wait(&acc_empty[slot], acc_phase ^ 1, wc)) break;
        tc_fence_after();
        for (int p = 0; p < A.n_parts; ++p) {
          const int n_mma = (p == A.n_parts - 1) ? (A.n_pad - p * 256) : 256;
          const uint32_t idesc = idesc_bf16_f32(128, n_mma, false, false);
          const uint32_t d_tmem = tmem_base + (uint32_t)((A.n_parts == 1 ? slot : p) * 256);
#pragma unroll
          for (int h = 0; h < HALVES; ++h) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              const uint64_t a_desc = smem_desc_sw128(k_base + stage * kStageBytes + h * kHalfBytes + kk * 32, 16, 1024);
              const uint64_t b_desc = smem_desc_sw128(q_base + h * q_half_bytes + p * A.box_rows * 128 + kk * 32, 16, 1024);
              mma_ss(d_tmem, a_desc, b_desc, idesc, (h | kk) ? 1u : 0u);
            }
          }
        }
        mma_commit(&empty[stage]);
        mma_commit(&acc_full[slot]);
        if (++stage == A.stages) { stage = 0; phase ^= 1; }
        if (++slot == slots) { slot = 0; acc_phase ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue: one key per thread.
    // Two groups of four warps take alternate tiles (group g = accumulator slot g), because one tile's epilogue
    // (key norm from shared memory, 128 accumulator columns from tensor memory) takes longer than the tile's
    // share of HBM time.  With a single accumulator slot (N > 256) only group 0 works.
    const int group = (warp - 2) >> 2;
    const int quarter = warp & 3;                       // TMEM lane quarter this warp may access
    const int row = quarter * 32 + lane;                // key row within the tile
    TileWalk w; w.seek(P, lo, hi);
    int stage = 0; uint32_t phase = 0; int slot = 0; uint32_t acc_phase = 0;
    int n_done = 0;                                     // tiles walked so far
    for (; w.valid(); w.next(P), ++n_done) {
      const bool mine = slots == 2 ? ((n_done & 1) == group) : (group == 0);
      if (!mine) {                                      // the other group's tile: only keep the ring position
        if (++stage == A.stages) { stage = 0; phase ^= 1; }
        continue;
      }
      slot = slots == 2 ? group : 0;
      acc_phase = slots == 2 ? (uint32_t)((n_done >> 1) & 1) : (uint32_t)(n_done & 1);
      if (!mbar_wait(&full[stage], phase, wc)) break;
      // 1/|k|: read from the caller's cache of inverse norms when there is one (the load is in flight under the
      // accumulator wait), else |k|^2 from the tile in shared memory (rotated 16-byte reads: conflict-free)
      const int T_s = __ldg(P.ctx_len + w.s);
      const int t = w.tile * kTileKeys + row;
      const bool own_norm = P.k_inv_norm == nullptr && !P.score_dot;
      float inv_cached = 1.f;
      if (P.k_inv_norm != nullptr && !P.score_dot)
        inv_cached = __ldg(P.k_inv_norm + kv_norm_index(P, w.s, w.kv, min(t, T_s - 1)));
      float nacc[4] = {0.f, 0.f, 0.f, 0.f};                 // independent partial sums: no 256-deep FMA chain
      const unsigned char* krow = k_smem + (size_t)stage * kStageBytes + row * 128;
      if (own_norm) {
#pragma unroll
      for (int h = 0; h < HALVES; ++h) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint4 v = *reinterpret_cast<const uint4*>(krow + h * kHalfBytes + (((c + row) & 7) << 4));
          const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float a = __uint_as_float(wds[i] << 16), b = __uint_as_float(wds[i] & 0xFFFF0000u);
            nacc[i] = fmaf(a, a, nacc[i]);
            nacc[i] = fmaf(b, b, nacc[i]);
          }
        }
      }
      }
      const float nn = (nacc[0] + nacc[1]) + (nacc[2] + nacc[3]);
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[stage]);
      if (!mbar_wait(&acc_full[slot], acc_phase, wc)) break;
      tc_fence_after();
      float bacc[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      float sacc[4] = {0.f, 0.f, 0.f, 0.f};               // mean-over-queries variant: columns >= N are exact zeros
      const bool agg_mean = P.agg_mean != 0;
      for (int p = 0; p < A.n_parts; ++p) {
        const int n_mma = (p == A.n_parts - 1) ? (A.n_pad - p * 256) : 256;
        const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((A.n_parts == 1 ? slot : p) * 256);
        int c0 = 0;
        for (; c0 + 64 <= n_mma; c0 += 64) {              // two loads in flight per wait
          uint32_t r0[32], r1[32];
          tmem_ld32(t_addr + c0, r0);
          tmem_ld32(t_addr + c0 + 32, r1);
          tmem_wait_ld();
          if (agg_mean) {
#pragma unroll
            for (int j = 0; j < 32; ++j) sacc[j & 3] += __uint_as_float(r0[j]) + __uint_as_float(r1[j]);
          }
          const int lim = A.n - (p * 256 + c0);
          if (lim >= 64) {
#pragma unroll
            for (int j = 0; j < 32; ++j) bacc[j & 3] = max3(bacc[j & 3], __uint_as_float(r0[j]), __uint_as_float(r1[j]));
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (j < lim) bacc[j & 3] = fmaxf(bacc[j & 3], __uint_as_float(r0[j]));
              if (j + 32 < lim) bacc[j & 3] = fmaxf(bacc[j & 3], __uint_as_float(r1[j]));
            }
          }
        }
        for (; c0 + 32 <= n_mma; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(t_addr + c0, r);
          tmem_wait_ld();
          if (agg_mean) {
#pragma unroll
            for (int j = 0; j < 32; ++j) sacc[j & 3] += __uint_as_float(r[j]);
          }
          const int lim = A.n - (p * 256 + c0);
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (j < lim) bacc[j & 3] = fmaxf(bacc[j & 3], __uint_as_float(r[j]));
        }
        if (c0 < n_mma) {
          uint32_t r[16];
          tmem_ld16(t_addr + c0, r);
          tmem_wait_ld();
          if (agg_mean) {
#pragma unroll
            for (int j = 0; j < 16; ++j) sacc[j & 3] += __uint_as_float(r[j]);
          }
          const int lim = A.n - (p * 256 + c0);
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (j < lim) bacc[j & 3] = fmaxf(bacc[j & 3], __uint_as_float(r[j]));
        }
      }
      const float best = agg_mean ? ((sacc[0] + sacc[1]) + (sacc[2] + sacc[3])) / (float)A.n
                                  : fmaxf(fmaxf(bacc[0], bacc[1]), fmaxf(bacc[2], bacc[3]));
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[slot]);
      if (t < T_s)
        scores[((long long)w.s * P.n_kv + w.kv) * P.max_ctx + t] =
            own_norm ? best / fmaxf(sqrtf(nn), kNormEps) : best * inv_cached;
      if (++stage == A.stages) { stage = 0; phase ^= 1; }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// ---------------------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
    if (qres != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

bool encode_tensor_map_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                            const uint64_t* strides_bytes, const uint32_t* box) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[5], gstr[4];
  cuuint32_t bdim[5], estr[5];
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bdim[i] = box[i]; estr[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr, bdim,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool encode_kv_tensor_map(CUtensorMap* out, const quoka_params* p, const void* cache, uint32_t box_rows) {
  const uint64_t dims[4] = {(uint64_t)p->head_dim, (uint64_t)(p->page_size ? kPage : p->kv_rows),
                            (uint64_t)p->n_kv_heads, (uint64_t)(p->page_size ? p->kv_rows : p->batch)};
  const uint64_t strides[3] = {(uint64_t)p->kv_stride_t * 2, (uint64_t)p->kv_stride_h * 2, (uint64_t)p->kv_stride_b * 2};
  const uint32_t box[4] = {64, box_rows, 1, 1};
  return encode_tensor_map_bf16(out, cache, 4, dims, strides, box);
}

bool score_keys_tc_supported(const quoka_params* p) {
  if (p->dtype != QUOKA_BF16) return false;
  const int N = p->n_retain < p->chunk_len ? p->n_retain : p->chunk_len;
  if (N > 512) return false;
  if (p->kv_stride_t != p->head_dim && (p->kv_stride_t * 2) % 16 != 0) return false;
  return true;
}

quoka_status launch_score_keys_tc(const quoka_params* p, const DevParams& P, const void* qbar, const void* k,
                                  float* scores, cudaStream_t st, bool chained) {
  const int N = P.n_sel;
  const ScoreSmemPlan pl = plan_score_smem(N, P.d);
  if (pl.stages < 2) return QUOKA_ERR_UNSUPPORTED;
  CUtensorMap tm_q, tm_k;
  {
    const uint64_t dims[3] = {(uint64_t)P.d, (uint64_t)N, (uint64_t)P.batch * P.n_kv};
    const uint64_t strides[2] = {(uint64_t)P.d * 2, (uint64_t)N * P.d * 2};
    const uint32_t box[3] = {64, (uint32_t)pl.box_rows, 1};
    if (!encode_tensor_map_bf16(&tm_q, qbar, 3, dims, strides, box)) return QUOKA_ERR_CUDA;
  }
  if (!encode_kv_tensor_map(&tm_k, p, k, 64)) return QUOKA_ERR_CUDA;
  ScoreArgs A{N, pl.n_pad, pl.n_parts, pl.box_rows, pl.q_rows, pl.stages, chained ? 1 : 0};
  const long long max_tiles = (long long)P.batch * P.n_kv * ((P.max_ctx + kTileKeys - 1) / kTileKeys);
  int grid = device_sm_count();
  if (grid <= 0) return QUOKA_ERR_CUDA;
  if (max_tiles < grid) grid = (int)max_tiles;
  if (grid <= 0) return QUOKA_OK;
  cudaError_t e;
  if (P.d == 128) {
    e = cudaFuncSetAttribute(score_keys_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.total);
    if (e != cudaSuccess) return QUOKA_ERR_CUDA;
    e = launch_kernel("score_keys_tc", score_keys_tc_kernel<2>, dim3(grid), dim3(kScoreThreads), pl.total, st, 1, chained, P, A, tm_q, tm_k, scores);
  } else {
    e = cudaFuncSetAttribute(score_keys_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.total);
    if (e != cudaSuccess) return QUOKA_ERR_CUDA;
    e = launch_kernel("score_keys_tc", score_keys_tc_kernel<1>, dim3(grid), dim3(kScoreThreads), pl.total, st, 1, chained, P, A, tm_q, tm_k, scores);
  }
  count_launch();
  return (e == cudaSuccess && cudaGetLastError() == cudaSuccess) ? QUOKA_OK : QUOKA_ERR_CUDA;
}

}  // namespace quoka
