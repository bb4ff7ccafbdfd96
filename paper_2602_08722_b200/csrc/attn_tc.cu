// Flash-style attention on the 5th-generation tensor cores over
//   [selected cached rows | the chunk's own causal rows]      (Algorithm 2's attention line, Eq. 2)
// or, without an index list, over every cached row (Eq. 2, dense chunk attention).  bf16 in, fp32
// softmax and accumulation, P rounded to bf16 for the PV product.
//
// One CTA owns 256 consecutive chunk rows of one query head as two 128-row Q tiles (A, B) and walks
// the key tiles (128 keys) once for both.  Roles:
//   warps 0-3 / 4-7  softmax of Q tile A / B: one thread per query row, S read from tensor memory,
//                    running max / sum in registers, P written back to tensor memory over S,
//                    lazy rescale of the O accumulator (only when the max grew by more than 2^32),
//                    final normalisation and the global store.
//   warps 8-10       loaders: every K / V row of a tile is fetched with 16-byte cp.async straight
//                    into the 128-byte-swizzled layout the MMA descriptors expect.  The row address
//                    comes from the selected-index list (the gather), the chunk offset, or the page
//                    table, so no compacted copy of K or V is ever made; rows past the end are
//                    zero-filled.  A slot's "full" barrier is armed by the copies themselves.
//   warp 11          MMA issuer (one thread): S = Q K^T (both operands in shared memory) and
//                    O += P V (P from tensor memory, V in shared memory, MN-major).
// Tensor memory (512 columns): S_A | S_B | O_A | O_B, P aliasing the first 64 columns of its S.
// K and V tiles share one ring of shared-memory slots in the order K0 V0 K1 V1 ...
// 384 threads and no register re-balancing between roles: every thread may use 168 registers
// (with 512 threads and setmaxnreg the compiler still scheduled the softmax for 128 registers,
// which halved its speed).
#include "attn_tiles.cuh"

namespace quoka {

template <int HALVES, bool SPARSE, bool SPLIT>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_tc_kernel(DevParams P, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __nv_bfloat16* __restrict__ kc,
               const __nv_bfloat16* __restrict__ vc, const int32_t* __restrict__ k_idx,
               const int32_t* __restrict__ k_cnt, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
  constexpr int D = HALVES * 64;
  constexpr uint32_t kHalfBytes = 128 * 128;                 // 128 rows x 128 B
  constexpr uint32_t kTileBytes = HALVES * kHalfBytes;       // one Q / K / V tile
  constexpr uint32_t S_COL[2] = {0, 128}, O_COL[2] = {256, 384};
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* q_smem = smem;                               // [2][HALVES][128][128 B]
  unsigned char* kv_smem = smem + 2 * kTileBytes;             // [kSlots][HALVES][128][128 B]
  uint64_t* bars = reinterpret_cast<uint64_t*>(kv_smem + (size_t)kSlots * kTileBytes);
  uint64_t* kv_full = bars;                 // [kSlots]  the loader threads' cp.async arrivals
  uint64_t* kv_empty = bars + kSlots;       // [kSlots]  MMA commit
  uint64_t* s_full = bars + 2 * kSlots;     // [2]       MMA commit
  uint64_t* p_full = s_full + 2;            // [2][2]    4 softmax warps arrive, per Q tile and half of the key tile
  uint64_t* o_full = p_full + 4;            // [2]       MMA commit after the last PV
  uint64_t* q_full = o_full + 2;            // TMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(q_full + 1);
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtx wc{&abort_flag, P.status};
  // grid = (heads, row blocks, batch): heads vary fastest so the CTAs resident together share a KV head's
  // rows in L2, and the row blocks run heaviest (most causal tiles) first, lightest last
  const int s = blockIdx.z, h = blockIdx.x, kv = h / P.group;
  // (SPLIT: grid.y = row blocks times the parts a row block's key tiles are cut into)
  const int n_parts = SPLIT ? P.attn_parts : 1;
  const int n_rb = gridDim.y / n_parts;
  const int rb = n_rb - 1 - blockIdx.y / n_parts;
  const int r0 = rb * 2 * kQTile;
  AttnGeom g = make_geom<SPARSE>(P, s, r0);
  // SPLIT: this CTA walks the tiles [t_lo, t_hi) of the row block's sequence only and leaves, per row, a partial
  // result; the part that finishes last adds the parts up.  The list length has to be known before the range is, so
  // nothing of the walk starts before the selection has ended.
  int t_lo = 0;
  if (SPLIT) {
    if (SPARSE) resolve(g, k_cnt, s);
    const int part = blockIdx.y % n_parts;
    t_lo = (int)(((long long)part * g.n_known) / n_parts);
    g.n_known = (int)(((long long)(part + 1) * g.n_known) / n_parts);
  }

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < kSlots; ++i) { mbar_init(&kv_full[i], kLoaderWarps * 32); mbar_init(&kv_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&o_full[i], 1); }
    for (int i = 0; i < 4; ++i) mbar_init(&p_full[i], 4);
    mbar_init(q_full, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
  }
  if (warp == kMmaWarp) tmem_alloc(tmem_slot, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp < 8) {
    // ================================================================== softmax + epilogue
    const int x = warp >> 2;                                  // Q tile A (0) or B (1)
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    const int row = r0 + x * kQTile + row_in_tile;            // chunk row
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t s_addr = lane_addr + S_COL[x], o_addr = lane_addr + O_COL[x];
    const float scale_log2 = P.scale * 1.4426950408889634f;
    float m_run = -INFINITY, l_run = 0.f;
    uint32_t phase = 0;
    bool ok = true;
    const int skip_x = max(x ? 0 : g.skip_a, t_lo);         // first tile this Q tile takes part in
    const bool active_x = (x ? g.active_b : true) && (!SPLIT || skip_x < g.n_known);
    for (int t = skip_x; active_x; ++t) {
      if (t == g.n_known) {                                   // end of what is known: the list length, or the end
        if (g.resolved) break;
        resolve(g, k_cnt, s);
        if (t == g.n_known) break;
      }
      if (!mbar_wait(&s_full[x], phase, wc)) { ok = false; break; }
      phase ^= 1;
      tc_fence_after();
      const int lim = visible_cols(tile_rows<SPARSE>(g, t), row);
      const bool masked = !__all_sync(0xFFFFFFFFu, lim >= kKeyTile);
      attn_softmax_tile<D>(s_addr, o_addr, lim, masked, scale_log2, t == skip_x, lane, m_run, l_run,
                           [&](int half) { mbar_arrive(&p_full[2 * x + half]); });
    }
    // ---- epilogue: O / l -> bf16 -> global
    if constexpr (!SPLIT) {
      if (ok && active_x && mbar_wait(&o_full[x], 0, wc)) {
        tc_fence_after();
        attn_store_row<D>(P, o_addr, m_run, l_run, s, h, row, out, lse);
      }
    } else {
      const bool have = ok && active_x && mbar_wait(&o_full[x], 0, wc);
      if (have) tc_fence_after();
      attn_split_epilogue<D>(P, (s * P.n_q + h) * n_rb + rb, blockIdx.y % n_parts, n_parts, x, quarter, lane, row_in_tile, row, have,
                             o_addr, m_run, l_run, s, h, out, lse);
    }
  } else if (warp < 8 + kLoaderWarps) {
    // ================================================================== K / V row loaders (gather)
    // One warp instruction copies 32 / PIECES whole rows (16 lanes x 16 bytes cover a 256-byte row); the
    // row groups of a tile are dealt round-robin to the loader warps.
    const int lw = warp - 8;
    constexpr int PIECES = D / 8;                             // 16-byte pieces per row (16 or 8)
    constexpr int ROWS_PER_INSTR = 32 / PIECES;               // 2 or 4
    constexpr int GROUPS = kKeyTile / ROWS_PER_INSTR;         // 64 or 32 row groups per tile
    constexpr int RPT = (GROUPS + kLoaderWarps - 1) / kLoaderWarps;   // row groups per warp (last one may be idle)
    const int c16 = lane % PIECES;                            // this thread's piece of the row
    const int rsub = lane / PIECES;
    const int32_t* idx = SPARSE ? k_idx + ((long long)s * P.n_kv + kv) * P.budget_cap : nullptr;
    uint32_t phase = 0;
    int slot = 0;
    const uint32_t kv_base = smem_u32(kv_smem);
    // Row addressing in 16-byte units, 32 bits wide (the host refuses caches beyond 2^32 units; strides are
    // multiples of 8 elements): sequence/head base plus this thread's piece, row stride, page stride.
    const uint32_t st16 = (uint32_t)(P.kv_st >> 3), sb16 = (uint32_t)(P.kv_sb >> 3);
    const uint32_t base16 = (uint32_t)(((P.page_size == 0 ? (long long)s * P.kv_sb : 0ll) + (long long)kv * P.kv_sh) >> 3) +
                            (uint32_t)c16;
    const int32_t* table = P.block_table + (long long)s * P.max_pages;
    // Row numbers of this warp's rows of a tile of the selected list (-1 past the end), `base` = the tile's first
    // list entry, `count` = entries left from there.  The warp's RPT * ROWS_PER_INSTR rows are numbered
    // p = i * ROWS_PER_INSTR + rsub; lane l keeps rows p = l and p = 32 + l (two registers instead of one per row
    // group), and the thread that copies row p fetches its number with a shuffle.  Except for the first list tile
    // they are fetched when the previous tile's copies have been issued and only looked at when this tile's copies
    // are issued (the loader normally waits for a free slot in between), so the loader does not wait on them.
    // The per-row code below is kept free of branches (clamped loads, selects): a branch per row costs a single
    // warp far more than the arithmetic it skips.
    constexpr int LIST_REGS = (RPT * ROWS_PER_INSTR + 31) / 32;
    static_assert(32 % ROWS_PER_INSTR == 0, "a row group's entries must sit in one register");
    int t_list[LIST_REGS];
    auto list_rows = [&](int base, int count) {
      const int last = min(count, kKeyTile) - 1;                   // last valid row of the tile
      if (last >= 0) {
#pragma unroll
        for (int k = 0; k < LIST_REGS; ++k) {
          const int pp = 32 * k + lane;
          const int rr = (lw + (pp / ROWS_PER_INSTR) * kLoaderWarps) * ROWS_PER_INSTR + pp % ROWS_PER_INSTR;
          const int v = __ldcg(idx + base + min(rr, last));        // written by the kernel before: L2, not the read-only path
          t_list[k] = rr <= last ? v : -1;
        }
      }
    };
#pragma unroll
    for (int k = 0; k < LIST_REGS; ++k) t_list[k] = -1;
    for (int tile = t_lo;; ++tile) {
      if (tile == g.n_known) {                                // end of what is known: the list length, or the end
        if (g.resolved) break;
        resolve(g, k_cnt, s);
        if (tile == g.n_known) break;
      }
      const TileRows tr = tile_rows<SPARSE>(g, tile);
      bool stop = false;
#pragma unroll 1
      for (int kvi = 0; kvi < 2; ++kvi) {                     // the tile's K rows, then its V rows
        if (!mbar_wait(&kv_empty[slot], phase ^ 1, wc)) { stop = true; break; }
        // A whole tile of consecutive rows (page-aligned in a paged cache) is fetched by the copy engine as 64-row
        // boxes: one thread issues them, the others only keep the barrier's arrival count.  Ragged tiles (rows past
        // the end must read as zeros, not as whatever the cache holds there) and listed rows take the copies below.
        if (!tr.from_list && tr.count >= kKeyTile && (P.page_size == 0 || (tr.first & (kPage - 1)) == 0)) {
          if (lw == 0 && lane == 0) {
            fence_proxy_async_smem();             // earlier contents of the slot were written through the generic proxy
            mbar_arrive_expect_tx(&kv_full[slot], kTileBytes);
            unsigned char* dst = kv_smem + (size_t)slot * kTileBytes;
            const CUtensorMap* tm = kvi ? &tm_v : &tm_k;
#pragma unroll
            for (int sub = 0; sub < 2; ++sub) {
              int c1 = tr.first + sub * 64, c3 = s;
              if (P.page_size != 0) { c1 = 0; c3 = __ldg(table + (tr.first >> 6) + sub); }
#pragma unroll
              for (int hh = 0; hh < HALVES; ++hh)
                tma_load_4d(dst + hh * kHalfBytes + sub * 64 * 128, tm, &kv_full[slot], hh * 64, c1, kv, c3);
            }
          } else {
            mbar_arrive(&kv_full[slot]);
          }
          if (++slot == kSlots) { slot = 0; phase ^= 1; }
          continue;
        }
        if (kvi == 0 && tr.from_list && tile == max(g.n_chunk, t_lo)) list_rows(tr.first, tr.count);   // first list tile
        const uint4* src_base = reinterpret_cast<const uint4*>(kvi ? vc : kc);
        const uint32_t dst_tile = kv_base + slot * kTileBytes + (c16 >> 3) * kHalfBytes;
        int t[RPT];                                               // row number, or -1
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
          const int rr = (lw + i * kLoaderWarps) * ROWS_PER_INSTR + rsub;
          const int listed = __shfl_sync(0xFFFFFFFFu, t_list[(i * ROWS_PER_INSTR) / 32], (i * ROWS_PER_INSTR + rsub) & 31);
          t[i] = tr.from_list ? listed : (rr < tr.count ? tr.first + rr : -1);
        }
#ifdef QUOKA_DEBUG
        // debug build: a listed row outside [0, T) is recorded and treated as absent (zero-filled) instead of read
#pragma unroll
        for (int i = 0; i < RPT; ++i)
          if (tr.from_list && (t[i] < -1 || t[i] >= g.T)) { atomicExch(P.status, (int32_t)QUOKA_ERR_BAD_INDEX); t[i] = -1; }
#endif
        uint32_t off[RPT];
        if (P.page_size == 0) {
#pragma unroll
          for (int i = 0; i < RPT; ++i) off[i] = base16 + (uint32_t)max(t[i], 0) * st16;
        } else {
#pragma unroll
          for (int i = 0; i < RPT; ++i) {
            const int tc = max(t[i], 0);
            int page = __ldg(table + (tc >> 6));
#ifdef QUOKA_DEBUG
            // debug build: a page id outside the pool is recorded and the row treated as absent
            if (t[i] >= 0 && (page < 0 || (long long)page >= P.kv_rows)) {
              atomicExch(P.status, (int32_t)QUOKA_ERR_BAD_INDEX);
              t[i] = -1;
            }
            if (page < 0 || (long long)page >= P.kv_rows) page = 0;
#endif
            off[i] = (uint32_t)page * sb16 + base16 + (uint32_t)(tc & (kPage - 1)) * st16;
          }
        }
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
          const int rr = (lw + i * kLoaderWarps) * ROWS_PER_INSTR + rsub;
          if (rr < kKeyTile)                                      // false only for the last group of some warps
            cp_async_16(dst_tile + rr * 128 + (((c16 & 7) ^ (rr & 7)) << 4), src_base + off[i], t[i] >= 0);
        }
        // this thread's share of the slot is signalled by the copy engine itself when the bytes have landed:
        // no wait in the loader, every slot of the ring can be in flight
        cp_async_mbar_arrive_noinc(&kv_full[slot]);
        if (kvi == 1 && tr.from_list) list_rows(tr.first + kKeyTile, tr.count - kKeyTile);   // next list tile
        if (++slot == kSlots) { slot = 0; phase ^= 1; }
      }
      if (stop) break;
    }
    cp_async_wait_all();                                      // nothing of this thread is in flight at exit
  } else if (lane == 0) {
    // ================================================================== MMA issuer (one thread)
    mbar_arrive_expect_tx(q_full, 2 * kTileBytes);
    for (int x = 0; x < 2; ++x)
      for (int hh = 0; hh < HALVES; ++hh)
        tma_load_4d(q_smem + x * kTileBytes + hh * kHalfBytes, &tm_q, q_full, hh * 64, r0 + x * kQTile, h, s);
    const uint32_t idesc_qk = idesc_bf16_f32(128, kKeyTile, false, false);
    const uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true);
    const uint32_t q_base = smem_u32(q_smem), kv_base = smem_u32(kv_smem);
    int slot = 0;
    uint32_t kv_phase = 0;
    uint32_t p_phase[2] = {0, 0};
    int k_slot = -1, v_slot = -1;
    bool ok = mbar_wait(q_full, 0, wc);
    auto acquire = [&]() -> int {           // next ring item (K or V) becomes readable
      if (!mbar_wait(&kv_full[slot], kv_phase, wc)) { ok = false; return 0; }
      fence_proxy_async_smem();             // cp.async wrote through the generic proxy, the MMA reads through the async one
      tc_fence_after();
      const int got = slot;
      if (++slot == kSlots) { slot = 0; kv_phase ^= 1; }
      return got;
    };
    // Operand descriptors are built once; a tile, slot or k-step offset is an addition to the 16-byte-unit
    // address field (shared memory addresses stay far below the field's 14 bits), which keeps the issuing
    // thread's instruction count per MMA small.
    const uint64_t desc_q = smem_desc_sw128(q_base, 16, 1024);
    const uint64_t desc_k = smem_desc_sw128(kv_base, 16, 1024);            // K-major rows (K tiles)
    const uint64_t desc_v = smem_desc_sw128(kv_base, kHalfBytes, 1024);    // MN-major rows (V tiles)
    auto issue_qk = [&](int x, int ks) {
      const uint64_t da = desc_q + (uint64_t)(x * (kTileBytes >> 4));
      const uint64_t db = desc_k + (uint64_t)((uint32_t)ks * (kTileBytes >> 4));
#pragma unroll
      for (int hh = 0; hh < HALVES; ++hh)
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const uint64_t off = (uint64_t)((hh * kHalfBytes + kk * 32) >> 4);
          mma_ss(tmem_base + S_COL[x], da + off, db + off, idesc_qk, (hh | kk) ? 1u : 0u);
        }
      mma_commit(&s_full[x]);
    };
    auto issue_pv = [&](int x, int vs, bool first) {
      const uint64_t dv = desc_v + (uint64_t)((uint32_t)vs * (kTileBytes >> 4));
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        if (!mbar_wait(&p_full[2 * x + half], p_phase[x], wc)) { ok = false; return; }
        tc_fence_after();
#pragma unroll
        for (int kk = half * 4; kk < half * 4 + 4; ++kk) {   // 16 keys per MMA: 8 packed columns of P, 16 rows of V
          mma_ts(tmem_base + O_COL[x], tmem_base + S_COL[x] + kk * 8, dv + (uint64_t)(kk * (2048 >> 4)), idesc_pv,
                 (!first || kk) ? 1u : 0u);
        }
      }
      p_phase[x] ^= 1;
    };
    // Tile t: O += P_t V_t for each Q tile taking part (as the two halves of P arrive), then S = Q K_{t+1}^T.
    // K_{t+1} and V_t are both acquired before the P waits, so those never sit on the P -> PV -> QK chain.
    // The sparse sequence's length is learnt (resolve) just before the look-ahead past the chunk's own tiles.
    const auto part = [&](int x, int t) { return x ? g.active_b : t >= g.skip_a; };
    if (ok && t_lo < g.n_known) {
      k_slot = acquire();
      if (ok) {
        if (part(0, t_lo)) issue_qk(0, k_slot);
        if (part(1, t_lo)) issue_qk(1, k_slot);
        mma_commit(&kv_empty[k_slot]);
      }
      for (int t = t_lo; ok; ++t) {
        if (t + 1 == g.n_known && !g.resolved) resolve(g, k_cnt, s);
        const bool more = t + 1 < g.n_known;
        v_slot = acquire();
        if (ok && more) k_slot = acquire();
        if (!ok) break;
        if (part(0, t)) {
          issue_pv(0, v_slot, t == max(g.skip_a, t_lo));
          if (!ok) break;
          if (!more) mma_commit(&o_full[0]);
        }
        if (more && part(0, t + 1)) issue_qk(0, k_slot);
        if (part(1, t)) {
          issue_pv(1, v_slot, t == t_lo);
          if (!ok) break;
          if (!more) mma_commit(&o_full[1]);
        }
        mma_commit(&kv_empty[v_slot]);
        if (!more) break;
        if (part(1, t + 1)) issue_qk(1, k_slot);
        mma_commit(&kv_empty[k_slot]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, 512);
}

// ---------------------------------------------------------------------------------------------- host
// Split attention.  A grid of fewer CTAs than SMs (short chunks, few heads) leaves part of the GPU idle while
// every CTA walks its whole key sequence; cutting each row block's tiles into parts, one CTA each, fills it.
// The number of parts minimises  waves(parts) * (tiles / parts + 6):  a part costs about six tiles' time of
// start-up, partial results and merge (the model fits the measured times of 1 to 5 parts on grids of 32 to 288 CTAs
// within 3 %), parts keep at least six tiles, and a split has to promise 3 % to be taken.  Grids of a wave or more
// stay whole: their sparse jobs are too short to gain, and the partial results of long dense ones would take
// hundreds of megabytes.
static long long attn_jobs(const quoka_params* p) {
  return (long long)p->n_q_heads * ((p->chunk_len + 2 * kQTile - 1) / (2 * kQTile)) * p->batch;
}
int attn_split_parts(const quoka_params* p, int tiles) {
  if (p->dtype != QUOKA_BF16) return 1;
  const long long jobs = attn_jobs(p), sms = device_sm_count();
  if (sms <= 0 || jobs >= sms) return 1;
  const double t = tiles + (p->chunk_len + 2 * kQTile - 1) / (2 * kQTile);   // plus the chunk's own tiles, on average
  int best = 1;
  double best_cost = t;
  for (int parts = 2; parts <= 8 && parts <= tiles / 6; ++parts) {
    const long long waves = (jobs * parts + sms - 1) / sms;
    const double cost = (double)waves * (t / parts + 6.0);
    if (cost < 0.97 * best_cost) { best = parts; best_cost = cost; }
  }
  return best;
}
size_t attn_split_partial_bytes(const quoka_params* p, int parts) {
  return parts <= 1 ? 0 : (size_t)attn_jobs(p) * parts * 2 * kSplitTileFloats * sizeof(float);
}
size_t attn_split_counter_bytes(const quoka_params* p) { return (size_t)attn_jobs(p) * 8 * sizeof(int32_t); }
// Parts of the launch at hand: `tiles` = key tiles of the longest row block the call can meet (the list or the
// cache, plus the chunk's own).  Without room for the partial results (the no-allocation entry point) nothing splits.
int attn_split_parts_for_launch(const quoka_params* p, const DevParams& P, bool sparse) {
  if (!P.attn_partials) return 1;
  return attn_split_parts(p, ((sparse ? P.budget_cap : P.max_ctx) + kKeyTile - 1) / kKeyTile + 1);
}

bool attn_tc_supported(const quoka_params* p) {
  if (p->dtype != QUOKA_BF16) return false;
  // the loaders address cache rows in 32-bit units of 16 bytes
  const int64_t extent = (p->page_size ? p->kv_rows : (int64_t)p->batch) * p->kv_stride_b;
  if (extent / 8 >= (int64_t)0xFFFFFFFFll) return false;
  return true;
}

quoka_status launch_attn_tc(const quoka_params* p, const DevParams& P, const void* q, const void* k, const void* v,
                            const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, cudaStream_t st,
                            bool after_selection) {
  if (attn_tc_pair_applies(P)) return launch_attn_tc_pair(p, P, q, k, v, k_idx, k_cnt, out, lse, st, after_selection);
  CUtensorMap tm_q;
  {
    const uint64_t dims[4] = {(uint64_t)P.d, (uint64_t)P.chunk, (uint64_t)P.n_q, (uint64_t)P.batch};
    const uint64_t strides[3] = {(uint64_t)P.q_st * 2, (uint64_t)P.q_sh * 2, (uint64_t)P.q_sb * 2};
    const uint32_t box[4] = {64, 128, 1, 1};
    if (!encode_tensor_map_bf16(&tm_q, q, 4, dims, strides, box)) return QUOKA_ERR_CUDA;
  }
  CUtensorMap tm_k, tm_v;
  if (!encode_kv_tensor_map(&tm_k, p, k, 64) || !encode_kv_tensor_map(&tm_v, p, v, 64)) return QUOKA_ERR_CUDA;
  const int halves = P.d / 64;
  const size_t tile = (size_t)halves * 128 * 128;
  const size_t smem = 1024 + (2 + kSlots) * tile + 512;
  const bool sparse = k_idx != nullptr;
  const int parts = attn_split_parts_for_launch(p, P, sparse);
  DevParams PP = P;
  PP.attn_parts = parts;
  dim3 grid(P.n_q, (P.chunk + 2 * kQTile - 1) / (2 * kQTile) * parts, P.batch);
  if (parts > 1 && !after_selection &&          // (the fused call clears the counters before its first kernel)
      cudaMemsetAsync(P.attn_counters, 0, attn_split_counter_bytes(p), st) != cudaSuccess)
    return QUOKA_ERR_CUDA;
  log_launch(sparse ? "attn_tc<sparse>" : "attn_tc<dense>", grid, dim3(kAttnThreads), smem, 1, sparse && after_selection);
  cudaError_t e = cudaSuccess;
  // Inside the fused call the sparse kernel is launched with programmatic stream serialisation: it may start
  // while the kernel before it on the stream (the key selection, which signals early and writes none of this
  // kernel's other inputs) still runs; it touches the selection's outputs only after its own
  // griddepcontrol.wait.  A stand-alone call keeps the ordinary stream order: whatever ran before it may have
  // written q, k or v.
#define QUOKA_ATTN_TC(H, S, X)                                                                                   \
  do {                                                                                                           \
    e = cudaFuncSetAttribute(attn_tc_kernel<H, S, X>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);   \
    if (e != cudaSuccess) return QUOKA_ERR_CUDA;                                                                 \
    cudaLaunchConfig_t cfg = {};                                                                                 \
    cfg.gridDim = grid;                                                                                          \
    cfg.blockDim = dim3(kAttnThreads);                                                                           \
    cfg.dynamicSmemBytes = smem;                                                                                 \
    cfg.stream = st;                                                                                             \
    cudaLaunchAttribute attr[1];                                                                                 \
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                             \
    attr[0].val.programmaticStreamSerializationAllowed = 1;                                                      \
    cfg.attrs = attr;                                                                                            \
    cfg.numAttrs = ((S) && after_selection) ? 1 : 0;                                                                                \
    e = cudaLaunchKernelEx(&cfg, attn_tc_kernel<H, S, X>, PP, tm_q, tm_k, tm_v, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, \
                           k_idx, k_cnt, (__nv_bfloat16*)out, lse);                                              \
    if (e != cudaSuccess) return QUOKA_ERR_CUDA;                                                                 \
  } while (0)
  if (parts > 1) {
    if (halves == 2) { if (sparse) QUOKA_ATTN_TC(2, true, true); else QUOKA_ATTN_TC(2, false, true); }
    else { if (sparse) QUOKA_ATTN_TC(1, true, true); else QUOKA_ATTN_TC(1, false, true); }
  } else {
    if (halves == 2) { if (sparse) QUOKA_ATTN_TC(2, true, false); else QUOKA_ATTN_TC(2, false, false); }
    else { if (sparse) QUOKA_ATTN_TC(1, true, false); else QUOKA_ATTN_TC(1, false, false); }
  }
#undef QUOKA_ATTN_TC
  count_launch();
  return cudaGetLastError() == cudaSuccess ? QUOKA_OK : QUOKA_ERR_CUDA;
}

}  // namespace quoka
