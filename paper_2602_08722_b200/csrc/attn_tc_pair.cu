// The tensor-core attention kernel for head_dim 128 with an even number of query heads per KV head: the CTAs of
// two query heads of one KV group run as a PAIR (a cluster of two on neighbouring SMs) and share every K / V tile.
//
// Both heads of a pair walk the same key tiles in the same order (the selected list, the chunk's own rows and the
// causal limits depend on the KV head and the chunk row only), so one `tcgen05.mma.cta_group::2` covers both:
// 256 rows of S (or O), 128 per CTA, with the K (or V) operand split between the two CTAs' shared memories.
//   S = Q K^T : each CTA supplies its own Q tile and 64 of the tile's 128 keys (all 128 elements of each).
//   O += P V  : each CTA supplies its own P (tensor memory) and 64 of V's 128 columns (all 128 keys).
// So a CTA fetches HALF of every K and V tile (the 16-byte cp.async gather of listed rows tops out near 20 bytes per
// clock and SM, which a one-CTA step of 64 KB all but needs), its loaders execute half the instructions, and per
// key tile and Q tile the tensor core reads 48 KB + 16 KB of a CTA's shared memory instead of 64 KB + 32 KB.  A
// step's time itself is set by one Q tile's chain S ready -> softmax -> P ready -> PV -> next QK^T and changes little:
// measured against the one-CTA kernel, 1 % (listed rows) to 4 % (whole tiles, paged serving mix) faster.
//
// Roles per CTA as in the one-CTA kernel (8 softmax warps, 3 loader warps, warp 11), except:
//   * only the first CTA's warp 11 issues MMAs.  A slot of its ring is ready when its own loaders AND the second
//     CTA's have filled it: warp 11 of the second CTA forwards its slots' "full" barriers, in ring order, to a
//     barrier of the first CTA;
//   * completions (S ready, slot free, O final) are delivered to both CTAs' barriers by one multicast commit;
//   * the softmax warps of both CTAs announce P on the first CTA's barriers;
//   * nobody leaves before a cluster barrier: the other CTA's MMAs read this one's shared and tensor memory.
// Tensor memory (512 columns per CTA): S_A | S_B | O_A | O_B, P aliasing the first 64 columns of its S.
// Ring slots are 16 KB: a K item holds [2 halves of d][64 keys][128 B], a V item [128 keys][128 B], both in the
// 128-byte-swizzled layout of the operand descriptors.
#include "attn_tiles.cuh"

namespace quoka {

constexpr int kPairSlots = 8;
constexpr int kPairLoaderWarps = 3;
constexpr uint32_t kPairSlotBytes = 16384;
constexpr uint32_t kPairQTileBytes = 32768;

template <bool SPARSE, bool SPLIT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kAttnThreads, 1)
attn_tc_pair_kernel(DevParams P, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __nv_bfloat16* __restrict__ kc,
                    const __nv_bfloat16* __restrict__ vc, const int32_t* __restrict__ k_idx,
                    const int32_t* __restrict__ k_cnt, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
  constexpr int D = 128;
  constexpr uint32_t S_COL[2] = {0, 128}, O_COL[2] = {256, 384};
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* q_smem = smem;                               // [2][2 halves][128][128 B]
  unsigned char* kv_smem = smem + 2 * kPairQTileBytes;        // [kPairSlots][16 KB]
  uint64_t* bars = reinterpret_cast<uint64_t*>(kv_smem + (size_t)kPairSlots * kPairSlotBytes);
  uint64_t* kv_full = bars;                       // [kPairSlots]  this CTA's loaders
  uint64_t* kv_empty = kv_full + kPairSlots;      // [kPairSlots]  MMA commit (both CTAs)
  uint64_t* peer_full = kv_empty + kPairSlots;    // [kPairSlots]  first CTA only: the second CTA's slot is full
  uint64_t* s_full = peer_full + kPairSlots;      // [2]           MMA commit (both CTAs)
  uint64_t* p_full = s_full + 2;                  // [2][2]        first CTA only: 4 softmax warps of each CTA
  uint64_t* o_full = p_full + 4;                  // [2]           MMA commit (both CTAs)
  uint64_t* q_full = o_full + 2;                  // this CTA's Q tiles (TMA)
  uint64_t* peer_q = q_full + 1;                  // first CTA only: the second CTA's Q tiles have landed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(peer_q + 1);
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtx wc{&abort_flag, P.status};
  const uint32_t rank = cluster_cta_rank();                   // 0: issues the MMAs; the pair is heads (2j, 2j + 1)
  const int s = blockIdx.z, h = blockIdx.x, kv = h / P.group;
  // grid.y = row blocks (heaviest first), times the parts a row block's key tiles are cut into (SPLIT)
  const int n_parts = SPLIT ? P.attn_parts : 1;
  const int n_rb = gridDim.y / n_parts;
  const int rb = n_rb - 1 - blockIdx.y / n_parts;
  const int r0 = rb * 2 * kQTile;
  AttnGeom g = make_geom<SPARSE>(P, s, r0);
  // SPLIT: this CTA walks the tiles [t_lo, t_hi) of the row block's sequence only and leaves, per row, a partial
  // result (reference point, sum, un-normalised output); the part that finishes last adds the parts up.  The list
  // length has to be known before the range is, so nothing of the walk starts before the selection has ended.
  int t_lo = 0;
  if (SPLIT) {
    if (SPARSE) resolve(g, k_cnt, s);
    const int part = blockIdx.y % n_parts;
    t_lo = (int)(((long long)part * g.n_known) / n_parts);
    g.n_known = (int)(((long long)(part + 1) * g.n_known) / n_parts);
  }

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < kPairSlots; ++i) {
      mbar_init(&kv_full[i], kPairLoaderWarps * 32);
      mbar_init(&kv_empty[i], 1);
      mbar_init(&peer_full[i], 1);
    }
    for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&o_full[i], 1); }
    for (int i = 0; i < 4; ++i) mbar_init(&p_full[i], 8);
    mbar_init(q_full, 1);
    mbar_init(peer_q, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
  }
  if (warp == kMmaWarp) tmem_alloc_pair(tmem_slot, 512);
  tc_fence_before();
  cluster_sync_all();                                         // both CTAs' barriers exist before anyone signals them
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
    const uint32_t p_bar0 = map_to_cta(smem_u32(&p_full[2 * x]), 0);   // the first CTA's barriers
    const uint32_t p_bar1 = map_to_cta(smem_u32(&p_full[2 * x + 1]), 0);
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
                           [&](int half) { mbar_arrive_cluster(half ? p_bar1 : p_bar0); });
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
  } else if (warp < 8 + kPairLoaderWarps) {
    // ================================================================== K / V loaders: this CTA's half of every tile
    // K item: tile rows [64 * rank, 64 * rank + 64), 256 bytes each (16 pieces, 2 rows per warp instruction).
    // V item: all 128 tile rows, bytes [128 * rank, 128 * rank + 128) of each (8 pieces, 4 rows per instruction).
    // Either way an item is 32 row groups, dealt round-robin to the loader warps.
    const int lw = warp - 8;
    constexpr int GROUPS = 32;
    constexpr int RPT = (GROUPS + kPairLoaderWarps - 1) / kPairLoaderWarps;   // row groups per warp (the last may be idle)
    const int kc16 = lane & 15, krsub = lane >> 4;
    const int vc16 = lane & 7, vrsub = lane >> 3;
    const int krow0 = (int)rank * 64;
    const int32_t* idx = SPARSE ? k_idx + ((long long)s * P.n_kv + kv) * P.budget_cap : nullptr;
    uint32_t phase = 0;
    int slot = 0;
    const uint32_t kv_base = smem_u32(kv_smem);
    // Row addressing in 16-byte units, 32 bits wide (the host refuses caches beyond 2^32 units; strides are
    // multiples of 8 elements): sequence/head base plus this thread's piece, row stride, page stride.
    const uint32_t st16 = (uint32_t)(P.kv_st >> 3), sb16 = (uint32_t)(P.kv_sb >> 3);
    const uint32_t head16 = (uint32_t)(((P.page_size == 0 ? (long long)s * P.kv_sb : 0ll) + (long long)kv * P.kv_sh) >> 3);
    const uint32_t kbase16 = head16 + (uint32_t)kc16, vbase16 = head16 + rank * 8u + (uint32_t)vc16;
    const int32_t* table = P.block_table + (long long)s * P.max_pages;
    // Row numbers of this warp's rows of a tile of the selected list (-1 past the end), fetched one tile ahead.
    // The warp's K rows are numbered p = 2 i + rsub (i = its i-th row group), its V rows p = 4 i + rsub; lane l
    // keeps K row p = l and V rows p = l, 32 + l, and the thread that copies a row fetches its number by shuffle.
    int tk_list = -1, tv_list[2] = {-1, -1};
    auto list_rows = [&](int base, int count) {
      const int last = min(count, kKeyTile) - 1;                   // last valid row of the tile
      if (last >= 0) {
        {
          const int gi = lw + (lane >> 1) * kPairLoaderWarps;
          const int rr = krow0 + gi * 2 + (lane & 1);
          const int v = __ldcg(idx + base + min(rr, last));        // written by the kernel before: L2, not the read-only path
          tk_list = (lane < 2 * RPT && gi < GROUPS && rr <= last) ? v : -1;
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int pp = 32 * k + lane;
          const int gi = lw + (pp >> 2) * kPairLoaderWarps;
          const int rr = gi * 4 + (pp & 3);
          const int v = __ldcg(idx + base + min(rr, last));
          tv_list[k] = (pp < 4 * RPT && gi < GROUPS && rr <= last) ? v : -1;
        }
      }
    };
    // One ring item of tile `tr`: K (is_v = false) or V.  Returns false when a wait gave up.
    auto item = [&](auto is_v_c, const TileRows& tr, bool first_list_tile) -> bool {
      constexpr bool V = decltype(is_v_c)::value;
      constexpr int RPI = V ? 4 : 2;                            // rows per warp instruction
      if (!mbar_wait(&kv_empty[slot], phase ^ 1, wc)) return false;
      // A whole tile of consecutive rows (page-aligned in a paged cache) is fetched by the copy engine as two
      // 8 KB boxes: one thread issues them, the others only keep the barrier's arrival count.  Ragged tiles (rows
      // past the end must read as zeros) and listed rows take the copies below.
      if (!tr.from_list && tr.count >= kKeyTile && (P.page_size == 0 || (tr.first & (kPage - 1)) == 0)) {
        if (lw == 0 && lane == 0) {
          fence_proxy_async_smem();             // earlier contents of the slot were written through the generic proxy
          mbar_arrive_expect_tx(&kv_full[slot], kPairSlotBytes);
          unsigned char* dst = kv_smem + (size_t)slot * kPairSlotBytes;
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            // K: box j = elements [64 j, 64 j + 64) of this CTA's 64 rows; V: box j = rows [64 j, 64 j + 64), this
            // CTA's 64 elements
            const int c0 = V ? (int)rank * 64 : j * 64;
            const int sub = V ? j : (int)rank;
            int c1 = tr.first + sub * 64, c3 = s;
            if (P.page_size != 0) { c1 = 0; c3 = __ldg(table + (tr.first >> 6) + sub); }
            tma_load_4d(dst + j * 8192, V ? &tm_v : &tm_k, &kv_full[slot], c0, c1, kv, c3);
          }
        } else {
          mbar_arrive(&kv_full[slot]);
        }
      } else {
        if (!V && first_list_tile) list_rows(tr.first, tr.count);
        const int c16 = V ? vc16 : kc16, rsub = V ? vrsub : krsub;
        const uint32_t base16 = V ? vbase16 : kbase16;
        const uint4* src_base = reinterpret_cast<const uint4*>(V ? vc : kc);
        const uint32_t dst_item = kv_base + (uint32_t)slot * kPairSlotBytes + (V ? 0u : (uint32_t)(c16 >> 3) * 8192u);
        int t[RPT];                                               // row number, or -1
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
          const int rr = (V ? 0 : krow0) + (lw + i * kPairLoaderWarps) * RPI + rsub;   // row of the tile
          const int listed = V ? __shfl_sync(0xFFFFFFFFu, tv_list[(i * 4) / 32], (i * 4 + rsub) & 31)
                               : __shfl_sync(0xFFFFFFFFu, tk_list, i * 2 + rsub);
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
          const int gi = lw + i * kPairLoaderWarps;
          const int lr = gi * RPI + rsub;                         // row of the item in shared memory
          if (gi < GROUPS)                                        // false only for the last group of some warps
            cp_async_16(dst_item + lr * 128 + (((c16 & 7) ^ (lr & 7)) << 4), src_base + off[i], t[i] >= 0);
        }
        // this thread's share of the slot is signalled by the copy engine itself when the bytes have landed
        cp_async_mbar_arrive_noinc(&kv_full[slot]);
        if (V && tr.from_list) list_rows(tr.first + kKeyTile, tr.count - kKeyTile);   // next list tile
      }
      if (++slot == kPairSlots) { slot = 0; phase ^= 1; }
      return true;
    };
    for (int tile = t_lo;; ++tile) {
      if (tile == g.n_known) {                                // end of what is known: the list length, or the end
        if (g.resolved) break;
        resolve(g, k_cnt, s);
        if (tile == g.n_known) break;
      }
      const TileRows tr = tile_rows<SPARSE>(g, tile);
      const bool first_list_tile = tr.from_list && tile == max(g.n_chunk, t_lo);
      if (!item(std::false_type{}, tr, first_list_tile)) break;
      if (!item(std::true_type{}, tr, first_list_tile)) break;
    }
    cp_async_wait_all();                                      // nothing of this thread is in flight at exit
  } else if (lane == 0) {
    // ================================================================== warp 11, one thread
    mbar_arrive_expect_tx(q_full, 2 * kPairQTileBytes);
    for (int x = 0; x < 2; ++x)
      for (int hh = 0; hh < 2; ++hh)
        tma_load_4d(q_smem + x * kPairQTileBytes + hh * 16384, &tm_q, q_full, hh * 64, r0 + x * kQTile, h, s);
    bool ok = mbar_wait(q_full, 0, wc);
    if (rank != 0) {
      // ---------------------------------------------------------------- second CTA: forward "full" to the first
      if (ok) mbar_arrive_cluster(map_to_cta(smem_u32(peer_q), 0));
      const uint32_t peer_full0 = map_to_cta(smem_u32(peer_full), 0);
      int slot = 0;
      uint32_t phase = 0;
      for (int tile = t_lo; ok; ++tile) {
        if (tile == g.n_known) {
          if (g.resolved) break;
          resolve(g, k_cnt, s);
          if (tile == g.n_known) break;
        }
#pragma unroll 1
        for (int kvi = 0; kvi < 2; ++kvi) {
          if (!mbar_wait(&kv_full[slot], phase, wc)) { ok = false; break; }
          fence_proxy_async_all();            // the loaders' cp.async wrote through the generic proxy
          mbar_arrive_cluster(peer_full0 + (uint32_t)slot * 8u);
          if (++slot == kPairSlots) { slot = 0; phase ^= 1; }
        }
      }
    } else {
      // ---------------------------------------------------------------- first CTA: MMA issuer for the pair
      const uint32_t idesc_qk = idesc_bf16_f32(256, kKeyTile, false, false);
      const uint32_t idesc_pv = idesc_bf16_f32(256, D, false, true);
      const uint32_t q_base = smem_u32(q_smem), kv_base = smem_u32(kv_smem);
      int slot = 0;
      uint32_t kv_phase = 0;
      uint32_t p_phase[2] = {0, 0};
      int k_slot = -1, v_slot = -1;
      if (ok) ok = mbar_wait(peer_q, 0, wc);
      auto acquire = [&]() -> int {           // next ring item (K or V) is readable in both CTAs
        if (!mbar_wait(&kv_full[slot], kv_phase, wc) || !mbar_wait(&peer_full[slot], kv_phase, wc)) {
          ok = false;
          return 0;
        }
        fence_proxy_async_smem();             // cp.async wrote through the generic proxy, the MMA reads through the async one
        tc_fence_after();
        const int got = slot;
        if (++slot == kPairSlots) { slot = 0; kv_phase ^= 1; }
        return got;
      };
      // Descriptors are built once; a tile, slot or k-step offset is an addition to the 16-byte-unit address field.
      const uint64_t desc_q = smem_desc_sw128(q_base, 16, 1024);
      const uint64_t desc_kv = smem_desc_sw128(kv_base, 16, 1024);
      auto issue_qk = [&](int x, int ks) {
        const uint64_t da = desc_q + (uint64_t)(x * (kPairQTileBytes >> 4));
        const uint64_t db = desc_kv + (uint64_t)((uint32_t)ks * (kPairSlotBytes >> 4));
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const uint64_t offa = (uint64_t)((hh * 16384 + kk * 32) >> 4);   // Q: halves of 128 rows
            const uint64_t offb = (uint64_t)((hh * 8192 + kk * 32) >> 4);    // K: halves of 64 rows
            mma_pair_ss(tmem_base + S_COL[x], da + offa, db + offb, idesc_qk, (hh | kk) ? 1u : 0u);
          }
        mma_pair_commit(&s_full[x]);
      };
      auto issue_pv = [&](int x, int vs, bool first) {
        const uint64_t dv = desc_kv + (uint64_t)((uint32_t)vs * (kPairSlotBytes >> 4));
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          if (!mbar_wait(&p_full[2 * x + half], p_phase[x], wc)) { ok = false; return; }
          tc_fence_after();
#pragma unroll
          for (int kk = half * 4; kk < half * 4 + 4; ++kk) {   // 16 keys per MMA: 8 packed columns of P, 16 rows of V
            mma_pair_ts(tmem_base + O_COL[x], tmem_base + S_COL[x] + kk * 8, dv + (uint64_t)(kk * (2048 >> 4)), idesc_pv,
                        (!first || kk) ? 1u : 0u);
          }
        }
        p_phase[x] ^= 1;
      };
      // Tile t: O += P_t V_t for each Q tile taking part (as the two halves of P arrive), then S = Q K_{t+1}^T.
      // K_{t+1} and V_t are both acquired before the P waits, so those never sit on the P -> PV -> QK chain.
      const auto part = [&](int x, int t) { return x ? g.active_b : t >= g.skip_a; };
      if (ok && t_lo < g.n_known) {
        k_slot = acquire();
        if (ok) {
          if (part(0, t_lo)) issue_qk(0, k_slot);
          if (part(1, t_lo)) issue_qk(1, k_slot);
          mma_pair_commit(&kv_empty[k_slot]);
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
            if (!more) mma_pair_commit(&o_full[0]);
          }
          if (more && part(0, t + 1)) issue_qk(0, k_slot);
          if (part(1, t)) {
            issue_pv(1, v_slot, t == t_lo);
            if (!ok) break;
            if (!more) mma_pair_commit(&o_full[1]);
          }
          mma_pair_commit(&kv_empty[v_slot]);
          if (!more) break;
          if (part(1, t + 1)) issue_qk(1, k_slot);
          mma_pair_commit(&kv_empty[k_slot]);
        }
      }
    }
  }
  tc_fence_before();
  cluster_sync_all();                                         // the other CTA's MMAs no longer read this CTA
  if (warp == kMmaWarp) tmem_dealloc_pair(tmem_base, 512);
}

// ---------------------------------------------------------------------------------------------- host
bool attn_tc_pair_applies(const DevParams& P) { return P.d == 128 && P.group % 2 == 0; }

quoka_status launch_attn_tc_pair(const quoka_params* p, const DevParams& P, const void* q, const void* k, const void* v,
                                 const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, cudaStream_t st,
                                 bool after_selection) {
  CUtensorMap tm_q;
  {
    const uint64_t dims[4] = {(uint64_t)P.d, (uint64_t)P.chunk, (uint64_t)P.n_q, (uint64_t)P.batch};
    const uint64_t strides[3] = {(uint64_t)P.q_st * 2, (uint64_t)P.q_sh * 2, (uint64_t)P.q_sb * 2};
    const uint32_t box[4] = {64, 128, 1, 1};
    if (!encode_tensor_map_bf16(&tm_q, q, 4, dims, strides, box)) return QUOKA_ERR_CUDA;
  }
  CUtensorMap tm_k, tm_v;
  if (!encode_kv_tensor_map(&tm_k, p, k, 64) || !encode_kv_tensor_map(&tm_v, p, v, 64)) return QUOKA_ERR_CUDA;
  const size_t smem = 1024 + 2 * kPairQTileBytes + (size_t)kPairSlots * kPairSlotBytes + 512;
  const bool sparse = k_idx != nullptr;
  const int parts = attn_split_parts_for_launch(p, P, sparse);
  DevParams PP = P;
  PP.attn_parts = parts;
  dim3 grid(P.n_q, (P.chunk + 2 * kQTile - 1) / (2 * kQTile) * parts, P.batch);   // n_q is even: clusters of (2, 1, 1)
  if (parts > 1 && !after_selection &&          // (the fused call clears the counters before its first kernel)
      cudaMemsetAsync(P.attn_counters, 0, attn_split_counter_bytes(p), st) != cudaSuccess)
    return QUOKA_ERR_CUDA;
  log_launch(sparse ? "attn_tc_pair<sparse>" : "attn_tc_pair<dense>", grid, dim3(kAttnThreads), smem, 2,
             sparse && after_selection);
  cudaError_t e = cudaSuccess;
  // Programmatic stream serialisation inside the fused call only, as for the one-CTA kernel.
#define QUOKA_ATTN_PAIR(S, X)                                                                                      \
  do {                                                                                                            \
    e = cudaFuncSetAttribute(attn_tc_pair_kernel<S, X>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
    if (e != cudaSuccess) return QUOKA_ERR_CUDA;                                                                  \
    cudaLaunchConfig_t cfg = {};                                                                                  \
    cfg.gridDim = grid;                                                                                           \
    cfg.blockDim = dim3(kAttnThreads);                                                                            \
    cfg.dynamicSmemBytes = smem;                                                                                  \
    cfg.stream = st;                                                                                              \
    cudaLaunchAttribute attr[1];                                                                                  \
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                              \
    attr[0].val.programmaticStreamSerializationAllowed = 1;                                                       \
    cfg.attrs = attr;                                                                                             \
    cfg.numAttrs = ((S) && after_selection) ? 1 : 0;                                                              \
    e = cudaLaunchKernelEx(&cfg, attn_tc_pair_kernel<S, X>, PP, tm_q, tm_k, tm_v, (const __nv_bfloat16*)k,        \
                           (const __nv_bfloat16*)v, k_idx, k_cnt, (__nv_bfloat16*)out, lse);                      \
    if (e != cudaSuccess) return QUOKA_ERR_CUDA;                                                                  \
  } while (0)
  if (parts > 1) { if (sparse) QUOKA_ATTN_PAIR(true, true); else QUOKA_ATTN_PAIR(false, true); }
  else { if (sparse) QUOKA_ATTN_PAIR(true, false); else QUOKA_ATTN_PAIR(false, false); }
#undef QUOKA_ATTN_PAIR
  count_launch();
  return cudaGetLastError() == cudaSuccess ? QUOKA_OK : QUOKA_ERR_CUDA;
}

}  // namespace quoka
