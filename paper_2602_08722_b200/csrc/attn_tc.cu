// Flash-style attention on the 5th-generation tensor cores over
//   [selected cached rows | the chunk's own causal rows]      (Algorithm 2's attention line, Eq. 2)
// or, without an index list, over every cached row (Eq. 2, dense chunk attention).  bf16 in, fp32
// softmax and accumulation, P rounded to bf16 for the PV product.
//
// One CTA owns 256 consecutive chunk rows of one query head as two 128-row Q tiles (A, B) and walks
// the key tiles (128 keys) once for both.  Roles:
//   warps 0-3 / 4-7  softmax of Q tile A / B: one thread per query row, S read from tensor memory,
//                    running max / sum in registers, P written back to tensor memory over S,
//                    lazy rescale of the O accumulator (only when the max grew by more than 2^8),
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
#include "sm100_ptx.cuh"
#include "tensor_kernels.cuh"

namespace quoka {

using namespace ptx;

constexpr int kAttnThreads = 12 * 32;
constexpr int kLoaderWarps = 3;
constexpr int kMmaWarp = 11;
constexpr int kQTile = 128;
constexpr int kKeyTile = 128;
constexpr int kSlots = 5;
constexpr float kRescaleThreshold = 8.0f;   // log2 units

bool encode_kv_tensor_map(CUtensorMap* out, const quoka_params* p, const void* cache, uint32_t box_rows);

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct AttnGeom {
  int T, cnt, n_sel;        // cached length, selected rows, selected tiles (sparse); cnt = T, n_sel unused (dense)
  int n_a, n_b, n_max;      // key tiles Q tile A / B take part in, and their maximum
};

template <bool SPARSE>
__device__ __forceinline__ AttnGeom make_geom(const DevParams& P, int s, int r0, const int32_t* k_cnt) {
  AttnGeom g;
  g.T = __ldg(P.ctx_len + s);
  const int C = P.chunk;
  const bool b_active = r0 + kQTile < C;
  if (SPARSE) {
    g.cnt = __ldg(k_cnt + s);
    g.n_sel = (g.cnt + kKeyTile - 1) / kKeyTile;
    g.n_a = g.n_sel + r0 / kQTile + 1;
    g.n_b = b_active ? g.n_a + 1 : 0;
  } else {
    g.cnt = g.T;
    g.n_sel = 0;
    const int last_a = min(r0 + kQTile - 1, C - 1), last_b = min(r0 + 2 * kQTile - 1, C - 1);
    g.n_a = (g.T + last_a) / kKeyTile + 1;
    g.n_b = b_active ? (g.T + last_b) / kKeyTile + 1 : 0;
  }
  g.n_max = max(g.n_a, g.n_b);
  return g;
}

// Number of visible columns of key tile j for chunk row `row` (columns [0, lim) are visible).
template <bool SPARSE>
__device__ __forceinline__ int visible_cols(const AttnGeom& g, int j, int row) {
  int lim;
  if (SPARSE) {
    if (j < g.n_sel) lim = g.cnt - j * kKeyTile;
    else lim = row - (j - g.n_sel) * kKeyTile + 1;
  } else {
    lim = g.T + row - j * kKeyTile + 1;
  }
  return max(0, min(kKeyTile, lim));
}

// Maximum of 32 score columns starting at col0; columns at and beyond `lim` are masked out.
__device__ __forceinline__ float max32(uint32_t (&v)[32], bool masked, int col0, int lim) {
  if (masked) {
#pragma unroll
    for (int i = 0; i < 32; ++i) if (col0 + i >= lim) v[i] = 0xFF800000u;    // -inf
  }
  float m0 = __uint_as_float(v[0]), m1 = __uint_as_float(v[1]);
#pragma unroll
  for (int i = 2; i < 30; i += 4) {
    m0 = max3(m0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
    m1 = max3(m1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
  }
  return max3(m0, m1, fmaxf(__uint_as_float(v[30]), __uint_as_float(v[31])));
}

template <int HALVES, bool SPARSE>
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_tc_kernel(DevParams P, const __grid_constant__ CUtensorMap tm_q, const __nv_bfloat16* __restrict__ kc,
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
  const int rb = gridDim.y - 1 - blockIdx.y;
  const int r0 = rb * 2 * kQTile;
  const AttnGeom g = make_geom<SPARSE>(P, s, r0, k_cnt);

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int i = 0; i < kSlots; ++i) { mbar_init(&kv_full[i], kLoaderWarps * 32); mbar_init(&kv_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&o_full[i], 1); }
    for (int i = 0; i < 4; ++i) mbar_init(&p_full[i], 4);
    mbar_init(q_full, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tm_q);
  }
  if (warp == kMmaWarp) tmem_alloc(tmem_slot, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp < 8) {
    // ================================================================== softmax + epilogue
    const int x = warp >> 2;                                  // Q tile A (0) or B (1)
    const int n_tiles = x ? g.n_b : g.n_a;
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    const int row = r0 + x * kQTile + row_in_tile;            // chunk row
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const uint32_t s_addr = lane_addr + S_COL[x], o_addr = lane_addr + O_COL[x];
    const float scale_log2 = P.scale * 1.4426950408889634f;
    float m_run = -INFINITY, l_run = 0.f;
    uint32_t phase = 0;
    bool ok = true;
    for (int j = 0; j < n_tiles; ++j) {
      if (!mbar_wait(&s_full[x], phase, wc)) { ok = false; break; }
      phase ^= 1;
      tc_fence_after();
      const int lim = visible_cols<SPARSE>(g, j, row);
      const bool masked = !__all_sync(0xFFFFFFFFu, lim >= kKeyTile);
      // ---- pass 1: the row maximum.  All four 32-column loads are issued together (one tensor-memory round
      // trip); the row is read once more, in 64-key blocks, by pass 2: tensor memory is cheap to re-read, and
      // not keeping the 128 values live leaves pass 2 the registers for a whole block of exponentials in flight.
      float mx;
      {
        uint32_t c0[32], c1[32], c2[32], c3[32];
        tmem_ld32(s_addr, c0);
        tmem_ld32(s_addr + 32, c1);
        tmem_ld32(s_addr + 64, c2);
        tmem_ld32(s_addr + 96, c3);
        tmem_wait_ld();
        mx = fmaxf(fmaxf(max32(c0, masked, 0, lim), max32(c1, masked, 32, lim)),
                   fmaxf(max32(c2, masked, 64, lim), max32(c3, masked, 96, lim)));
      }
      const float m_tile = mx * scale_log2;
      // ---- lazy rescale of the accumulator: only when some row's maximum grew by more than the threshold
      const bool grow = m_tile > m_run + kRescaleThreshold;
      if (__any_sync(0xFFFFFFFFu, grow)) {
        const float m_new = fmaxf(m_run, m_tile);
        if (j > 0) {
          const float alpha = (m_run == -INFINITY) ? 0.f : ex2(m_run - m_new);
          l_run *= alpha;
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(o_addr + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st32(o_addr + c * 32, r);
          }
          tmem_wait_st();
        }
        m_run = m_new;
      }
      const float m_use = (m_run == -INFINITY) ? 0.f : m_run;
      // ---- pass 2: p = 2^(s*scale - m) in two blocks of 64 keys.  bf16 P goes over the first 64 columns of
      // S (block h of P lands on columns 32h..32h+31, all of them read already) and each block is handed to the
      // MMA issuer as soon as it is stored, so the first PV products run under the second block's arithmetic.
      const uint64_t sc2 = pack2(scale_log2, scale_log2), nm2 = pack2(-m_use, -m_use);
      uint64_t psa[2] = {0ull, 0ull};                           // four running sums as two packed pairs
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t v[64], pk[32];
        tmem_ld32(s_addr + half * 64, v);
        tmem_ld32(s_addr + half * 64 + 32, v + 32);
        tmem_wait_ld();
        if (masked) {
#pragma unroll
          for (int i = 0; i < 64; ++i) if (half * 64 + i >= lim) v[i] = 0xFF800000u;   // -inf: exp2 gives exactly 0
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float x0, x1;
          unpack2(fma2(pack2u(v[2 * i], v[2 * i + 1]), sc2, nm2), x0, x1);
          const float p0 = ex2(x0), p1 = ex2(x1);
          psa[i & 1] = add2(psa[i & 1], pack2(p0, p1));
          const __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);
          pk[i] = *reinterpret_cast<const uint32_t*>(&b2);
        }
        tmem_st32(s_addr + half * 32, pk);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[2 * x + half]);
      }
      float ps0, ps1, ps2, ps3;
      unpack2(psa[0], ps0, ps1);
      unpack2(psa[1], ps2, ps3);
      l_run += (ps0 + ps1) + (ps2 + ps3);
    }
    // ---- epilogue: O / l -> bf16 -> global
    if (ok && n_tiles > 0 && mbar_wait(&o_full[x], 0, wc)) {
      tc_fence_after();
      const float inv = 1.f / l_run;
      const bool store = row < P.chunk;
      __nv_bfloat16* orow = out + (long long)s * P.o_sb + (long long)h * P.o_sh + (long long)row * P.o_st;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(o_addr + c * 32, r);
        tmem_wait_ld();
        if (store) {
#pragma unroll
          for (int v4 = 0; v4 < 4; ++v4) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(r[v4 * 8 + 2 * i]) * inv,
                                                               __uint_as_float(r[v4 * 8 + 2 * i + 1]) * inv);
              w[i] = *reinterpret_cast<const uint32_t*>(&b2);
            }
            *reinterpret_cast<uint4*>(orow + c * 32 + v4 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      if (store && lse)
        lse[((long long)s * P.n_q + h) * P.chunk + row] = (m_run + log2f(l_run)) * 0.6931471805599453f;
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
    const int n_items = 2 * g.n_max;
    uint32_t phase = 0;
    int slot = 0;
    const uint32_t kv_base = smem_u32(kv_smem);
    // Row addressing in 16-byte units, 32 bits wide (the host refuses caches beyond 2^32 units; strides are
    // multiples of 8 elements): sequence/head base plus this thread's piece, row stride, page stride.
    const uint32_t st16 = (uint32_t)(P.kv_st >> 3), sb16 = (uint32_t)(P.kv_sb >> 3);
    const uint32_t base16 = (uint32_t)(((P.page_size == 0 ? (long long)s * P.kv_sb : 0ll) + (long long)kv * P.kv_sh) >> 3) +
                            (uint32_t)c16;
    const int32_t* table = P.block_table + (long long)s * P.max_pages;
    // Row numbers of this thread's rows of a tile of the selected list (-1 past the end).  They are fetched one
    // tile ahead and only looked at when that tile's copies are issued, so the loader never waits on them.
    // The per-row code below is kept free of branches (clamped loads, selects): a branch per row costs a single
    // warp far more than the arithmetic it skips.
    auto list_rows = [&](int j, int (&t)[RPT]) {
      if (SPARSE && j < g.n_sel) {
        const int last = g.cnt - 1 - j * kKeyTile;                 // last valid row of this tile (>= 0)
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
          const int rr = (lw + i * kLoaderWarps) * ROWS_PER_INSTR + rsub;
          const int v = __ldg(idx + j * kKeyTile + min(rr, last));
          t[i] = rr <= last ? v : -1;
        }
      }
    };
    int t_cur[RPT], t_next[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i) t_next[i] = -1;
    list_rows(0, t_next);
    for (int it = 0; it < n_items; ++it) {
      if (!mbar_wait(&kv_empty[slot], phase ^ 1, wc)) break;
      const int j = it >> 1;
      const bool from_list = SPARSE && j < g.n_sel;
      if (!(it & 1)) {
#pragma unroll
        for (int i = 0; i < RPT; ++i) t_cur[i] = t_next[i];
      }
      // rows outside the list are consecutive: row_first + r for r < row_count (the chunk's own rows, or all rows)
      int row_first, row_count;
      if (SPARSE) { row_first = g.T + (j - g.n_sel) * kKeyTile; row_count = P.chunk - (j - g.n_sel) * kKeyTile; }
      else { row_first = j * kKeyTile; row_count = g.T + P.chunk - j * kKeyTile; }
      const uint4* src_base = reinterpret_cast<const uint4*>((it & 1) ? vc : kc);
      const uint32_t dst_tile = kv_base + slot * kTileBytes + (c16 >> 3) * kHalfBytes;
      int t[RPT];                                                 // row number, or -1
#pragma unroll
      for (int i = 0; i < RPT; ++i) {
        const int rr = (lw + i * kLoaderWarps) * ROWS_PER_INSTR + rsub;
        t[i] = from_list ? t_cur[i] : (rr < row_count ? row_first + rr : -1);
      }
      uint32_t off[RPT];
      if (P.page_size == 0) {
#pragma unroll
        for (int i = 0; i < RPT; ++i) off[i] = base16 + (uint32_t)max(t[i], 0) * st16;
      } else {
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
          const int tc = max(t[i], 0);
          off[i] = (uint32_t)__ldg(table + (tc >> 6)) * sb16 + base16 + (uint32_t)(tc & (kPage - 1)) * st16;
        }
      }
#pragma unroll
      for (int i = 0; i < RPT; ++i) {
        const int rr = (lw + i * kLoaderWarps) * ROWS_PER_INSTR + rsub;
        if (rr < kKeyTile)                                        // false only for the last group of some warps
          cp_async_16(dst_tile + rr * 128 + (((c16 & 7) ^ (rr & 7)) << 4), src_base + off[i], t[i] >= 0);
      }
      // this thread's share of the slot is signalled by the copy engine itself when the bytes have landed:
      // no wait in the loader, every slot of the ring can be in flight
      cp_async_mbar_arrive_noinc(&kv_full[slot]);
      if (!(it & 1)) list_rows(j + 1, t_next);
      if (++slot == kSlots) { slot = 0; phase ^= 1; }
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
    auto issue_pv = [&](int x, int vs, int j) {
      const uint64_t dv = desc_v + (uint64_t)((uint32_t)vs * (kTileBytes >> 4));
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        if (!mbar_wait(&p_full[2 * x + half], p_phase[x], wc)) { ok = false; return; }
        tc_fence_after();
#pragma unroll
        for (int kk = half * 4; kk < half * 4 + 4; ++kk) {   // 16 keys per MMA: 8 packed columns of P, 16 rows of V
          mma_ts(tmem_base + O_COL[x], tmem_base + S_COL[x] + kk * 8, dv + (uint64_t)(kk * (2048 >> 4)), idesc_pv,
                 (j | kk) ? 1u : 0u);
        }
      }
      p_phase[x] ^= 1;
    };
    if (ok && g.n_max > 0) {
      k_slot = acquire();
      if (ok) {
        if (g.n_a > 0) issue_qk(0, k_slot);
        if (g.n_b > 0) issue_qk(1, k_slot);
        mma_commit(&kv_empty[k_slot]);
      }
      for (int j = 0; ok && j < g.n_max; ++j) {
        const bool more = j + 1 < g.n_max;
        v_slot = acquire();
        if (ok && more) k_slot = acquire();     // both are normally there already: keeps the waits off the P -> PV -> QK chain
        if (!ok) break;
        if (j < g.n_a) {
          issue_pv(0, v_slot, j);
          if (!ok) break;
          if (j + 1 == g.n_a) mma_commit(&o_full[0]);
        }
        if (more && j + 1 < g.n_a) issue_qk(0, k_slot);
        if (j < g.n_b) {
          issue_pv(1, v_slot, j);
          if (!ok) break;
          if (j + 1 == g.n_b) mma_commit(&o_full[1]);
        }
        mma_commit(&kv_empty[v_slot]);
        if (more) {
          if (j + 1 < g.n_b) issue_qk(1, k_slot);
          mma_commit(&kv_empty[k_slot]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, 512);
}

// ---------------------------------------------------------------------------------------------- host
bool attn_tc_supported(const quoka_params* p) {
  if (p->dtype != QUOKA_BF16) return false;
  // the loaders address cache rows in 32-bit units of 16 bytes
  const int64_t extent = (p->page_size ? p->kv_rows : (int64_t)p->batch) * p->kv_stride_b;
  if (extent / 8 >= (int64_t)0xFFFFFFFFll) return false;
  return true;
}

quoka_status launch_attn_tc(const quoka_params* p, const DevParams& P, const void* q, const void* k, const void* v,
                            const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, cudaStream_t st) {
  CUtensorMap tm_q;
  {
    const uint64_t dims[4] = {(uint64_t)P.d, (uint64_t)P.chunk, (uint64_t)P.n_q, (uint64_t)P.batch};
    const uint64_t strides[3] = {(uint64_t)P.q_st * 2, (uint64_t)P.q_sh * 2, (uint64_t)P.q_sb * 2};
    const uint32_t box[4] = {64, 128, 1, 1};
    if (!encode_tensor_map_bf16(&tm_q, q, 4, dims, strides, box)) return QUOKA_ERR_CUDA;
  }
  const int halves = P.d / 64;
  const size_t tile = (size_t)halves * 128 * 128;
  const size_t smem = 1024 + (2 + kSlots) * tile + 512;
  dim3 grid(P.n_q, (P.chunk + 2 * kQTile - 1) / (2 * kQTile), P.batch);
  const bool sparse = k_idx != nullptr;
  cudaError_t e = cudaSuccess;
#define QUOKA_ATTN_TC(H, S)                                                                                      \
  do {                                                                                                           \
    e = cudaFuncSetAttribute(attn_tc_kernel<H, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);      \
    if (e != cudaSuccess) return QUOKA_ERR_CUDA;                                                                 \
    attn_tc_kernel<H, S><<<grid, kAttnThreads, smem, st>>>(P, tm_q, (const __nv_bfloat16*)k,                     \
                                                           (const __nv_bfloat16*)v, k_idx, k_cnt,                \
                                                           (__nv_bfloat16*)out, lse);                            \
  } while (0)
  if (halves == 2) { if (sparse) QUOKA_ATTN_TC(2, true); else QUOKA_ATTN_TC(2, false); }
  else { if (sparse) QUOKA_ATTN_TC(1, true); else QUOKA_ATTN_TC(1, false); }
#undef QUOKA_ATTN_TC
  count_launch();
  return cudaGetLastError() == cudaSuccess ? QUOKA_OK : QUOKA_ERR_CUDA;
}

}  // namespace quoka
