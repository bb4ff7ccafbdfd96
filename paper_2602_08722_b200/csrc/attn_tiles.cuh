// Pieces shared by the tensor-core attention kernels: tile geometry of a CTA's walk over the key tiles,
// the rows a tile holds, the causal limit, and small softmax helpers.
#pragma once

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
// The reference point m of the exponentials 2^(s - m) is raised, and O and l rescaled, only when a row's maximum
// exceeds it by more than this many powers of two.  Until then P, l and O are simply larger by a common factor of at
// most 2^32, which floating point carries without loss (bf16 and fp32 both reach 2^127; l <= 2^32 * keys and
// |O| <= l * max|v| stay far below that); the quotient O / l does not change.  With 8 the rescale (a read-modify-
// write of the whole accumulator row on the softmax -> PV chain) still ran often enough to cost 1-2 % of the kernel.
constexpr float kRescaleThreshold = 32.0f;   // log2 units

bool encode_kv_tensor_map(CUtensorMap* out, const quoka_params* p, const void* cache, uint32_t box_rows);

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Every CTA walks ONE sequence of key tiles t = 0 .. n_total-1 for both of its Q tiles; Q tile x takes part in
// the tiles t >= skip[x] (a suffix, so both finish on the same tile).
//   dense : the tiles of rows [0, T + C) in DESCENDING order (the tiles only Q tile B sees come first).
//   sparse: first the chunk's own tiles (the one only B sees, then tiles 0 .. c_a-1), THEN the tiles of the
//           selected list.  The chunk's tiles do not depend on the key selection, so this kernel is launched
//           with programmatic stream serialisation: it starts while the selection kernel still runs, works
//           through the chunk tiles, and only then waits for the selection (`resolve`) to learn the list length.
struct AttnGeom {
  int T, C;
  int n_chunk;        // sparse: tiles of the chunk's own rows in the sequence; dense: 0
  int c_a;            // sparse: chunk tiles Q tile A sees
  int b_first;        // sparse: 1 when the sequence starts with the tile only B sees
  int skip_a;         // first tile Q tile A takes part in (B takes part in all); scalars, not arrays: the struct
  bool active_b;      // must live in registers (an indexed member would put it in local memory)
  int n_known;        // tiles known so far (sparse: n_chunk until resolved, then n_chunk + n_sel)
  int cnt;            // sparse: selected rows (valid once resolved)
  int n_dense;        // dense: number of tiles
  bool resolved;
};

template <bool SPARSE>
__device__ __forceinline__ AttnGeom make_geom(const DevParams& P, int s, int r0) {
  AttnGeom g;
  g.T = __ldg(P.ctx_len + s);
  g.C = P.chunk;
  const bool b_active = r0 + kQTile < g.C;
  g.active_b = b_active;
  g.cnt = 0;
  if (SPARSE) {
    g.c_a = r0 / kQTile + 1;
    g.b_first = b_active ? 1 : 0;
    g.n_chunk = g.c_a + g.b_first;
    g.skip_a = g.b_first;
    g.n_known = g.n_chunk;
    g.n_dense = 0;
    g.resolved = false;
  } else {
    const int last_a = min(r0 + kQTile - 1, g.C - 1), last_b = min(r0 + 2 * kQTile - 1, g.C - 1);
    const int n_a = (g.T + last_a) / kKeyTile + 1;
    const int n_b = b_active ? (g.T + last_b) / kKeyTile + 1 : 0;
    g.n_dense = max(n_a, n_b);
    g.skip_a = g.n_dense - n_a;
    g.n_chunk = 0; g.c_a = 0; g.b_first = 0;
    g.n_known = g.n_dense;
    g.resolved = true;
  }
  return g;
}

// Sparse: wait for the selection kernel (a no-op when this kernel was not launched early) and read the list length.
__device__ __forceinline__ void resolve(AttnGeom& g, const int32_t* k_cnt, int s) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  g.cnt = __ldcg(k_cnt + s);
  g.n_known = g.n_chunk + (g.cnt + kKeyTile - 1) / kKeyTile;
  g.resolved = true;
}

// Rows of tile t: from the selected list (`from_list`, rows list[base .. base + count)), or the consecutive cache
// rows first .. first + count - 1.  `diag` = chunk position of the tile's first row minus one tile-relative
// offset, used by the causal limit: row r sees columns [0, r - col0 + 1).
struct TileRows {
  bool from_list;       // addressing: rows list[first .. first + count), else the consecutive cache rows first ..
  bool causal;          // masking: row r sees columns [0, r - col0 + 1), else columns [0, count)
  int first, count;     // consecutive rows (count may exceed the tile or be <= 0), or list base and remaining count
  int col0;             // causal tiles: chunk position (dense: position in [0, T + C)) of column 0
};

template <bool SPARSE>
__device__ __forceinline__ TileRows tile_rows(const AttnGeom& g, int t) {
  TileRows r;
  if (SPARSE) {
    if (t < g.n_chunk) {
      const int ct = g.b_first ? (t == 0 ? g.c_a : t - 1) : t;
      r.from_list = false;
      r.causal = true;
      r.first = g.T + ct * kKeyTile;
      r.count = g.C - ct * kKeyTile;
      r.col0 = ct * kKeyTile;
    } else {
      // a list as long as the cache is the identity (the budget covers the cache): its tiles are plain row ranges
      const int st = t - g.n_chunk;
      r.from_list = g.cnt != g.T;
      r.causal = false;
      r.first = st * kKeyTile;
      r.count = g.cnt - st * kKeyTile;
      r.col0 = 0;
    }
  } else {
    const int j = g.n_dense - 1 - t;
    r.from_list = false;
    r.causal = true;
    r.first = j * kKeyTile;
    r.count = g.T + g.C - j * kKeyTile;
    r.col0 = j * kKeyTile - g.T;            // chunk position of column 0 (negative inside the cache)
  }
  return r;
}

// Number of visible columns of tile t for chunk row `row` (columns [0, lim) are visible).
__device__ __forceinline__ int visible_cols(const TileRows& tr, int row) {
  const int lim = tr.causal ? row - tr.col0 + 1 : tr.count;
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

// ---------------------------------------------------------------------------------------------- softmax of one tile
// One thread = one query row of a 128-row Q tile against one 128-key tile: S is read from tensor memory at s_addr,
// bf16 P written back over its first 64 columns, the running reference point m_run (log2 units) and sum l_run kept
// up, the accumulator at o_addr rescaled when the reference point moves.  `lim` = visible columns of this row,
// `masked` = some row of the warp sees fewer than all; `announce(half)` (lane 0) tells the MMA issuer that a half of
// P is in place.  first_tile: nothing has been accumulated yet.
template <int D, typename Announce>
__device__ __forceinline__ void attn_softmax_tile(uint32_t s_addr, uint32_t o_addr, int lim, bool masked, float scale_log2,
                                                  bool first_tile, int lane, float& m_run, float& l_run,
                                                  Announce&& announce) {
  // ---- pass 1: the row maximum.  All four 32-column loads are issued together (one tensor-memory round
  // trip).  The first 96 scores stay in registers for pass 2, the last 32 are read once more there (under the
  // third block's exponentials): all 128 alive next to a block of exponentials in flight do not fit the 168
  // registers, and 96 fit only because P is stored 16 columns at a time and the rare rescale below works in
  // 8-column pieces.
  float mx;
  uint32_t v0[96];                                         // the first 96 scores stay in registers for pass 2
  {
    uint32_t c3[32];
    tmem_ld32(s_addr, v0);
    tmem_ld32(s_addr + 32, v0 + 32);
    tmem_ld32(s_addr + 64, v0 + 64);
    tmem_ld32(s_addr + 96, c3);
    tmem_wait_ld();
    uint32_t (&a0)[32] = *reinterpret_cast<uint32_t (*)[32]>(v0);
    uint32_t (&a1)[32] = *reinterpret_cast<uint32_t (*)[32]>(v0 + 32);
    uint32_t (&a2)[32] = *reinterpret_cast<uint32_t (*)[32]>(v0 + 64);
    mx = fmaxf(fmaxf(max32(a0, masked, 0, lim), max32(a1, masked, 32, lim)),
               fmaxf(max32(a2, masked, 64, lim), max32(c3, masked, 96, lim)));
  }
  const float m_tile = mx * scale_log2;
  // ---- lazy rescale of the accumulator: only when some row's maximum grew by more than the threshold
  const bool grow = m_tile > m_run + kRescaleThreshold;
  if (__any_sync(0xFFFFFFFFu, grow)) {
    const float m_new = fmaxf(m_run, m_tile);
    if (!first_tile) {
      const float alpha = (m_run == -INFINITY) ? 0.f : ex2(m_run - m_new);
      l_run *= alpha;
#pragma unroll 1
      for (int c = 0; c < D / 8; ++c) {                       // rare: small pieces, few registers
        uint32_t r[8];
        tmem_ld8(o_addr + c * 8, r);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 8; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
        tmem_st8(o_addr + c * 8, r);
      }
      tmem_wait_st();
    }
    m_run = m_new;
  }
  const float m_use = (m_run == -INFINITY) ? 0.f : m_run;
  // ---- pass 2: p = 2^(s*scale - m) in four blocks of 32 keys.  bf16 P goes over the first 64 columns of S
  // (block b of P lands on columns 16b..16b+15, all of them read already) and each half of the tile is handed to
  // the MMA issuer as soon as it is stored, so the first PV products run under the second half's arithmetic.
  const uint64_t sc2 = pack2(scale_log2, scale_log2), nm2 = pack2(-m_use, -m_use);
  uint64_t psa[2] = {0ull, 0ull};                           // four running sums as two packed pairs
  uint32_t vb[32];
#pragma unroll
  for (int blk = 0; blk < 4; ++blk) {
    if (blk == 2) tmem_ld32(s_addr + 96, vb);              // under the third block's exponentials
    if (blk == 3) {
      tmem_wait_ld();
      if (masked) {
#pragma unroll
        for (int i = 0; i < 32; ++i) if (96 + i >= lim) vb[i] = 0xFF800000u;   // -inf: exp2 gives exactly 0
      }
    }
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint32_t e0 = blk < 3 ? v0[blk * 32 + 2 * i] : vb[2 * i], e1 = blk < 3 ? v0[blk * 32 + 2 * i + 1] : vb[2 * i + 1];
      float x0, x1;
      unpack2(fma2(pack2u(e0, e1), sc2, nm2), x0, x1);
      const float p0 = ex2(x0), p1 = ex2(x1);
      psa[i & 1] = add2(psa[i & 1], pack2(p0, p1));
      const __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);
      pk[i] = *reinterpret_cast<const uint32_t*>(&b2);
    }
    tmem_st16(s_addr + blk * 16, pk);
    if (blk & 1) {
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) announce(blk >> 1);
    }
  }
  float ps0, ps1, ps2, ps3;
  unpack2(psa[0], ps0, ps1);
  unpack2(psa[1], ps2, ps3);
  l_run += (ps0 + ps1) + (ps2 + ps3);
}

// Epilogue of a softmax thread: its row of O from tensor memory, divided by l, to global memory as bf16 (and the
// row's log-sum-exp when asked for).
template <int D>
__device__ __forceinline__ void attn_store_row(const DevParams& P, uint32_t o_addr, float m_run, float l_run, int s, int h,
                                               int row, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
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

// ---------------------------------------------------------------------------------------------- split attention
// A launch whose grid is far smaller than the GPU cuts every row block's key tiles into parts, one CTA (pair) each.
constexpr int kSplitTileFloats = 130 * 128;     // one part's partial result of a 128-row Q tile

// Epilogue of a softmax warp of a split launch.
template <int D>
__device__ __forceinline__ void attn_split_epilogue(const DevParams& P, int job, int part, int n_parts, int x, int quarter,
                                                    int lane, int row_in_tile, int row, bool have, uint32_t o_addr,
                                                    float m_run, float l_run, int s, int h, __nv_bfloat16* out,
                                                    float* lse) {
  // ---- this part's partial result (reference point m, sum l, un-normalised O; a part without tiles for this
  // Q tile leaves m = -inf), then the merge by whichever part's warp arrives last.  One counter per (row block
  // of a head, softmax warp); nobody waits for anybody.  The parts are added up in part order, so the result
  // does not depend on which part came last.
  constexpr int kTile = kSplitTileFloats;                   // [D columns of O | m | l][128 rows], D <= 128
  float* tile0 = P.attn_partials + ((size_t)job * n_parts * 2 + x) * kTile;
  float* mine = tile0 + (size_t)part * 2 * kTile;
  if (have) {
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
      uint32_t r[32];
      tmem_ld32(o_addr + c * 32, r);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) mine[(c * 32 + i) * 128 + row_in_tile] = __uint_as_float(r[i]);
    }
  }
  mine[D * 128 + row_in_tile] = have ? m_run : -INFINITY;
  mine[(D + 1) * 128 + row_in_tile] = have ? l_run : 0.f;
  __threadfence();
  __syncwarp();
  int32_t* counter = P.attn_counters + (job * 2 + x) * 4 + quarter;
  int arrived = 0;
  if (lane == 0) arrived = atomicAdd(counter, 1);
  arrived = __shfl_sync(0xFFFFFFFFu, arrived, 0);
  if (arrived == n_parts - 1) {
    if (lane == 0) *counter = 0;                            // as the next launch expects it
    __threadfence();
    float wgt[8];
    float M = -INFINITY;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      wgt[q] = q < n_parts ? __ldcg(tile0 + (size_t)q * 2 * kTile + D * 128 + row_in_tile) : -INFINITY;
      M = fmaxf(M, wgt[q]);
    }
    float l = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float w = wgt[q] == -INFINITY ? 0.f : ex2(wgt[q] - M);
      if (q < n_parts) l += w * __ldcg(tile0 + (size_t)q * 2 * kTile + (D + 1) * 128 + row_in_tile);
      wgt[q] = w;
    }
    const float inv = 1.f / l;
    const bool store = row < P.chunk;
    __nv_bfloat16* orow = out + (long long)s * P.o_sb + (long long)h * P.o_sh + (long long)row * P.o_st;
#pragma unroll 1
    for (int c = 0; c < D / 32; ++c) {
      float acc[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) acc[i] = 0.f;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        if (q < n_parts && wgt[q] != 0.f) {
          const float* src = tile0 + (size_t)q * 2 * kTile + (c * 32) * 128 + row_in_tile;
#pragma unroll
          for (int i = 0; i < 32; ++i) acc[i] = fmaf(wgt[q], __ldcg(src + i * 128), acc[i]);
        }
      }
      if (store) {
#pragma unroll
        for (int v4 = 0; v4 < 4; ++v4) {
          uint32_t w[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 b2 = __floats2bfloat162_rn(acc[v4 * 8 + 2 * i] * inv, acc[v4 * 8 + 2 * i + 1] * inv);
            w[i] = *reinterpret_cast<const uint32_t*>(&b2);
          }
          *reinterpret_cast<uint4*>(orow + c * 32 + v4 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
    }
    if (store && lse) lse[((long long)s * P.n_q + h) * P.chunk + row] = (M + log2f(l)) * 0.6931471805599453f;
  }
}

}  // namespace quoka
