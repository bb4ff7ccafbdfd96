// Shared device-side definitions for the QuoKA kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "quoka.h"

namespace quoka {

constexpr float kNormEps = 1e-12f;
constexpr int kPage = 64;

// Device copy of the launch-invariant part of quoka_params.
struct DevParams {
  int batch, n_q, n_kv, group, d;
  int chunk;        // C
  int n_sel;        // N = min(N_Q, C)
  int n_retain;     // N_Q as given
  int kv_budget;    // B_SA or <= 0
  float budget_frac;
  float scale;      // softmax scale
  int max_ctx;
  int budget_cap;   // row pitch of k_idx
  const int32_t* ctx_len;
  int64_t q_sb, q_sh, q_st;
  int64_t o_sb, o_sh, o_st;
  int page_size, max_pages;
  const int32_t* block_table;
  int64_t kv_sb, kv_sh, kv_st;
  int32_t* status;  // device status word
  int score_dot;    // 1: raw dot products (no normalisation of queries or keys)
  int agg_mean;     // 1: mean over the retained queries instead of the maximum
  const float* k_inv_norm;  // cached 1/|k| per cache row, or null
  int64_t kv_rows;  // rows per (sequence, head) when contiguous
  // split attention (small grids): room for the parts' partial results and their arrival counters, or null
  float* attn_partials;
  int32_t* attn_counters;
  int attn_parts;   // parts per row block of the launch at hand (set by the launcher), 1 = no split
};

// B_s of one sequence: min(B_SA, T) or floor(frac*T + 0.5) in double.
__host__ __device__ inline int key_budget(int T, int kv_budget, float frac) {
  if (kv_budget > 0) return kv_budget < T ? kv_budget : T;
  int B = (int)floor((double)frac * (double)T + 0.5);
  if (B < 0) B = 0;
  return B < T ? B : T;
}

// Element offset of row t of (sequence s, KV head h) in a contiguous or paged cache.
__device__ __forceinline__ int64_t kv_row_offset(const DevParams& P, int s, int h, int t) {
  if (P.page_size == 0) return (int64_t)s * P.kv_sb + (int64_t)h * P.kv_sh + (int64_t)t * P.kv_st;
  const int page = __ldg(P.block_table + (int64_t)s * P.max_pages + (t >> 6));
  return (int64_t)page * P.kv_sb + (int64_t)h * P.kv_sh + (int64_t)(t & (kPage - 1)) * P.kv_st;
}

// Index of row t of (sequence s, KV head h) in the cached inverse-norm array (the cache's layout without head_dim).
__device__ __forceinline__ int64_t kv_norm_index(const DevParams& P, int s, int h, int t) {
  if (P.page_size == 0) return ((int64_t)s * P.n_kv + h) * P.kv_rows + t;
  const int page = __ldg(P.block_table + (int64_t)s * P.max_pages + (t >> 6));
  return ((int64_t)page * P.n_kv + h) * kPage + (t & (kPage - 1));
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Load NE consecutive elements (NE*sizeof(T) is 8, 16 or 32 bytes, pointer aligned to min(16, that)) as floats.
template <typename T, int NE>
__device__ __forceinline__ void load_vec(const T* __restrict__ p, float (&out)[NE]) {
  if constexpr (sizeof(T) == 4) {
    if constexpr (NE % 4 == 0) {
#pragma unroll
      for (int i = 0; i < NE / 4; ++i) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(p) + i);
        out[4 * i + 0] = v.x; out[4 * i + 1] = v.y; out[4 * i + 2] = v.z; out[4 * i + 3] = v.w;
      }
    } else {
      static_assert(NE % 2 == 0, "NE");
#pragma unroll
      for (int i = 0; i < NE / 2; ++i) {
        const float2 v = __ldg(reinterpret_cast<const float2*>(p) + i);
        out[2 * i] = v.x; out[2 * i + 1] = v.y;
      }
    }
  } else {
    if constexpr (NE % 8 == 0) {
#pragma unroll
      for (int i = 0; i < NE / 8; ++i) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(p) + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          out[8 * i + 2 * j] = __uint_as_float(w[j] << 16);
          out[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
        }
      }
    } else if constexpr (NE % 4 == 0) {
#pragma unroll
      for (int i = 0; i < NE / 4; ++i) {
        const uint2 v = __ldg(reinterpret_cast<const uint2*>(p) + i);
        out[4 * i + 0] = __uint_as_float(v.x << 16); out[4 * i + 1] = __uint_as_float(v.x & 0xFFFF0000u);
        out[4 * i + 2] = __uint_as_float(v.y << 16); out[4 * i + 3] = __uint_as_float(v.y & 0xFFFF0000u);
      }
    } else {
      static_assert(NE % 2 == 0, "NE");
#pragma unroll
      for (int i = 0; i < NE / 2; ++i) {
        const uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(p) + i);
        out[2 * i] = __uint_as_float(v << 16); out[2 * i + 1] = __uint_as_float(v & 0xFFFF0000u);
      }
    }
  }
}

template <typename T, int NE>
__device__ __forceinline__ void store_vec(T* __restrict__ p, const float (&v)[NE]) {
#pragma unroll
  for (int i = 0; i < NE; ++i) p[i] = from_f32<T>(v[i]);
}

// Monotone map float -> uint32 (ascending); -0 and +0 map to the same code.
__device__ __forceinline__ uint32_t float_order_key(float f) {
  uint32_t b = __float_as_uint(f);
  if ((b << 1) == 0) b = 0;
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Inverse of float_order_key.
__device__ __forceinline__ float order_key_to_float(uint32_t c) {
  return __uint_as_float((c & 0x80000000u) ? (c & 0x7FFFFFFFu) : ~c);
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
  return x;
}

// ---- programmatic dependent launch ------------------------------------------------------------------
// The kernels of one fused call form a chain on one stream, each reading what the one before it wrote.  A kernel
// launched with programmatic stream serialisation may become resident while the kernel before it still runs;
// it must then execute grid_dependency_wait() before its first access to anything that kernel writes (the wait
// returns once that grid has completed and its writes are visible; without the launch attribute it returns at
// once).  A kernel lets the one after it start early with grid_launch_dependents(), which every CTA executes at
// its start; the dependent grid is launched when all of them have, so it never holds resources that this
// grid's own CTAs still need.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launch with optional thread-block cluster width and, if `chained`, programmatic stream serialisation.
void log_launch(const char* kernel, dim3 grid, dim3 block, size_t smem, int cluster, bool chained);
int device_sm_count();

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(const char* name, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t st, int cluster, bool chained, Args&&... args) {
  log_launch(name, grid, block, smem, cluster, chained);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (chained) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- launch functions implemented in the .cu files (host side) -------------------------------
// `chained`: the kernel before it on the stream is the one of the same fused call whose output it reads (see above).
cudaError_t launch_rank_queries(const DevParams& P, int dtype, const void* q, int32_t* q_idx, cudaStream_t st);
cudaError_t launch_aggregate_queries(const DevParams& P, int dtype, const void* q, int32_t* q_idx, void* qbar,
                                     cudaStream_t st, bool chained = false);
cudaError_t launch_score_keys_simt(const DevParams& P, int dtype, const void* qbar, const void* k, float* scores,
                                   cudaStream_t st);
cudaError_t launch_key_norms(const DevParams& P, int dtype, const void* k, float* k_inv_norm, int all_rows,
                             cudaStream_t st);
cudaError_t launch_select_keys(const DevParams& P, const float* scores, int32_t* k_idx, int32_t* k_cnt,
                               cudaStream_t st, bool chained = false);
cudaError_t launch_attn_simt(const DevParams& P, int dtype, const void* q, const void* k, const void* v,
                             const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, cudaStream_t st);

// Generation phase (chunk of one query): matrix-vector scoring and a gather attention kernel.
bool decode_path_applies(const DevParams& P);
bool decode_attn_fits(const DevParams& P, bool with_list);
cudaError_t launch_score_keys_gemv(const DevParams& P, int dtype, const void* qbar, const void* k, float* scores,
                                   cudaStream_t st, bool chained);
cudaError_t launch_decode_attn(const DevParams& P, int dtype, const void* q, const void* k, const void* v,
                               const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, cudaStream_t st,
                               bool chained);
cudaError_t launch_append_kv(const DevParams& P, int dtype, const void* k_new, const void* v_new, void* k_cache,
                             void* v_cache, cudaStream_t st);

// Host checks shared by the fused entry points (everything but the workspace); nothing is enqueued before they pass.
quoka_status check_prefill_args(const quoka_params* p, const void* q, const void* k_cache, const void* v_cache,
                                const void* out);
// the fused call behind quoka_prefill_chunk, and its workspace need, with or without the split-attention scratch
quoka_status prefill_chunk_impl(const quoka_params* p, const void* q, const void* k_cache, const void* v_cache, void* out,
                                int32_t* k_idx_out, int32_t* k_cnt_out, void* ws, size_t ws_bytes, void* stream,
                                bool with_split);
size_t workspace_bytes(const quoka_params* p, bool with_split);
// Device address of the built-in scratch array on the current device (looked up once per device).
quoka_status static_scratch_for_current_device(void** out);

void count_launch(int n = 1);
// QUOKA_LOG=1 in the environment: one line per kernel launch (grid, block, shared memory) on stderr.
bool log_enabled();
void log_launch(const char* kernel, dim3 grid, dim3 block, size_t smem, int cluster, bool chained);

}  // namespace quoka
