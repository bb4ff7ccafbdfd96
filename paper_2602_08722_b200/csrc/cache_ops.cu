// Appending a chunk's keys and values to the cache (Algorithm 2, "append K_i, V_i to the cache").
//
// The chunk's K_i, V_i arrive dense, [b][n_KV][C][d]; row r of (sequence s, KV head h) goes to cache row
// T_s + r, whose address comes from the strides or, in a paged cache, from the block table.  T_s is read on
// the device, so a loop over chunks needs no host round trip.  One thread moves 16 bytes of K and the same 16
// bytes of V; a warp covers whole rows, so both the reads and the writes are full-width.  HBM-bound:
// 2 * b * n_KV * C * d * es bytes read and as many written.
#include "common.cuh"

namespace quoka {

template <int ES>   // element size in bytes
__global__ void __launch_bounds__(256) append_kv_kernel(DevParams P, const uint4* __restrict__ k_new,
                                                         const uint4* __restrict__ v_new, uint4* __restrict__ k_cache,
                                                         uint4* __restrict__ v_cache) {
  const int wpr = P.d * ES / 16;                                     // 16-byte words per row
  const int64_t total = (int64_t)P.batch * P.n_kv * P.chunk * wpr;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int w = (int)(e % wpr);
    const int64_t row = e / wpr;
    const int r = (int)(row % P.chunk);
    const int h = (int)((row / P.chunk) % P.n_kv);
    const int s = (int)(row / ((int64_t)P.chunk * P.n_kv));
    const int T = __ldg(P.ctx_len + s);
    const int64_t dst = kv_row_offset(P, s, h, T + r) * ES / 16 + w;   // strides are multiples of 8 elements
    k_cache[dst] = __ldg(k_new + e);
    v_cache[dst] = __ldg(v_new + e);
  }
}

cudaError_t launch_append_kv(const DevParams& P, int dtype, const void* k_new, const void* v_new, void* k_cache,
                             void* v_cache, cudaStream_t st) {
  const int es = dtype == QUOKA_BF16 ? 2 : 4;
  const int64_t total = (int64_t)P.batch * P.n_kv * P.chunk * (P.d * es / 16);
  if (total <= 0) return cudaSuccess;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  log_launch("append_kv", dim3((unsigned)blocks), dim3(256), 0, 1, false);
  if (es == 2)
    append_kv_kernel<2><<<(unsigned)blocks, 256, 0, st>>>(P, (const uint4*)k_new, (const uint4*)v_new, (uint4*)k_cache, (uint4*)v_cache);
  else
    append_kv_kernel<4><<<(unsigned)blocks, 256, 0, st>>>(P, (const uint4*)k_new, (const uint4*)v_new, (uint4*)k_cache, (uint4*)v_cache);
  count_launch();
  return cudaGetLastError();
}

}  // namespace quoka
