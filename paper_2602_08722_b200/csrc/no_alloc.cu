// quoka_prefill_chunk_static: the fused per-chunk call for callers that cannot hand the library a
// workspace because they cannot allocate device memory at all.
//
// Who that is: a serving process that gave every free byte of HBM to its KV-cache pool at start-up
// (any later cudaMalloc fails or forces the pool to shrink), and code on a latency-critical path
// where cudaMalloc / cudaFree are off limits because they synchronise the whole device.  For them the
// intermediates of the chunk (retained-query ranks, Qbar, key scores, selected indices) live in a
// fixed array that is part of the library image: every GPU that loads the library holds
// QUOKA_STATIC_SCRATCH_BYTES of it until the process exits, whether or not this entry point is used.
#include <mutex>

#include "common.cuh"

namespace quoka {

static __device__ __align__(256) unsigned char g_static_scratch[QUOKA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static std::mutex g_setup_mutex;
static void* g_scratch_addr[kMaxDevices] = {};

// The array's name is only a host-side handle; the address kernels can use has to be asked for,
// once per device, with that device current.  The address is remembered for the life of the
// process: after cudaDeviceReset (or any teardown of the device's primary context) it is stale,
// and this entry point must not be used again in that process.
quoka_status static_scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return QUOKA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return QUOKA_ERR_CUDA;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return QUOKA_OK;
}

}  // namespace quoka

extern "C" quoka_status quoka_prefill_chunk_static(const quoka_params* p, const void* q, const void* k_cache,
                                                   const void* v_cache, void* out, int32_t* k_idx_out,
                                                   int32_t* k_cnt_out, void* stream) {
  // every host-side refusal comes before the first thing put on the stream (the memset below)
  quoka_status st = quoka::check_prefill_args(p, q, k_cache, v_cache, out);
  if (st != QUOKA_OK) return st;
  // the array has no room for the scratch of the split attention kernel: small grids run unsplit here
  if (quoka::workspace_bytes(p, /*with_split=*/false) > (size_t)QUOKA_STATIC_SCRATCH_BYTES) return QUOKA_ERR_STATIC_LIMIT;
  void* scratch = nullptr;
  if ((st = quoka::static_scratch_for_current_device(&scratch)) != QUOKA_OK) return st;
  // The array keeps whatever the previous call left.  Only the status word has to start at zero;
  // everything else is written before it is read.
  if (cudaMemsetAsync(scratch, 0, 256, static_cast<cudaStream_t>(stream)) != cudaSuccess) return QUOKA_ERR_CUDA;
  return quoka::prefill_chunk_impl(p, q, k_cache, v_cache, out, k_idx_out, k_cnt_out, scratch,
                                   (size_t)QUOKA_STATIC_SCRATCH_BYTES, stream, /*with_split=*/false);
}
