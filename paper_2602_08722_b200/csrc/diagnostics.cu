// Diagnostics: launch-geometry logging (QUOKA_LOG=1), the host-side block-table check, and a self-test of the
// bounded device wait that every tensor-core kernel relies on.
#include <cstdio>
#include <cstdlib>
#include <vector>

#include "sm100_ptx.cuh"
#include "common.cuh"

namespace quoka {

bool log_enabled() {
  static const bool on = []() {
    const char* e = std::getenv("QUOKA_LOG");
    return e && e[0] && e[0] != '0';
  }();
  return on;
}

void log_launch(const char* kernel, dim3 grid, dim3 block, size_t smem, int cluster, bool chained) {
  if (!log_enabled()) return;
  std::fprintf(stderr, "[quoka] %-28s grid (%u,%u,%u) block %u smem %zu B cluster %d%s\n", kernel, grid.x, grid.y, grid.z,
               block.x, smem, cluster, chained ? " programmatic-launch" : "");
}

// One warp waits on an mbarrier that nobody ever arrives on.  The wait must give up after `limit` cycles, record
// QUOKA_ERR_TIMEOUT in the status word and return; the CTA then leaves normally.  No copy engine, tensor core
// or tensor memory is involved, so nothing is in flight when the wait runs out.
__global__ void __launch_bounds__(32) wait_timeout_selftest_kernel(int32_t* status, long long limit, int32_t* gave_up) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(&bar, 1);
    ptx::fence_mbar_init();
  }
  __syncwarp();
  const ptx::WaitCtx wc{&abort_flag, status, limit};
  const bool ok = ptx::mbar_wait(&bar, 0, wc);
  if (threadIdx.x == 0) *gave_up = ok ? 0 : 1;
}

// SMs of the current device (looked up once per process).
int device_sm_count() {
  static int n = []() {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return v;
  }();
  return n;
}

}  // namespace quoka

using namespace quoka;

extern "C" {

quoka_status quoka_selftest_wait_timeout(void* ws, int64_t limit_cycles, int32_t* gave_up, void* stream) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0) return QUOKA_ERR_WORKSPACE;
  if (!gave_up || limit_cycles <= 0 || limit_cycles > 2000000000LL) return QUOKA_ERR_INVALID_ARG;
  log_launch("wait_timeout_selftest", dim3(1), dim3(32), 0, 1, false);
  wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<int32_t*>(ws),
                                                                                 (long long)limit_cycles, gave_up);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? QUOKA_OK : QUOKA_ERR_CUDA;
}

quoka_status quoka_check_block_table(const quoka_params* p, const int32_t* ctx_len_host,
                                     const int32_t* block_table_host) {
  if (!p || !ctx_len_host || !block_table_host) return QUOKA_ERR_INVALID_ARG;
  if (p->page_size != kPage || p->batch <= 0 || p->max_pages_per_seq <= 0 || p->kv_rows <= 0 || p->chunk_len <= 0)
    return QUOKA_ERR_INVALID_ARG;
  std::vector<unsigned char> used((size_t)p->kv_rows, 0);
  for (int s = 0; s < p->batch; ++s) {
    const int64_t T = ctx_len_host[s];
    if (T < 0 || T > p->max_ctx_len) return QUOKA_ERR_INVALID_ARG;
    const int64_t pages = (T + p->chunk_len + kPage - 1) / kPage;
    if (pages > p->max_pages_per_seq) return QUOKA_ERR_INVALID_ARG;
    for (int64_t i = 0; i < pages; ++i) {
      const int32_t page = block_table_host[(int64_t)s * p->max_pages_per_seq + i];
      if (page < 0 || page >= p->kv_rows) return QUOKA_ERR_INVALID_ARG;      // outside the pool
      if (used[(size_t)page]) return QUOKA_ERR_INVALID_ARG;                    // two logical pages on one physical page
      used[(size_t)page] = 1;
    }
  }
  return QUOKA_OK;
}

}  // extern "C"
