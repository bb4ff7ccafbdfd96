// Host side of the C ABI: argument validation, workspace carving, launch sequencing.
// Nothing here allocates device memory or synchronises (except quoka_last_device_status).
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>

#include <mutex>

#include "common.cuh"
#include "tensor_kernels.cuh"

namespace quoka {

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

struct Workspace {
  int32_t* status;
  int32_t* q_idx;
  void* qbar;
  float* scores;
  int32_t* k_idx;
  int32_t* k_cnt;
  float* attn_partials;      // split attention of small grids: partial results and arrival counters, or null
  int32_t* attn_counters;
  size_t total;
};

static int budget_cap_of(const quoka_params* p) {
  int cap = key_budget(p->max_ctx_len, p->kv_budget, p->budget_frac);
  return cap < 1 ? 1 : cap;
}

// Parts the attention kernels may cut a row block into for this problem (the larger of the sparse and the dense call's).
static int attn_parts_bound(const quoka_params* p) {
  if (p->impl == QUOKA_IMPL_SIMT || p->chunk_len <= 1) return 1;
  const int cap = budget_cap_of(p);
  const int sparse = attn_split_parts(p, (cap + 127) / 128 + 1), dense = attn_split_parts(p, (p->max_ctx_len + 127) / 128 + 1);
  return sparse > dense ? sparse : dense;
}

// with_split = false: the layout without the split-attention scratch (every call still works, small grids unsplit)
static Workspace carve(const quoka_params* p, void* ws, bool with_split = true) {
  Workspace w{};
  const size_t es = p->dtype == QUOKA_BF16 ? 2 : 4;
  const int N = p->n_retain < p->chunk_len ? p->n_retain : p->chunk_len;
  const int cap = budget_cap_of(p);
  char* base = static_cast<char*>(ws);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    char* r = base ? base + off : nullptr;
    off += align_up(bytes);
    return r;
  };
  w.status = reinterpret_cast<int32_t*>(take(256));
  w.q_idx = reinterpret_cast<int32_t*>(take((size_t)p->batch * p->n_q_heads * N * 4));
  w.qbar = take((size_t)p->batch * p->n_kv_heads * N * p->head_dim * es);
  w.scores = reinterpret_cast<float*>(take((size_t)p->batch * p->n_kv_heads * (size_t)(p->max_ctx_len > 0 ? p->max_ctx_len : 1) * 4));
  w.k_idx = reinterpret_cast<int32_t*>(take((size_t)p->batch * p->n_kv_heads * cap * 4));
  w.k_cnt = reinterpret_cast<int32_t*>(take((size_t)p->batch * 4));
  const int parts = with_split ? attn_parts_bound(p) : 1;
  if (parts > 1) {
    w.attn_counters = reinterpret_cast<int32_t*>(take(attn_split_counter_bytes(p)));
    w.attn_partials = reinterpret_cast<float*>(take(attn_split_partial_bytes(p, parts)));
  }
  w.total = off;
  return w;
}

static quoka_status validate(const quoka_params* p) {
  if (!p) return QUOKA_ERR_INVALID_ARG;
  if (p->batch <= 0 || p->n_q_heads <= 0 || p->n_kv_heads <= 0 || p->chunk_len <= 0 || p->n_retain <= 0)
    return QUOKA_ERR_INVALID_ARG;
  if (p->n_q_heads % p->n_kv_heads != 0) return QUOKA_ERR_INVALID_ARG;
  if (p->max_ctx_len < 0 || !p->ctx_len) return QUOKA_ERR_INVALID_ARG;
  if (p->kv_budget <= 0 && !(p->budget_frac >= 0.f && p->budget_frac <= 1.f)) return QUOKA_ERR_INVALID_ARG;
  if (p->dtype != QUOKA_BF16 && p->dtype != QUOKA_F32) return QUOKA_ERR_INVALID_ARG;
  if (p->impl < QUOKA_IMPL_AUTO || p->impl > QUOKA_IMPL_TENSOR) return QUOKA_ERR_INVALID_ARG;
  if (p->score_mode < QUOKA_SCORE_COSINE || p->score_mode > QUOKA_SCORE_DOT) return QUOKA_ERR_INVALID_ARG;
  if (p->query_agg < QUOKA_AGG_MAX || p->query_agg > QUOKA_AGG_MEAN) return QUOKA_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return QUOKA_ERR_UNSUPPORTED;
  if (p->page_size != 0 && p->page_size != kPage) return QUOKA_ERR_UNSUPPORTED;
  if (p->page_size == kPage && (!p->block_table || p->max_pages_per_seq <= 0)) return QUOKA_ERR_INVALID_ARG;
  if (p->page_size == kPage && (int64_t)p->max_pages_per_seq * kPage < (int64_t)p->max_ctx_len + p->chunk_len)
    return QUOKA_ERR_INVALID_ARG;
  if (p->page_size == 0 && p->kv_rows < (int64_t)p->max_ctx_len + p->chunk_len) return QUOKA_ERR_INVALID_ARG;
  if (p->chunk_len > p->n_retain && p->chunk_len > 8192) return QUOKA_ERR_UNSUPPORTED;
  if (p->impl == QUOKA_IMPL_TENSOR && p->dtype != QUOKA_BF16) return QUOKA_ERR_UNSUPPORTED;
  const int64_t strides[] = {p->q_stride_b, p->q_stride_h, p->q_stride_t, p->o_stride_b, p->o_stride_h,
                             p->o_stride_t, p->kv_stride_b, p->kv_stride_h, p->kv_stride_t};
  for (int64_t s : strides)
    if (s < 0 || (s % 8) != 0) return QUOKA_ERR_INVALID_ARG;
  if (p->q_stride_t < p->head_dim || p->o_stride_t < p->head_dim || p->kv_stride_t < p->head_dim)
    return QUOKA_ERR_INVALID_ARG;
  return QUOKA_OK;
}

static bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15) == 0; }

// Everything the fused call checks before it touches the stream, except the workspace.
quoka_status check_prefill_args(const quoka_params* p, const void* q, const void* k_cache, const void* v_cache,
                                const void* out) {
  quoka_status st = validate(p);
  if (st != QUOKA_OK) return st;
  if (!q || !k_cache || !v_cache || !out) return QUOKA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out)) return QUOKA_ERR_INVALID_ARG;
  return QUOKA_OK;
}

static quoka_status check_ws(const quoka_params* p, void* ws, size_t ws_bytes, bool with_split = true) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255) != 0) return QUOKA_ERR_WORKSPACE;
  if (ws_bytes < carve(p, nullptr, with_split).total) return QUOKA_ERR_WORKSPACE;
  return QUOKA_OK;
}

size_t workspace_bytes(const quoka_params* p, bool with_split) { return carve(p, nullptr, with_split).total; }

static DevParams make_dev(const quoka_params* p, void* ws, bool with_split = true) {
  DevParams P{};
  P.batch = p->batch; P.n_q = p->n_q_heads; P.n_kv = p->n_kv_heads; P.group = p->n_q_heads / p->n_kv_heads;
  P.d = p->head_dim; P.chunk = p->chunk_len; P.n_retain = p->n_retain;
  P.n_sel = p->n_retain < p->chunk_len ? p->n_retain : p->chunk_len;
  P.kv_budget = p->kv_budget; P.budget_frac = p->budget_frac;
  P.scale = p->softmax_scale != 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
  P.max_ctx = p->max_ctx_len; P.budget_cap = budget_cap_of(p);
  P.ctx_len = p->ctx_len;
  P.q_sb = p->q_stride_b; P.q_sh = p->q_stride_h; P.q_st = p->q_stride_t;
  P.o_sb = p->o_stride_b; P.o_sh = p->o_stride_h; P.o_st = p->o_stride_t;
  P.page_size = p->page_size; P.max_pages = p->max_pages_per_seq; P.block_table = p->block_table;
  P.kv_sb = p->kv_stride_b; P.kv_sh = p->kv_stride_h; P.kv_st = p->kv_stride_t;
  P.status = static_cast<int32_t*>(ws);
  P.score_dot = p->score_mode == QUOKA_SCORE_DOT ? 1 : 0;
  P.agg_mean = p->query_agg == QUOKA_AGG_MEAN ? 1 : 0;
  P.k_inv_norm = p->k_inv_norm;
  P.kv_rows = p->kv_rows;
  const Workspace w = carve(p, ws, with_split);
  P.attn_partials = w.attn_partials; P.attn_counters = w.attn_counters; P.attn_parts = 1;
  return P;
}

static bool use_tensor(const quoka_params* p) {
  if (p->impl == QUOKA_IMPL_SIMT) return false;
  if (p->dtype != QUOKA_BF16) return false;
  return true;
}

#define QUOKA_TRY_CUDA(expr)                          \
  do {                                                \
    cudaError_t e_ = (expr);                          \
    if (e_ != cudaSuccess) return QUOKA_ERR_CUDA;     \
  } while (0)

static quoka_status run_select_queries(const quoka_params* p, const DevParams& P, const void* q, int32_t* q_idx,
                                       void* qbar, cudaStream_t st) {
  QUOKA_TRY_CUDA(launch_rank_queries(P, p->dtype, q, q_idx, st));
  QUOKA_TRY_CUDA(launch_aggregate_queries(P, p->dtype, q, q_idx, qbar, st, /*chained=*/true));
  return QUOKA_OK;
}

// chained: the aggregation kernel of the same call is the kernel before it on the stream
static quoka_status run_score_keys(const quoka_params* p, const DevParams& P, const void* qbar, const void* k,
                                   float* scores, cudaStream_t st, bool chained = false) {
  if (p->max_ctx_len == 0) return QUOKA_OK;
  if (p->impl == QUOKA_IMPL_AUTO && decode_path_applies(P)) {       // one query: a matrix-vector product
    QUOKA_TRY_CUDA(launch_score_keys_gemv(P, p->dtype, qbar, k, scores, st, chained));
    return QUOKA_OK;
  }
  if (use_tensor(p) && score_keys_tc_supported(p)) return launch_score_keys_tc(p, P, qbar, k, scores, st, chained);
  if (p->impl == QUOKA_IMPL_TENSOR) return QUOKA_ERR_UNSUPPORTED;
  QUOKA_TRY_CUDA(launch_score_keys_simt(P, p->dtype, qbar, k, scores, st));
  return QUOKA_OK;
}

static quoka_status run_attn(const quoka_params* p, const DevParams& P, const void* q, const void* k, const void* v,
                             const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, cudaStream_t st,
                             bool after_selection = false) {
  if (p->impl == QUOKA_IMPL_AUTO && P.chunk == 1 && decode_attn_fits(P, k_idx != nullptr)) {
    QUOKA_TRY_CUDA(launch_decode_attn(P, p->dtype, q, k, v, k_idx, k_cnt, out, lse, st, after_selection));
    return QUOKA_OK;
  }
  if (use_tensor(p) && attn_tc_supported(p))
    return launch_attn_tc(p, P, q, k, v, k_idx, k_cnt, out, lse, st, after_selection);
  if (p->impl == QUOKA_IMPL_TENSOR) return QUOKA_ERR_UNSUPPORTED;
  QUOKA_TRY_CUDA(launch_attn_simt(P, p->dtype, q, k, v, k_idx, k_cnt, out, lse, st));
  return QUOKA_OK;
}

// Two side streams and the events that tie them to the caller's stream, made once per device: the host-buffer entry
// point brings the next slice of a chunk in and takes the previous one out while the current one is computed.
struct HostPipe {
  cudaStream_t h2d = nullptr, d2h = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr, in[4] = {}, done[4] = {};
  bool ok = false, tried = false;
};
static HostPipe* host_pipe_for_current_device() {
  constexpr int kMaxDev = 64;
  static HostPipe pipes[kMaxDev];
  static std::mutex mu;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  HostPipe& hp = pipes[dev];
  if (!hp.tried) {
    hp.tried = true;
    bool good = cudaStreamCreateWithFlags(&hp.h2d, cudaStreamNonBlocking) == cudaSuccess &&
                cudaStreamCreateWithFlags(&hp.d2h, cudaStreamNonBlocking) == cudaSuccess &&
                cudaEventCreateWithFlags(&hp.fork, cudaEventDisableTiming) == cudaSuccess &&
                cudaEventCreateWithFlags(&hp.join, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 4 && good; ++i)
      good = cudaEventCreateWithFlags(&hp.in[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&hp.done[i], cudaEventDisableTiming) == cudaSuccess;
    hp.ok = good;
  }
  return hp.ok ? &hp : nullptr;
}

// The fused loop body.  with_split = false keeps to the workspace layout without the split-attention scratch (the
// built-in array of the no-allocation entry point has no room for it).
quoka_status prefill_chunk_impl(const quoka_params* p, const void* q, const void* k_cache, const void* v_cache, void* out,
                                int32_t* k_idx_out, int32_t* k_cnt_out, void* ws, size_t ws_bytes, void* stream,
                                bool with_split) {
  quoka_status st = check_prefill_args(p, q, k_cache, v_cache, out);
  if (st != QUOKA_OK) return st;
  if ((st = check_ws(p, ws, ws_bytes, with_split)) != QUOKA_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  DevParams P = make_dev(p, ws, with_split);
  Workspace w = carve(p, ws, with_split);
  int32_t* k_idx = k_idx_out ? k_idx_out : w.k_idx;
  int32_t* k_cnt = k_cnt_out ? k_cnt_out : w.k_cnt;
  // the split attention's arrival counters start at zero; cleared here so that nothing sits between the selection
  // kernel and the attention kernel on the stream
  if (w.attn_counters) QUOKA_TRY_CUDA(cudaMemsetAsync(w.attn_counters, 0, attn_split_counter_bytes(p), cs));
  if (p->max_ctx_len > 0) {
    if ((st = run_select_queries(p, P, q, w.q_idx, w.qbar, cs)) != QUOKA_OK) return st;
    if ((st = run_score_keys(p, P, w.qbar, k_cache, w.scores, cs, /*chained=*/true)) != QUOKA_OK) return st;
  }
  // with an empty cache the selection kernel only writes k_cnt = 0 and the -1 padding
  QUOKA_TRY_CUDA(launch_select_keys(P, w.scores, k_idx, k_cnt, cs, /*chained=*/p->max_ctx_len > 0));
  return run_attn(p, P, q, k_cache, v_cache, k_idx, k_cnt, out, nullptr, cs, /*after_selection=*/true);
}

}  // namespace quoka

using namespace quoka;

extern "C" {

quoka_status quoka_kv_budget_cap(const quoka_params* p, int32_t* cap) {
  if (!p || !cap) return QUOKA_ERR_INVALID_ARG;
  *cap = budget_cap_of(p);
  return QUOKA_OK;
}

quoka_status quoka_workspace_size(const quoka_params* p, size_t* bytes) {
  if (!bytes) return QUOKA_ERR_INVALID_ARG;
  quoka_status st = validate(p);
  if (st != QUOKA_OK) return st;
  *bytes = carve(p, nullptr).total;
  return QUOKA_OK;
}

quoka_status quoka_select_queries(const quoka_params* p, const void* q, int32_t* q_idx, void* qbar, void* ws,
                                  size_t ws_bytes, void* stream) {
  quoka_status st = validate(p);
  if (st != QUOKA_OK) return st;
  if (!q || !q_idx || !qbar || !aligned16(q) || !aligned16(qbar)) return QUOKA_ERR_INVALID_ARG;
  if ((st = check_ws(p, ws, ws_bytes)) != QUOKA_OK) return st;
  return run_select_queries(p, make_dev(p, ws), q, q_idx, qbar, static_cast<cudaStream_t>(stream));
}

quoka_status quoka_score_keys(const quoka_params* p, const void* qbar, const void* k_cache, float* scores, void* ws,
                              size_t ws_bytes, void* stream) {
  quoka_status st = validate(p);
  if (st != QUOKA_OK) return st;
  if (!qbar || !k_cache || !scores || !aligned16(qbar) || !aligned16(k_cache)) return QUOKA_ERR_INVALID_ARG;
  if ((st = check_ws(p, ws, ws_bytes)) != QUOKA_OK) return st;
  return run_score_keys(p, make_dev(p, ws), qbar, k_cache, scores, static_cast<cudaStream_t>(stream));
}

quoka_status quoka_update_key_norms(const quoka_params* p, const void* k_cache, float* k_inv_norm, int32_t all_rows,
                                    void* ws, size_t ws_bytes, void* stream) {
  quoka_status st = validate(p);
  if (st != QUOKA_OK) return st;
  if (!k_cache || !k_inv_norm || !aligned16(k_cache)) return QUOKA_ERR_INVALID_ARG;
  if ((st = check_ws(p, ws, ws_bytes)) != QUOKA_OK) return st;
  QUOKA_TRY_CUDA(launch_key_norms(make_dev(p, ws), p->dtype, k_cache, k_inv_norm, all_rows ? 1 : 0,
                                  static_cast<cudaStream_t>(stream)));
  return QUOKA_OK;
}

quoka_status quoka_select_keys(const quoka_params* p, const float* scores, int32_t* k_idx, int32_t* k_cnt, void* ws,
                               size_t ws_bytes, void* stream) {
  quoka_status st = validate(p);
  if (st != QUOKA_OK) return st;
  if (!scores || !k_idx || !k_cnt) return QUOKA_ERR_INVALID_ARG;
  if ((st = check_ws(p, ws, ws_bytes)) != QUOKA_OK) return st;
  DevParams P = make_dev(p, ws);
  QUOKA_TRY_CUDA(launch_select_keys(P, scores, k_idx, k_cnt, static_cast<cudaStream_t>(stream)));
  return QUOKA_OK;
}

quoka_status quoka_sparse_attn(const quoka_params* p, const void* q, const void* k_cache, const void* v_cache,
                               const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, void* ws,
                               size_t ws_bytes, void* stream) {
  quoka_status st = validate(p);
  if (st != QUOKA_OK) return st;
  if (!q || !k_cache || !v_cache || !k_idx || !k_cnt || !out) return QUOKA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out)) return QUOKA_ERR_INVALID_ARG;
  if ((st = check_ws(p, ws, ws_bytes)) != QUOKA_OK) return st;
  return run_attn(p, make_dev(p, ws), q, k_cache, v_cache, k_idx, k_cnt, out, lse,
                  static_cast<cudaStream_t>(stream));
}

quoka_status quoka_dense_chunk_attn(const quoka_params* p, const void* q, const void* k_cache, const void* v_cache,
                                    void* out, float* lse, void* ws, size_t ws_bytes, void* stream) {
  quoka_status st = validate(p);
  if (st != QUOKA_OK) return st;
  if (!q || !k_cache || !v_cache || !out) return QUOKA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out)) return QUOKA_ERR_INVALID_ARG;
  if ((st = check_ws(p, ws, ws_bytes)) != QUOKA_OK) return st;
  return run_attn(p, make_dev(p, ws), q, k_cache, v_cache, nullptr, nullptr, out, lse,
                  static_cast<cudaStream_t>(stream));
}

quoka_status quoka_prefill_chunk(const quoka_params* p, const void* q, const void* k_cache, const void* v_cache,
                                 void* out, int32_t* k_idx_out, int32_t* k_cnt_out, void* ws, size_t ws_bytes,
                                 void* stream) {
  return prefill_chunk_impl(p, q, k_cache, v_cache, out, k_idx_out, k_cnt_out, ws, ws_bytes, stream, /*with_split=*/true);
}

quoka_status quoka_prefill_chunk_host(const quoka_params* p, const int32_t* ctx_len_host, const void* q_host,
                                      const void* k_new_host, const void* v_new_host, void* out_host, void* q_dev,
                                      void* k_cache, void* v_cache, void* out_dev, void* ws, size_t ws_bytes,
                                      void* stream) {
  quoka_status st = validate(p);
  if (st != QUOKA_OK) return st;
  if (p->page_size != 0) return QUOKA_ERR_UNSUPPORTED;
  if (!ctx_len_host || !q_host || !k_new_host || !v_new_host || !out_host || !q_dev || !k_cache || !v_cache ||
      !out_dev)
    return QUOKA_ERR_INVALID_ARG;
  const size_t es = p->dtype == QUOKA_BF16 ? 2 : 4;
  const int64_t C = p->chunk_len, d = p->head_dim;
  if (p->q_stride_t != d || p->q_stride_h != C * d || p->q_stride_b != (int64_t)p->n_q_heads * C * d ||
      p->o_stride_t != d || p->o_stride_h != C * d || p->o_stride_b != (int64_t)p->n_q_heads * C * d ||
      p->kv_stride_t != d)
    return QUOKA_ERR_INVALID_ARG;
  for (int s = 0; s < p->batch; ++s)
    if (ctx_len_host[s] < 0 || ctx_len_host[s] > p->max_ctx_len) return QUOKA_ERR_INVALID_ARG;
  if ((st = check_ws(p, ws, ws_bytes)) != QUOKA_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  // Copies of the KV heads [kv0, kv0 + n_kv) and their query heads; every (sequence, head) block is contiguous on
  // both sides, the sequences are `pitch` apart.
  const int G = p->n_q_heads / p->n_kv_heads;
  const size_t head_bytes = (size_t)C * d * es;
  auto copy_in = [&](int kv0, int n_kv, cudaStream_t on) -> cudaError_t {
    cudaError_t e = cudaMemcpy2DAsync(static_cast<char*>(q_dev) + (size_t)kv0 * G * head_bytes, (size_t)p->q_stride_b * es,
                                      static_cast<const char*>(q_host) + (size_t)kv0 * G * head_bytes,
                                      (size_t)p->n_q_heads * head_bytes, (size_t)n_kv * G * head_bytes, p->batch,
                                      cudaMemcpyHostToDevice, on);
    for (int s = 0; s < p->batch && e == cudaSuccess; ++s) {
      const size_t dst_off = ((size_t)s * p->kv_stride_b + (size_t)kv0 * p->kv_stride_h + (size_t)ctx_len_host[s] * p->kv_stride_t) * es;
      const size_t src_off = ((size_t)s * p->n_kv_heads + kv0) * head_bytes;
      e = cudaMemcpy2DAsync(static_cast<char*>(k_cache) + dst_off, (size_t)p->kv_stride_h * es,
                            static_cast<const char*>(k_new_host) + src_off, head_bytes, head_bytes, n_kv,
                            cudaMemcpyHostToDevice, on);
      if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(static_cast<char*>(v_cache) + dst_off, (size_t)p->kv_stride_h * es,
                              static_cast<const char*>(v_new_host) + src_off, head_bytes, head_bytes, n_kv,
                              cudaMemcpyHostToDevice, on);
    }
    return e;
  };
  auto copy_out = [&](int kv0, int n_kv, cudaStream_t on) -> cudaError_t {
    return cudaMemcpy2DAsync(static_cast<char*>(out_host) + (size_t)kv0 * G * head_bytes, (size_t)p->n_q_heads * head_bytes,
                             static_cast<const char*>(out_dev) + (size_t)kv0 * G * head_bytes, (size_t)p->o_stride_b * es,
                             (size_t)n_kv * G * head_bytes, p->batch, cudaMemcpyDeviceToHost, on);
  };
  // A large chunk is cut into slices of whole KV groups (the selection and the attention of a KV group need nothing
  // of another group): slice i + 1 comes in and slice i - 1 goes out while slice i is computed.  Only for problems
  // the attention kernels would not split (a slice must give the same bits as the whole), without a cache of key
  // norms (indexed by the whole problem's head count), and when the side streams exist.
  int slices = 1;
  const size_t q_bytes = (size_t)p->batch * p->n_q_heads * head_bytes;
  if (!p->k_inv_norm && attn_parts_bound(p) == 1 && q_bytes >= ((size_t)8 << 20)) {
    if (p->n_kv_heads % 4 == 0) slices = 4;
    else if (p->n_kv_heads % 2 == 0) slices = 2;
  }
  HostPipe* hp = slices > 1 ? host_pipe_for_current_device() : nullptr;
  if (!hp) {
    QUOKA_TRY_CUDA(copy_in(0, p->n_kv_heads, cs));
    st = quoka_prefill_chunk(p, q_dev, k_cache, v_cache, out_dev, nullptr, nullptr, ws, ws_bytes, stream);
    if (st != QUOKA_OK) return st;
    QUOKA_TRY_CUDA(copy_out(0, p->n_kv_heads, cs));
    return QUOKA_OK;
  }
  const int kv_per = p->n_kv_heads / slices;
  quoka_params sub = *p;
  sub.n_kv_heads = kv_per;
  sub.n_q_heads = kv_per * G;
  QUOKA_TRY_CUDA(cudaEventRecord(hp->fork, cs));
  QUOKA_TRY_CUDA(cudaStreamWaitEvent(hp->h2d, hp->fork, 0));
  for (int i = 0; i < slices; ++i) {
    const int kv0 = i * kv_per;
    QUOKA_TRY_CUDA(copy_in(kv0, kv_per, hp->h2d));
    QUOKA_TRY_CUDA(cudaEventRecord(hp->in[i], hp->h2d));
    QUOKA_TRY_CUDA(cudaStreamWaitEvent(cs, hp->in[i], 0));
    st = prefill_chunk_impl(&sub, static_cast<char*>(q_dev) + (size_t)kv0 * G * head_bytes,
                            static_cast<char*>(k_cache) + (size_t)kv0 * p->kv_stride_h * es,
                            static_cast<char*>(v_cache) + (size_t)kv0 * p->kv_stride_h * es,
                            static_cast<char*>(out_dev) + (size_t)kv0 * G * head_bytes, nullptr, nullptr, ws, ws_bytes,
                            stream, /*with_split=*/false);
    if (st != QUOKA_OK) return st;
    QUOKA_TRY_CUDA(cudaEventRecord(hp->done[i], cs));
    QUOKA_TRY_CUDA(cudaStreamWaitEvent(hp->d2h, hp->done[i], 0));
    QUOKA_TRY_CUDA(copy_out(kv0, kv_per, hp->d2h));
  }
  QUOKA_TRY_CUDA(cudaEventRecord(hp->join, hp->d2h));
  QUOKA_TRY_CUDA(cudaStreamWaitEvent(cs, hp->join, 0));
  return QUOKA_OK;
}

quoka_status quoka_append_kv(const quoka_params* p, const void* k_new, const void* v_new, void* k_cache,
                             void* v_cache, float* k_inv_norm, void* ws, size_t ws_bytes, void* stream) {
  quoka_status st = validate(p);
  if (st != QUOKA_OK) return st;
  if (!k_new || !v_new || !k_cache || !v_cache) return QUOKA_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_cache) || !aligned16(v_cache)) return QUOKA_ERR_INVALID_ARG;
  if ((st = check_ws(p, ws, ws_bytes)) != QUOKA_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const DevParams P = make_dev(p, ws);
  QUOKA_TRY_CUDA(launch_append_kv(P, p->dtype, k_new, v_new, k_cache, v_cache, cs));
  if (k_inv_norm) QUOKA_TRY_CUDA(launch_key_norms(P, p->dtype, k_cache, k_inv_norm, 0, cs));
  return QUOKA_OK;
}

quoka_status quoka_last_device_status(void* ws, void* stream, int32_t* status_out) {
  if (!status_out) return QUOKA_ERR_INVALID_ARG;
  if (!ws) {                                  // the built-in scratch array of quoka_prefill_chunk_static
    quoka_status st = static_scratch_for_current_device(&ws);
    if (st != QUOKA_OK) return st;
  }
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  int32_t h = 0;
  QUOKA_TRY_CUDA(cudaMemcpyAsync(&h, ws, sizeof(h), cudaMemcpyDeviceToHost, cs));
  QUOKA_TRY_CUDA(cudaStreamSynchronize(cs));
  QUOKA_TRY_CUDA(cudaMemsetAsync(ws, 0, sizeof(int32_t), cs));
  *status_out = h;
  return QUOKA_OK;
}

const char* quoka_status_string(quoka_status s) {
  switch (s) {
    case QUOKA_OK: return "ok";
    case QUOKA_ERR_INVALID_ARG: return "invalid argument";
    case QUOKA_ERR_UNSUPPORTED: return "unsupported configuration";
    case QUOKA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case QUOKA_ERR_CUDA: return "CUDA call failed";
    case QUOKA_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case QUOKA_ERR_STATIC_LIMIT: return "problem needs more scratch than the built-in static array holds";
    case QUOKA_ERR_BAD_INDEX: return "a selected row or page id was out of range (debug build)";
    default: return "unknown status";
  }
}

int64_t quoka_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
