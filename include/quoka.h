/*
 * quoka.h - C ABI of the B200 (sm_100a) implementation of QuoKA's per-chunk
 * sparse prefill attention ("QuoKA: Query-oriented KV selection for efficient
 * LLM prefill", Algorithm 1 and Algorithm 2).
 *
 * One call sequence handles ONE attention layer and ONE prefill chunk of every
 * sequence in a batch:
 *
 *   quoka_select_queries   Alg. 1 "Query Sub-selection" + normalisation + GQA pre-aggregation
 *   quoka_score_keys       Alg. 1  S = Qbar K^T on normalised keys,  S^ = max over queries
 *   quoka_select_keys      Alg. 1  I = topk(S^, B_SA)
 *   quoka_sparse_attn      Alg. 2  Attention(Q_i, [K^ | K_i], [V^ | V_i])   (Eq. 1, Eq. 2)
 *   quoka_prefill_chunk    all four, back to back on one stream
 *   quoka_dense_chunk_attn Eq. 2 without selection (the speed-up denominator)
 *
 * Symbols: b batch, n_Q query heads, n_KV KV heads, G = n_Q / n_KV, d head_dim,
 * T_s cached length of sequence s (K_<i), C = B_CP chunk length, N = min(N_Q, C)
 * retained queries, B_s = key budget of sequence s.
 *
 * Pointers.  Unless a parameter is marked HOST, every data pointer is a DEVICE
 * pointer into memory the caller allocated; the library allocates nothing, keeps
 * no state between calls (except the entry point marked otherwise) and only
 * writes the outputs and the workspace.  `stream` is a cudaStream_t passed as
 * void* (NULL = the legacy default stream).  Calls are asynchronous: they
 * enqueue work on `stream` and return.
 *
 * Cache layout.  The caller has ALREADY written the chunk's own K_i, V_i at rows
 * [T_s, T_s + C) of the cache (Alg. 2 appends after attention; appending before
 * is equivalent because selection only reads rows < T_s).  Contiguous cache:
 * element (s, h, t, x) at  s*kv_stride_b + h*kv_stride_h + t*kv_stride_t + x.
 * Paged cache (page_size == 64): logical row t of sequence s lives in page
 * p = block_table[s*max_pages_per_seq + t/64] at
 * p*kv_stride_b + h*kv_stride_h + (t%64)*kv_stride_t + x.   Strides are in
 * elements; head_dim is contiguous.  All base pointers 16-byte aligned, all
 * strides multiples of 8 elements.
 *
 * Errors.  Every call validates its arguments on the host before launching
 * anything and returns a status; nothing is launched on error.  Problems only
 * the device can see (a bounded wait that ran out) are recorded in a status word
 * inside the workspace: read it with quoka_last_device_status.  No entry point
 * throws, traps or blocks.
 *
 * Determinism.  The same inputs give bit-identical outputs from run to run.
 */
#ifndef QUOKA_H_
#define QUOKA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  QUOKA_OK = 0,
  QUOKA_ERR_INVALID_ARG = 1,  /* null pointer, non-positive size, n_Q % n_KV != 0, misaligned stride */
  QUOKA_ERR_UNSUPPORTED = 2,  /* head_dim not in {64,128}, page_size not in {0,64}, chunk_len > 8192 with selection */
  QUOKA_ERR_WORKSPACE = 3,    /* workspace pointer null / misaligned / smaller than quoka_workspace_size */
  QUOKA_ERR_CUDA = 4,         /* a CUDA runtime or driver call failed (launch, tensor-map encode) */
  QUOKA_ERR_TIMEOUT = 5,      /* device status word: a bounded wait inside a kernel ran out */
  QUOKA_ERR_STATIC_LIMIT = 6, /* quoka_prefill_chunk_static: the problem needs more scratch than the built-in array */
  QUOKA_ERR_BAD_INDEX = 7     /* device status word (debug build): a selected row or a page id was out of range */
} quoka_status;

typedef enum { QUOKA_BF16 = 0, QUOKA_F32 = 1 } quoka_dtype;

/* Which kernels serve the contraction steps (scoring, attention). */
typedef enum {
  QUOKA_IMPL_AUTO = 0,   /* tcgen05 tensor-core kernels for bf16, scalar kernels for f32 */
  QUOKA_IMPL_SIMT = 1,   /* scalar fp32 kernels (any dtype); the on-device cross-check */
  QUOKA_IMPL_TENSOR = 2  /* tcgen05 kernels; QUOKA_ERR_UNSUPPORTED if dtype is f32 */
} quoka_impl;

/* How a cached key is scored against the retained queries (the paper's ablations, Appendix "Ablations").
 * The defaults are the method as published: cosine similarity, maximum over the retained queries. */
typedef enum {
  QUOKA_SCORE_COSINE = 0,  /* Alg. 1: queries and keys divided by their norms before the product          */
  QUOKA_SCORE_DOT = 1      /* ablation: raw dot products, neither queries nor keys are normalised         */
} quoka_score_mode;
typedef enum {
  QUOKA_AGG_MAX = 0,       /* Alg. 1: S^ = max over the retained queries                                  */
  QUOKA_AGG_MEAN = 1       /* ablation: S^ = mean over the retained queries                               */
} quoka_query_agg;

typedef struct {
  int32_t batch, n_q_heads, n_kv_heads, head_dim;
  int32_t chunk_len;     /* C = B_CP                                                          */
  int32_t n_retain;      /* N_Q; >= chunk_len means no query sub-selection (Alg. 1, the `if`)  */
  int32_t kv_budget;     /* B_SA in keys, B_s = min(B_SA, T_s); <= 0 selects budget_frac       */
  float budget_frac;     /* B_s = floor(budget_frac * T_s + 0.5), evaluated in double          */
  int32_t dtype;         /* quoka_dtype of q, k_cache, v_cache, qbar, out                      */
  int32_t impl;          /* quoka_impl                                                         */
  float softmax_scale;   /* 0 selects 1/sqrt(head_dim) (Eq. 1)                                 */
  int32_t max_ctx_len;   /* HOST upper bound on every T_s: sizes grids, buffers and workspace  */
  const int32_t* ctx_len;      /* DEVICE [batch]: T_s; rows [0,T_s) are the selectable cache    */
  /* q and out: element (s, h, r, x) at s*stride_b + h*stride_h + r*stride_t + x               */
  int64_t q_stride_b, q_stride_h, q_stride_t;
  int64_t o_stride_b, o_stride_h, o_stride_t;
  /* KV cache, see "Cache layout" above                                                        */
  int32_t page_size;           /* 0 = contiguous, 64 = paged                                    */
  int32_t max_pages_per_seq;
  const int32_t* block_table;  /* DEVICE [batch][max_pages_per_seq], NULL when contiguous       */
  int64_t kv_stride_b, kv_stride_h, kv_stride_t;   /* kv_stride_b is the page stride when paged */
  int64_t kv_rows;             /* rows allocated per (sequence, head) when contiguous (>= T_s+C);
                                  number of pages in the pool when paged                        */
  int32_t score_mode;          /* quoka_score_mode; affects qbar (normalised or raw) and the scores */
  int32_t query_agg;           /* quoka_query_agg                                                 */
  const float* k_inv_norm;     /* DEVICE, may be NULL: 1/max(|k|,1e-12) of every cache row, kept by the caller with
                                  quoka_update_key_norms.  Indexed like the cache without head_dim: contiguous
                                  [b][n_KV][kv_rows], paged [page][n_KV][64].  When given, quoka_score_keys and
                                  quoka_prefill_chunk read it instead of recomputing the norms of all T_s keys  */
} quoka_params;

/* Row pitch of k_idx: the largest B_s any sequence can have, from max_ctx_len. */
quoka_status quoka_kv_budget_cap(const quoka_params* p, int32_t* cap);

/* Bytes of workspace that every call below accepts (256-byte aligned pointer).
 * The first 256 bytes hold the device status word, which the caller sets to zero
 * once after allocating; the rest is scratch whose contents mean nothing between
 * calls.  Two calls that share a workspace must not overlap on the GPU.
 * For problems whose attention grid is smaller than the GPU (few heads, a short
 * chunk) the size includes room for the partial results of the split attention
 * kernel (each row block's keys are cut into up to 8 parts, one CTA each, and added
 * up in part order: results are reproducible from run to run, and differ from the
 * unsplit kernel's in the last bits only). */
quoka_status quoka_workspace_size(const quoka_params* p, size_t* bytes);

/* Alg. 1, "Query Sub-selection", then the normalisation and the mean over the G
 * heads of each KV group.  Per query head: M = mean over the chunk of the raw
 * queries; c_r = CosSim(q_r, M); if C > N_Q keep the N_Q rows of LOWEST c_r,
 * most dissimilar first, equal values earlier position first, else keep all rows
 * in order.  Then Qbar[kv][j] = (1/G) sum_g  q^_{kvG+g, pi_g(j)}  with
 * q^ = q / max(|q|, 1e-12), accumulated in fp32 and rounded once to `dtype`.
 *   q      in  [b][n_Q][C][d] by strides
 *   q_idx  out [b][n_Q][N] int32, ordered by rank
 *   qbar   out [b][n_KV][N][d] dense, `dtype` */
quoka_status quoka_select_queries(const quoka_params* p, const void* q, int32_t* q_idx, void* qbar,
                                  void* ws, size_t ws_bytes, void* stream);

/* Alg. 1, scoring and max over the query axis: for every cached row t < T_s,
 * scores[s][kv][t] = max_j (Qbar[s][kv][j] . k_t) / max(|k_t|, 1e-12).  The
 * N x T score matrix is never written to memory.
 *   scores out [b][n_KV][max_ctx_len] fp32; entries t >= T_s are not written */
quoka_status quoka_score_keys(const quoka_params* p, const void* qbar, const void* k_cache, float* scores,
                              void* ws, size_t ws_bytes, void* stream);

/* Alg. 1 normalises every cached key in every chunk ("K <- K / norm(K)"); a cached key never changes, so its
 * inverse norm can be computed once, when the key is appended, and kept beside the cache (the cost the paper's
 * conclusion names as what is left to reduce is this pass over all T keys).  Writes
 * k_inv_norm[row] = 1 / max(|k_row|, 1e-12) for rows [T_s, T_s + C) of every (sequence, KV head) (the chunk just
 * appended), or for rows [0, T_s + C) when all_rows is non-zero (first use on an existing cache).
 * p->k_inv_norm is ignored here; the output pointer is the argument. */
quoka_status quoka_update_key_norms(const quoka_params* p, const void* k_cache, float* k_inv_norm, int32_t all_rows,
                                    void* ws, size_t ws_bytes, void* stream);

/* Alg. 1, I = topk(S^, B_SA) per (sequence, KV head): the B_s rows with the
 * largest score; among equal scores at the threshold the lower row wins; the
 * list is written ascending by row.  T_s <= B_s gives 0..T_s-1.
 *   k_idx out [b][n_KV][cap] int32 (cap from quoka_kv_budget_cap), entries >= B_s set to -1
 *   k_cnt out [b] int32 = B_s */
quoka_status quoka_select_keys(const quoka_params* p, const float* scores, int32_t* k_idx, int32_t* k_cnt,
                               void* ws, size_t ws_bytes, void* stream);

/* Alg. 2, the attention line, with Eq. 1/Eq. 2 semantics: row r of query head h
 * attends rows k_idx[s][h/G][0..k_cnt[s]) of the ORIGINAL cache plus the chunk's
 * own rows T_s..T_s+r (causal, diagonal included); softmax in fp32.  The rows are
 * gathered inside the kernel; no compacted copy of K or V is made.
 *   out [b][n_Q][C][d] by strides, `dtype`;  lse [b][n_Q][C] fp32 natural-log-sum-exp of
 *   the scaled logits, may be NULL */
quoka_status quoka_sparse_attn(const quoka_params* p, const void* q, const void* k_cache, const void* v_cache,
                               const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse,
                               void* ws, size_t ws_bytes, void* stream);

/* Eq. 2: the chunk attends all T_s cached rows and its own rows causally. */
quoka_status quoka_dense_chunk_attn(const quoka_params* p, const void* q, const void* k_cache,
                                    const void* v_cache, void* out, float* lse,
                                    void* ws, size_t ws_bytes, void* stream);

/* Alg. 2, loop body: the four steps above on `stream` with the intermediates in
 * the workspace.  k_idx_out ([b][n_KV][cap]) and k_cnt_out ([b]) may be NULL; when
 * given they receive the selection that was used.  The kernels of one call are
 * launched so that each may become resident while the one before it still runs
 * (each waits for its producer itself); towards everything else on `stream` the
 * call is ordered like a single kernel: it starts after the work before it and
 * the work after it starts when its last kernel has completed. */
quoka_status quoka_prefill_chunk(const quoka_params* p, const void* q, const void* k_cache, const void* v_cache,
                                 void* out, int32_t* k_idx_out, int32_t* k_cnt_out,
                                 void* ws, size_t ws_bytes, void* stream);

/* The same loop body for a caller whose chunk lives in HOST memory (pinned for
 * the copies to be asynchronous): copies q_host -> q_dev, the chunk's K_i, V_i
 * ([b][n_KV][C][d] dense, HOST) into rows [T_s, T_s+C) of the contiguous device
 * cache, runs quoka_prefill_chunk, and copies out_dev -> out_host
 * ([b][n_Q][C][d] dense), all on `stream`.  ctx_len_host is a HOST copy of T_s.
 * Paged caches are not supported here (QUOKA_ERR_UNSUPPORTED).  q_dev / out_dev
 * must be dense [b][n_Q][C][d] and p's q/o strides must describe them.
 * A chunk of 8 MiB of queries or more is cut into 2 or 4 slices of whole KV
 * groups, and slice i+1 is copied in and slice i-1 copied out on two streams of
 * the library's own (made on first use, one set per device) while slice i is
 * computed on `stream`; the result is the same bits as the unsliced call's.
 * Towards `stream` the call is still ordered like one operation (it forks from
 * `stream` at its start and joins it at its end, also under stream capture).
 * Two such calls must not overlap on one device (they share the side streams
 * and their events), whatever streams they are given. */
quoka_status quoka_prefill_chunk_host(const quoka_params* p, const int32_t* ctx_len_host,
                                      const void* q_host, const void* k_new_host, const void* v_new_host,
                                      void* out_host, void* q_dev, void* k_cache, void* v_cache, void* out_dev,
                                      void* ws, size_t ws_bytes, void* stream);

/* Alg. 2, "append K_i, V_i to the cache": copies the chunk's keys and values, dense [b][n_KV][C][d] in DEVICE
 * memory, into rows [T_s, T_s + C) of the cache (contiguous by strides, or paged through the block table), with
 * T_s read from p->ctx_len on the device.  Call it before the chunk's quoka_prefill_chunk (see "Cache layout").
 * When k_inv_norm is not NULL the inverse norms of the appended rows are written as quoka_update_key_norms
 * would.  The caller advances ctx_len by C after the chunk's attention. */
quoka_status quoka_append_kv(const quoka_params* p, const void* k_new, const void* v_new, void* k_cache,
                             void* v_cache, float* k_inv_norm, void* ws, size_t ws_bytes, void* stream);

/* (The paper has no counterpart of this call: it is a deployment variant of quoka_prefill_chunk.)
 * The same loop body for callers that cannot allocate device memory and so have no workspace to
 * pass: a process whose KV-cache pool already owns all of HBM, or a latency-critical loop in which
 * cudaMalloc/cudaFree (which synchronise the device) are forbidden.  The intermediates live in an
 * array of QUOKA_STATIC_SCRATCH_BYTES that is part of the library image; every GPU that loads the
 * library holds that much memory until the process exits.  Inputs and outputs are still the
 * caller's.  The call allocates nothing and frees nothing.
 *   - Problems whose intermediates exceed QUOKA_STATIC_SCRATCH_BYTES are refused with
 *     QUOKA_ERR_STATIC_LIMIT before anything is launched (for scale: 32 q / 8 kv heads, d 128,
 *     131072 cached rows, N_Q 256 needs about 5.1 MiB; a batch of 8 at 65536 rows does not fit).
 *     The array has no room for the split attention kernel's partial results: small grids run
 *     unsplit here, so on those the output may differ from quoka_prefill_chunk's in the last bits.
 *   - The first call on each device looks up the array's device address (that device must be
 *     current); make that first call before any stream capture begins.
 *   - All calls in the process share the one array per device, and it keeps the previous call's
 *     contents.  The status word is cleared at the start of every call; nothing else needs to start
 *     at zero.  Two calls whose work overlaps on the same GPU (different streams, or different host
 *     threads) race on the array: serialise them.
 *   - The array's status word is read (and cleared) with quoka_last_device_status(NULL, stream, &st);
 *     read it before the next static call, which clears it.
 *   - The array's address is looked up once per device and remembered: after cudaDeviceReset the
 *     process must not use this entry point again. */
#define QUOKA_STATIC_SCRATCH_BYTES (8u << 20)
quoka_status quoka_prefill_chunk_static(const quoka_params* p, const void* q, const void* k_cache,
                                        const void* v_cache, void* out, int32_t* k_idx_out, int32_t* k_cnt_out,
                                        void* stream);

/* Copies the device status word of `ws` to the host (synchronises `stream`) and
 * clears it.  *status_out is a quoka_status.  ws == NULL reads the status word of the built-in
 * array that quoka_prefill_chunk_static uses on the current device.  After a QUOKA_ERR_TIMEOUT the
 * outputs of the call that hit it are undefined (the kernel left its loops and ran its teardown
 * with work possibly still outstanding). */
quoka_status quoka_last_device_status(void* ws, void* stream, int32_t* status_out);

const char* quoka_status_string(quoka_status s);

/* Number of kernels this library has launched in this process (all entry points). */
int64_t quoka_launch_count(void);

/* ---- diagnostics (no counterpart in the paper) ------------------------------------------------
 * QUOKA_LOG=1 in the environment prints one line per kernel launch (name, grid, block, dynamic
 * shared memory, cluster width) on stderr.
 *
 * A build with -DQUOKA_DEBUG (python -m paper_2602_08722_b200.build --debug, libquoka_debug.so)
 * range-checks every selected-row index and every block-table entry the attention kernel is about
 * to use; a bad one records QUOKA_ERR_BAD_INDEX in the status word and the row is treated as
 * absent (zero-filled, masked) instead of being read. */

/* HOST-side check of a paged cache's block table before it is uploaded: ctx_len_host [batch] and
 * block_table_host [batch][max_pages_per_seq] are HOST arrays.  Every page that rows
 * [0, T_s + C) of a sequence need must lie inside the pool (0 <= page < kv_rows) and no physical
 * page may be used twice.  Returns QUOKA_ERR_INVALID_ARG otherwise.  Launches nothing. */
quoka_status quoka_check_block_table(const quoka_params* p, const int32_t* ctx_len_host,
                                     const int32_t* block_table_host);

/* Self-test of the bounded device wait: launches one warp that waits on a barrier nobody signals,
 * with a limit of limit_cycles SM cycles (1 .. 2e9).  The wait must give up: *gave_up (DEVICE
 * int32) becomes 1, the status word of `ws` becomes QUOKA_ERR_TIMEOUT, and the kernel returns.
 * Exercises exactly the wait every tensor-core kernel of the library uses. */
quoka_status quoka_selftest_wait_timeout(void* ws, int64_t limit_cycles, int32_t* gave_up, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QUOKA_H_ */
