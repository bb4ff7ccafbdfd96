// Host-side entry points of the tcgen05 (5th-generation tensor core) kernels.
#pragma once

#include "common.cuh"

namespace quoka {

// Whether the tensor-core kernel covers this configuration (bf16, supported N / head_dim / layout).
bool score_keys_tc_supported(const quoka_params* p);
quoka_status launch_score_keys_tc(const quoka_params* p, const DevParams& P, const void* qbar, const void* k,
                                  float* scores, cudaStream_t st, bool chained);

bool attn_tc_supported(const quoka_params* p);
quoka_status launch_attn_tc(const quoka_params* p, const DevParams& P, const void* q, const void* k, const void* v,
                            const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, cudaStream_t st,
                            bool after_selection);
// head_dim 128 with an even GQA ratio: the CTAs of two heads of a KV group work as a pair (cta_group::2)
bool attn_tc_pair_applies(const DevParams& P);
// Small grids: the key tiles of every row block are cut into this many parts, one CTA each (1 = no split).
// `tiles` = key tiles of the longest row block the call can meet.  Scratch for the partial results:
int attn_split_parts(const quoka_params* p, int tiles);
size_t attn_split_partial_bytes(const quoka_params* p, int parts);
size_t attn_split_counter_bytes(const quoka_params* p);
int attn_split_parts_for_launch(const quoka_params* p, const DevParams& P, bool sparse);
quoka_status launch_attn_tc_pair(const quoka_params* p, const DevParams& P, const void* q, const void* k, const void* v,
                                 const int32_t* k_idx, const int32_t* k_cnt, void* out, float* lse, cudaStream_t st,
                                 bool after_selection);

}  // namespace quoka
