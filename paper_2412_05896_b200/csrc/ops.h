// Internal launchers behind the C ABI; arguments are already validated by xkv_api.cu.
#pragma once

#include <cuda_runtime.h>

#include "../../include/xkv.h"

namespace xkv {

size_t score_workspace_bytes(const xkv_dims* d, int max_seqlen, int64_t total_tokens);
xkv_status score(const xkv_dims* d, const void* q_win, const void* k, const int32_t* cu_seqlens,
                 int64_t total_tokens, int max_seqlen, float* scores, float* sorted, float* gains, float* mass,
                 int curve_len, void* workspace, size_t workspace_bytes, cudaStream_t st,
                 const float* lse = nullptr);
// 1 when the shape is one the scoring pass from given row normalisers covers
int score_lse_supported(const xkv_dims* d, int max_seqlen);

size_t prefill_workspace_bytes();
xkv_status prefill_attn(const xkv_dims* d, const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                        int64_t total_tokens, int max_seqlen, void* out, float* lse, void* workspace,
                        cudaStream_t st);

size_t select_workspace_bytes(const xkv_dims* d, int max_seqlen, int64_t total_tokens);
xkv_status select_compact(const xkv_dims* d, int layer, const int32_t* budget, int per_sequence,
                          const float* scores, const float* sorted, const void* k, const void* v,
                          const int32_t* cu_seqlens, int64_t total_tokens, int max_seqlen, const xkv_cache* c,
                          int32_t* sel, int sel_stride, void* workspace, size_t workspace_bytes, cudaStream_t st);

xkv_status build_block_table(const int32_t* first_page, const int32_t* n_pages_lb, int n_lb, int32_t* block_table,
                             int max_pages_per_seq, cudaStream_t st);
xkv_status batch_curves(const float* gains, int n_layers, int batch, int curve_len, double scale, float* out,
                        cudaStream_t st);

xkv_status head_curves(const xkv_dims* d, const float* scores, const float* sorted, const int32_t* cu_seqlens,
                       int64_t total_tokens, int max_seqlen, float* out, int curve_len, cudaStream_t st);

size_t decode_workspace_bytes(const xkv_dims* d, int n_layers, int max_cache_len, int chunk_rows);
xkv_status decode_attn(const xkv_dims* d, const xkv_cache* c, int layer_begin, int layer_end, const void* q,
                       const void* k_new, const void* v_new, void* out, float* lse, int chunk_rows,
                       void* workspace, size_t workspace_bytes, cudaStream_t st, bool clear_status = false);

xkv_status decode_attn_static(const xkv_dims* d, const xkv_cache* c, int layer_begin, int layer_end,
                              const void* q, const void* k_new, const void* v_new, void* out, float* lse,
                              int chunk_rows, int32_t* status_out, cudaStream_t st);
void set_profile_events(cudaEvent_t start, cudaEvent_t stop);

}  // namespace xkv
