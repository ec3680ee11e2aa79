// Parameters shared by the scoring kernels (xkv_score.cu, xkv_score_tc.cu).
#pragma once

#include "common.cuh"

namespace xkv {

struct ScoreParams {
  const __nv_bfloat16* q_win;
  const __nv_bfloat16* k;
  const int32_t* cu_seqlens;
  float* scores;
  float* sorted;
  float* gains;
  float* mass;
  float* u;            // [Hkv][T] un-pooled column sums
  float* tmp_sorted;   // [Hkv][T] ping-pong buffer of the merge passes
  float2* stats_part;  // [units][n_splits][M]
  float* mrow;         // [units][M]
  float* part_sum;     // [units][n_chunks]
  WorkspaceHeader* hdr;
  int32_t* unit_ticket;  // [units] pass-1 items of the unit that have finished
  int32_t* unit_ready;   // [units] 1 once mrow of the unit is final
  int32_t slice_tiles, n_work;
  int64_t total_tokens, stride_token, stride_head;
  int32_t batch, n_q_heads, n_kv_heads, group, window, M, pool_kernel, pool_mode;
  int32_t M_real;      // G*W; M is M_real rounded up to a multiple of 16 (the padding rows never contribute)
  int32_t split_keys, n_splits, n_chunks, curve_len;
  int32_t max_seqlen;  // host bound of every prompt length; longer prompts are cut to it and reported
  float scale_log2;
  uint64_t wait_ns;    // limit of every bounded wait
};

// tcgen05 variant of the two logit passes (xkv_score_tc.cu).  Returns XKV_ERR_UNSUPPORTED when the shape
// is outside what it covers; the caller then uses the mma.sync kernels.
xkv_status score_tc_passes(const ScoreParams& p, int head_dim, int max_seqlen, cudaStream_t st);
// The column-sum pass alone, for row normalisers that are already in p.mrow (same shapes as score_tc_passes).
xkv_status score_tc_pass2(const ScoreParams& p, int head_dim, int max_seqlen, cudaStream_t st);
// Key split the tcgen05 variant uses (0 if it does not cover the shape).
int score_tc_split_keys(int M, int head_dim, int units, int max_seqlen);

// Single-launch variant (xkv_score_fused.cu): a thread-block cluster per unit keeps the unit's logits in tensor
// memory between the statistics and the column sums, so the keys are read once.  Covers G*W = 32 and prompts of
// at most 8192 tokens.
bool score_fused_covers(int M, int head_dim, int units, int max_seqlen);
xkv_status score_fused_pass(const ScoreParams& p, int head_dim, int max_seqlen, cudaStream_t st);

}  // namespace xkv
