// Internal interface of the token filter (shared by the C entry point and vit_forward).
#pragma once
#include "common.cuh"

// cls_score_topk_filter with the number of kept tokens given instead of derived from keep_ratio
// (1 <= k <= n_patch; desc->keep_ratio is ignored).  vit_forward ranks a later stage over the whole grid, with
// the absent positions' scores set to NaN (they rank last), and keeps as many as that stage leaves.
int32_t spv_filter_run_k(spv_ctx* ctx, const spv_filter_desc* desc, int32_t k, const float* scores,
                         const void* tokens_in, void* tokens_out, int32_t* kept_idx, float* mean_scores,
                         const int32_t* pos_in, int32_t* pos_out, void* workspace, size_t workspace_bytes,
                         cudaStream_t stream);

// Fused front end of the filter inside vit_forward: the CLS->patch softmax weights are evaluated from the global
// row's scaled logits and per-head (maximum, 1 / sum) in the same pass that averages them over the heads and forms
// the ranking keys, so the [batch, heads, n_patch] score tensor is never written.  Same arithmetic, in the same
// order, as the score kernel followed by the head-mean kernel: the kept set is bit-identical.
//   logits [batch * n_global][heads][n_tok] (row of global token 0 used), head_stats [batch][heads][2];
//   cur_pos [batch][n_tok - n_global] original position of each present patch (NULL = identity);
//   np_grid positions are ranked (absent ones rank last), kept_idx [batch][k] ascending original positions.
int32_t spv_filter_rank_logits(spv_ctx* ctx, int32_t batch, int32_t heads, int32_t n_global, int32_t n_tok,
                               int32_t np_grid, int32_t k, const float* logits, const float* head_stats,
                               const int32_t* cur_pos, int32_t* kept_idx, void* workspace, size_t workspace_bytes,
                               cudaStream_t stream);
