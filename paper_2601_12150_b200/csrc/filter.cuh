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
