// Internal interface of the sparse-attention module (shared by the C entry point and vit_forward).
#pragma once
#include "common.cuh"

// Block-major view of one token layout: patch tokens grouped by spatial block (blocks in row-major
// order over the block grid), so that the neighbour blocks of one block row are one contiguous
// token range.  All arrays live in the caller's workspace.
struct SpvAttnPlan {
  int32_t batch, grid_h, grid_w, block, radius, n_global, n_patch;
  int32_t nby, nbx, nb;
  int32_t segs_per_block, nseg;     // search segments used to build the plan
  int32_t tiles_per_row, tiles_per_image;
  int32_t identity;                 // tokens already block-major: no regrouping copy, bm_src unused
  int32_t* seg_lo;                  // [B][nseg]
  int32_t* seg_cnt;                 // [B][nseg]
  int32_t* seg_off;                 // [B][nseg+1]
  int32_t* block_off;               // [B][nb+1]  first block-major ordinal of each block
  int32_t* tok_blk;                 // [B][n_patch] block id of block-major ordinal t
  int32_t* bm_src;                  // [B][n_patch] input patch ordinal of block-major ordinal t
  int4* tiles;                      // [B][tiles_per_image] {q_begin, q_end, by, bx_first | bx_last << 16}
};

size_t spv_attn_plan_bytes(int32_t batch, int32_t grid_h, int32_t grid_w, int32_t block, int32_t n_patch,
                           int32_t token_order);

// Build the plan on `stream` (three small kernels).  patch_pos as in spv_attn_desc; check_positions adds a
// kernel that verifies a caller's patch_pos (range and order) and latches a violation in the status word.
int32_t spv_attn_plan_build(spv_ctx* ctx, int32_t batch, int32_t grid_h, int32_t grid_w, int32_t block,
                            int32_t radius, int32_t n_global, int32_t n_patch, const int32_t* patch_pos,
                            int32_t token_order, void* ws, size_t ws_bytes, cudaStream_t stream,
                            SpvAttnPlan* plan, bool check_positions = false);

struct SpvAttnIO {
  const void *q, *k, *v;            // bf16, tokens in BLOCK-MAJOR order (globals first)
  int64_t sb, st, sh;               // element strides of q/k/v
  void* o;                          // bf16 output
  int64_t o_sb, o_st, o_sh;
  const int32_t* o_tok;             // [B][n_patch] output patch ordinal of block-major ordinal t; NULL = t
  int32_t heads;
  float scale;                      // softmax scale (already defaulted)
};

// Patch-query rows: the tcgen05 flash kernel.
int32_t spv_attn_run_patches(spv_ctx* ctx, const SpvAttnPlan* plan, const SpvAttnIO* io, cudaStream_t stream);

// Global-query rows (dense rows, memory-bound) and optional CLS->patch scores.
// scores: fp32 [B][heads][score_stride], the weight of block-major ordinal t written at score_idx[b][t]
// (NULL = t); score_stride >= the largest index + 1 (the patch count, or the grid size when the indices
// are original positions).
size_t spv_attn_global_bytes(int32_t batch, int32_t n_global, int32_t heads, int32_t n_tok);
// head_stats (optional): fp32 [B][heads][2] = (row maximum of the scaled logits, 1 / row sum) of global token 0;
// logits_out then receives the scaled logits [B*G][heads][n_tok] inside `ws` (valid until `ws` is written again):
// weight of token t = exp(logit[t] - maximum) / sum, which the fused ranking of the token filter evaluates itself.
int32_t spv_attn_run_globals(spv_ctx* ctx, const SpvAttnPlan* plan, const SpvAttnIO* io, float* scores,
                             const int32_t* score_idx, int32_t score_stride, void* ws, size_t ws_bytes,
                             cudaStream_t stream, float* head_stats = nullptr, const float** logits_out = nullptr);
