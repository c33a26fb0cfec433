/*
 * CPU oracle for the large-resolution ViT inference path (test infrastructure).
 *
 * This is TEST INFRASTRUCTURE, not a product path: a plain, slow, single-source
 * C restatement of what the method computes, written from the paper's
 * definitions.  Only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it.  It shares no code, header, table or helper with the CUDA
 * library.
 *
 * Numeric policy: tensors are stored as fp32; every reduction (dot products,
 * softmax sums, LayerNorm statistics, GEMM accumulation) is carried in fp64.
 * The one exception is the head average of the token filter, which is the
 * fp32 sequential sum the ranking rule is defined on (it decides an integer
 * result, so both sides must take it in the same precision).
 *
 * Pins (tests/test_oracle_*.py): hand-enumerated neighbour sets on 4x4 grids,
 * closed-form pair counts, equality with an independently written dense softmax
 * attention when the neighbourhood covers the grid, a library masked attention
 * in fp64, one-hot / constant V identities, numpy.lexsort for the ranking, and
 * an independent fp64 restatement of the whole forward on tiny models.
 * Paper-level accuracy / time / memory tables need the paper's datasets and
 * trained weights: parity unpinned for those.
 *
 * Token order: index 0..G-1 are the global tokens (CLS first), then patch
 * tokens.  Patch token t (0-based among patches) sits at original grid
 * position pos = patch_pos ? patch_pos[t] : t, with y = pos / W, x = pos % W.
 */
#ifndef SPV_ORACLE_H
#define SPV_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int32_t batch, grid_h, grid_w;
  int32_t block, radius;       /* block edge b in patches; radius r in blocks  */
  int32_t n_global;            /* G leading global tokens                      */
  int32_t heads, head_dim;
  float softmax_scale;         /* 0 => 1/sqrt(head_dim)                        */
  int32_t n_patch;             /* patch tokens present                         */
  const int32_t* patch_pos;    /* [batch, n_patch] original y*W+x, or NULL     */
} spvo_attn_desc;

/* Sec. 3.2: may query token i attend key token j?  (image `bi` of the batch) */
int32_t spvo_allowed(const spvo_attn_desc* d, int32_t bi, int32_t i, int32_t j);

/* Sec. 3.2: masked softmax attention by the definition, one query at a time.
 * q,k,v,o: fp32 [batch, N, heads, head_dim] contiguous, N = G + n_patch.
 * cls_scores: optional fp32 [batch, heads, n_patch]: softmax row of token 0 at
 * the patch columns (Sec. 3.3 importance scores before head averaging).
 * rows / n_rows: optional list of query token indices to compute (all when
 * rows == NULL); other rows of o are left untouched. */
int32_t spvo_attention(const spvo_attn_desc* d, const float* q, const float* k,
                       const float* v, float* o, float* cls_scores,
                       const int32_t* rows, int32_t n_rows);

/* Plain dense softmax attention, written separately (pins spvo_attention). */
int32_t spvo_dense_attention(int32_t batch, int32_t n_tok, int32_t heads,
                             int32_t head_dim, float scale, const float* q,
                             const float* k, const float* v, float* o);

/* Sec. 3.3: number of patch tokens kept, k = ceil(keep_ratio * n_patch). */
int32_t spvo_keep_count(int32_t n_patch, double keep_ratio);

/* Sec. 3.3: head average (fp32, heads summed in index order, then divided),
 * rank by (mean desc, index asc), keep the first k, emit indices ascending and
 * gather token rows (2-byte elements, copied as bytes), globals first.
 * scores [batch, heads, n_patch]; tokens_in [batch, G+n_patch, dim] (uint16);
 * tokens_out [batch, G+k, dim]; kept_idx [batch, k]; mean_scores optional
 * [batch, n_patch].  tokens_in/tokens_out may be NULL (indices only). */
int32_t spvo_filter(int32_t batch, int32_t heads, int32_t n_patch,
                    int32_t n_global, int32_t dim, double keep_ratio,
                    const float* scores, const uint16_t* tokens_in,
                    uint16_t* tokens_out, int32_t* kept_idx,
                    float* mean_scores);

enum { SPVO_MLP_GELU = 0, SPVO_MLP_SWIGLU = 1 };
enum { SPVO_ATTN_DENSE = 0, SPVO_ATTN_SPARSE = 1 };

typedef struct {
  int32_t layers, dim, heads, mlp_hidden, mlp_kind, patch, n_global;
  int32_t has_layerscale;
  float ln_eps;
  int32_t attn_mode, block, radius;
  int32_t filter_layer;        /* 0 = off; f => after block f (1-based)        */
  double keep_ratio;
  /* Several filter stages (Sec. 3.3 applied more than once): stage s runs
   * after block filter_layers[s] (1-based, strictly increasing) and keeps
   * ceil(keep_ratios[s] * tokens present).  n_filters == 0: the single stage
   * (filter_layer, keep_ratio) above, if filter_layer > 0. */
  int32_t n_filters;
  int32_t filter_layers[4];
  double keep_ratios[4];
} spvo_vit_config;

typedef struct {
  const float *ln1_g, *ln1_b;      /* [dim]                                    */
  const float *w_qkv, *b_qkv;      /* [3*dim, dim], [3*dim]; rows: q | k | v,
                                      each head-major (head*head_dim + e)      */
  const float *w_o, *b_o;          /* [dim, dim], [dim]                        */
  const float *ls1;                /* [dim] or NULL                            */
  const float *ln2_g, *ln2_b;
  const float *w_fc1, *b_fc1;      /* [hidden, dim]                            */
  const float *w_fc3, *b_fc3;      /* SwiGLU second input projection, or NULL  */
  const float *w_fc2, *b_fc2;      /* [dim, hidden]                            */
  const float *ls2;
} spvo_layer_weights;

typedef struct {
  const float *w_pe, *b_pe;        /* [dim, 3*patch*patch] (c, py, px), [dim]  */
  const float *cls;                /* [G, dim]                                 */
  const float *pos;                /* [G + H*W, dim], already at the grid size */
  const float *lnf_g, *lnf_b;
  const spvo_layer_weights* layer; /* [layers]                                 */
} spvo_vit_weights;

/* Whole forward.  image fp32 [batch, 3, H*patch, W*patch].
 * out_tokens fp32 [batch, G+k, dim] after the final LayerNorm (k = tokens left
 * by the last stage; H*W when the filter is off).  kept_idx optional
 * [batch, k_1 + ... + k_S]: per image the kept sets of the stages one after
 * the other, each as ascending ORIGINAL grid positions.  forced_keep optional,
 * same layout: bypass the ranking of every stage (teacher forcing).
 * tap_layer / tap_x optional: copy of the residual stream [batch, N_l, dim]
 * after block tap_layer (1-based; 0 = after patch embedding). */
int32_t spvo_vit_forward(const spvo_vit_config* c, const spvo_vit_weights* w,
                         const float* image, int32_t batch, int32_t grid_h,
                         int32_t grid_w, float* out_tokens, int32_t* kept_idx,
                         const int32_t* forced_keep, int32_t tap_layer,
                         float* tap_x);

/* Building blocks of the forward, exported so that each can be pinned alone. */
void spvo_layernorm(const float* x, int64_t rows, int32_t dim, const float* g,
                    const float* b, float eps, float* y);
void spvo_linear(const float* x, int64_t rows, int32_t in_dim, int32_t out_dim,
                 const float* w /*[out,in]*/, const float* bias, float* y);
float spvo_gelu(float x);
float spvo_silu(float x);
/* The same two activations over arrays: y[i] = gelu(a[i]);  y[i] = silu(a[i]) * b[i]. */
void spvo_gelu_n(const float* a, int64_t n, float* y);
void spvo_silu_mul_n(const float* a, const float* b, int64_t n, float* y);

int32_t spvo_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
