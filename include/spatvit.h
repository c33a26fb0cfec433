/*
 * libspatvit -- large-resolution ViT inference hot path for NVIDIA B200 (sm_100a).
 *
 * Two computations from the paper plus the ViT block around them:
 *   Sec. 3.2  spatially-aware neighbouring-block sparse attention with global tokens
 *             (spatial_block_attention);
 *   Sec. 3.3  global-attention-score token filter: CLS->patch scores averaged over heads,
 *             rank, discard the lowest share, compact the survivors (cls_score_topk_filter);
 *   Sec. 3 / Sec. 4.1  the unchanged ViT backbone run with both (vit_forward).
 *
 * Conventions for every entry point
 *   - plain C ABI; every function returns an int32_t status (SPV_OK == 0);
 *   - every tensor pointer is a DEVICE pointer owned by the caller unless the comment says
 *     host; the library never frees or keeps them after the call returns (weights excepted:
 *     see spv_vit_weights);
 *   - scratch memory is a caller-provided device workspace sized by the matching
 *     *_workspace_size query (device memory, 256-byte aligned);
 *   - `stream` is a cudaStream_t passed as void*; calls only enqueue work on it.  Argument
 *     errors are reported synchronously by the return value; device-side errors (a bounded
 *     wait that expired) are latched in the context and returned by spv_check();
 *   - token order: index 0..G-1 are the global tokens (CLS first), then patch tokens.  Patch
 *     token t sits at original grid position pos = patch_pos ? patch_pos[t] : t, y = pos / W,
 *     x = pos % W.  Spatial block of a patch: (y / block, x / block); edge blocks may be
 *     partial;
 *   - bf16 tensors are raw 2-byte values; all tensors 16-byte aligned.
 */
#ifndef SPATVIT_H
#define SPATVIT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  SPV_OK = 0,
  SPV_ERR_INVALID_ARG = 1, /* a size, ratio or pointer is out of its documented range      */
  SPV_ERR_UNSUPPORTED = 2, /* valid request outside this build (e.g. head_dim != 64)       */
  SPV_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or smaller than the query says */
  SPV_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed                          */
  SPV_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (reported by spv_check)   */
  SPV_ERR_ALIGNMENT = 6,   /* a tensor base or stride breaks the 16-byte rule              */
  SPV_ERR_STATIC_LIMIT = 7 /* request larger than the library's built-in scratch array     */
};

typedef struct spv_ctx spv_ctx; /* device id, device status word, cached driver entry points */

/* Create / destroy a context for CUDA device `device` (host calls; create allocates a few
 * bytes of device memory for the status words).  A context belongs to that device: every entry
 * point that takes it returns SPV_ERR_INVALID_ARG when another device is current on the calling
 * thread.  One context per device and per host thread that issues calls. */
int32_t spv_create(spv_ctx** out, int32_t device);
int32_t spv_destroy(spv_ctx* ctx);
/* Static description of a status code (host string, never NULL). */
const char* spv_status_string(int32_t status);
/* Synchronise `stream`, then return and clear the latched device-side status. */
int32_t spv_check(spv_ctx* ctx, void* stream);
/* Site code of the bounded wait that the last failing spv_check() reported (0 = none): the
 * kernel and barrier that gave up, for diagnosis. */
uint32_t spv_last_wait_site(const spv_ctx* ctx);
/* Self-test of the bounded-wait path (no counterpart in the paper): launches one CTA in which one
 * thread waits on a barrier that nobody arrives on.  The wait gives up after limit_ns (clamped to
 * 1 ms), latches site code 0x5E1F and the kernel returns; the next spv_check() on the stream
 * returns SPV_ERR_TIMEOUT, spv_last_wait_site() 0x5E1F, and the context stays usable. */
int32_t spv_selftest_wait(spv_ctx* ctx, uint32_t limit_ns, void* stream);
/* Number of kernels this context has launched so far (host counter, for accounting). */
int64_t spv_launch_count(const spv_ctx* ctx);

/* ------------------------------------------------------------------------------------------
 * Sec. 3.2 -- spatially-aware neighbouring-block sparse attention.
 *
 * For a patch query i in spatial block (by, bx) the key set is
 *   {global tokens}  U  {patch tokens whose block (cy, cx) has |cy-by| <= radius and
 *                        |cx-bx| <= radius}  (neighbourhood clipped at the grid border),
 * for a global query it is every token.  O_i = sum_j softmax_j(scale * <q_i, k_j>) v_j.
 * radius >= max(#block rows, #block cols) - 1 gives dense attention.  The N x N score matrix is
 * never materialised.
 * ---------------------------------------------------------------------------------------- */
enum { SPV_TOKENS_ROW_MAJOR = 0, SPV_TOKENS_BLOCK_MAJOR = 1 };

typedef struct {
  int32_t batch, grid_h, grid_w; /* patch grid H x W of the ORIGINAL image                      */
  int32_t block, radius;         /* block edge b in patches (the paper's window size); r blocks */
  int32_t n_global;              /* G >= 1 leading global tokens                                */
  int32_t heads, head_dim;       /* head_dim must be 64                                         */
  float softmax_scale;           /* 0 => 1/sqrt(head_dim)                                       */
  int32_t n_patch;               /* patch tokens present per image (== H*W when patch_pos NULL) */
  const int32_t* patch_pos;      /* device [batch, n_patch] original positions y*W+x, each
                                    position at most once per image, in the order token_order
                                    states (checked on the device: a violation is latched, the
                                    patch rows of o are then not written, and spv_check()
                                    reports SPV_ERR_INVALID_ARG and clears it); NULL = full grid */
  int32_t token_order;           /* SPV_TOKENS_ROW_MAJOR: patch tokens in ascending position.
                                    SPV_TOKENS_BLOCK_MAJOR: patch tokens sorted by (block row,
                                    block column, position); avoids the internal regrouping copy */
  int64_t stride_b, stride_tok, stride_head; /* in elements, shared by q, k, v and o; head_dim is
                                    contiguous; stride_tok and stride_head multiples of 8        */
} spv_attn_desc;

/* Bytes of device workspace spatial_block_attention needs for `desc` (host call). */
int32_t spv_attn_workspace_size(const spv_attn_desc* desc, size_t* bytes);

/* q, k, v: bf16 device tensors addressed as base + b*stride_b + tok*stride_tok +
 * head*stride_head + e.  o: bf16, same addressing, every token row is written.
 * cls_scores: optional fp32 device [batch, heads, n_patch]: softmax weights of query token 0
 * at the patch columns, indexed like the patch tokens (the importance scores of Sec. 3.3
 * before head averaging).  Asynchronous on `stream`. */
int32_t spatial_block_attention(spv_ctx* ctx, const spv_attn_desc* desc, const void* q,
                                const void* k, const void* v, void* o, float* cls_scores,
                                void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Sec. 3.3 -- global-attention-score token filter.
 *
 * mean_j = (sum over heads, in head order, fp32) / heads;  rank patch tokens by
 * (mean descending, index ascending) -- +0 and -0 tie, NaN ranks last;  keep the first
 * k = ceil(keep_ratio * n_patch) (discarding the floor(p * n_patch) lowest, keep_ratio = 1-p);
 * emit their indices in ascending order and copy their rows, global tokens first.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
  int32_t batch, heads, n_patch, n_global;
  int32_t dim;                       /* elements per token row (bf16), multiple of 8            */
  double keep_ratio;                 /* in (0, 1]                                               */
  int64_t in_stride_b, out_stride_b; /* elements between images; 0 => densely packed            */
} spv_filter_desc;

/* Host, pure: k for (n_patch, keep_ratio); SPV_ERR_INVALID_ARG outside (0, 1] or n_patch < 1. */
int32_t spv_filter_keep_count(int32_t n_patch, double keep_ratio, int32_t* k);
int32_t spv_filter_workspace_size(const spv_filter_desc* desc, size_t* bytes);

/* scores: fp32 device [batch, heads, n_patch].
 * tokens_in: bf16 device [batch, n_global + n_patch, dim]; tokens_out: bf16 device
 * [batch, n_global + k, dim]; both may be NULL together (indices only).
 * kept_idx: int32 device [batch, k], ascending patch indices in [0, n_patch).
 * mean_scores: optional fp32 device [batch, n_patch].
 * pos_in / pos_out: optional int32 device [batch, n_patch] / [batch, k]: pos_out[t] =
 * pos_in[kept_idx[t]] (carries original grid positions through the filter).
 * Asynchronous on `stream`. */
int32_t cls_score_topk_filter(spv_ctx* ctx, const spv_filter_desc* desc, const float* scores,
                              const void* tokens_in, void* tokens_out, int32_t* kept_idx,
                              float* mean_scores, const int32_t* pos_in, int32_t* pos_out,
                              void* workspace, size_t workspace_bytes, void* stream);

/* The token filter for callers that must not allocate device memory (the paper has no
 * counterpart; this is a packaging variant of cls_score_topk_filter, same kernels, same results).
 *
 * Who needs it: code that runs after an application has handed out all of its device memory
 * and forbids further allocation (an inference server with a fixed memory plan, a plug-in
 * inside a host program that owns the allocator), and code in a latency-critical loop where
 * cudaMalloc / cudaFree would synchronise the whole device.  Such callers can neither size a
 * workspace and allocate it nor create an spv_ctx (spv_create allocates), so this entry point
 * takes no context and no workspace: the head means and ranking keys live in a file-scope
 * device array of SPV_FILTER_STATIC_BYTES that every GPU holds from the moment the library is
 * loaded until the process exits.
 *
 * Limits and rules
 *   - batch * round_up(n_patch, 4) * 8 bytes must fit in SPV_FILTER_STATIC_BYTES (2 MiB: e.g.
 *     4 images of a 256 x 256 patch grid); larger requests return SPV_ERR_STATIC_LIMIT and
 *     launch nothing;
 *   - works on the CUDA device that is current on the calling thread.  The first call on a
 *     device looks up the array's device address (one cudaGetSymbolAddress, no allocation) and
 *     keeps it; make that first call before any stream capture begins;
 *   - all calls on one device share the array, and it keeps what the previous call left there.
 *     The kernels write every element they later read, so no clearing is needed, but two calls
 *     whose kernels can overlap on the GPU (different streams without an ordering) race on it:
 *     order them;
 *   - the call itself performs no cudaMalloc, cudaFree or other allocating routine; inputs and
 *     outputs are the caller's, exactly as for cls_score_topk_filter.  Asynchronous on `stream`;
 *   - having no context, its launches appear neither in spv_launch_count() nor in the per-class
 *     timing of spv_profile_enable(), and its errors are all returned by the call itself. */
#define SPV_FILTER_STATIC_BYTES (2u << 20)
int32_t cls_score_topk_filter_static(const spv_filter_desc* desc, const float* scores,
                                     const void* tokens_in, void* tokens_out, int32_t* kept_idx,
                                     float* mean_scores, const int32_t* pos_in, int32_t* pos_out,
                                     void* stream);

/* ------------------------------------------------------------------------------------------
 * Sec. 3 / Sec. 4.1 -- the ViT backbone run with sparse attention and the filter.
 *
 * Pre-LayerNorm encoder: x = patch_embed(image) + pos;  per block
 *   x += ls1 * (Attn(LN1 x) W_o + b_o);  x += ls2 * MLP(LN2 x);
 * after block `filter_layer` the residual stream is filtered with the CLS scores of that
 * block's attention (Sec. 3.3: the pruning comes after a few initial layers and shortens the
 * sequence for all later ones); output = final LayerNorm of the surviving tokens, global tokens
 * first, patches in ascending original position.  The filter may be applied at up to
 * SPV_MAX_FILTERS blocks: every stage ranks the tokens still present by that block's CLS
 * attention and keeps ceil(keep * present); survivors keep their original grid positions for
 * the neighbourhood rule of Sec. 3.2.
 * ---------------------------------------------------------------------------------------- */
enum { SPV_MLP_GELU = 0, SPV_MLP_SWIGLU = 1 };
enum { SPV_ATTN_DENSE = 0, SPV_ATTN_SPARSE = 1 };
enum { SPV_MAX_FILTERS = 4 };

typedef struct {
  int32_t layers, dim, heads, mlp_hidden;
  int32_t mlp_kind;       /* SPV_MLP_GELU (exact erf GELU) | SPV_MLP_SWIGLU (silu(xW1+b1)*(xW3+b3)) */
  int32_t patch;          /* patch edge in pixels                                               */
  int32_t n_global;
  int32_t has_layerscale;
  float ln_eps;
  int32_t attn_mode;      /* SPV_ATTN_DENSE | SPV_ATTN_SPARSE                                   */
  int32_t block, radius;
  int32_t filter_layer;   /* 0 = off; f => filter after block f (1-based)                       */
  double keep_ratio;
  int32_t n_filters;      /* 0: the single stage (filter_layer, keep_ratio) above.  s > 0: stage i
                             runs after block filter_layers[i] (1-based, strictly increasing) with
                             keep_ratios[i] in (0, 1]; filter_layer / keep_ratio are ignored      */
  int32_t filter_layers[SPV_MAX_FILTERS];
  double keep_ratios[SPV_MAX_FILTERS];
  int32_t unfused_filter; /* 0 (default): the CLS->patch weights are evaluated, averaged over the heads
                             and turned into ranking keys in one kernel; 1: the score tensor
                             [batch, heads, patches] is written first and then averaged (the two
                             standalone steps).  Same kept set either way                        */
} spv_vit_config;

/* Per-layer weights: matrices bf16 [out_features, in_features] row-major; vectors fp32. */
typedef struct {
  const float *ln1_g, *ln1_b;
  const void* w_qkv; const float* b_qkv; /* [3*dim, dim]: q | k | v, each head-major          */
  const void* w_o;   const float* b_o;   /* [dim, dim]                                         */
  const float* ls1;                      /* [dim] or NULL                                      */
  const float *ln2_g, *ln2_b;
  const void* w_fc1; const float* b_fc1; /* [hidden, dim]                                      */
  const void* w_fc3; const float* b_fc3; /* SwiGLU second input projection, else NULL          */
  const void* w_fc2; const float* b_fc2; /* [dim, hidden]                                      */
  const float* ls2;
} spv_layer_weights;

/* All pointers device pointers the caller keeps alive for the duration of the call; `layer`
 * is a HOST array of `layers` entries. */
typedef struct {
  const void* w_pe; const float* b_pe;   /* bf16 [dim, 3*patch*patch] (channel, py, px), [dim] */
  const float* cls;                      /* fp32 [G, dim]                                      */
  const float* pos;                      /* fp32 [G + H*W, dim], already at the grid size      */
  const float *lnf_g, *lnf_b;
  const spv_layer_weights* layer;        /* host [layers]                                      */
} spv_vit_weights;

int32_t spv_vit_workspace_size(const spv_vit_config* cfg, int32_t batch, int32_t grid_h,
                               int32_t grid_w, size_t* bytes);

/* image: fp32 device [batch, 3, grid_h*patch, grid_w*patch], already normalised.
 * out_tokens: bf16 device [batch, n_global + k, dim], k = tokens left by the last filter stage
 * (grid_h*grid_w when the filter is off).
 * kept_idx: optional int32 device [batch, k_1 + ... + k_S]: per image the kept sets of the S
 * stages one after the other, each as ascending original patch indices (one stage: [batch, k]).
 * forced_keep: optional int32 device array of the same layout that replaces the ranking of every
 * stage (teacher forcing for parity checks): each stage's entries strictly ascending, inside the
 * grid and a subset of the stage before; a violation is found on the device and reported by
 * spv_check() as SPV_ERR_INVALID_ARG (the output is then undefined).  Asynchronous on `stream`. */
int32_t vit_forward(spv_ctx* ctx, const spv_vit_config* cfg, const spv_vit_weights* weights,
                    const float* image, int32_t batch, int32_t grid_h, int32_t grid_w,
                    void* out_tokens, int32_t* kept_idx, const int32_t* forced_keep,
                    void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * Building blocks of vit_forward, exported so that each can be checked and timed alone.
 * ---------------------------------------------------------------------------------------- */
enum {
  SPV_EPI_BIAS = 0,        /* out bf16 = acc + bias                                          */
  SPV_EPI_BIAS_GELU = 1,   /* out bf16 = gelu(acc + bias)                                    */
  SPV_EPI_BIAS_SILU = 2,   /* out bf16 = silu(acc + bias)                                    */
  SPV_EPI_BIAS_MUL = 3,    /* out bf16 = (acc + bias) * aux   (aux bf16 [M, N])              */
  SPV_EPI_BIAS_SCALE_RESID = 4, /* resid fp32 [M, N] += scale[n] * (acc + bias) (scale NULL => 1) */
  SPV_EPI_BIAS_ADDROW = 5  /* resid fp32 [M, N] = acc + bias + addrow[(m % rows_per_image)]  */
};

/* The residual epilogue adds into `out` with fp32 add-reduce operations issued by the kernel (each
 * element receives exactly one add per call, so the result is deterministic); `out` must not be
 * read or written by other work on the GPU while the call runs.
 * C[M, N] = A[M, K] * W[N, K]^T (+ epilogue).  a, w: bf16 device, row-major with leading
 * dimensions lda, ldw (elements, multiples of 8); K multiple of 8.  out: bf16 [M, ldo] for the
 * bf16 epilogues, fp32 residual [M, ldo] for the residual ones.  bias fp32 [N] or NULL. */
typedef struct {
  int32_t m, n, k;
  int64_t lda, ldw, ldo;
  int32_t epilogue;
  const float* bias;
  const void* aux;        /* SPV_EPI_BIAS_MUL: bf16 [M, ldaux]                                */
  int64_t ldaux;
  const float* scale;     /* SPV_EPI_BIAS_SCALE_RESID: fp32 [N] or NULL                       */
  const float* addrow;    /* SPV_EPI_BIAS_ADDROW: fp32 [rows_per_image, ldadd]                */
  int64_t ldadd;
  int32_t rows_per_image;
} spv_gemm_desc;
int32_t spv_gemm_bf16(spv_ctx* ctx, const spv_gemm_desc* desc, const void* a, const void* w,
                      void* out, void* stream);

/* y bf16 [rows, dim] = LayerNorm(x fp32 [rows, dim]) * gamma + beta; dim multiple of 8.
 * out_row: optional int32 device [rows] destination row of each input row (NULL = identity). */
int32_t spv_layernorm(spv_ctx* ctx, const float* x, int64_t rows, int32_t dim, const float* gamma,
                      const float* beta, float eps, void* y, const int32_t* out_row, void* stream);

/* ------------------------------------------------------------------------------------------
 * Per-kernel-class device timing (CUDA events recorded on the launch stream around every
 * launch while enabled; a few hundred nanoseconds per launch).  Off by default.
 * ---------------------------------------------------------------------------------------- */
enum {
  SPV_K_GEMM = 0,          /* tcgen05 GEMMs (QKV, out-proj, MLP, patch embedding)              */
  SPV_K_ATTN_PATCH = 1,    /* sparse-attention flash kernel, patch queries                     */
  SPV_K_ATTN_GLOBAL = 2,   /* global-token rows and CLS->patch scores                          */
  SPV_K_ATTN_PLAN = 3,     /* block offsets / query tiles / regrouping copy                    */
  SPV_K_LAYERNORM = 4,
  SPV_K_FILTER_SELECT = 5, /* head mean + ranking                                              */
  SPV_K_FILTER_GATHER = 6, /* compaction copy of the surviving rows                            */
  SPV_K_MISC = 7,          /* im2col, position tables, output row map                          */
  SPV_K_COUNT = 8
};
typedef struct {
  int64_t launches;  /* timed launch groups of this class                                      */
  double ms;         /* summed device time                                                     */
  double work;       /* summed algorithmic work: FLOP for SPV_K_GEMM, bytes for LayerNorm and
                        the filter kernels, 0 where the caller has to count it                 */
} spv_kernel_stat;
/* enable != 0: start timing (and clear the accumulated figures); 0: stop. */
int32_t spv_profile_enable(spv_ctx* ctx, int32_t enable);
/* Wait for the recorded events, add them into `out` (host array of SPV_K_COUNT entries) and
 * clear the record. */
int32_t spv_profile_read(spv_ctx* ctx, spv_kernel_stat* out);

/* ------------------------------------------------------------------------------------------
 * Hardware rate probes (no counterpart in the paper): the rates the attention kernel's design is
 * argued from, measured on the device the context was created on.  Each probe runs its kernel twice
 * and times the second run; the call is synchronous on `stream`.
 *   SPV_MB_EX2           ex2.approx.ftz.f32, eight independent chains per thread; units = operations
 *   SPV_MB_SOFTMAX_BODY  inner body of the online softmax on 64 scores per thread (scale, 2^x, row
 *                        sum, bf16 pack); poly_per_8 in {0, 2, 4, 8} of every eight exponentials are
 *                        evaluated as a cubic on the multiply-add pipe; units = scores
 *   SPV_MB_MMA_SS / _TS  tcgen05.mma kind::f16 of m x n x 16 (m 64 or 128, n multiple of 16 up to
 *                        256), A from shared memory / from TMEM, one issuing thread per CTA, iters x 4
 *                        instructions rotating over `accumulators` TMEM accumulators; units = FLOP
 *   SPV_MB_L2_TMA        TMA tile loads of box_rows x 128 bytes from a buffer of at most 32 MB (so
 *                        that it stays in L2), `stages` loads in flight per CTA; units = bytes
 * buffer: device scratch, 256-byte aligned; SPV_MB_L2_TMA walks over it (give it 32 MB + 64 KB), the
 * other probes need 64 KB.  Contents are not preserved.
 * ---------------------------------------------------------------------------------------- */
enum { SPV_MB_EX2 = 0, SPV_MB_SOFTMAX_BODY = 1, SPV_MB_MMA_SS = 2, SPV_MB_MMA_TS = 3, SPV_MB_L2_TMA = 4 };
typedef struct {
  int32_t kind;
  int32_t ctas_per_sm; /* grid = SM count x this (1..4)                                          */
  int32_t threads;     /* per CTA, EX2 / SOFTMAX_BODY only                                       */
  int32_t iters;       /* loop trips per thread / issuing thread                                 */
  int32_t m, n;        /* MMA shape                                                              */
  int32_t box_rows, stages; /* L2_TMA                                                            */
  int32_t poly_per_8;  /* SOFTMAX_BODY                                                           */
  int32_t accumulators; /* MMA: consecutive instructions rotate over this many accumulators (1..8;
                           1 = the dependent chain of a K loop)                                  */
  int32_t issue_mode;   /* MMA: 0 = one thread alone runs the issue loop; 1 = its whole warp runs the
                           loop and an elected lane issues                                       */
  int32_t issuers;      /* MMA: warps of the CTA that issue concurrently, each on its own
                           accumulators (1..4)                                                   */
} spv_microbench_desc;
typedef struct {
  double ms;      /* CUDA-event time of the timed run                                            */
  double cycles;  /* SM cycles of the slowest CTA (clock64)                                      */
  double units;   /* work of the timed run, see above                                            */
  int32_t sm_count;
} spv_microbench_result;
int32_t spv_microbench(spv_ctx* ctx, const spv_microbench_desc* desc, void* buffer, size_t buffer_bytes,
                       void* stream, spv_microbench_result* out);

#ifdef __cplusplus
}
#endif
#endif /* SPATVIT_H */
