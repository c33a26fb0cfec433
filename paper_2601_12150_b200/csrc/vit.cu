// Sec. 3 / Sec. 4.1 -- the ViT backbone run with neighbouring-block sparse attention (Sec. 3.2)
// and the global-attention-score token filter (Sec. 3.3): a fixed kernel sequence on one stream.
//
// Internal token order: global tokens first, then patch tokens in BLOCK-MAJOR order (grouped by
// spatial block, blocks row-major over the block grid, ascending position inside a block).  The
// attention kernel then reads Q/K/V straight out of the QKV GEMM's output with no regrouping
// copy in any layer, and the filter's stable compaction keeps the order block-major.  Only the
// final LayerNorm scatters rows back to ascending original position, the exported order.
// The filter may run after several blocks (up to SPV_MAX_FILTERS stages): every stage ranks over the whole
// grid (positions that are gone rank last), marks the kept positions, compacts the residual stream and the
// position list into the other of two buffers and rebuilds the attention plan from the new positions.
//
// The residual stream stays fp32 (LayerNorm reads it, the GEMM epilogues add into it); every
// GEMM operand is bf16.
#include "attention.cuh"
#include "filter.cuh"

namespace {

// ------------------------------------------------------------------------------------------
// small kernels around the GEMMs
// ------------------------------------------------------------------------------------------

// Block-major ordinal t of the full grid -> original position, and the inverse table.
__global__ void vit_bm_tables(int H, int W, int b, int nbx, int32_t* __restrict__ bm_pos,
                              int32_t* __restrict__ bm_of_pos, int batch) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int np = H * W;
  if (t >= np) return;
  const int row_tokens = b * W;                 // every block row above the last one is full height
  const int by = t / row_tokens;
  int rem = t - by * row_tokens;
  const int bh = min(b, H - by * b);
  int bx = rem / (bh * b);
  if (bx > nbx - 1) bx = nbx - 1;
  rem -= bx * bh * b;
  const int bw = min(b, W - bx * b);
  const int pos = (by * b + rem / bw) * W + bx * b + rem % bw;
  for (int i = 0; i < batch; ++i) bm_pos[(size_t)i * np + t] = pos;
  bm_of_pos[pos] = t;
}

// pos_bm[t, :] = pos[G + bm_pos[t], :]   (fp32 rows, 128-bit copies)
__global__ void vit_permute_pos(const float4* __restrict__ pos, const int32_t* __restrict__ bm_pos, int n_global,
                                int np, int dvec, float4* __restrict__ pos_bm) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)np * dvec) return;
  const int t = (int)(i / dvec), c = (int)(i % dvec);
  pos_bm[i] = __ldg(pos + (int64_t)(n_global + __ldg(bm_pos + t)) * dvec + c);
}

// Global token rows of the embedding: x[b, g, :] = cls[g, :] + pos[g, :]
__global__ void vit_global_rows(const float* __restrict__ cls, const float* __restrict__ pos, int n_global, int dim,
                                int64_t n_tok, float* __restrict__ x) {
  const int b = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_global * dim) return;
  x[(int64_t)b * n_tok * dim + i] = cls[i] + pos[i];
}

// im2col of non-overlapping patches into bf16 rows ordered block-major:
//   A[b * np + bm_of_pos[y/P * W + x/P], (c * P + y % P) * P + x % P] = image[b, c, y, x]
// One thread per pixel; reads are coalesced along x, writes are runs of P consecutive bf16.
__global__ void __launch_bounds__(256) vit_im2col(const float* __restrict__ image, int P, int gh, int gw,
                                                  const int32_t* __restrict__ bm_of_pos, int kpad,
                                                  __nv_bfloat16* __restrict__ a) {
  const int wpix = gw * P, hpix = gh * P;
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  const int y = blockIdx.y;
  const int bc = blockIdx.z;          // b * 3 + c
  if (x >= wpix) return;
  const int b = bc / 3, c = bc % 3;
  const float v = __ldg(image + ((int64_t)bc * hpix + y) * wpix + x);
  const int t = __ldg(bm_of_pos + (y / P) * gw + x / P);
  a[((int64_t)b * gh * gw + t) * kpad + (c * P + y % P) * P + x % P] = __float2bfloat16(v);
}

// The same for patch sizes that are multiples of 8: one thread per 8 pixels of a patch row
// (two 128-bit loads, one 128-bit store).
__global__ void __launch_bounds__(256) vit_im2col_x8(const float* __restrict__ image, int P, int gh, int gw,
                                                     const int32_t* __restrict__ bm_of_pos, int kpad,
                                                     __nv_bfloat16* __restrict__ a) {
  const int wpix = gw * P, hpix = gh * P;
  const int x = (blockIdx.x * blockDim.x + threadIdx.x) * 8;
  const int y = blockIdx.y;
  const int bc = blockIdx.z;          // b * 3 + c
  if (x >= wpix) return;
  const int b = bc / 3, c = bc % 3;
  const float4* src = reinterpret_cast<const float4*>(image + ((int64_t)bc * hpix + y) * wpix + x);
  const float4 v0 = __ldcs(src), v1 = __ldcs(src + 1);
  const int t = __ldg(bm_of_pos + (y / P) * gw + x / P);
  uint4 o;
  o.x = spv::pack_bf16(v0.x, v0.y); o.y = spv::pack_bf16(v0.z, v0.w);
  o.z = spv::pack_bf16(v1.x, v1.y); o.w = spv::pack_bf16(v1.z, v1.w);
  *reinterpret_cast<uint4*>(a + ((int64_t)b * gh * gw + t) * kpad + (c * P + y % P) * P + x % P) = o;
}

// Zero the padding columns kp .. kpad-1 of a [rows, kpad] bf16 matrix.
__global__ void vit_zero_pad(__nv_bfloat16* __restrict__ a, int64_t rows, int kp, int kpad) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int npad = kpad - kp;
  if (i >= rows * npad) return;
  a[(i / npad) * kpad + kp + i % npad] = __float2bfloat16(0.f);
}

// w_pad[d, 0..kpad) = w[d, 0..kp) padded with zeros (row stride becomes a multiple of 16 bytes)
__global__ void vit_pad_weight(const __nv_bfloat16* __restrict__ w, int rows, int kp, int kpad,
                               __nv_bfloat16* __restrict__ w_pad) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)rows * kpad) return;
  const int r = (int)(i / kpad), c = (int)(i % kpad);
  w_pad[i] = c < kp ? w[(int64_t)r * kp + c] : __float2bfloat16(0.f);
}

// mark[b, pos] = 1 for every kept original position (mark zeroed beforehand).  kept: [batch] rows of k
// entries, `stride` apart.  The entries have to be inside the grid, strictly ascending and, for a later
// stage, marked by the stage before (prev_mark); the first violation is latched in the status word.
__global__ void vit_mark_kept(const int32_t* __restrict__ kept, int64_t stride, int k, int np,
                              float* __restrict__ mark, const float* __restrict__ prev_mark,
                              uint32_t* __restrict__ status) {
  const int b = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= k) return;
  const int pos = __ldg(kept + (size_t)b * stride + i);
  bool ok = pos >= 0 && pos < np;
  if (ok && i > 0) ok = __ldg(kept + (size_t)b * stride + i - 1) < pos;
  if (ok && prev_mark) ok = prev_mark[(size_t)b * np + pos] != 0.0f;
  if (ok) mark[(size_t)b * np + pos] = 1.0f;
  else atomicCAS(status, 0u, SPV_SITE_BAD_KEPT_INDEX);
}

// mask_bm[b, t] = mark[b, cur_pos[b, t]] for the n_cur tokens present: the kept set as a one-head score
// row over the internal token order; ranking it keeps exactly the marked tokens, in internal order.
__global__ void vit_mask_to_order(const float* __restrict__ mark, const int32_t* __restrict__ cur_pos, int n_cur,
                                  int np_grid, float* __restrict__ mask_bm) {
  const int b = blockIdx.y;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_cur) return;
  mask_bm[(size_t)b * n_cur + t] = mark[(size_t)b * np_grid + __ldg(cur_pos + (size_t)b * n_cur + t)];
}

// Destination row of every internal row for the final LayerNorm.  Unfiltered: G + position.
__global__ void vit_out_rows_full(const int32_t* __restrict__ bm_pos, int n_global, int np,
                                  int32_t* __restrict__ out_row) {
  const int b = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int n = n_global + np;
  if (i >= n) return;
  out_row[(size_t)b * n + i] = b * n + (i < n_global ? i : n_global + __ldg(bm_pos + (size_t)b * np + i - n_global));
}

// Filtered: rank of each kept position among the kept positions (exclusive scan of the marks
// over the grid), one CTA per image.
__global__ void __launch_bounds__(1024) vit_out_rows_kept(const float* __restrict__ mark, int np_grid,
                                                          const int32_t* __restrict__ pos_kept, int k, int n_global,
                                                          int32_t* __restrict__ rank_ws,
                                                          int32_t* __restrict__ out_row) {
  __shared__ int warp_sums[32];
  __shared__ int carry_s;
  const int b = blockIdx.x;
  const float* mk = mark + (size_t)b * np_grid;
  int32_t* rk = rank_ws + (size_t)b * np_grid;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < np_grid; base += 1024) {
    const int i = base + threadIdx.x;
    const int v = (i < np_grid && mk[i] != 0.0f) ? 1 : 0;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int n = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += n; }
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      int w = warp_sums[lane], s = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { int n = __shfl_up_sync(0xffffffffu, s, o); if (lane >= o) s += n; }
      warp_sums[lane] = s - w;
    }
    __syncthreads();
    const int excl = carry_s + warp_sums[warp] + inc - v;
    if (i < np_grid) rk[i] = excl;
    __syncthreads();
    if (threadIdx.x == 1023) carry_s = excl + v;
    __syncthreads();
  }
  const int n = n_global + k;
  for (int i = threadIdx.x; i < n; i += 1024)
    out_row[(size_t)b * n + i] =
        b * n + (i < n_global ? i : n_global + rk[__ldg(pos_kept + (size_t)b * k + i - n_global)]);
}

// ------------------------------------------------------------------------------------------
// workspace layout
// ------------------------------------------------------------------------------------------
struct VitLayout {
  int32_t np0, n0, k, k1, n1, kp, kpad, nbx, nby;
  // filter stages: block after which each runs, tokens it keeps, entries per image over all stages
  int32_t n_stage, st_layer[SPV_MAX_FILTERS], st_k[SPV_MAX_FILTERS], k_total;
  size_t x0, x1, h, qkv, o, h1, h3, im2col, w_pe_pad, pos_bm, scores, mask, mark, mark2, rank, bm_pos, bm_of_pos, pos2,
      pos3, kept_bm, kept_rm, out_row, head_stats, plan, plan_bytes, glob, glob_bytes, filt, filt_bytes, total;
};

int32_t vit_layout(const spv_vit_config* c, int32_t batch, int32_t gh, int32_t gw, VitLayout* L) {
  if (!c || batch < 1 || gh < 1 || gw < 1) return SPV_ERR_INVALID_ARG;
  if (c->layers < 1 || c->dim < 64 || c->heads < 1 || c->mlp_hidden < 8 || c->patch < 1) return SPV_ERR_INVALID_ARG;
  if (c->dim != c->heads * 64) return SPV_ERR_UNSUPPORTED;               // head_dim 64 only
  if (c->dim % 8 || c->mlp_hidden % 8) return SPV_ERR_ALIGNMENT;
  if (c->n_global < 1 || c->n_global > 16) return SPV_ERR_UNSUPPORTED;
  if (c->mlp_kind != SPV_MLP_GELU && c->mlp_kind != SPV_MLP_SWIGLU) return SPV_ERR_INVALID_ARG;
  if (c->attn_mode != SPV_ATTN_DENSE && c->attn_mode != SPV_ATTN_SPARSE) return SPV_ERR_INVALID_ARG;
  if (c->block < 1 || c->radius < 0) return SPV_ERR_INVALID_ARG;
  if ((int64_t)gh * gw > (1 << 24)) return SPV_ERR_UNSUPPORTED;
  const int32_t G = c->n_global, D = c->dim, HID = c->mlp_hidden;
  L->np0 = gh * gw;
  L->n0 = G + L->np0;
  // the filter stages
  double st_keep[SPV_MAX_FILTERS];
  L->n_stage = 0;
  if (c->n_filters < 0 || c->n_filters > SPV_MAX_FILTERS) return SPV_ERR_INVALID_ARG;
  if (c->n_filters == 0) {
    if (c->filter_layer < 0 || c->filter_layer > c->layers) return SPV_ERR_INVALID_ARG;
    if (c->filter_layer > 0) { L->n_stage = 1; L->st_layer[0] = c->filter_layer; st_keep[0] = c->keep_ratio; }
  } else {
    L->n_stage = c->n_filters;
    for (int s = 0; s < L->n_stage; ++s) {
      L->st_layer[s] = c->filter_layers[s];
      st_keep[s] = c->keep_ratios[s];
      if (L->st_layer[s] < 1 || L->st_layer[s] > c->layers) return SPV_ERR_INVALID_ARG;
      if (s > 0 && L->st_layer[s] <= L->st_layer[s - 1]) return SPV_ERR_INVALID_ARG;
    }
  }
  L->k = L->np0;
  L->k_total = 0;
  for (int s = 0; s < L->n_stage; ++s) {
    int32_t st = spv_filter_keep_count(L->k, st_keep[s], &L->st_k[s]);
    if (st != SPV_OK) return st;
    L->k = L->st_k[s];
    L->k_total += L->k;
  }
  L->k1 = L->n_stage > 0 ? L->st_k[0] : L->np0;      // the longest sequence after a filter
  L->n1 = G + L->k1;
  L->kp = 3 * c->patch * c->patch;
  L->kpad = (int32_t)spv_align_up((size_t)L->kp, 8);
  L->nby = (gh + c->block - 1) / c->block;
  L->nbx = (gw + c->block - 1) / c->block;
  const size_t rows = (size_t)batch * L->n0;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t r = off; off += spv_align_up(bytes, 256); return r; };
  L->x0 = take(rows * D * 4);
  L->x1 = take(L->n_stage > 0 ? (size_t)batch * L->n1 * D * 4 : 0);
  L->h = take(rows * D * 2);
  L->qkv = take(rows * 3 * D * 2);
  L->o = take(rows * D * 2);
  const size_t im2col_bytes = (size_t)batch * L->np0 * L->kpad * 2;
  const size_t h1_bytes = rows * HID * 2;
  L->h1 = take(h1_bytes > im2col_bytes ? h1_bytes : im2col_bytes);   // the im2col matrix lives here first
  L->im2col = L->h1;
  L->h3 = take(c->mlp_kind == SPV_MLP_SWIGLU ? rows * HID * 2 : 0);
  L->w_pe_pad = take((size_t)D * L->kpad * 2);
  L->pos_bm = take((size_t)L->np0 * D * 4);
  L->scores = take(c->unfused_filter ? (size_t)batch * c->heads * L->np0 * 4 : 0);
  L->head_stats = take((size_t)batch * c->heads * 2 * 4);
  L->mask = take((size_t)batch * L->np0 * 4);
  L->mark = take((size_t)batch * L->np0 * 4);
  L->mark2 = take(L->n_stage > 1 ? (size_t)batch * L->np0 * 4 : 0);
  L->rank = take((size_t)batch * L->np0 * 4);
  L->bm_pos = take((size_t)batch * L->np0 * 4);
  L->bm_of_pos = take((size_t)L->np0 * 4);
  L->pos2 = take((size_t)batch * L->k1 * 4);
  L->pos3 = take(L->n_stage > 1 ? (size_t)batch * L->k1 * 4 : 0);
  L->kept_bm = take((size_t)batch * L->k1 * 4);
  L->kept_rm = take((size_t)batch * L->k1 * 4);
  L->out_row = take(rows * 4);
  L->plan_bytes = spv_attn_plan_bytes(batch, gh, gw, c->block, L->np0, SPV_TOKENS_BLOCK_MAJOR);
  L->plan = take(L->plan_bytes);
  L->glob_bytes = spv_attn_global_bytes(batch, G, c->heads, L->n0);
  L->glob = take(L->glob_bytes);
  spv_filter_desc fd{};
  fd.batch = batch; fd.heads = c->heads; fd.n_patch = L->np0; fd.n_global = G; fd.dim = 2 * D;
  fd.keep_ratio = 1.0;
  size_t fb = 0;
  int32_t st = spv_filter_workspace_size(&fd, &fb);
  if (st != SPV_OK) return st;
  L->filt_bytes = fb;
  L->filt = take(fb);
  L->total = off;
  return SPV_OK;
}

inline unsigned cdiv(int64_t a, int64_t b) { return (unsigned)((a + b - 1) / b); }

}  // namespace

extern "C" int32_t spv_vit_workspace_size(const spv_vit_config* cfg, int32_t batch, int32_t grid_h, int32_t grid_w,
                                          size_t* bytes) {
  if (!bytes) return SPV_ERR_INVALID_ARG;
  VitLayout L;
  int32_t st = vit_layout(cfg, batch, grid_h, grid_w, &L);
  if (st != SPV_OK) return st;
  *bytes = L.total;
  return SPV_OK;
}

extern "C" int32_t vit_forward(spv_ctx* ctx, const spv_vit_config* c, const spv_vit_weights* w, const float* image,
                               int32_t batch, int32_t gh, int32_t gw, void* out_tokens, int32_t* kept_idx,
                               const int32_t* forced_keep, void* workspace, size_t workspace_bytes, void* stream_) {
  if (!ctx || !w || !image || !out_tokens || !w->layer) return SPV_ERR_INVALID_ARG;
  if (spv_on_device(ctx) != SPV_OK) return SPV_ERR_INVALID_ARG;
  VitLayout L;
  int32_t st = vit_layout(c, batch, gh, gw, &L);
  if (st != SPV_OK) return st;
  if (!workspace || workspace_bytes < L.total || ((uintptr_t)workspace & 255u)) return SPV_ERR_WORKSPACE;
  if (forced_keep && L.n_stage == 0) return SPV_ERR_INVALID_ARG;
  if (!w->w_pe || !w->cls || !w->pos || !w->lnf_g || !w->lnf_b) return SPV_ERR_INVALID_ARG;
  if (((uintptr_t)image & 15u) || ((uintptr_t)out_tokens & 15u)) return SPV_ERR_ALIGNMENT;
  cudaStream_t stream = (cudaStream_t)stream_;
  char* ws = (char*)workspace;
  const int32_t G = c->n_global, D = c->dim, HID = c->mlp_hidden, P = c->patch, H = c->heads;
  const int32_t np0 = L.np0;
  float* x = (float*)(ws + L.x0);
  float* x_alt = (float*)(ws + L.x1);
  __nv_bfloat16* hbuf = (__nv_bfloat16*)(ws + L.h);
  __nv_bfloat16* qkv = (__nv_bfloat16*)(ws + L.qkv);
  __nv_bfloat16* obuf = (__nv_bfloat16*)(ws + L.o);
  __nv_bfloat16* h1 = (__nv_bfloat16*)(ws + L.h1);
  __nv_bfloat16* h3 = (__nv_bfloat16*)(ws + L.h3);
  __nv_bfloat16* acol = (__nv_bfloat16*)(ws + L.im2col);
  __nv_bfloat16* w_pe_pad = (__nv_bfloat16*)(ws + L.w_pe_pad);
  float* pos_bm = (float*)(ws + L.pos_bm);
  float* scores = (float*)(ws + L.scores);
  float* head_stats = (float*)(ws + L.head_stats);
  const float* cls_logits = nullptr;
  float* mask = (float*)(ws + L.mask);
  float* mark = (float*)(ws + L.mark);
  float* mark2 = (float*)(ws + L.mark2);
  int32_t* rank = (int32_t*)(ws + L.rank);
  int32_t* bm_pos = (int32_t*)(ws + L.bm_pos);
  int32_t* bm_of_pos = (int32_t*)(ws + L.bm_of_pos);
  int32_t* pos2 = (int32_t*)(ws + L.pos2);
  int32_t* pos3 = (int32_t*)(ws + L.pos3);
  int32_t* kept_bm = (int32_t*)(ws + L.kept_bm);
  int32_t* kept_rm = (int32_t*)(ws + L.kept_rm);
  int32_t* out_row = (int32_t*)(ws + L.out_row);

  // ---- token order tables, patch embedding (a1)
  SpvProfScope* prof_misc = new SpvProfScope(ctx, SPV_K_MISC, stream);
  vit_bm_tables<<<cdiv(np0, 256), 256, 0, stream>>>(gh, gw, c->block, L.nbx, bm_pos, bm_of_pos, batch);
  vit_permute_pos<<<cdiv((int64_t)np0 * (D / 4), 256), 256, 0, stream>>>((const float4*)w->pos, bm_pos, G, np0,
                                                                          D / 4, (float4*)pos_bm);
  vit_global_rows<<<dim3(cdiv(G * D, 256), batch), 256, 0, stream>>>(w->cls, w->pos, G, D, L.n0, x);
  if (P % 8 == 0)
    vit_im2col_x8<<<dim3(cdiv(gw * P / 8, 256), gh * P, batch * 3), 256, 0, stream>>>(image, P, gh, gw, bm_of_pos,
                                                                                     L.kpad, acol);
  else
    vit_im2col<<<dim3(cdiv(gw * P, 256), gh * P, batch * 3), 256, 0, stream>>>(image, P, gh, gw, bm_of_pos, L.kpad,
                                                                              acol);
  int launches = 4;
  const void* w_pe = w->w_pe;
  if (L.kpad != L.kp) {
    vit_zero_pad<<<cdiv((int64_t)batch * np0 * (L.kpad - L.kp), 256), 256, 0, stream>>>(acol, (int64_t)batch * np0,
                                                                                       L.kp, L.kpad);
    vit_pad_weight<<<cdiv((int64_t)D * L.kpad, 256), 256, 0, stream>>>((const __nv_bfloat16*)w->w_pe, D, L.kp,
                                                                        L.kpad, w_pe_pad);
    w_pe = w_pe_pad;
    launches += 2;
  }
  delete prof_misc;
  if ((st = spv_launch_ok(ctx, launches)) != SPV_OK) return st;
  for (int b = 0; b < batch; ++b) {
    spv_gemm_desc g{};
    g.m = np0; g.n = D; g.k = L.kpad; g.lda = L.kpad; g.ldw = L.kpad; g.ldo = D;
    g.epilogue = SPV_EPI_BIAS_ADDROW; g.bias = w->b_pe; g.addrow = pos_bm; g.ldadd = D; g.rows_per_image = np0;
    if ((st = spv_gemm_bf16(ctx, &g, acol + (size_t)b * np0 * L.kpad, w_pe, x + ((size_t)b * L.n0 + G) * D,
                            stream)) != SPV_OK)
      return st;
  }

  // ---- attention plan of the full grid
  const int radius = c->attn_mode == SPV_ATTN_DENSE ? (L.nby > L.nbx ? L.nby : L.nbx) : c->radius;
  SpvAttnPlan plan;
  if ((st = spv_attn_plan_build(ctx, batch, gh, gw, c->block, radius, G, np0, nullptr, SPV_TOKENS_BLOCK_MAJOR,
                                ws + L.plan, L.plan_bytes, stream, &plan)) != SPV_OK)
    return st;

  int32_t np = np0;            // patch tokens currently present
  int64_t n = L.n0;            // tokens per image
  const int32_t* cur_pos = bm_pos;
  int stage = 0;               // next filter stage
  int32_t k_before = 0;        // entries of the earlier stages in kept_idx / forced_keep
  const float* last_mark = nullptr;
  for (int l = 1; l <= c->layers; ++l) {
    const spv_layer_weights* lw = &w->layer[l - 1];
    if (!lw->ln1_g || !lw->ln1_b || !lw->w_qkv || !lw->w_o || !lw->ln2_g || !lw->ln2_b || !lw->w_fc1 || !lw->w_fc2)
      return SPV_ERR_INVALID_ARG;
    if (c->mlp_kind == SPV_MLP_SWIGLU && !lw->w_fc3) return SPV_ERR_INVALID_ARG;
    const int64_t rows = (int64_t)batch * n;
    // attention branch: x += ls1 * (Attn(LN1 x) W_o^T + b_o)      (a2, a3, a4, a5, a6)
    if ((st = spv_layernorm(ctx, x, rows, D, lw->ln1_g, lw->ln1_b, c->ln_eps, hbuf, nullptr, stream)) != SPV_OK)
      return st;
    {
      spv_gemm_desc g{};
      g.m = (int32_t)rows; g.n = 3 * D; g.k = D; g.lda = D; g.ldw = D; g.ldo = 3 * D;
      g.epilogue = SPV_EPI_BIAS; g.bias = lw->b_qkv;
      if ((st = spv_gemm_bf16(ctx, &g, hbuf, lw->w_qkv, qkv, stream)) != SPV_OK) return st;
    }
    {
      SpvAttnIO io;
      io.q = qkv; io.k = qkv + D; io.v = qkv + 2 * D;
      io.sb = n * 3 * D; io.st = 3 * D; io.sh = 64;
      io.o = obuf; io.o_sb = n * D; io.o_st = D; io.o_sh = 64; io.o_tok = nullptr;
      io.heads = H; io.scale = 0.125f;
      if ((st = spv_attn_run_patches(ctx, &plan, &io, stream)) != SPV_OK) return st;
      // CLS->patch scores land at the tokens' ORIGINAL positions, so that the ranking breaks
      // ties by the lower original index
      const bool want_scores = stage < L.n_stage && l == L.st_layer[stage] && !forced_keep;
      if (want_scores && !c->unfused_filter) {
        // fused: the global kernels leave the logits and per-head (maximum, 1 / sum); the filter's first kernel
        // evaluates the weights itself, so the [batch, heads, patches] score tensor is never written
        if ((st = spv_attn_run_globals(ctx, &plan, &io, nullptr, nullptr, np0, ws + L.glob, L.glob_bytes, stream,
                                       head_stats, &cls_logits)) != SPV_OK)
          return st;
      } else {
        // a later stage ranks over the whole grid: positions that are gone hold NaN, which ranks last
        if (want_scores && stage > 0)
          SPV_CUDA_OK(cudaMemsetAsync(scores, 0xFF, (size_t)batch * H * np0 * 4, stream));
        if ((st = spv_attn_run_globals(ctx, &plan, &io, want_scores ? scores : nullptr,
                                       want_scores ? cur_pos : nullptr, np0, ws + L.glob, L.glob_bytes, stream)) != SPV_OK)
          return st;
      }
    }
    {
      spv_gemm_desc g{};
      g.m = (int32_t)rows; g.n = D; g.k = D; g.lda = D; g.ldw = D; g.ldo = D;
      g.epilogue = SPV_EPI_BIAS_SCALE_RESID; g.bias = lw->b_o; g.scale = c->has_layerscale ? lw->ls1 : nullptr;
      if ((st = spv_gemm_bf16(ctx, &g, obuf, lw->w_o, x, stream)) != SPV_OK) return st;
    }
    // MLP branch: x += ls2 * MLP(LN2 x)                               (a2, a7)
    if ((st = spv_layernorm(ctx, x, rows, D, lw->ln2_g, lw->ln2_b, c->ln_eps, hbuf, nullptr, stream)) != SPV_OK)
      return st;
    const __nv_bfloat16* mlp_act = h1;
    {
      spv_gemm_desc g{};
      g.m = (int32_t)rows; g.n = HID; g.k = D; g.lda = D; g.ldw = D; g.ldo = HID;
      g.epilogue = c->mlp_kind == SPV_MLP_SWIGLU ? SPV_EPI_BIAS_SILU : SPV_EPI_BIAS_GELU; g.bias = lw->b_fc1;
      if ((st = spv_gemm_bf16(ctx, &g, hbuf, lw->w_fc1, h1, stream)) != SPV_OK) return st;
      if (c->mlp_kind == SPV_MLP_SWIGLU) {
        g.epilogue = SPV_EPI_BIAS_MUL; g.bias = lw->b_fc3; g.aux = h1; g.ldaux = HID;
        if ((st = spv_gemm_bf16(ctx, &g, hbuf, lw->w_fc3, h3, stream)) != SPV_OK) return st;
        mlp_act = h3;
      }
    }
    {
      spv_gemm_desc g{};
      g.m = (int32_t)rows; g.n = D; g.k = HID; g.lda = HID; g.ldw = HID; g.ldo = D;
      g.epilogue = SPV_EPI_BIAS_SCALE_RESID; g.bias = lw->b_fc2; g.scale = c->has_layerscale ? lw->ls2 : nullptr;
      if ((st = spv_gemm_bf16(ctx, &g, mlp_act, lw->w_fc2, x, stream)) != SPV_OK) return st;
    }

    // ---- Sec. 3.3: after a stage's block the lowest-scored patches leave the sequence (a8-a10)
    if (stage < L.n_stage && l == L.st_layer[stage]) {
      const int32_t k = L.st_k[stage];
      const int32_t* kept_positions;
      int64_t kept_stride;
      if (forced_keep) {
        kept_positions = forced_keep + k_before;
        kept_stride = L.k_total;
      } else {
        // rank on the head-averaged scores in original-position order -> ascending original indices
        if (!c->unfused_filter) {
          if ((st = spv_filter_rank_logits(ctx, batch, H, G, (int32_t)n, np0, k, cls_logits, head_stats, cur_pos,
                                           kept_rm, ws + L.filt, L.filt_bytes, stream)) != SPV_OK)
            return st;
        } else {
          spv_filter_desc fd{};
          fd.batch = batch; fd.heads = H; fd.n_patch = np0; fd.n_global = G; fd.dim = 0; fd.keep_ratio = 1.0;
          if ((st = spv_filter_run_k(ctx, &fd, k, scores, nullptr, nullptr, kept_rm, nullptr, nullptr, nullptr,
                                     ws + L.filt, L.filt_bytes, stream)) != SPV_OK)
            return st;
        }
        kept_positions = kept_rm;
        kept_stride = k;
      }
      // the kept set as a one-head score row over the internal order; ranking it compacts the
      // residual stream (fp32 rows copied as 2*D 16-bit elements) and the positions, order kept
      float* mk = (stage & 1) ? mark2 : mark;
      {
        SpvProfScope prof(ctx, SPV_K_MISC, stream);
        SPV_CUDA_OK(cudaMemsetAsync(mk, 0, (size_t)batch * np0 * 4, stream));
        vit_mark_kept<<<dim3(cdiv(k, 256), batch), 256, 0, stream>>>(kept_positions, kept_stride, k, np0, mk, last_mark,
                                                                     ctx->d_status + 1);
        vit_mask_to_order<<<dim3(cdiv(np, 256), batch), 256, 0, stream>>>(mk, cur_pos, np, np0, mask);
      }
      if ((st = spv_launch_ok(ctx, 2)) != SPV_OK) return st;
      float* x_next = (x == (float*)(ws + L.x0)) ? x_alt : (float*)(ws + L.x0);
      int32_t* pos_next = (cur_pos == pos2) ? pos3 : pos2;
      spv_filter_desc fd{};
      fd.batch = batch; fd.heads = 1; fd.n_patch = np; fd.n_global = G; fd.dim = 2 * D; fd.keep_ratio = 1.0;
      fd.in_stride_b = n * 2 * D; fd.out_stride_b = (int64_t)(G + k) * 2 * D;
      if ((st = spv_filter_run_k(ctx, &fd, k, mask, x, x_next, kept_bm, nullptr, cur_pos, pos_next, ws + L.filt,
                                 L.filt_bytes, stream)) != SPV_OK)
        return st;
      if (kept_idx)
        SPV_CUDA_OK(cudaMemcpy2DAsync(kept_idx + k_before, (size_t)L.k_total * 4, kept_positions,
                                      (size_t)kept_stride * 4, (size_t)k * 4, (size_t)batch, cudaMemcpyDeviceToDevice,
                                      stream));
      x = x_next;
      np = k;
      n = G + k;
      cur_pos = pos_next;
      last_mark = mk;
      k_before += k;
      ++stage;
      if ((st = spv_attn_plan_build(ctx, batch, gh, gw, c->block, radius, G, np, cur_pos, SPV_TOKENS_BLOCK_MAJOR,
                                    ws + L.plan, L.plan_bytes, stream, &plan)) != SPV_OK)
        return st;
    }
  }

  // ---- final LayerNorm, rows scattered back to ascending original position (a12)
  {
    SpvProfScope prof(ctx, SPV_K_MISC, stream);
    if (L.n_stage > 0) {
      vit_out_rows_kept<<<batch, 1024, 0, stream>>>(last_mark, np0, cur_pos, L.k, G, rank, out_row);
    } else {
      vit_out_rows_full<<<dim3(cdiv(L.n0, 256), batch), 256, 0, stream>>>(bm_pos, G, np0, out_row);
    }
  }
  if ((st = spv_launch_ok(ctx)) != SPV_OK) return st;
  return spv_layernorm(ctx, x, (int64_t)batch * n, D, w->lnf_g, w->lnf_b, c->ln_eps, out_tokens, out_row, stream);
}
