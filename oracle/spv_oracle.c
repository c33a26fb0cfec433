/*
 * CPU oracle (test infrastructure; see spv_oracle.h for the policy and pins).
 *
 * Every routine is the definition written out: explicit loops, fp64
 * reductions, no tiling, no neighbour lists, no fused steps.  OpenMP only
 * spreads independent rows over threads.
 */
#include "spv_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int32_t spvo_num_threads(void) {
#ifdef _OPENMP
  return (int32_t)omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/* Sec. 3.2 -- which (query, key) pairs survive the sparsification.           */
/*                                                                           */
/* Local windowed attention: a patch token attends to the patch tokens that  */
/* are spatially adjacent in the original pixel space; "adjacent" is read as */
/* "lies in a spatial block within `radius` blocks of the query's block, in  */
/* both directions, clipped at the image border" (the abstract's            */
/* neighbouring blocks).  Global attention: global tokens attend to every    */
/* token, and (BigBird-style, which Sec. 3.2 cites) every token attends to   */
/* the global tokens.                                                        */
/* ------------------------------------------------------------------------- */
static int32_t token_pos(const spvo_attn_desc* d, int32_t bi, int32_t tok) {
  int32_t t = tok - d->n_global;
  return d->patch_pos ? d->patch_pos[(int64_t)bi * d->n_patch + t] : t;
}

int32_t spvo_allowed(const spvo_attn_desc* d, int32_t bi, int32_t i, int32_t j) {
  if (i < d->n_global || j < d->n_global) return 1;
  int32_t pi = token_pos(d, bi, i), pj = token_pos(d, bi, j);
  int32_t yi = pi / d->grid_w, xi = pi % d->grid_w;
  int32_t yj = pj / d->grid_w, xj = pj % d->grid_w;
  int32_t dby = yi / d->block - yj / d->block;
  int32_t dbx = xi / d->block - xj / d->block;
  if (dby < 0) dby = -dby;
  if (dbx < 0) dbx = -dbx;
  return (dby <= d->radius && dbx <= d->radius) ? 1 : 0;
}

static double attn_scale(float s, int32_t head_dim) {
  return s != 0.0f ? (double)s : 1.0 / sqrt((double)head_dim);
}

/* Sec. 3.2 -- masked softmax attention, one (image, head, query) at a time:  */
/*   s_j = scale * <q_i, k_j> for allowed j;  p = softmax(s);  o_i = sum p_j v_j */
/* Sec. 3.3 -- the importance scores are the global token's attention        */
/* weights: p of query token 0 at the patch columns.                         */
int32_t spvo_attention(const spvo_attn_desc* d, const float* q, const float* k,
                       const float* v, float* o, float* cls_scores,
                       const int32_t* rows, int32_t n_rows) {
  const int32_t G = d->n_global, N = G + d->n_patch, H = d->heads, E = d->head_dim;
  if (d->batch < 1 || N < 1 || H < 1 || E < 1 || d->block < 1 || d->radius < 0) return 1;
  const double scale = attn_scale(d->softmax_scale, E);
  const int32_t nq = rows ? n_rows : N;
  const int64_t work = (int64_t)d->batch * H * nq;
  int32_t bad = 0;
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)N);
    double* acc = (double*)malloc(sizeof(double) * (size_t)E);
#pragma omp for schedule(dynamic, 16)
    for (int64_t wi = 0; wi < work; ++wi) {
      const int32_t qi = (int32_t)(wi % nq);
      const int32_t h = (int32_t)((wi / nq) % H);
      const int32_t bi = (int32_t)(wi / ((int64_t)nq * H));
      const int32_t i = rows ? rows[qi] : qi;
      if (i < 0 || i >= N) {
#pragma omp atomic write
        bad = 1;
        continue;
      }
      const float* qv = q + (((int64_t)bi * N + i) * H + h) * E;
      double mx = -INFINITY;
      for (int32_t j = 0; j < N; ++j) {
        if (!spvo_allowed(d, bi, i, j)) { s[j] = -INFINITY; continue; }
        const float* kv = k + (((int64_t)bi * N + j) * H + h) * E;
        double dot = 0.0;
        for (int32_t e = 0; e < E; ++e) dot += (double)qv[e] * (double)kv[e];
        s[j] = scale * dot;
        if (s[j] > mx) mx = s[j];
      }
      double den = 0.0;
      for (int32_t j = 0; j < N; ++j) {
        s[j] = (s[j] == -INFINITY) ? 0.0 : exp(s[j] - mx);
        den += s[j];
      }
      for (int32_t e = 0; e < E; ++e) acc[e] = 0.0;
      for (int32_t j = 0; j < N; ++j) {
        if (s[j] == 0.0) continue;
        const double p = s[j] / den;
        const float* vv = v + (((int64_t)bi * N + j) * H + h) * E;
        for (int32_t e = 0; e < E; ++e) acc[e] += p * (double)vv[e];
      }
      float* ov = o + (((int64_t)bi * N + i) * H + h) * E;
      for (int32_t e = 0; e < E; ++e) ov[e] = (float)acc[e];
      if (cls_scores && i == 0) {
        float* cs = cls_scores + ((int64_t)bi * H + h) * d->n_patch;
        for (int32_t j = G; j < N; ++j) cs[j - G] = (float)(s[j] / den);
      }
    }
    free(s);
    free(acc);
  }
  return bad;
}

/* Textbook dense attention, softmax(scale * Q K^T) V, written on its own so  */
/* that it can pin spvo_attention when the neighbourhood covers the grid.    */
int32_t spvo_dense_attention(int32_t batch, int32_t n_tok, int32_t heads,
                             int32_t head_dim, float scale_in, const float* q,
                             const float* k, const float* v, float* o) {
  const double scale = attn_scale(scale_in, head_dim);
  const int64_t work = (int64_t)batch * heads * n_tok;
#pragma omp parallel
  {
    double* w = (double*)malloc(sizeof(double) * (size_t)n_tok);
#pragma omp for schedule(dynamic, 16)
    for (int64_t wi = 0; wi < work; ++wi) {
      const int64_t i = wi % n_tok, h = (wi / n_tok) % heads, b = wi / ((int64_t)n_tok * heads);
      const float* qv = q + ((b * n_tok + i) * heads + h) * head_dim;
      double top = -INFINITY;
      for (int64_t j = 0; j < n_tok; ++j) {
        const float* kv = k + ((b * n_tok + j) * heads + h) * head_dim;
        double a = 0.0;
        for (int32_t e = 0; e < head_dim; ++e) a += (double)kv[e] * (double)qv[e];
        w[j] = a * scale;
        top = w[j] > top ? w[j] : top;
      }
      double z = 0.0;
      for (int64_t j = 0; j < n_tok; ++j) { w[j] = exp(w[j] - top); z += w[j]; }
      float* ov = o + ((b * n_tok + i) * heads + h) * head_dim;
      for (int32_t e = 0; e < head_dim; ++e) {
        double a = 0.0;
        for (int64_t j = 0; j < n_tok; ++j)
          a += w[j] * (double)v[((b * n_tok + j) * heads + h) * head_dim + e];
        ov[e] = (float)(a / z);
      }
    }
    free(w);
  }
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Sec. 3.3 -- token filter.                                                 */
/* Tokens are ranked by importance and the share p with the lowest scores is */
/* dropped for good: floor(p * N_p) tokens go, so with keep = 1 - p the      */
/* number kept is ceil(keep * N_p) (a 1e-9 guard absorbs the fp64            */
/* representation error of keep * N_p), at least 1 and at most N_p.          */
/* ------------------------------------------------------------------------- */
int32_t spvo_keep_count(int32_t n_patch, double keep_ratio) {
  if (n_patch < 1 || !(keep_ratio > 0.0) || keep_ratio > 1.0) return -1;
  double kd = ceil(keep_ratio * (double)n_patch - 1e-9);
  int32_t k = (int32_t)kd;
  if (k < 1) k = 1;
  if (k > n_patch) k = n_patch;
  return k;
}

typedef struct { float m; int32_t j; } rank_item;

/* Total order: larger mean first; equal means (+0 == -0) -> lower index
 * first; NaN ranks below every number. */
static int rank_cmp(const void* pa, const void* pb) {
  const rank_item* a = (const rank_item*)pa;
  const rank_item* b = (const rank_item*)pb;
  const int an = isnan(a->m), bn = isnan(b->m);
  if (an != bn) return an ? 1 : -1;
  if (!an) {
    if (a->m > b->m) return -1;
    if (a->m < b->m) return 1;
  }
  return (a->j > b->j) - (a->j < b->j);
}

static int int_cmp(const void* pa, const void* pb) {
  const int32_t a = *(const int32_t*)pa, b = *(const int32_t*)pb;
  return (a > b) - (a < b);
}

int32_t spvo_filter(int32_t batch, int32_t heads, int32_t n_patch,
                    int32_t n_global, int32_t dim, double keep_ratio,
                    const float* scores, const uint16_t* tokens_in,
                    uint16_t* tokens_out, int32_t* kept_idx,
                    float* mean_scores) {
  const int32_t k = spvo_keep_count(n_patch, keep_ratio);
  if (k < 0 || batch < 1 || heads < 1 || n_global < 0) return 1;
  rank_item* it = (rank_item*)malloc(sizeof(rank_item) * (size_t)n_patch);
  for (int32_t b = 0; b < batch; ++b) {
    for (int32_t j = 0; j < n_patch; ++j) {
      /* head average: fp32, heads added in index order, one division */
      volatile float sum = 0.0f;
      for (int32_t h = 0; h < heads; ++h)
        sum = sum + scores[((int64_t)b * heads + h) * n_patch + j];
      volatile float mean = sum / (float)heads;
      it[j].m = mean;
      it[j].j = j;
      if (mean_scores) mean_scores[(int64_t)b * n_patch + j] = mean;
    }
    qsort(it, (size_t)n_patch, sizeof(rank_item), rank_cmp);
    int32_t* kk = kept_idx + (int64_t)b * k;
    for (int32_t t = 0; t < k; ++t) kk[t] = it[t].j;
    qsort(kk, (size_t)k, sizeof(int32_t), int_cmp);
    if (tokens_in && tokens_out) {
      const uint16_t* src = tokens_in + (int64_t)b * (n_global + n_patch) * dim;
      uint16_t* dst = tokens_out + (int64_t)b * (n_global + k) * dim;
      for (int32_t g = 0; g < n_global; ++g)
        memcpy(dst + (int64_t)g * dim, src + (int64_t)g * dim, sizeof(uint16_t) * (size_t)dim);
      for (int32_t t = 0; t < k; ++t)
        memcpy(dst + (int64_t)(n_global + t) * dim, src + (int64_t)(n_global + kk[t]) * dim,
               sizeof(uint16_t) * (size_t)dim);
    }
  }
  free(it);
  return 0;
}

/* ------------------------------------------------------------------------- */
/* The surrounding ViT block (a standard pre-LayerNorm Transformer encoder;  */
/* the paper keeps the backbone unchanged, Sec. 4.1 Settings).               */
/* ------------------------------------------------------------------------- */
void spvo_layernorm(const float* x, int64_t rows, int32_t dim, const float* g,
                    const float* b, float eps, float* y) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    const float* xr = x + r * dim;
    double mu = 0.0;
    for (int32_t i = 0; i < dim; ++i) mu += (double)xr[i];
    mu /= (double)dim;
    double var = 0.0;
    for (int32_t i = 0; i < dim; ++i) { double t = (double)xr[i] - mu; var += t * t; }
    var /= (double)dim;
    const double rstd = 1.0 / sqrt(var + (double)eps);
    for (int32_t i = 0; i < dim; ++i)
      y[r * dim + i] = (float)(((double)xr[i] - mu) * rstd * (double)g[i] + (double)b[i]);
  }
}

/* y[r, o] = sum_i x[r, i] * w[o, i] + bias[o].  The weight is transposed once
 * so that the inner loop runs over independent outputs (each output still
 * adds its terms in index order, in fp64). */
void spvo_linear(const float* x, int64_t rows, int32_t in_dim, int32_t out_dim,
                 const float* w, const float* bias, float* y) {
  float* wt = (float*)malloc(sizeof(float) * (size_t)in_dim * (size_t)out_dim);
#pragma omp parallel for schedule(static)
  for (int32_t i = 0; i < in_dim; ++i)
    for (int32_t o = 0; o < out_dim; ++o) wt[(int64_t)i * out_dim + o] = w[(int64_t)o * in_dim + i];
#pragma omp parallel
  {
    double* acc = (double*)malloc(sizeof(double) * (size_t)out_dim);
#pragma omp for schedule(dynamic, 8)
    for (int64_t r = 0; r < rows; ++r) {
      for (int32_t o = 0; o < out_dim; ++o) acc[o] = bias ? (double)bias[o] : 0.0;
      const float* xr = x + r * in_dim;
      for (int32_t i = 0; i < in_dim; ++i) {
        const double a = (double)xr[i];
        const float* wr = wt + (int64_t)i * out_dim;
        for (int32_t o = 0; o < out_dim; ++o) acc[o] += a * (double)wr[o];
      }
      for (int32_t o = 0; o < out_dim; ++o) y[r * out_dim + o] = (float)acc[o];
    }
    free(acc);
  }
  free(wt);
}

/* exact (erf) GELU and SiLU */
float spvo_gelu(float x) { return (float)(0.5 * (double)x * (1.0 + erf((double)x / sqrt(2.0)))); }
float spvo_silu(float x) { return (float)((double)x / (1.0 + exp(-(double)x))); }

void spvo_gelu_n(const float* a, int64_t n, float* y) {
  for (int64_t i = 0; i < n; ++i) y[i] = spvo_gelu(a[i]);
}
void spvo_silu_mul_n(const float* a, const float* b, int64_t n, float* y) {
  for (int64_t i = 0; i < n; ++i) y[i] = spvo_silu(a[i]) * b[i];
}

int32_t spvo_vit_forward(const spvo_vit_config* c, const spvo_vit_weights* w,
                         const float* image, int32_t batch, int32_t gh, int32_t gw,
                         float* out_tokens, int32_t* kept_idx,
                         const int32_t* forced_keep, int32_t tap_layer, float* tap_x) {
  const int32_t D = c->dim, G = c->n_global, P = c->patch, NP0 = gh * gw;
  const int32_t hd = D / c->heads, KP = 3 * P * P, HID = c->mlp_hidden;
  if (c->layers < 1 || D % c->heads != 0 || batch < 1 || NP0 < 1) return 1;
  /* the filter stages: (layer, keep ratio) pairs, layers strictly increasing */
  int32_t n_stage = 0, st_layer[4];
  double st_keep[4];
  if (c->n_filters < 0 || c->n_filters > 4) return 1;
  if (c->n_filters == 0) {
    if (c->filter_layer < 0 || c->filter_layer > c->layers) return 1;
    if (c->filter_layer > 0) { n_stage = 1; st_layer[0] = c->filter_layer; st_keep[0] = c->keep_ratio; }
  } else {
    n_stage = c->n_filters;
    for (int32_t s = 0; s < n_stage; ++s) {
      st_layer[s] = c->filter_layers[s];
      st_keep[s] = c->keep_ratios[s];
      if (st_layer[s] < 1 || st_layer[s] > c->layers) return 1;
      if (s > 0 && st_layer[s] <= st_layer[s - 1]) return 1;
    }
  }
  int32_t k_total = 0;                    /* entries per image in kept_idx / forced_keep */
  {
    int32_t cur = NP0;
    for (int32_t s = 0; s < n_stage; ++s) {
      cur = spvo_keep_count(cur, st_keep[s]);
      if (cur < 0) return 3;
      k_total += cur;
    }
  }
  int32_t stage = 0, k_before = 0;        /* next stage; entries of earlier stages */
  int32_t np = NP0;                       /* patch tokens currently present */
  int64_t N = G + np;
  const int64_t Wpix = (int64_t)gw * P, Hpix = (int64_t)gh * P;

  /* patch embedding: token(G + y*W + x) = W_pe . patch(y, x) + b_pe + pos   */
  float* x = (float*)malloc(sizeof(float) * (size_t)(batch * N * D));
  {
    float* cols = (float*)malloc(sizeof(float) * (size_t)((int64_t)batch * NP0 * KP));
    for (int32_t b = 0; b < batch; ++b)
      for (int32_t t = 0; t < NP0; ++t) {
        const int32_t py0 = (t / gw) * P, px0 = (t % gw) * P;
        float* cr = cols + ((int64_t)b * NP0 + t) * KP;
        for (int32_t ch = 0; ch < 3; ++ch)
          for (int32_t py = 0; py < P; ++py)
            for (int32_t px = 0; px < P; ++px)
              cr[(ch * P + py) * P + px] =
                  image[(((int64_t)b * 3 + ch) * Hpix + (py0 + py)) * Wpix + (px0 + px)];
      }
    float* emb = (float*)malloc(sizeof(float) * (size_t)((int64_t)batch * NP0 * D));
    spvo_linear(cols, (int64_t)batch * NP0, KP, D, w->w_pe, w->b_pe, emb);
    for (int32_t b = 0; b < batch; ++b) {
      for (int32_t g = 0; g < G; ++g)
        for (int32_t i = 0; i < D; ++i)
          x[((int64_t)b * N + g) * D + i] = w->cls[(int64_t)g * D + i] + w->pos[(int64_t)g * D + i];
      for (int32_t t = 0; t < NP0; ++t)
        for (int32_t i = 0; i < D; ++i)
          x[((int64_t)b * N + G + t) * D + i] =
              emb[((int64_t)b * NP0 + t) * D + i] + w->pos[(int64_t)(G + t) * D + i];
    }
    free(cols);
    free(emb);
  }
  if (tap_x && tap_layer == 0) memcpy(tap_x, x, sizeof(float) * (size_t)(batch * N * D));

  int32_t* pos = NULL;                    /* [batch, np] after the filter   */
  for (int32_t l = 1; l <= c->layers; ++l) {
    const spvo_layer_weights* lw = &w->layer[l - 1];
    const int64_t R = (int64_t)batch * N;
    float* hbuf = (float*)malloc(sizeof(float) * (size_t)(R * D));
    float* qkv = (float*)malloc(sizeof(float) * (size_t)(R * 3 * D));
    float* qb = (float*)malloc(sizeof(float) * (size_t)(R * D));
    float* kb = (float*)malloc(sizeof(float) * (size_t)(R * D));
    float* vb = (float*)malloc(sizeof(float) * (size_t)(R * D));
    float* ab = (float*)malloc(sizeof(float) * (size_t)(R * D));
    float* pb = (float*)malloc(sizeof(float) * (size_t)(R * D));
    const int is_stage = stage < n_stage && l == st_layer[stage];
    float* sc = is_stage ? (float*)malloc(sizeof(float) * (size_t)((int64_t)batch * c->heads * np)) : NULL;

    /* attention branch: x += ls1 * (Attn(LN1(x)) W_o^T + b_o) */
    spvo_layernorm(x, R, D, lw->ln1_g, lw->ln1_b, c->ln_eps, hbuf);
    spvo_linear(hbuf, R, D, 3 * D, lw->w_qkv, lw->b_qkv, qkv);
    for (int64_t r = 0; r < R; ++r)
      for (int32_t i = 0; i < D; ++i) {
        qb[r * D + i] = qkv[r * 3 * D + i];
        kb[r * D + i] = qkv[r * 3 * D + D + i];
        vb[r * D + i] = qkv[r * 3 * D + 2 * D + i];
      }
    spvo_attn_desc ad;
    ad.batch = batch; ad.grid_h = gh; ad.grid_w = gw; ad.block = c->block;
    ad.radius = c->radius; ad.n_global = G; ad.heads = c->heads; ad.head_dim = hd;
    ad.softmax_scale = 0.0f; ad.n_patch = np; ad.patch_pos = pos;
    if (c->attn_mode == SPVO_ATTN_DENSE) {
      /* dense baseline: a neighbourhood that covers the whole grid */
      ad.block = 1;
      ad.radius = gh > gw ? gh : gw;
    }
    if (spvo_attention(&ad, qb, kb, vb, ab, sc, NULL, 0)) return 2;
    spvo_linear(ab, R, D, D, lw->w_o, lw->b_o, pb);
    for (int64_t r = 0; r < R; ++r)
      for (int32_t i = 0; i < D; ++i)
        x[r * D + i] += (lw->ls1 ? lw->ls1[i] : 1.0f) * pb[r * D + i];

    /* MLP branch: x += ls2 * MLP(LN2(x)) */
    spvo_layernorm(x, R, D, lw->ln2_g, lw->ln2_b, c->ln_eps, hbuf);
    float* h1 = (float*)malloc(sizeof(float) * (size_t)(R * HID));
    spvo_linear(hbuf, R, D, HID, lw->w_fc1, lw->b_fc1, h1);
    if (c->mlp_kind == SPVO_MLP_SWIGLU) {
      float* h3 = (float*)malloc(sizeof(float) * (size_t)(R * HID));
      spvo_linear(hbuf, R, D, HID, lw->w_fc3, lw->b_fc3, h3);
      for (int64_t e = 0; e < R * HID; ++e) h1[e] = spvo_silu(h1[e]) * h3[e];
      free(h3);
    } else {
      for (int64_t e = 0; e < R * HID; ++e) h1[e] = spvo_gelu(h1[e]);
    }
    spvo_linear(h1, R, HID, D, lw->w_fc2, lw->b_fc2, pb);
    for (int64_t r = 0; r < R; ++r)
      for (int32_t i = 0; i < D; ++i)
        x[r * D + i] += (lw->ls2 ? lw->ls2[i] : 1.0f) * pb[r * D + i];
    free(h1);

    /* Sec. 3.3: after a stage's block, the lowest-scored patches leave the
     * residual stream for all later blocks.  The ranking is over the tokens
     * present (ties: lower index, i.e. lower original position, first);
     * survivors keep their original grid positions. */
    if (is_stage) {
      const int32_t k = spvo_keep_count(np, st_keep[stage]);
      if (k < 0) return 3;
      int32_t* keep = (int32_t*)malloc(sizeof(int32_t) * (size_t)((int64_t)batch * k));  /* indices into the present tokens */
      if (forced_keep) {
        /* given as original positions: look each one up among the present tokens */
        for (int32_t b = 0; b < batch; ++b)
          for (int32_t t = 0; t < k; ++t) {
            const int32_t want = forced_keep[(int64_t)b * k_total + k_before + t];
            int32_t found = -1;
            if (!pos) found = (want >= 0 && want < np) ? want : -1;
            else
              for (int32_t j = 0; j < np; ++j)
                if (pos[(int64_t)b * np + j] == want) { found = j; break; }
            if (found < 0) return 4;
            keep[(int64_t)b * k + t] = found;
          }
      } else {
        if (spvo_filter(batch, c->heads, np, G, D, st_keep[stage], sc, NULL, NULL, keep, NULL))
          return 3;
      }
      const int64_t N2 = G + k;
      float* x2 = (float*)malloc(sizeof(float) * (size_t)(batch * N2 * D));
      int32_t* pos2 = (int32_t*)malloc(sizeof(int32_t) * (size_t)((int64_t)batch * k));
      for (int32_t b = 0; b < batch; ++b) {
        memcpy(x2 + (int64_t)b * N2 * D, x + (int64_t)b * N * D, sizeof(float) * (size_t)(G * D));
        for (int32_t t = 0; t < k; ++t) {
          const int32_t j = keep[(int64_t)b * k + t];
          if (j < 0 || j >= np) return 4;
          memcpy(x2 + ((int64_t)b * N2 + G + t) * D, x + ((int64_t)b * N + G + j) * D,
                 sizeof(float) * (size_t)D);
          /* before the first stage the index is the grid position itself */
          pos2[(int64_t)b * k + t] = pos ? pos[(int64_t)b * np + j] : j;
          if (kept_idx) kept_idx[(int64_t)b * k_total + k_before + t] = pos2[(int64_t)b * k + t];
        }
      }
      free(keep);
      free(x);
      if (pos) free(pos);
      x = x2;
      pos = pos2;
      np = k;
      N = N2;
      k_before += k;
      ++stage;
    }
    free(hbuf); free(qkv); free(qb); free(kb); free(vb); free(ab); free(pb);
    if (sc) free(sc);
    if (tap_x && tap_layer == l) memcpy(tap_x, x, sizeof(float) * (size_t)(batch * N * D));
  }
  spvo_layernorm(x, (int64_t)batch * N, D, w->lnf_g, w->lnf_b, c->ln_eps, out_tokens);
  free(x);
  if (pos) free(pos);
  return 0;
}
