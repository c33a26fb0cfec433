// Sec. 3.2 -- spatially-aware neighbouring-block sparse attention with global tokens.
//
// Layout idea: patch tokens are handled in BLOCK-MAJOR order (grouped by spatial block, blocks in
// row-major order over the block grid).  The key blocks of one neighbour block row, columns
// bx-r .. bx+r, are then ONE contiguous token range, so a key tile is a plain TMA box of
// consecutive rows and the sparsity mask of a query row is a column interval of the tile.  The
// same path serves full grids, ragged edge blocks and filtered token sets (blocks that lost
// tokens just have shorter ranges).  Neighbour ranges are computed on the fly from block
// coordinates and the per-block offsets; no N x N object and no neighbour list exists.
//
// Kernels
//   attn_plan_*        per-block token counts (binary search in the sorted positions), scan,
//                      each block row cut into 128-row query tiles
//   attn_regroup       row-major -> block-major copy of Q, K, V (only for row-major callers)
//   attn_patch_kernel  flash-style tcgen05 kernel: S = Q K^T of a 128-row query tile and a 32-key tile into
//                      one of three TMEM buffers, online softmax by 128 row-owning threads whose four warps
//                      advance independently (a warp whose rows have no key in a tile writes P = 0 and moves
//                      on; warps meet only when O has to be rescaled), P written over its own S as bf16,
//                      O += P V with V as an MN-major shared-memory operand; Q K^T is issued by two threads
//                      (even / odd key tiles), P V by one; the global tokens' keys and values join the softmax state in the epilogue
//                      (dot products on the CUDA cores while the last P V runs), so key tiles stay multiples
//                      of the MMA shape
//   attn_global_*      the dense rows of the global (CLS) queries and the CLS->patch scores
#include "attention.cuh"

namespace {

using namespace spv;

constexpr int TQ = 128;            // query rows per tile (MMA M)
constexpr int TK = 32;             // keys per tile (MMA N of S, K extent of P V): three S buffers of 32 columns and
                                   // O make 160 TMEM columns, so three CTAs fit an SM
constexpr int HD = 64;             // head_dim
constexpr int KST = 6;             // K / V smem stages (Q K^T runs up to two key tiles ahead of P V; an even count, so
                                   // that each of the two Q K^T issuers always meets the same stages)
constexpr int NSB = 3;             // S / P buffers in TMEM: a softmax warp may be two key tiles ahead of the slowest
constexpr int ATT_THREADS = 256;   // warps 0-3 softmax (one warpgroup), 4 TMA, 5-7 MMA issue: the second warpgroup
                                   // hands most of its registers to the first
constexpr int TILE_BYTES = 128 * 128;  // Q tile
constexpr int KV_BYTES = TK * 128;      // K or V tile
constexpr int MAXG = 16;           // global tokens: they are the first key tile of every query tile (at most TK).
                                   // (Adding them per query row in the epilogue with fp32 arithmetic instead was
                                   // measured: equal at one global token, 5 / 17 / 28 % slower at 2 / 5 / 8.)
// Shared memory of a CTA: Q tile, K / V stages, alignment slack, barriers.
constexpr int ATT_SMEM = TILE_BYTES + 2 * KST * KV_BYTES + 1024 /*align*/ + 512 /*barriers*/;
// two TMEM allocations per CTA, 160 columns in all, so that three CTAs share an SM's 512: O and two S buffers in
// the first, the third S buffer in the second.  A row's P (bf16, 16 columns) is written over its own S.
constexpr uint32_t TMEM_COLS = 128, TMEM_S2_COLS = 32;
constexpr uint32_t O_COL = 0, S_COL = 64;

// ------------------------------------------------------------------------------------------
// plan
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ int lower_bound_i32(const int32_t* a, int n, int key) {
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(a + mid) < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ int block_of_pos(int pos, int W, int b, int nbx) {
  return ((pos / W) / b) * nbx + (pos % W) / b;
}

// first ordinal t whose block id is >= blk (token order block-major, so block ids are sorted)
__device__ __forceinline__ int lower_bound_blk(const int32_t* pos, int n, int blk, int W, int b, int nbx) {
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (block_of_pos(__ldg(pos + mid), W, b, nbx) < blk) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// The caller's positions have to be inside the grid and strictly ascending: by position for row-major
// callers, by (block, position) for block-major ones (the searches below rely on it).  The first violation
// is latched in the status word.
__global__ void attn_check_positions(SpvAttnPlan p, const int32_t* __restrict__ patch_pos, int token_order,
                                     uint32_t* __restrict__ status) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = blockIdx.y;
  if (t >= p.n_patch) return;
  const int32_t* pos = patch_pos + (size_t)b * p.n_patch;
  const int cur = __ldg(pos + t);
  bool ok = cur >= 0 && cur < p.grid_h * p.grid_w;
  if (ok && t > 0) {
    const int prev = __ldg(pos + t - 1);
    if (prev < 0 || prev >= p.grid_h * p.grid_w) ok = false;
    else if (token_order == SPV_TOKENS_ROW_MAJOR) ok = prev < cur;
    else {
      const int bp = block_of_pos(prev, p.grid_w, p.block, p.nbx), bc = block_of_pos(cur, p.grid_w, p.block, p.nbx);
      ok = bp < bc || (bp == bc && prev < cur);
    }
  }
  if (!ok) atomicCAS(status, 0u, SPV_SITE_BAD_PATCH_POS);
}

// One thread per search segment.  Row-major callers: segment = (block, row inside block): its
// tokens are one run of the position-sorted input.  Block-major callers: segment = block.
// `bad` (optional): the word in which attn_check_positions latches a violation; when it is set the plan is
// built empty (no segment has a token, so no query tile exists and the patch kernel does nothing) instead of
// being searched for in positions that are not in order.
__global__ void attn_plan_segments(SpvAttnPlan p, const int32_t* __restrict__ patch_pos, int token_order,
                                   const uint32_t* __restrict__ bad) {
  const int seg = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = blockIdx.y;
  if (seg >= p.nseg) return;
  if (bad && *bad != 0u) {
    p.seg_lo[(size_t)b * p.nseg + seg] = 0;
    p.seg_cnt[(size_t)b * p.nseg + seg] = 0;
    return;
  }
  const int blk = seg / p.segs_per_block, yy = seg % p.segs_per_block;
  const int by = blk / p.nbx, bx = blk % p.nbx;
  const int32_t* pos = patch_pos ? patch_pos + (size_t)b * p.n_patch : nullptr;
  int lo, cnt;
  if (token_order == SPV_TOKENS_ROW_MAJOR) {
    const int y = by * p.block + yy;
    const int x0 = bx * p.block, x1 = min(x0 + p.block, p.grid_w);
    if (y >= p.grid_h) { lo = 0; cnt = 0; }
    else if (pos) {
      lo = lower_bound_i32(pos, p.n_patch, y * p.grid_w + x0);
      cnt = lower_bound_i32(pos, p.n_patch, y * p.grid_w + x1) - lo;
    } else { lo = y * p.grid_w + x0; cnt = x1 - x0; }
  } else {
    if (pos) {
      lo = lower_bound_blk(pos, p.n_patch, blk, p.grid_w, p.block, p.nbx);
      cnt = lower_bound_blk(pos, p.n_patch, blk + 1, p.grid_w, p.block, p.nbx) - lo;
    } else {   // full grid already grouped by block: sizes follow from the geometry
      const int bh = min(p.block, p.grid_h - by * p.block), bw = min(p.block, p.grid_w - bx * p.block);
      cnt = bh * bw;
      lo = 0;   // filled by the scan (identity)
    }
  }
  p.seg_lo[(size_t)b * p.nseg + seg] = lo;
  p.seg_cnt[(size_t)b * p.nseg + seg] = max(cnt, 0);
}

// One CTA per image: exclusive scan of the segment counts, block offsets, then the query tiles.
__global__ void __launch_bounds__(1024) attn_plan_scan(SpvAttnPlan p) {
  __shared__ int warp_sums[32];
  __shared__ int carry;
  const int b = blockIdx.x;
  const int32_t* cnt = p.seg_cnt + (size_t)b * p.nseg;
  int32_t* off = p.seg_off + (size_t)b * (p.nseg + 1);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base < p.nseg; base += 1024) {
    const int i = base + threadIdx.x;
    const int v = i < p.nseg ? cnt[i] : 0;
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
    const int excl = carry + warp_sums[warp] + inc - v;
    if (i < p.nseg) off[i] = excl;
    __syncthreads();
    if (threadIdx.x == 1023) carry = excl + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) off[p.nseg] = carry;
  __syncthreads();
  int32_t* boff = p.block_off + (size_t)b * (p.nb + 1);
  for (int blk = threadIdx.x; blk <= p.nb; blk += 1024) boff[blk] = off[min(blk * p.segs_per_block, p.nseg)];
  __syncthreads();
  // query tiles: the tokens of one block row cut into runs of TQ (a block may straddle two tiles;
  // every row looks up its own block), each with the first and last block it touches
  int4* tiles = p.tiles + (size_t)b * p.tiles_per_image;
  for (int by = threadIdx.x; by < p.nby; by += 1024) {
    int4* t = tiles + (size_t)by * p.tiles_per_row;
    int nt = 0;
    const int row_end = boff[(by + 1) * p.nbx];
    int bx = 0;
    for (int s = boff[by * p.nbx]; s < row_end; s += TQ) {
      const int e = min(s + TQ, row_end);
      while (boff[by * p.nbx + bx + 1] <= s) ++bx;
      const int first = bx;
      int last = bx;
      while (boff[by * p.nbx + last + 1] < e) ++last;
      t[nt++] = make_int4(s, e, by, first | (last << 16));
    }
    for (; nt < p.tiles_per_row; ++nt) t[nt] = make_int4(0, 0, 0, 0);
  }
}

__global__ void attn_plan_fill(SpvAttnPlan p) {
  const int seg = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = blockIdx.y;
  if (seg >= p.nseg) return;
  const int off = p.seg_off[(size_t)b * (p.nseg + 1) + seg];
  const int cnt = p.seg_cnt[(size_t)b * p.nseg + seg];
  const int lo = p.seg_lo[(size_t)b * p.nseg + seg];
  const int blk = seg / p.segs_per_block;
  for (int e = 0; e < cnt; ++e) {
    p.tok_blk[(size_t)b * p.n_patch + off + e] = blk;
    if (!p.identity) p.bm_src[(size_t)b * p.n_patch + off + e] = lo + e;
  }
}

// Q, K, V rows of every (token, head) copied into block-major order: 8 lanes move one 128-byte row.
__global__ void __launch_bounds__(256) attn_regroup(const __nv_bfloat16* __restrict__ q,
                                                    const __nv_bfloat16* __restrict__ k,
                                                    const __nv_bfloat16* __restrict__ v, int64_t sb, int64_t st,
                                                    int64_t sh, __nv_bfloat16* __restrict__ qo,
                                                    __nv_bfloat16* __restrict__ ko, __nv_bfloat16* __restrict__ vo,
                                                    const int32_t* __restrict__ bm_src, int batch, int n_global,
                                                    int n_patch, int heads, const uint32_t* __restrict__ bad) {
  if (*bad != 0u) return;        // the plan is empty (positions out of order): bm_src holds nothing
  const int n_tok = n_global + n_patch;
  const int64_t total = (int64_t)batch * n_tok * heads;
  const int sub = threadIdx.x & 7;
  for (int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 3; r < total;
       r += ((int64_t)gridDim.x * blockDim.x) >> 3) {
    const int h = (int)(r % heads);
    const int64_t bt = r / heads;
    const int t = (int)(bt % n_tok), b = (int)(bt / n_tok);
    const int src = t < n_global ? t : n_global + __ldg(bm_src + (size_t)b * n_patch + (t - n_global));
    const int64_t so = b * sb + (int64_t)src * st + (int64_t)h * sh + sub * 8;
    const int64_t dof = (((int64_t)b * n_tok + t) * heads + h) * HD + sub * 8;
    *reinterpret_cast<uint4*>(qo + dof) = __ldg(reinterpret_cast<const uint4*>(q + so));
    *reinterpret_cast<uint4*>(ko + dof) = __ldg(reinterpret_cast<const uint4*>(k + so));
    *reinterpret_cast<uint4*>(vo + dof) = __ldg(reinterpret_cast<const uint4*>(v + so));
  }
}

// ------------------------------------------------------------------------------------------
// patch-query kernel
// ------------------------------------------------------------------------------------------
struct PatchParams {
  const int32_t* block_off;
  const int32_t* tok_blk;
  const int4* tiles;
  const int32_t* o_tok;
  const __nv_bfloat16 *k, *v;
  int64_t sb, st, sh;
  __nv_bfloat16* o;
  int64_t o_sb, o_st, o_sh;
  int nbx, nby, nb, radius, n_global, n_patch, tiles_per_image;
  float scale_log2;
  uint32_t* status;
  // global-query form (template parameter GLOB): the query tile is the global tokens' rows, a CTA takes the key
  // chunk blockIdx.x and leaves its (reference maximum, sum, sum p*v) per row for attn_global_combine
  int chunk_len, n_chunks;
  float scale;                     // natural-logarithm scale of the logits
  float* logits;                   // [batch * G * heads, n_tok] scaled logits of global token 0's rows, or NULL
  float* part_ml;                  // [batch * G * heads, n_chunks, 2]
  float* part_o;                   // [batch * G * heads, n_chunks, 64]
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

__device__ __forceinline__ void unpack8(const uint4& u, float* f) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 h = *reinterpret_cast<const __nv_bfloat162*>(&w[i]);
    f[2 * i] = __low2float(h);
    f[2 * i + 1] = __high2float(h);
  }
}

template <bool GLOB>
__global__ void __launch_bounds__(ATT_THREADS, 3)
attn_patch_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                  const PatchParams p) {
  const int b = blockIdx.z, h = blockIdx.y;
  // patch coordinates: key (and query) kb is token G + kb, so the global tokens are [-G, 0)
  int4 tile = make_int4(-p.n_global, 0, 0, 0);           // global-query form: the query rows are the global tokens
  if constexpr (!GLOB) tile = __ldg(p.tiles + (size_t)b * p.tiles_per_image + blockIdx.x);
  const int q_begin = tile.x, q_end = tile.y;
  if (q_begin >= q_end) return;                          // unused slot of the tile table
  const int by = tile.z, bx_first = tile.w & 0xFFFF, bx_last = tile.w >> 16;
  // global-query form: this CTA's chunk of the keys (all of them are allowed)
  const int gk0 = -p.n_global + (int)blockIdx.x * p.chunk_len, gk1 = min(gk0 + p.chunk_len, p.n_patch);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = smem + TILE_BYTES;
  uint8_t* sV = sK + KST * KV_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sV + KST * KV_BYTES);
  uint64_t* q_full = bars;
  uint64_t* k_full = bars + 1;
  uint64_t* k_empty = k_full + KST;
  uint64_t* v_full = k_empty + KST;
  uint64_t* v_empty = v_full + KST;
  uint64_t* s_full = v_empty + KST;      // [NSB] Q K^T of the buffer's key tile has completed
  uint64_t* p_full = s_full + NSB;       // [NSB] all 128 rows have written P (and read S) of the buffer
  uint64_t* pv_done = p_full + NSB;      // [NSB] P V of the buffer's key tile (and all before it) has completed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pv_done + NSB);
  volatile uint32_t* abort_flag = tmem_slot + 3;
  static_assert(1 + 4 * KST + 3 * NSB + 2 <= 64, "barrier area");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = p.radius, G = p.n_global;
  // the key ranges are walked block row by block row; the global-query form has one range, its chunk
  const int cy0 = GLOB ? 1 : max(by - r, 0), cy1 = GLOB ? 0 : min(by + r, p.nby - 1);
  const int cxl = max(bx_first - r, 0), cxh = min(bx_last + r, p.nbx - 1);
  const int32_t* boff = p.block_off + (size_t)b * (p.nb + 1);

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < KST; ++s) {
      mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1);
      mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
    }
    for (int s = 0; s < NSB; ++s) { mbar_init(&s_full[s], 1); mbar_init(&p_full[s], 128); mbar_init(&pv_done[s], 1); }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 5) {
    tmem_alloc(tmem_slot, TMEM_COLS);
    tmem_alloc(tmem_slot + 2, TMEM_S2_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot, tmem_s2 = tmem_slot[2];
  // S buffer b of the three: two sit behind O in the first allocation, the third is the second allocation
  auto s_col = [&](uint32_t buf) { return buf < 2 ? tmem + S_COL + buf * TK : tmem_s2; };

  // the softmax warpgroup holds a score row of the key tile per thread; the other warpgroup needs few
  // registers (the kernel starts with 80 per thread: 80 + (80 - 24) = 136)
  if (warp >= 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 24;");
  if (warp == 4) {
    // ---------------- TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v);
      mbar_expect_tx(q_full, TILE_BYTES);
      tma_load_4d(sQ, &tm_q, q_full, 0, G + q_begin, h, b);
      // The global tokens are the first key tile of every query tile: in the patch coordinates used here (key kb
      // is token G + kb) they are the keys [-G, 0), a block row of their own in front of the neighbourhood's.
      uint32_t j = 0;
      for (int cy = cy0 - 1; cy <= cy1; ++cy) {
        int ks = GLOB ? gk0 : -G, ke = GLOB ? gk1 : 0;
        if (cy >= cy0) { ks = __ldg(boff + cy * p.nbx + cxl); ke = __ldg(boff + cy * p.nbx + cxh + 1); }
        for (int kb = ks; kb < ke; kb += TK, ++j) {
          const int s = j % KST;
          const uint32_t ph = ((j / KST) & 1) ^ 1;
          mbar_wait(&k_empty[s], ph, abort_flag, p.status, 0x1100 + s);
          mbar_expect_tx(&k_full[s], KV_BYTES);
          tma_load_4d(sK + s * KV_BYTES, &tm_k, &k_full[s], 0, G + kb, h, b);
          mbar_wait(&v_empty[s], ph, abort_flag, p.status, 0x1200 + s);
          mbar_expect_tx(&v_full[s], KV_BYTES);
          tma_load_4d(sV + s * KV_BYTES, &tm_v, &v_full[s], 0, G + kb, h, b);
        }
      }
    }
  } else {
    // ---------------- MMA issuers.  One thread gets a tcgen05.mma of these small shapes issued only about every
    // 120 cycles (measured): S = Q K^T has two issuing threads (warp 5 the even key tiles, warp 7 the odd ones;
    // consecutive tiles go to different S buffers) and O += P V one (warp 6; its instructions accumulate into the
    // same O and stay in one thread's order).
    if (lane == 0) {
      uint32_t n_kv = GLOB ? (uint32_t)((gk1 - gk0 + TK - 1) / TK) : 1u;   // (patch form: the global tokens' tile)
      for (int cy = cy0; cy <= cy1; ++cy) {
        const int ks = __ldg(boff + cy * p.nbx + cxl), ke = __ldg(boff + cy * p.nbx + cxh + 1);
        n_kv += (uint32_t)((ke - ks + TK - 1) / TK);
      }
      if (warp != 6) {
        constexpr uint32_t idesc_s = idesc_bf16(TQ, TK, false);
        const uint64_t dq = smem_desc_sw128(smem_u32(sQ));
        mbar_wait(q_full, 0, abort_flag, p.status, 0x1000);
        // Q K^T of key tile t goes to S buffer t % 3, up to two tiles ahead of the softmax, as soon as P V of
        // tile t - 3, which read its P from that buffer, has completed
        for (uint32_t t = warp == 5 ? 0 : 1; t < n_kv; t += 2) {
          const int s = t % KST;
          const uint32_t sb = t % NSB;
          mbar_wait(&k_full[s], (t / KST) & 1, abort_flag, p.status, 0x1300 + s);
          if (t >= NSB) mbar_wait(&pv_done[sb], ((t - NSB) / NSB) & 1, abort_flag, p.status, 0x1400 + sb);
          tc_fence_after();
          const uint64_t dk = smem_desc_sw128(smem_u32(sK + s * KV_BYTES));
          const uint32_t d_s = s_col(sb);
#pragma unroll
          for (int kk = 0; kk < HD / 16; ++kk)
            mma_ss(d_s, dq + (uint64_t)(kk * 2), dk + (uint64_t)(kk * 2), idesc_s, kk != 0);
          tc_commit(&s_full[sb]);
          tc_commit(&k_empty[s]);
        }
      } else {
        constexpr uint32_t idesc_o = idesc_bf16(TQ, HD, true);
        for (uint32_t j = 0; j < n_kv; ++j) {
          const int s = j % KST;
          const uint32_t sb = j % NSB;
          mbar_wait(&v_full[s], (j / KST) & 1, abort_flag, p.status, 0x1500 + s);
          mbar_wait(&p_full[sb], (j / NSB) & 1, abort_flag, p.status, 0x1600 + sb);
          tc_fence_after();
          const uint64_t dv = smem_desc_sw128(smem_u32(sV + s * KV_BYTES));
          const uint32_t a_p = s_col(sb);
#pragma unroll
          for (int kk = 0; kk < TK / 16; ++kk)
            mma_ts(tmem + O_COL, a_p + kk * 8, dv + (uint64_t)(kk * 128), idesc_o, (j | kk) != 0);
          tc_commit(&pv_done[sb]);
          tc_commit(&v_empty[s]);
        }
      }
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 136;");
    // ---------------- softmax + epilogue: thread `row` owns query row `row` (TMEM lane `row`)
    const int row = threadIdx.x;
    const int tok = q_begin + row;
    const bool valid = tok < q_end;
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    const uint32_t lane_addr = tmem + lane_off;
    int bxq = bx_first;
    if (!GLOB && valid) bxq = __ldg(p.tok_blk + (size_t)b * p.n_patch + tok) % p.nbx;
    const int rlo = max(bxq - r, 0), rhi = min(bxq + r, p.nbx - 1);
    const float sl2 = p.scale_log2;

    // The running maximum starts at a finite floor instead of -inf, so that a tile in which this
    // row has no allowed key (all scores masked to -inf) gives p = 2^(-inf) = 0 and not 2^(nan).
    // The first key tile holds the global tokens (allowed for every row), so l > 0 from then on.
    float m = -1.0e30f;
    float l = 0.f;

    uint32_t j = 0;
    for (int cy = cy0 - 1; cy <= cy1; ++cy) {
      int ks = -G, ke = 0, lo = -G, hi = 0;                // the global tokens' tile: keys [-G, 0) for every row
      if constexpr (GLOB) { ks = lo = gk0; ke = hi = gk1; }
      if (GLOB || cy >= cy0) {
        if constexpr (!GLOB) {
          ks = __ldg(boff + cy * p.nbx + cxl); ke = __ldg(boff + cy * p.nbx + cxh + 1);
          lo = __ldg(boff + cy * p.nbx + rlo); hi = __ldg(boff + cy * p.nbx + rhi + 1);
        }
        // Rows past the end of the tile are never stored: they take the key range of the warp's
        // first row, so that the warp stays uniform (valid rows are a prefix of the tile).
        const int lo0 = __shfl_sync(0xffffffffu, lo, 0), hi0 = __shfl_sync(0xffffffffu, hi, 0);
        const bool v0 = __shfl_sync(0xffffffffu, (int)valid, 0) != 0;
        if (!valid) { lo = lo0; hi = v0 ? hi0 : lo0; }
      }
      // over the warp's rows: a superset of the union of the allowed ranges (keys outside it are not even
      // read) and a subset of their intersection (keys inside it need no mask), once per block row
      const int ulo = __reduce_min_sync(0xffffffffu, lo), uhi = __reduce_max_sync(0xffffffffu, hi);
      const int ilo = __reduce_max_sync(0xffffffffu, lo), ihi = __reduce_min_sync(0xffffffffu, hi);
      for (int kb = ks; kb < ke; kb += TK, ++j) {
        const uint32_t sbuf = j % NSB, sph = (j / NSB) & 1;
        const uint32_t s_addr = s_col(sbuf) + lane_off;
        mbar_wait(&s_full[sbuf], sph, abort_flag, p.status, 0x1800 + sbuf);
        tc_fence_after();
        if (uhi <= kb || ulo >= kb + TK) {
          // no row of this warp has a key in the tile: P = 0 for its 32 rows and on to the next tile, without
          // waiting for the other warps (their rows' P V needs this warp's rows of P all the same)
          uint32_t z[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) z[i] = 0u;
          tmem_st16(s_addr, z);
          tc_wait_st();
          tc_fence_before();
          mbar_arrive(&p_full[sbuf]);
          continue;
        }
        uint32_t sr[TK];
        tmem_ld32(s_addr, sr);
        tc_wait_ld();
        if constexpr (GLOB) {
          // the scaled logits of global token 0 (query row 0) for the consumer of the CLS->patch scores
          if (p.logits && row == 0) {
            float* lg = p.logits + ((size_t)(b * G) * gridDim.y + h) * (size_t)(G + p.n_patch) + (G + kb);
#pragma unroll
            for (int i = 0; i < TK; ++i)
              if (kb + i < ke) lg[i] = __uint_as_float(sr[i]) * p.scale;
          }
        }
        // a tile that is not inside every row's range is masked in registers: column c is allowed iff
        // c_lo <= c < c_hi, one unsigned compare
        if (!(kb >= ilo && kb + TK <= ihi)) {
          const int c_lo = min(max(lo - kb, 0), TK), c_hi = min(max(hi - kb, 0), TK);
          // bit i of the row's mask word = column i is allowed (bits [c_lo, c_hi))
          const uint32_t below_hi = c_hi >= 32 ? 0xffffffffu : (1u << c_hi) - 1u;
          const uint32_t below_lo = c_lo >= 32 ? 0xffffffffu : (1u << c_lo) - 1u;
          const uint32_t mw = below_hi & ~below_lo;
#pragma unroll
          for (int i = 0; i < TK; ++i)
            if (!(mw & (1u << i))) sr[i] = 0xff800000u;
        }
        float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
        for (int i = 0; i < TK; i += 8) {
          m0 = fmax3(m0, __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
          m1 = fmax3(m1, __uint_as_float(sr[i + 2]), __uint_as_float(sr[i + 3]));
          m2 = fmax3(m2, __uint_as_float(sr[i + 4]), __uint_as_float(sr[i + 5]));
          m3 = fmax3(m3, __uint_as_float(sr[i + 6]), __uint_as_float(sr[i + 7]));
        }
        const float mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
        // lazy rescale: the running maximum only moves when it would grow by more than 2^8
        const float m_t = mx * sl2;
        const bool need = m_t > m + 8.0f;
        const float m_new = need ? m_t : m;
        const float alpha = need ? fast_exp2(m - m_new) : 1.0f;
        // O has to be rescaled only where something has been accumulated (l > 0); that is the one place where a
        // warp waits for the P V of the previous key tile, i.e. for the other warps
        if (__any_sync(0xffffffffu, need && l > 0.f)) {
          const uint32_t pj = j - 1;                       // l > 0 implies j > 0
          mbar_wait(&pv_done[pj % NSB], (pj / NSB) & 1, abort_flag, p.status, 0x1900);
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < HD / 32; ++c) {
            uint32_t orr[32];
            tmem_ld32(lane_addr + O_COL + 32 * c, orr);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * alpha);
            tmem_st32(lane_addr + O_COL + 32 * c, orr);
          }
        }
        // p = 2^(s*scale - m), packed to bf16 pairs and written over the first half of this row's S (masked
        // scores are -inf, so p = 0); two scores per packed fp32x2 multiply-add and add
        float2 rs_a = make_float2(0.f, 0.f), rs_b = make_float2(0.f, 0.f);
        const float2 sl2_2 = make_float2(sl2, sl2), nm_2 = make_float2(-m_new, -m_new);
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < TK; i += 4) {
          const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(sr[i]), __uint_as_float(sr[i + 1])), sl2_2, nm_2);
          const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(sr[i + 2]), __uint_as_float(sr[i + 3])), sl2_2, nm_2);
          const float2 p0 = make_float2(fast_exp2(x0.x), fast_exp2(x0.y));
          const float2 p1 = make_float2(fast_exp2(x1.x), fast_exp2(x1.y));
          rs_a = __fadd2_rn(rs_a, p0);
          rs_b = __fadd2_rn(rs_b, p1);
          pk[i / 2] = pack_bf16(p0.x, p0.y);
          pk[i / 2 + 1] = pack_bf16(p1.x, p1.y);
        }
        tmem_st16(s_addr, pk);
        l = l * alpha + ((rs_a.x + rs_a.y) + (rs_b.x + rs_b.y));
        m = m_new;
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(&p_full[sbuf]);
      }
    }
    // ---------------- epilogue: O / l once the last P V has completed (l > 0: every row saw the global keys)
    const float inv = 1.0f / l;
    mbar_wait(&pv_done[(j - 1) % NSB], ((j - 1) / NSB) & 1, abort_flag, p.status, 0x1A00);
    tc_fence_after();
    if constexpr (GLOB) {
      // the chunk's partial state of the global rows, in the units attn_global_combine merges: reference maximum
      // as a natural-logarithm logit (any reference does: sums and values are relative to it), sum, sum p * v
      if (warp == 0) {                                     // the G <= 16 valid rows are rows of warp 0
        const size_t pidx = ((size_t)(b * G + min(row, G - 1)) * gridDim.y + h) * p.n_chunks + blockIdx.x;
        if (valid) {
          p.part_ml[pidx * 2] = m * 0.6931471805599453f;
          p.part_ml[pidx * 2 + 1] = l;
        }
#pragma unroll
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t orr[32];
          tmem_ld32(lane_addr + O_COL + 32 * c, orr);
          tc_wait_ld();
          if (valid) {
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              *reinterpret_cast<uint4*>(p.part_o + pidx * HD + 32 * c + i) = make_uint4(orr[i], orr[i + 1], orr[i + 2], orr[i + 3]);
          }
        }
      }
    } else {
    float of[HD];
#pragma unroll
    for (int c = 0; c < HD / 32; ++c) {
      uint32_t orr[32];
      tmem_ld32(lane_addr + O_COL + 32 * c, orr);
      tc_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) of[32 * c + i] = __uint_as_float(orr[i]) * inv;
    }
    // stage the bf16 row in the (now dead) Q tile, same 128-byte swizzle; each warp then stores its
    // own 32 rows, eight lanes per 128-byte row
    {
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint4 w;
        w.x = pack_bf16(of[8 * c], of[8 * c + 1]);
        w.y = pack_bf16(of[8 * c + 2], of[8 * c + 3]);
        w.z = pack_bf16(of[8 * c + 4], of[8 * c + 5]);
        w.w = pack_bf16(of[8 * c + 6], of[8 * c + 7]);
        *reinterpret_cast<uint4*>(sQ + row * 128 + ((c ^ (row & 7)) << 4)) = w;
      }
    }
    if (p.o_tok == nullptr && 32 * warp + 32 <= q_end - q_begin) {
      // all 32 rows of this warp are valid and consecutive in the output: one TMA tile store of the
      // warp's staged rows (four swizzle atoms of eight rows), no waiting for the other warps
      fence_async_smem();
      __syncwarp();
      if (lane == 0) {
        tma_store_4d(&tm_o, sQ + warp * (32 * 128), 0, G + q_begin + 32 * warp, h, b);
        bulk_commit();
        bulk_wait_read<0>();
      }
    } else {
      __syncwarp();
      {
        const int r0 = 32 * warp + (lane >> 3), cc = lane & 7;
        __nv_bfloat16* obase = p.o + b * p.o_sb + (int64_t)G * p.o_st + (int64_t)h * p.o_sh + cc * 8;
        uint4 w[8];
        int ot[8];
#pragma unroll
        for (int q4 = 0; q4 < 8; ++q4) {
          const int rr = r0 + 4 * q4, tk = q_begin + rr;
          w[q4] = *reinterpret_cast<const uint4*>(sQ + rr * 128 + ((cc ^ (rr & 7)) << 4));
          ot[q4] = (p.o_tok && tk < q_end) ? __ldg(p.o_tok + (size_t)b * p.n_patch + tk) : tk;
        }
#pragma unroll
        for (int q4 = 0; q4 < 8; ++q4)
          if (q_begin + r0 + 4 * q4 < q_end) *reinterpret_cast<uint4*>(obase + (int64_t)ot[q4] * p.o_st) = w[q4];
      }
    }
    }  // !GLOB
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 5) {
    tmem_dealloc(tmem, TMEM_COLS);
    tmem_dealloc(tmem_s2, TMEM_S2_COLS);
  }
}

// ------------------------------------------------------------------------------------------
// global-query rows
// ------------------------------------------------------------------------------------------
constexpr int GCH = 128;   // fewest keys per CTA (bounds the number of chunk partials)
constexpr int GLOB_TENSOR_MIN = 3;   // from this many global tokens on, their rows run as a query tile of the tensor-core
                                     // kernel (measured equal at two, 1.6 to 5 times faster from three to sixteen)

// grid (heads, chunks, batch * ceil(G / GQ)).  One pass over the chunk's keys serves GQ global queries (GQ = 1 is
// what runs: with four queries per pass K and V cross HBM once per four queries, but the eight-lane dot products
// and their shuffles then make the kernel instruction-bound -- 3.5 ms instead of 4.0 per step for five global
// tokens, 5.8 instead of 4.5 for nine; the later queries' passes find K and V in L2 anyway): every group of
// eight lanes walks keys k0 + grp, k0 + grp + 32, ...
// with its own running (max, sum, sum p*v) per query -- the key and the value row of a key are loaded together,
// so twice as many loads are in flight as with a score pass followed by a value pass -- and the 32 group states
// are merged through shared memory, query after query.  Writes the chunk's (max, sum, sum p*v) of every query
// and, when the scores are wanted, the scaled logits of global token 0.
template <bool kLogits, int GQ>
__global__ void __launch_bounds__(256, 2) attn_global_partial(const __nv_bfloat16* __restrict__ q,
                                                           const __nv_bfloat16* __restrict__ k,
                                                           const __nv_bfloat16* __restrict__ v, int64_t sb,
                                                           int64_t st, int64_t sh, int n_tok, int n_global,
                                                           int heads, float scale, float* __restrict__ logits,
                                                           float* __restrict__ part_ml, float* __restrict__ part_o,
                                                           int n_chunks, int chunk_len) {
  __shared__ float s_m[32], s_l[32];
  __shared__ float s_o[32][HD + 1];
  // heads fastest: the CTAs running together read whole token rows (all heads) of one key chunk
  const int h = blockIdx.x, chunk = blockIdx.y;
  const int g_chunks = (n_global + GQ - 1) / GQ;
  const int b = blockIdx.z / g_chunks, g0 = (blockIdx.z % g_chunks) * GQ;
  const int k0 = chunk * chunk_len, k1 = min(k0 + chunk_len, n_tok);
  const int sub = threadIdx.x & 7, grp = threadIdx.x >> 3;   // 8 lanes per key, 32 keys in flight
  float qf[GQ][8];
#pragma unroll
  for (int gq = 0; gq < GQ; ++gq) {
    const int g = min(g0 + gq, n_global - 1);                // past the last query: a copy of it, never written
    unpack8(__ldg(reinterpret_cast<const uint4*>(q + b * sb + (int64_t)g * st + (int64_t)h * sh) + sub), qf[gq]);
  }
  float* lg = logits + ((size_t)(b * n_global) * heads + h) * n_tok;     // row of global token 0
  float m[GQ], l[GQ], acc[GQ][8];
#pragma unroll
  for (int gq = 0; gq < GQ; ++gq) {
    m[gq] = -INFINITY; l[gq] = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[gq][i] = 0.f;
  }
  // the trip count is the same for every lane (the shuffles name the whole warp); keys past the
  // end of the chunk are predicated off.  The loads of the next GU keys (key and value rows) are in flight
  // while the current ones are used.
  constexpr int GU = GQ == 1 ? 4 : 2;
  auto load_batch = [&](int kk0, uint4* ku, uint4* vu) {
#pragma unroll
    for (int u = 0; u < GU; ++u) {
      const int kk = kk0 + u * 32 + grp;
      ku[u] = make_uint4(0u, 0u, 0u, 0u);
      vu[u] = make_uint4(0u, 0u, 0u, 0u);
      if (kk < k1) {
        const int64_t off = b * sb + (int64_t)kk * st + (int64_t)h * sh;
        ku[u] = __ldg(reinterpret_cast<const uint4*>(k + off) + sub);
        vu[u] = __ldg(reinterpret_cast<const uint4*>(v + off) + sub);
      }
    }
  };
  uint4 kn[GU], vn[GU];
  load_batch(k0, kn, vn);
#pragma unroll 1
  for (int kk0 = k0; kk0 < k1; kk0 += 32 * GU) {
    uint4 ku[GU], vu[GU];
#pragma unroll
    for (int u = 0; u < GU; ++u) { ku[u] = kn[u]; vu[u] = vn[u]; }
    if (kk0 + 32 * GU < k1) load_batch(kk0 + 32 * GU, kn, vn);
    float kf[GU][8], vf[GU][8];
#pragma unroll
    for (int u = 0; u < GU; ++u) { unpack8(ku[u], kf[u]); unpack8(vu[u], vf[u]); }
#pragma unroll
    for (int gq = 0; gq < GQ; ++gq) {
      float d[GU];
#pragma unroll
      for (int u = 0; u < GU; ++u) {
        d[u] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) d[u] = fmaf(qf[gq][i], kf[u][i], d[u]);
      }
#pragma unroll
      for (int u = 0; u < GU; ++u) {
        d[u] += __shfl_xor_sync(0xffffffffu, d[u], 1);
        d[u] += __shfl_xor_sync(0xffffffffu, d[u], 2);
        d[u] += __shfl_xor_sync(0xffffffffu, d[u], 4);
        d[u] = (kk0 + u * 32 + grp < k1) ? d[u] * scale : -INFINITY;
      }
      if (kLogits && g0 + gq == 0 && sub < GU) {
        // lane u of the group writes key u's logit
        float mine = d[0];
#pragma unroll
        for (int u = 1; u < GU; ++u) mine = sub == u ? d[u] : mine;
        const int kk = kk0 + sub * 32 + grp;
        if (kk < k1) lg[kk] = mine;
      }
      float mx = d[0];
#pragma unroll
      for (int u = 1; u < GU; ++u) mx = fmaxf(mx, d[u]);
      if (mx > m[gq]) {                      // the same decision in all eight lanes of the group
        const float a = __expf(m[gq] - mx);  // m = -inf on the first batch: a = 0, the state is empty
        l[gq] *= a;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[gq][i] *= a;
        m[gq] = mx;
      }
      const float mref = m[gq] == -INFINITY ? 0.f : m[gq];   // a group that has seen no key yet: every p below is 0
#pragma unroll
      for (int u = 0; u < GU; ++u) {
        const float pw = __expf(d[u] - mref);          // 0 for a key past the end of the chunk
        l[gq] += pw;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[gq][i] = fmaf(pw, vf[u][i], acc[gq][i]);
      }
    }
  }
#pragma unroll
  for (int gq = 0; gq < GQ; ++gq) {
    if (g0 + gq >= n_global) break;                          // uniform over the CTA
    if (gq > 0) __syncthreads();                             // the previous query's merge has read the arrays
    if (sub == 0) { s_m[grp] = m[gq]; s_l[grp] = l[gq]; }
#pragma unroll
    for (int i = 0; i < 8; ++i) s_o[grp][sub * 8 + i] = acc[gq][i];
    __syncthreads();
    float cmax = -INFINITY;
#pragma unroll
    for (int gI = 0; gI < 32; ++gI) cmax = fmaxf(cmax, s_m[gI]);
    const size_t pidx = ((size_t)(b * n_global + g0 + gq) * heads + h) * n_chunks + chunk;
    if (threadIdx.x < HD) {
      float t = 0.f;
#pragma unroll
      for (int gI = 0; gI < 32; ++gI)
        if (s_m[gI] > -INFINITY) t += s_o[gI][threadIdx.x] * __expf(s_m[gI] - cmax);
      part_o[pidx * HD + threadIdx.x] = t;
    }
    if (threadIdx.x == 0) {
      float t = 0.f;
#pragma unroll
      for (int gI = 0; gI < 32; ++gI)
        if (s_m[gI] > -INFINITY) t += s_l[gI] * __expf(s_m[gI] - cmax);
      part_ml[pidx * 2] = cmax;
      part_ml[pidx * 2 + 1] = t;
    }
  }
}

// grid (heads, batch * G): merge the chunk partials, write the output row and (g == 0) the
// CLS->patch softmax weights.
__global__ void __launch_bounds__(256) attn_global_combine(const float* __restrict__ logits,
                                                           const float* __restrict__ part_ml,
                                                           const float* __restrict__ part_o, int n_chunks,
                                                           int n_tok, int n_global, int heads,
                                                           __nv_bfloat16* __restrict__ o, int64_t o_sb,
                                                           int64_t o_st, int64_t o_sh, float* __restrict__ scores,
                                                           const int32_t* __restrict__ score_idx, int score_stride,
                                                           float* __restrict__ head_stats) {
  __shared__ float s_m, s_l;
  __shared__ float s_red[16];
  const int h = blockIdx.x, bg = blockIdx.y;
  const int b = bg / n_global, g = bg % n_global;
  const size_t pbase = ((size_t)bg * heads + h) * n_chunks;
  float mx = -INFINITY;
  for (int c = threadIdx.x; c < n_chunks; c += 256) mx = fmaxf(mx, part_ml[(pbase + c) * 2]);
#pragma unroll
  for (int o2 = 16; o2 > 0; o2 >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o2));
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = s_red[0];
    for (int w = 1; w < 8; ++w) t = fmaxf(t, s_red[w]);
    s_m = t;
  }
  __syncthreads();
  const float M = s_m;
  float ls = 0.f;
  for (int c = threadIdx.x; c < n_chunks; c += 256)
    ls += part_ml[(pbase + c) * 2 + 1] * __expf(part_ml[(pbase + c) * 2] - M);
#pragma unroll
  for (int o2 = 16; o2 > 0; o2 >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o2);
  if ((threadIdx.x & 31) == 0) s_red[8 + (threadIdx.x >> 5)] = ls;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += s_red[8 + w];
    s_l = t;
  }
  __syncthreads();
  const float inv = 1.0f / s_l;
  if (threadIdx.x < HD) {
    float acc = 0.f;
    for (int c = 0; c < n_chunks; ++c)
      acc += part_o[(pbase + c) * HD + threadIdx.x] * __expf(part_ml[(pbase + c) * 2] - M);
    o[b * o_sb + (int64_t)g * o_st + (int64_t)h * o_sh + threadIdx.x] = __float2bfloat16(acc * inv);
  }
  // (row maximum of the scaled logits, 1 / row sum) of global token 0: with the logits they give the softmax
  // weights to a consumer that folds them into its own pass (the fused ranking of the token filter)
  if (head_stats && g == 0 && threadIdx.x == 0) {
    head_stats[((size_t)b * heads + h) * 2] = M;
    head_stats[((size_t)b * heads + h) * 2 + 1] = inv;
  }
  if (scores && g == 0) {
    const float* lg = logits + ((size_t)bg * heads + h) * n_tok;
    const int n_patch = n_tok - n_global;
    float* sc = scores + ((size_t)b * heads + h) * score_stride;
    for (int t = threadIdx.x; t < n_patch; t += 256) {
      const int dst = score_idx ? __ldg(score_idx + (size_t)b * n_patch + t) : t;
      sc[dst] = __expf(lg[n_global + t] - M) * inv;
    }
  }
}

int32_t make_qkv_map(spv_ctx* ctx, CUtensorMap* m, const void* base, int64_t sb, int64_t st, int64_t sh, int n_tok,
                     int heads, int batch, int rows) {
  const uint64_t dims[4] = {(uint64_t)HD, (uint64_t)n_tok, (uint64_t)heads, (uint64_t)batch};
  const uint64_t str[3] = {(uint64_t)st * 2, (uint64_t)sh * 2, (uint64_t)sb * 2};
  const uint32_t box[4] = {(uint32_t)HD, (uint32_t)rows, 1, 1};
  return spv_make_tmap_bf16(ctx, m, base, 4, dims, str, box);
}

}  // namespace

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
static void plan_geometry(SpvAttnPlan* p, int token_order) {
  p->nby = (p->grid_h + p->block - 1) / p->block;
  p->nbx = (p->grid_w + p->block - 1) / p->block;
  p->nb = p->nby * p->nbx;
  p->segs_per_block = token_order == SPV_TOKENS_ROW_MAJOR ? p->block : 1;
  p->nseg = p->nb * p->segs_per_block;
  const int64_t rowcap = (int64_t)(p->block < p->grid_h ? p->block : p->grid_h) * p->grid_w;
  p->tiles_per_row = (int32_t)((rowcap + TQ - 1) / TQ);
  p->tiles_per_image = p->tiles_per_row * p->nby;
  p->identity = token_order == SPV_TOKENS_BLOCK_MAJOR;
}

size_t spv_attn_plan_bytes(int32_t batch, int32_t grid_h, int32_t grid_w, int32_t block, int32_t n_patch,
                           int32_t token_order) {
  SpvAttnPlan p{};
  p.batch = batch; p.grid_h = grid_h; p.grid_w = grid_w; p.block = block; p.n_patch = n_patch;
  plan_geometry(&p, token_order);
  size_t n = 0;
  n += spv_align_up((size_t)batch * p.nseg * 4, 256) * 2;
  n += spv_align_up((size_t)batch * (p.nseg + 1) * 4, 256);
  n += spv_align_up((size_t)batch * (p.nb + 1) * 4, 256);
  n += spv_align_up((size_t)batch * n_patch * 4, 256) * 2;
  n += spv_align_up((size_t)batch * p.tiles_per_image * sizeof(int4), 256);
  return n;
}

int32_t spv_attn_plan_build(spv_ctx* ctx, int32_t batch, int32_t grid_h, int32_t grid_w, int32_t block,
                            int32_t radius, int32_t n_global, int32_t n_patch, const int32_t* patch_pos,
                            int32_t token_order, void* ws, size_t ws_bytes, cudaStream_t stream,
                            SpvAttnPlan* plan, bool check_positions) {
  SpvAttnPlan p{};
  p.batch = batch; p.grid_h = grid_h; p.grid_w = grid_w; p.block = block; p.n_global = n_global;
  p.n_patch = n_patch;
  plan_geometry(&p, token_order);
  const int reach = (p.nby > p.nbx ? p.nby : p.nbx);
  p.radius = radius < reach ? radius : reach;
  if (p.nbx >= 65536) return SPV_ERR_UNSUPPORTED;
  if (ws_bytes < spv_attn_plan_bytes(batch, grid_h, grid_w, block, n_patch, token_order)) return SPV_ERR_WORKSPACE;
  char* w = (char*)ws;
  auto take = [&](size_t bytes) { void* r = w; w += spv_align_up(bytes, 256); return r; };
  p.seg_lo = (int32_t*)take((size_t)batch * p.nseg * 4);
  p.seg_cnt = (int32_t*)take((size_t)batch * p.nseg * 4);
  p.seg_off = (int32_t*)take((size_t)batch * (p.nseg + 1) * 4);
  p.block_off = (int32_t*)take((size_t)batch * (p.nb + 1) * 4);
  p.tok_blk = (int32_t*)take((size_t)batch * n_patch * 4);
  p.bm_src = (int32_t*)take((size_t)batch * n_patch * 4);
  p.tiles = (int4*)take((size_t)batch * p.tiles_per_image * sizeof(int4));
  const dim3 sgrid((p.nseg + 255) / 256, batch);
  SpvProfScope prof(ctx, SPV_K_ATTN_PLAN, stream);
  int launches = 3;
  if (check_positions && patch_pos) {
    attn_check_positions<<<dim3((n_patch + 255) / 256, batch), 256, 0, stream>>>(p, patch_pos, token_order,
                                                                              ctx->d_status + 1);
    ++launches;
  }
  attn_plan_segments<<<sgrid, 256, 0, stream>>>(p, patch_pos, token_order,
                                                (check_positions && patch_pos) ? ctx->d_status + 1 : nullptr);
  attn_plan_scan<<<batch, 1024, 0, stream>>>(p);
  attn_plan_fill<<<sgrid, 256, 0, stream>>>(p);
  *plan = p;
  return spv_launch_ok(ctx, launches);
}

static int32_t attn_configure(spv_ctx* ctx) {
  if (!ctx->attn_configured) {
    SPV_CUDA_OK(cudaFuncSetAttribute(attn_patch_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM));
    SPV_CUDA_OK(cudaFuncSetAttribute(attn_patch_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM));
    ctx->attn_configured = 1;
  }
  return SPV_OK;
}

int32_t spv_attn_run_patches(spv_ctx* ctx, const SpvAttnPlan* plan, const SpvAttnIO* io, cudaStream_t stream) {
  int32_t st;
  if ((st = attn_configure(ctx)) != SPV_OK) return st;
  const int n_tok = plan->n_global + plan->n_patch;
  CUtensorMap tq, tk, tv;
  if ((st = make_qkv_map(ctx, &tq, io->q, io->sb, io->st, io->sh, n_tok, io->heads, plan->batch, TQ)) != SPV_OK) return st;
  if ((st = make_qkv_map(ctx, &tk, io->k, io->sb, io->st, io->sh, n_tok, io->heads, plan->batch, TK)) != SPV_OK) return st;
  if ((st = make_qkv_map(ctx, &tv, io->v, io->sb, io->st, io->sh, n_tok, io->heads, plan->batch, TK)) != SPV_OK) return st;
  PatchParams pp;
  pp.block_off = plan->block_off; pp.tok_blk = plan->tok_blk; pp.tiles = plan->tiles; pp.o_tok = io->o_tok;
  pp.k = (const __nv_bfloat16*)io->k; pp.v = (const __nv_bfloat16*)io->v;
  pp.sb = io->sb; pp.st = io->st; pp.sh = io->sh;
  pp.o = (__nv_bfloat16*)io->o; pp.o_sb = io->o_sb; pp.o_st = io->o_st; pp.o_sh = io->o_sh;
  pp.nbx = plan->nbx; pp.nby = plan->nby; pp.nb = plan->nb; pp.radius = plan->radius;
  pp.n_global = plan->n_global; pp.n_patch = plan->n_patch; pp.tiles_per_image = plan->tiles_per_image;
  pp.scale_log2 = io->scale * 1.4426950408889634f;
  pp.status = ctx->d_status;
  pp.chunk_len = 0; pp.n_chunks = 0; pp.scale = io->scale; pp.logits = nullptr; pp.part_ml = nullptr; pp.part_o = nullptr;
  const dim3 grid(plan->tiles_per_image, io->heads, plan->batch);
  SpvProfScope prof(ctx, SPV_K_ATTN_PATCH, stream);
  // the output as a tensor map (same row order as Q, boxes of 32 rows): warps whose rows are all valid store by TMA
  CUtensorMap to;
  if ((st = make_qkv_map(ctx, &to, io->o, io->o_sb, io->o_st, io->o_sh, n_tok, io->heads, plan->batch, 32)) != SPV_OK) return st;
  attn_patch_kernel<false><<<grid, ATT_THREADS, ATT_SMEM, stream>>>(tq, tk, tv, to, pp);
  return spv_launch_ok(ctx);
}

size_t spv_attn_global_bytes(int32_t batch, int32_t n_global, int32_t heads, int32_t n_tok) {
  const size_t rows = (size_t)batch * n_global * heads;
  const size_t chunks = (n_tok + GCH - 1) / GCH;
  return spv_align_up(rows * n_tok * 4, 256) + spv_align_up(rows * chunks * 2 * 4, 256) +
         spv_align_up(rows * chunks * HD * 4, 256);
}

int32_t spv_attn_run_globals(spv_ctx* ctx, const SpvAttnPlan* plan, const SpvAttnIO* io, float* scores,
                             const int32_t* score_idx, int32_t score_stride, void* ws, size_t ws_bytes,
                             cudaStream_t stream, float* head_stats, const float** logits_out) {
  const int n_tok = plan->n_global + plan->n_patch, G = plan->n_global, B = plan->batch;
  if (ws_bytes < spv_attn_global_bytes(B, G, io->heads, n_tok)) return SPV_ERR_WORKSPACE;
  const size_t rows = (size_t)B * G * io->heads;
  if (G >= GLOB_TENSOR_MIN) {
    // Several global tokens: their rows are one query tile of the tensor-core kernel (global-query form), the keys
    // split into chunks so that the CTAs fill the GPU about once (three per SM); the chunk partials are merged by
    // the same combine kernel.  One pass serves all G queries, so the time does not grow with G.
    int32_t st;
    if ((st = attn_configure(ctx)) != SPV_OK) return st;
    int chunks = (int)(((size_t)ctx->sm_count * 3 + (size_t)B * io->heads - 1) / ((size_t)B * io->heads));
    int chunk_len = ((n_tok + chunks - 1) / chunks + TK - 1) / TK * TK;
    if (chunk_len < 2 * GCH) chunk_len = 2 * GCH;
    chunks = (n_tok + chunk_len - 1) / chunk_len;
    char* w = (char*)ws;
    float* logits = (float*)w; w += spv_align_up(rows * n_tok * 4, 256);
    float* part_ml = (float*)w; w += spv_align_up(rows * chunks * 2 * 4, 256);
    float* part_o = (float*)w;
    if (logits_out) *logits_out = logits;
    CUtensorMap tq, tk, tv;
    if ((st = make_qkv_map(ctx, &tq, io->q, io->sb, io->st, io->sh, n_tok, io->heads, B, TQ)) != SPV_OK) return st;
    if ((st = make_qkv_map(ctx, &tk, io->k, io->sb, io->st, io->sh, n_tok, io->heads, B, TK)) != SPV_OK) return st;
    if ((st = make_qkv_map(ctx, &tv, io->v, io->sb, io->st, io->sh, n_tok, io->heads, B, TK)) != SPV_OK) return st;
    PatchParams pp;
    pp.block_off = plan->block_off; pp.tok_blk = plan->tok_blk; pp.tiles = plan->tiles; pp.o_tok = nullptr;
    pp.k = (const __nv_bfloat16*)io->k; pp.v = (const __nv_bfloat16*)io->v;
    pp.sb = io->sb; pp.st = io->st; pp.sh = io->sh;
    pp.o = (__nv_bfloat16*)io->o; pp.o_sb = io->o_sb; pp.o_st = io->o_st; pp.o_sh = io->o_sh;
    pp.nbx = 1; pp.nby = 1; pp.nb = 0; pp.radius = 0;
    pp.n_global = G; pp.n_patch = plan->n_patch; pp.tiles_per_image = 0;
    pp.scale_log2 = io->scale * 1.4426950408889634f;
    pp.status = ctx->d_status;
    pp.chunk_len = chunk_len; pp.n_chunks = chunks; pp.scale = io->scale;
    pp.logits = (scores || head_stats) ? logits : nullptr; pp.part_ml = part_ml; pp.part_o = part_o;
    SpvProfScope prof(ctx, SPV_K_ATTN_GLOBAL, stream);
    attn_patch_kernel<true><<<dim3(chunks, io->heads, B), ATT_THREADS, ATT_SMEM, stream>>>(tq, tk, tv, tq, pp);
    attn_global_combine<<<dim3(io->heads, B * G), 256, 0, stream>>>(logits, part_ml, part_o, chunks, n_tok, G,
                                                                   io->heads, (__nv_bfloat16*)io->o, io->o_sb,
                                                                   io->o_st, io->o_sh, scores, score_idx, score_stride,
                                                                   head_stats);
    return spv_launch_ok(ctx, 2);
  }
  // as many chunks as fill the GPU once (two CTAs of this kernel per SM), none shorter than GCH keys
  const int max_chunks = (n_tok + GCH - 1) / GCH;
  const size_t ctas_per_chunk = (size_t)B * G * io->heads;
  int chunks = (int)((size_t)ctx->sm_count * 2 / ctas_per_chunk);
  chunks = chunks < 1 ? 1 : (chunks > max_chunks ? max_chunks : chunks);
  const int chunk_len = ((n_tok + chunks - 1) / chunks + 127) / 128 * 128;
  chunks = (n_tok + chunk_len - 1) / chunk_len;
  char* w = (char*)ws;
  float* logits = (float*)w; w += spv_align_up(rows * n_tok * 4, 256);
  float* part_ml = (float*)w; w += spv_align_up(rows * chunks * 2 * 4, 256);
  float* part_o = (float*)w;
  SpvProfScope prof(ctx, SPV_K_ATTN_GLOBAL, stream);
  if (logits_out) *logits_out = logits;
  const bool lg_on = scores || head_stats;
#define SPV_GLOBAL_PARTIAL(LG, GQ_)                                                                                  \
  attn_global_partial<LG, GQ_><<<dim3(io->heads, chunks, B * ((G + GQ_ - 1) / GQ_)), 256, 0, stream>>>(              \
      (const __nv_bfloat16*)io->q, (const __nv_bfloat16*)io->k, (const __nv_bfloat16*)io->v, io->sb, io->st, io->sh, \
      n_tok, G, io->heads, io->scale, logits, part_ml, part_o, chunks, chunk_len)
  if (lg_on) SPV_GLOBAL_PARTIAL(true, 1); else SPV_GLOBAL_PARTIAL(false, 1);
#undef SPV_GLOBAL_PARTIAL
  attn_global_combine<<<dim3(io->heads, B * G), 256, 0, stream>>>(logits, part_ml, part_o, chunks, n_tok, G,
                                                                 io->heads, (__nv_bfloat16*)io->o, io->o_sb,
                                                                 io->o_st, io->o_sh, scores, score_idx, score_stride,
                                                                 head_stats);
  return spv_launch_ok(ctx, 2);
}

// ------------------------------------------------------------------------------------------
// C entry points
// ------------------------------------------------------------------------------------------
static int32_t validate_desc(const spv_attn_desc* d) {
  if (!d) return SPV_ERR_INVALID_ARG;
  if (d->batch < 1 || d->grid_h < 1 || d->grid_w < 1 || d->block < 1 || d->radius < 0 || d->heads < 1)
    return SPV_ERR_INVALID_ARG;
  if (d->n_patch < 1 || d->n_patch > d->grid_h * d->grid_w) return SPV_ERR_INVALID_ARG;
  if (!d->patch_pos && d->n_patch != d->grid_h * d->grid_w) return SPV_ERR_INVALID_ARG;
  if (d->token_order != SPV_TOKENS_ROW_MAJOR && d->token_order != SPV_TOKENS_BLOCK_MAJOR)
    return SPV_ERR_INVALID_ARG;
  if (d->head_dim != HD) return SPV_ERR_UNSUPPORTED;
  if (d->n_global < 1 || d->n_global > MAXG) return SPV_ERR_UNSUPPORTED;
  if (d->stride_tok % 8 || d->stride_head % 8 || d->stride_b % 8) return SPV_ERR_ALIGNMENT;
  if (d->stride_tok < HD || d->stride_head < HD) return SPV_ERR_INVALID_ARG;
  return SPV_OK;
}

static size_t regroup_bytes(const spv_attn_desc* d) {
  if (d->token_order == SPV_TOKENS_BLOCK_MAJOR) return 0;
  return 3 * spv_align_up((size_t)d->batch * (d->n_global + d->n_patch) * d->heads * HD * 2, 256);
}

extern "C" int32_t spv_attn_workspace_size(const spv_attn_desc* d, size_t* bytes) {
  int32_t st = validate_desc(d);
  if (st != SPV_OK) return st;
  if (!bytes) return SPV_ERR_INVALID_ARG;
  *bytes = spv_attn_plan_bytes(d->batch, d->grid_h, d->grid_w, d->block, d->n_patch, d->token_order) +
           regroup_bytes(d) + spv_attn_global_bytes(d->batch, d->n_global, d->heads, d->n_global + d->n_patch);
  return SPV_OK;
}

extern "C" int32_t spatial_block_attention(spv_ctx* ctx, const spv_attn_desc* d, const void* q, const void* k,
                                           const void* v, void* o, float* cls_scores, void* workspace,
                                           size_t workspace_bytes, void* stream_) {
  if (!ctx) return SPV_ERR_INVALID_ARG;
  int32_t st = validate_desc(d);
  if (spv_on_device(ctx) != SPV_OK) return SPV_ERR_INVALID_ARG;
  if (st != SPV_OK) return st;
  if (!q || !k || !v || !o) return SPV_ERR_INVALID_ARG;
  if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)o) & 15u) return SPV_ERR_ALIGNMENT;
  size_t need;
  spv_attn_workspace_size(d, &need);
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255u)) return SPV_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)stream_;
  char* w = (char*)workspace;
  const size_t plan_b = spv_attn_plan_bytes(d->batch, d->grid_h, d->grid_w, d->block, d->n_patch, d->token_order);
  SpvAttnPlan plan;
  st = spv_attn_plan_build(ctx, d->batch, d->grid_h, d->grid_w, d->block, d->radius, d->n_global, d->n_patch,
                           d->patch_pos, d->token_order, w, plan_b, stream, &plan, true);
  if (st != SPV_OK) return st;
  w += plan_b;
  const int n_tok = d->n_global + d->n_patch;
  const float scale = d->softmax_scale != 0.f ? d->softmax_scale : 0.125f;
  SpvAttnIO io;
  io.heads = d->heads; io.scale = scale;
  io.o = o; io.o_sb = d->stride_b; io.o_st = d->stride_tok; io.o_sh = d->stride_head;
  // global-query rows read the caller's tensors directly (a dense row needs no grouping)
  SpvAttnIO gio = io;
  gio.q = q; gio.k = k; gio.v = v; gio.sb = d->stride_b; gio.st = d->stride_tok; gio.sh = d->stride_head;
  gio.o_tok = nullptr;
  if (d->token_order == SPV_TOKENS_ROW_MAJOR) {
    const size_t one = spv_align_up((size_t)d->batch * n_tok * d->heads * HD * 2, 256);
    __nv_bfloat16* qb = (__nv_bfloat16*)w; w += one;
    __nv_bfloat16* kb = (__nv_bfloat16*)w; w += one;
    __nv_bfloat16* vb = (__nv_bfloat16*)w; w += one;
    const int64_t total = (int64_t)d->batch * n_tok * d->heads;
    int64_t blocks = (total * 8 + 255) / 256;
    const int64_t cap = (int64_t)ctx->sm_count * 16;
    if (blocks > cap) blocks = cap;
    SpvProfScope prof(ctx, SPV_K_ATTN_PLAN, stream);
    attn_regroup<<<(unsigned)blocks, 256, 0, stream>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k,
                                                      (const __nv_bfloat16*)v, d->stride_b, d->stride_tok,
                                                      d->stride_head, qb, kb, vb, plan.bm_src, d->batch,
                                                      d->n_global, d->n_patch, d->heads, ctx->d_status + 1);
    if ((st = spv_launch_ok(ctx)) != SPV_OK) return st;
    io.q = qb; io.k = kb; io.v = vb;
    io.st = (int64_t)d->heads * HD; io.sh = HD; io.sb = (int64_t)n_tok * d->heads * HD;
    io.o_tok = plan.bm_src;
  } else {
    io.q = q; io.k = k; io.v = v; io.sb = d->stride_b; io.st = d->stride_tok; io.sh = d->stride_head;
    io.o_tok = nullptr;
  }
  if ((st = spv_attn_run_patches(ctx, &plan, &io, stream)) != SPV_OK) return st;
  return spv_attn_run_globals(ctx, &plan, &gio, cls_scores, nullptr, d->n_patch, w,
                              spv_attn_global_bytes(d->batch, d->n_global, d->heads, n_tok), stream);
}
