// Sec. 3.3 -- global-attention-score token filter: head average, exact deterministic top-k
// (ties to the lower index) and compaction of the surviving token rows.
//
// Three kernels on one stream:
//   filter_mean_key   head average in fp32 (heads added in index order, one division) and an
//                     order-preserving 32-bit key per patch; filter_mean_key_logits is the same with the
//                     softmax weights evaluated on the fly from the global row's logits (the fused front end
//                     inside vit_forward: the [batch, heads, patches] score tensor is never written);
//   filter_select     one CTA per image: 4-pass radix select of the k-th largest key, then an
//                     ordered two-counter scan that emits the kept indices in ascending order;
//   filter_gather     128-bit row copy of the global tokens and the kept rows.
#include "filter.cuh"

namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelItems = 4;

// Larger mean -> larger key.  +0 and -0 share a key; NaN gets key 0 (ranks last).
__device__ __forceinline__ uint32_t rank_key(float m) {
  if (m != m) return 0u;
  if (m == 0.0f) m = 0.0f;   // folds -0 into +0
  uint32_t u = __float_as_uint(m);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(256) filter_mean_key(const float* __restrict__ scores, int heads, int n_patch,
                                                       int npad, float* __restrict__ mean_ws,
                                                       uint32_t* __restrict__ key_ws,
                                                       float* __restrict__ mean_out) {
  const int b = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= npad) return;
  if (j >= n_patch) {          // padding of the key array: below every real key, never selected
    key_ws[(size_t)b * npad + j] = 0u;
    return;
  }
  const float* s = scores + (size_t)b * heads * n_patch + j;
  float sum = 0.0f;
  for (int h = 0; h < heads; ++h) sum = __fadd_rn(sum, __ldg(s + (size_t)h * n_patch));
  const float mean = __fdiv_rn(sum, (float)heads);
  mean_ws[(size_t)b * npad + j] = mean;
  key_ws[(size_t)b * npad + j] = rank_key(mean);
  if (mean_out) mean_out[(size_t)b * n_patch + j] = mean;
}

// The same head mean and key, with the softmax weight of every head evaluated here from the global row's
// scaled logits: p = exp(logit - max_h) * inv_sum_h, summed in head order.  One thread per present patch; the
// mean and key land at the patch's original position (keys of absent positions were zeroed beforehand).
__global__ void __launch_bounds__(256) filter_mean_key_logits(const float* __restrict__ logits,
                                                              const float* __restrict__ head_stats, int heads,
                                                              int n_global, int n_tok,
                                                              const int32_t* __restrict__ cur_pos, int npad,
                                                              float* __restrict__ mean_ws,
                                                              uint32_t* __restrict__ key_ws) {
  const int b = blockIdx.y;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int n_cur = n_tok - n_global;
  if (t >= n_cur) return;
  const float* lg = logits + (size_t)b * n_global * heads * n_tok + n_global + t;
  const float* hs = head_stats + (size_t)b * heads * 2;
  float sum = 0.0f;
  for (int h = 0; h < heads; ++h) {
    const float p = __expf(__ldg(lg + (size_t)h * n_tok) - __ldg(hs + 2 * h)) * __ldg(hs + 2 * h + 1);
    sum = __fadd_rn(sum, p);
  }
  const float mean = __fdiv_rn(sum, (float)heads);
  const int pos = cur_pos ? __ldg(cur_pos + (size_t)b * n_cur + t) : t;
  mean_ws[(size_t)b * npad + pos] = mean;
  key_ws[(size_t)b * npad + pos] = rank_key(mean);
}

// Block-wide exclusive scan of two counters; returns this thread's exclusive prefixes and the
// block totals.  Called by all kSelThreads threads.
__device__ __forceinline__ void block_scan2(int a, int b, int& ea, int& eb, int& ta, int& tb, int (*warp_tot)[2]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int na = __shfl_up_sync(0xffffffffu, ia, o), nb = __shfl_up_sync(0xffffffffu, ib, o);
    if (lane >= o) { ia += na; ib += nb; }
  }
  if (lane == 31) { warp_tot[warp][0] = ia; warp_tot[warp][1] = ib; }
  __syncthreads();
  if (warp == 0) {
    int wa = warp_tot[lane][0], wb = warp_tot[lane][1];
    int sa = wa, sb = wb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int na = __shfl_up_sync(0xffffffffu, sa, o), nb = __shfl_up_sync(0xffffffffu, sb, o);
      if (lane >= o) { sa += na; sb += nb; }
    }
    warp_tot[lane][0] = sa - wa;   // exclusive warp offsets
    warp_tot[lane][1] = sb - wb;
    if (lane == 31) { warp_tot[32][0] = sa; warp_tot[32][1] = sb; }
  }
  __syncthreads();
  ea = warp_tot[warp][0] + ia - a;
  eb = warp_tot[warp][1] + ib - b;
  ta = warp_tot[32][0];
  tb = warp_tot[32][1];
  __syncthreads();
}

__global__ void __launch_bounds__(kSelThreads) filter_select(const uint32_t* __restrict__ key_ws, int n_patch,
                                                             int npad, int k, int32_t* __restrict__ kept_idx,
                                                             const int32_t* __restrict__ pos_in,
                                                             int32_t* __restrict__ pos_out) {
  __shared__ int hist[256];
  __shared__ int warp_tot[33][2];
  __shared__ uint32_t s_prefix;
  __shared__ int s_remaining;
  const int b = blockIdx.x;
  const uint32_t* keys = key_ws + (size_t)b * npad;
  const uint4* keys4 = reinterpret_cast<const uint4*>(keys);
  const int n4 = npad >> 2;
  if (threadIdx.x == 0) { s_prefix = 0u; s_remaining = k; }

  // ---- radix select: the k-th largest key, 8 bits per pass from the top
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
    for (int i = threadIdx.x; i < n4; i += kSelThreads) {
      const uint4 v = keys4[i];
      const uint32_t e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int t = 0; t < 4; ++t)
        if (4 * i + t < n_patch && (e[t] & himask) == prefix) atomicAdd(&hist[(e[t] >> shift) & 255u], 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int rem = s_remaining, bin = 255;
      for (; bin > 0; --bin) {
        if (hist[bin] >= rem) break;
        rem -= hist[bin];
      }
      s_prefix = prefix | ((uint32_t)bin << shift);
      s_remaining = rem;
    }
    __syncthreads();
  }
  const uint32_t thr = s_prefix;     // k-th largest key
  const int need_eq = s_remaining;   // how many keys equal to it are kept (lowest indices first)

  // ---- ordered compaction: keep j iff key > thr, or key == thr and fewer than need_eq equal
  //      keys precede j.  prefix_keep = prefix_gt + min(prefix_eq, need_eq).
  int base_gt = 0, base_eq = 0;
  int32_t* kout = kept_idx + (size_t)b * k;
  for (int tile0 = 0; tile0 < n4; tile0 += kSelThreads) {
    const int i = tile0 + threadIdx.x;
    uint32_t e[4] = {0u, 0u, 0u, 0u};
    if (i < n4) {
      const uint4 v = keys4[i];
      e[0] = v.x; e[1] = v.y; e[2] = v.z; e[3] = v.w;
    }
    int gt = 0, eq = 0;
#pragma unroll
    for (int t = 0; t < kSelItems; ++t) {
      const bool valid = i < n4 && 4 * i + t < n_patch;
      gt += (valid && e[t] > thr) ? 1 : 0;
      eq += (valid && e[t] == thr) ? 1 : 0;
    }
    int egt, eeq, tgt, teq;
    block_scan2(gt, eq, egt, eeq, tgt, teq, warp_tot);
    int pgt = base_gt + egt, peq = base_eq + eeq;
#pragma unroll
    for (int t = 0; t < kSelItems; ++t) {
      const int j = 4 * i + t;
      const bool valid = i < n4 && j < n_patch;
      const bool is_gt = valid && e[t] > thr, is_eq = valid && e[t] == thr;
      if (is_gt || (is_eq && peq < need_eq)) {
        const int dst = pgt + min(peq, need_eq);
        kout[dst] = j;
        if (pos_out) pos_out[(size_t)b * k + dst] = pos_in ? pos_in[(size_t)b * n_patch + j] : j;
      }
      pgt += is_gt ? 1 : 0;
      peq += is_eq ? 1 : 0;
    }
    base_gt += tgt;
    base_eq += teq;
  }
}

// Row copy with 128-bit accesses: output row r of image b comes from input row r (global
// tokens) or n_global + kept_idx[r - n_global].  One warp per row, rows strided over the grid.
__global__ void __launch_bounds__(256) filter_gather(const uint4* __restrict__ in, uint4* __restrict__ out,
                                                     const int32_t* __restrict__ kept_idx, int batch, int n_global,
                                                     int k, int row_vec, int64_t in_stride_b_vec,
                                                     int64_t out_stride_b_vec) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
  const int rows_per_image = n_global + k;
  const int64_t total = (int64_t)batch * rows_per_image;
  for (int64_t r = warp; r < total; r += nwarps) {
    const int b = (int)(r / rows_per_image);
    const int t = (int)(r - (int64_t)b * rows_per_image);
    const int src_row = t < n_global ? t : n_global + __ldg(kept_idx + (size_t)b * k + (t - n_global));
    const uint4* src = in + b * in_stride_b_vec + (int64_t)src_row * row_vec;
    uint4* dst = out + b * out_stride_b_vec + (int64_t)t * row_vec;
    int c = lane;
    for (; c + 96 < row_vec; c += 128) {
      const uint4 v0 = __ldcs(src + c), v1 = __ldcs(src + c + 32), v2 = __ldcs(src + c + 64),
                  v3 = __ldcs(src + c + 96);
      __stcs(dst + c, v0);
      __stcs(dst + c + 32, v1);
      __stcs(dst + c + 64, v2);
      __stcs(dst + c + 96, v3);
    }
    for (; c < row_vec; c += 32) __stcs(dst + c, __ldcs(src + c));
  }
}

int32_t validate(const spv_filter_desc* d, int32_t* k) {
  if (!d || d->batch < 1 || d->heads < 1 || d->n_patch < 1 || d->n_global < 0) return SPV_ERR_INVALID_ARG;
  if (d->dim < 0 || (d->dim % 8) != 0) return SPV_ERR_ALIGNMENT;
  if (d->in_stride_b % 8 != 0 || d->out_stride_b % 8 != 0) return SPV_ERR_ALIGNMENT;
  return spv_filter_keep_count(d->n_patch, d->keep_ratio, k);
}

}  // namespace

extern "C" int32_t spv_filter_keep_count(int32_t n_patch, double keep_ratio, int32_t* k) {
  if (!k || n_patch < 1 || !(keep_ratio > 0.0) || keep_ratio > 1.0) return SPV_ERR_INVALID_ARG;
  // discard floor(p * n) lowest  <=>  keep ceil(keep * n); the guard absorbs the representation
  // error of keep * n in double
  double kd = __builtin_ceil(keep_ratio * (double)n_patch - 1e-9);
  int32_t kk = (int32_t)kd;
  if (kk < 1) kk = 1;
  if (kk > n_patch) kk = n_patch;
  *k = kk;
  return SPV_OK;
}

extern "C" int32_t spv_filter_workspace_size(const spv_filter_desc* d, size_t* bytes) {
  int32_t k;
  int32_t st = validate(d, &k);
  if (st != SPV_OK) return st;
  if (!bytes) return SPV_ERR_INVALID_ARG;
  const size_t npad = spv_align_up((size_t)d->n_patch, 4);
  *bytes = spv_align_up((size_t)d->batch * npad * sizeof(float), 256) +
           spv_align_up((size_t)d->batch * npad * sizeof(uint32_t), 256);
  return SPV_OK;
}

extern "C" int32_t cls_score_topk_filter(spv_ctx* ctx, const spv_filter_desc* d, const float* scores,
                                         const void* tokens_in, void* tokens_out, int32_t* kept_idx,
                                         float* mean_scores, const int32_t* pos_in, int32_t* pos_out,
                                         void* workspace, size_t workspace_bytes, void* stream_) {
  if (!ctx) return SPV_ERR_INVALID_ARG;
  int32_t k;
  int32_t st = validate(d, &k);
  if (st != SPV_OK) return st;
  return spv_filter_run_k(ctx, d, k, scores, tokens_in, tokens_out, kept_idx, mean_scores, pos_in, pos_out, workspace,
                          workspace_bytes, (cudaStream_t)stream_);
}

int32_t spv_filter_run_k(spv_ctx* ctx, const spv_filter_desc* d, int32_t k, const float* scores,
                         const void* tokens_in, void* tokens_out, int32_t* kept_idx, float* mean_scores,
                         const int32_t* pos_in, int32_t* pos_out, void* workspace, size_t workspace_bytes,
                         cudaStream_t stream) {
  if (!ctx || !d || k < 1 || k > d->n_patch) return SPV_ERR_INVALID_ARG;
  if (spv_on_device(ctx) != SPV_OK) return SPV_ERR_INVALID_ARG;
  if (!scores || !kept_idx) return SPV_ERR_INVALID_ARG;
  if ((tokens_in == nullptr) != (tokens_out == nullptr)) return SPV_ERR_INVALID_ARG;
  if (tokens_in && d->dim == 0) return SPV_ERR_INVALID_ARG;
  if (((uintptr_t)scores & 15u) || ((uintptr_t)tokens_in & 15u) || ((uintptr_t)tokens_out & 15u))
    return SPV_ERR_ALIGNMENT;
  const size_t need = spv_align_up((size_t)d->batch * spv_align_up((size_t)d->n_patch, 4) * sizeof(float), 256) * 2;
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255u)) return SPV_ERR_WORKSPACE;
  const int npad = (int)spv_align_up((size_t)d->n_patch, 4);
  float* mean_ws = (float*)workspace;
  uint32_t* key_ws =
      (uint32_t*)((char*)workspace + spv_align_up((size_t)d->batch * npad * sizeof(float), 256));

  {
    SpvProfScope prof(ctx, SPV_K_FILTER_SELECT, stream,
                      (double)d->batch * ((double)d->heads * d->n_patch * 4.0 + (double)k * 4.0));
    filter_mean_key<<<dim3((npad + 255) / 256, d->batch), 256, 0, stream>>>(scores, d->heads, d->n_patch, npad,
                                                                          mean_ws, key_ws, mean_scores);
    filter_select<<<d->batch, kSelThreads, 0, stream>>>(key_ws, d->n_patch, npad, k, kept_idx, pos_in, pos_out);
  }
  int launches = 2;
  if (tokens_in) {
    const int64_t rows = (int64_t)d->batch * (d->n_global + k);
    const int row_vec = d->dim / 8;
    const int64_t in_sb = d->in_stride_b ? d->in_stride_b : (int64_t)(d->n_global + d->n_patch) * d->dim;
    const int64_t out_sb = d->out_stride_b ? d->out_stride_b : (int64_t)(d->n_global + k) * d->dim;
    int64_t blocks = (rows + 7) / 8;
    const int64_t cap = (int64_t)ctx->sm_count * 8;
    if (blocks > cap) blocks = cap;
    SpvProfScope prof(ctx, SPV_K_FILTER_GATHER, stream, 2.0 * (double)rows * d->dim * 2.0);
    filter_gather<<<(unsigned)blocks, 256, 0, stream>>>((const uint4*)tokens_in, (uint4*)tokens_out, kept_idx,
                                                       d->batch, d->n_global, k, row_vec, in_sb / 8, out_sb / 8);
    ++launches;
  }
  return spv_launch_ok(ctx, launches);
}

int32_t spv_filter_rank_logits(spv_ctx* ctx, int32_t batch, int32_t heads, int32_t n_global, int32_t n_tok,
                               int32_t np_grid, int32_t k, const float* logits, const float* head_stats,
                               const int32_t* cur_pos, int32_t* kept_idx, void* workspace, size_t workspace_bytes,
                               cudaStream_t stream) {
  if (!ctx || !logits || !head_stats || !kept_idx || batch < 1 || heads < 1 || n_global < 1) return SPV_ERR_INVALID_ARG;
  const int n_cur = n_tok - n_global;
  if (n_cur < 1 || n_cur > np_grid || k < 1 || k > n_cur) return SPV_ERR_INVALID_ARG;
  const int npad = (int)spv_align_up((size_t)np_grid, 4);
  const size_t half = spv_align_up((size_t)batch * npad * sizeof(float), 256);
  if (!workspace || workspace_bytes < 2 * half || ((uintptr_t)workspace & 255u)) return SPV_ERR_WORKSPACE;
  float* mean_ws = (float*)workspace;
  uint32_t* key_ws = (uint32_t*)((char*)workspace + half);
  SpvProfScope prof(ctx, SPV_K_FILTER_SELECT, stream,
                    (double)batch * ((double)heads * n_cur * 4.0 + (double)k * 4.0));
  // key 0 ranks below every real key: padding and positions that are no longer present
  SPV_CUDA_OK(cudaMemsetAsync(key_ws, 0, (size_t)batch * npad * sizeof(uint32_t), stream));
  filter_mean_key_logits<<<dim3((n_cur + 255) / 256, batch), 256, 0, stream>>>(logits, head_stats, heads, n_global,
                                                                             n_tok, cur_pos, npad, mean_ws, key_ws);
  filter_select<<<batch, kSelThreads, 0, stream>>>(key_ws, np_grid, npad, k, kept_idx, nullptr, nullptr);
  return spv_launch_ok(ctx, 2);
}

// ------------------------------------------------------------------------------------------
// Variant for callers that cannot allocate: the scratch (head means + ranking keys) is a
// file-scope device array instead of a caller workspace.  In host code `g_filter_scratch` is only
// a stand-in for the symbol, not a device address: the address is looked up once per device with
// cudaGetSymbolAddress and that pointer is what the kernels receive.
// ------------------------------------------------------------------------------------------
#include <mutex>

static __device__ __align__(256) unsigned char g_filter_scratch[SPV_FILTER_STATIC_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices];     // device address of g_filter_scratch on each device
int g_static_sms[kMaxDevices];

// Set-up of the current device (first call only): symbol address and SM count.  No allocation.
int32_t static_scratch(int* device_out, void** ptr_out, int* sms_out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPV_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_filter_scratch) != cudaSuccess || !p) return SPV_ERR_CUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
      return SPV_ERR_CUDA;
    g_static_sms[dev] = sms;
    g_static_ptr[dev] = p;
  }
  *device_out = dev;
  *ptr_out = g_static_ptr[dev];
  *sms_out = g_static_sms[dev];
  return SPV_OK;
}
}  // namespace

extern "C" int32_t cls_score_topk_filter_static(const spv_filter_desc* d, const float* scores, const void* tokens_in,
                                                void* tokens_out, int32_t* kept_idx, float* mean_scores,
                                                const int32_t* pos_in, int32_t* pos_out, void* stream_) {
  int32_t k;
  int32_t st = validate(d, &k);
  if (st != SPV_OK) return st;
  if (!scores || !kept_idx) return SPV_ERR_INVALID_ARG;
  if ((tokens_in == nullptr) != (tokens_out == nullptr)) return SPV_ERR_INVALID_ARG;
  if (tokens_in && d->dim == 0) return SPV_ERR_INVALID_ARG;
  if (((uintptr_t)scores & 15u) || ((uintptr_t)tokens_in & 15u) || ((uintptr_t)tokens_out & 15u))
    return SPV_ERR_ALIGNMENT;
  const size_t npad = spv_align_up((size_t)d->n_patch, 4);
  const size_t half = spv_align_up((size_t)d->batch * npad * sizeof(float), 256);
  if (2 * half > (size_t)SPV_FILTER_STATIC_BYTES) return SPV_ERR_STATIC_LIMIT;
  int dev, sms;
  void* scratch;
  if ((st = static_scratch(&dev, &scratch, &sms)) != SPV_OK) return st;
  cudaStream_t stream = (cudaStream_t)stream_;
  float* mean_ws = (float*)scratch;
  uint32_t* key_ws = (uint32_t*)((char*)scratch + half);
  // every element of [0, npad) per image is written by filter_mean_key before filter_select reads
  // it, so what an earlier call left in the array is never seen
  filter_mean_key<<<dim3((unsigned)((npad + 255) / 256), d->batch), 256, 0, stream>>>(
      scores, d->heads, d->n_patch, (int)npad, mean_ws, key_ws, mean_scores);
  filter_select<<<d->batch, kSelThreads, 0, stream>>>(key_ws, d->n_patch, (int)npad, k, kept_idx, pos_in, pos_out);
  if (tokens_in) {
    const int64_t rows = (int64_t)d->batch * (d->n_global + k);
    const int row_vec = d->dim / 8;
    const int64_t in_sb = d->in_stride_b ? d->in_stride_b : (int64_t)(d->n_global + d->n_patch) * d->dim;
    const int64_t out_sb = d->out_stride_b ? d->out_stride_b : (int64_t)(d->n_global + k) * d->dim;
    int64_t blocks = (rows + 7) / 8;
    const int64_t cap = (int64_t)sms * 8;
    if (blocks > cap) blocks = cap;
    filter_gather<<<(unsigned)blocks, 256, 0, stream>>>((const uint4*)tokens_in, (uint4*)tokens_out, kept_idx,
                                                       d->batch, d->n_global, k, row_vec, in_sb / 8, out_sb / 8);
  }
  return cudaGetLastError() == cudaSuccess ? SPV_OK : SPV_ERR_CUDA;
}
