// Rate probes for the three hardware limits the sparse-attention kernel is designed against:
//   - special-function unit: ex2.approx per clock and SM, alone and inside the softmax inner body
//     (scale, exponential, row sum, bf16 pack), optionally with part of the exponentials evaluated
//     as a polynomial on the multiply-add pipe;
//   - tensor pipe: tcgen05.mma issue rate for the tile shapes in question (M = 64 / 128, several N),
//     A operand from shared memory or from TMEM;
//   - L2 -> shared memory: TMA tile loads of an L2-resident buffer with a ring of stages in flight.
// Every kernel is bounded (fixed trip counts, bounded mbarrier waits) and touches only its own
// buffers.  The paper has no counterpart; the numbers feed the kernel design notes.
#include "common.cuh"

namespace {

using namespace spv;

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// out[0 .. grid) = cycles of each CTA
__global__ void __launch_bounds__(1024) mb_ex2_kernel(int iters, float seed, float* sink, long long* cyc) {
  float x[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = seed + 0.01f * (float)(i + threadIdx.x % 7);
  __syncthreads();
  const long long t0 = clock64();
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = ex2f(-x[i]);     // stays in (0.5, 1]
  }
  const long long t1 = clock64();
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) s += x[i];
  if (s == 123.456f) sink[0] = s;
  if (threadIdx.x == 0) cyc[blockIdx.x] = t1 - t0;
}

// 2^x for x <= 0 on the multiply-add pipe: round to nearest integer by the magic-number add, cubic
// in the remainder r in [-0.5, 0.5] (equal-ripple fit of the relative error), exponent added as an
// integer.  Used here only to measure what such an evaluation costs next to ex2.approx.
__device__ __forceinline__ float exp2_poly(float x) {
  x = fmaxf(x, -120.0f);
  const float t = x + 12582912.0f;                       // 1.5 * 2^23: low mantissa bits = round(x)
  const float r = x - (t - 12582912.0f);
  float p = fmaf(5.5171661e-2f, r, 2.4261113e-1f);
  p = fmaf(p, r, 6.9326097e-1f);
  p = fmaf(p, r, 9.9992806e-1f);                         // relative error below 7.5e-5
  return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}

// The inner body of the online softmax on `cols` scores per thread held in registers: p = 2^(s*scale - m),
// row sum, bf16 pack.  poly_per_8 of every eight exponentials go to the polynomial.
template <int POLY>
__global__ void __launch_bounds__(1024) mb_softmax_body_kernel(int iters, float seed, uint32_t* sink, long long* cyc) {
  constexpr int COLS = 64;
  float s[COLS];
#pragma unroll
  for (int i = 0; i < COLS; ++i) s[i] = -seed * (float)((i * 37 + threadIdx.x) % 19);
  float l = 0.f;
  uint32_t acc = 0;
  const float sl2 = 0.18f;
  __syncthreads();
  const long long t0 = clock64();
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
    const float m = seed * (float)it;
    const float2 sl2_2 = make_float2(sl2, sl2), nm_2 = make_float2(-m, -m);
    float2 rs = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < COLS; i += 2) {
      const float2 x = __ffma2_rn(make_float2(s[i], s[i + 1]), sl2_2, nm_2);
      float2 pp;
      if ((i % 8) < POLY) { pp.x = exp2_poly(x.x); pp.y = exp2_poly(x.y); }
      else { pp.x = ex2f(x.x); pp.y = ex2f(x.y); }
      rs = __fadd2_rn(rs, pp);
      acc ^= pack_bf16(pp.x, pp.y);
    }
    l += rs.x + rs.y;
  }
  const long long t1 = clock64();
  if (l == 123.456f || acc == 0x12345u) sink[0] = acc;
  if (threadIdx.x == 0) cyc[blockIdx.x] = t1 - t0;
}

// tcgen05.mma rate: one thread issues iters x 4 MMAs of M x N x 16 (operands: whatever the zero-filled
// shared memory / TMEM holds), one commit at the end.  Consecutive instructions rotate over n_acc
// accumulators: n_acc = 1 is the dependent chain of a K loop, larger values show what independent
// instructions reach.
struct MmaArgs { int m, n, iters, a_from_tmem, tmem_cols, n_acc, issue_mode, issuers; uint32_t* status; long long* cyc; };

__global__ void __launch_bounds__(128) mb_mma_kernel(MmaArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;                 // 128 rows x 128 B
  uint8_t* sB = smem + 16384;         // 256 rows x 128 B
  uint64_t* bar = reinterpret_cast<uint64_t*>(sB + 32768);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar + 4);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  for (int i = threadIdx.x; i < (16384 + 32768) / 16; i += blockDim.x)
    reinterpret_cast<uint4*>(smem)[i] = make_uint4(0u, 0u, 0u, 0u);
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) { for (int i = 0; i < 4; ++i) mbar_init(&bar[i], 1); *abort_flag = 0; mbar_fence_init(); }
  if (warp == 0) { tmem_alloc(tmem_slot, (uint32_t)a.tmem_cols); tmem_relinquish(); }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t idesc = idesc_bf16(a.m, a.n, false);
  const uint64_t da = smem_desc_sw128(smem_u32(sA)), db = smem_desc_sw128(smem_u32(sB));
  const uint32_t a_tmem = tmem + (uint32_t)a.tmem_cols - 32;    // 4 x 8 columns of bf16 A
  if (a.issue_mode == 0) {
    // one thread of each of the first `issuers` warps runs its own issue loop (divergent branch), on its own
    // accumulators and its own mbarrier
    if ((threadIdx.x & 31) == 0 && warp < a.issuers) {
      const long long t0 = clock64();
      const uint32_t base = tmem + (uint32_t)(warp * a.n_acc * a.n);
      uint32_t acc = 0;
#pragma unroll 1
      for (int it = 0; it < a.iters; ++it) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const uint32_t d_col = base + acc * (uint32_t)a.n;
          acc = acc + 1 == (uint32_t)a.n_acc ? 0u : acc + 1;
          if (a.a_from_tmem) mma_ts(d_col, a_tmem + kk * 8, db + (uint64_t)(kk * 2), idesc, 1u);
          else mma_ss(d_col, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, 1u);
        }
      }
      tc_commit(&bar[warp]);
      mbar_wait(&bar[warp], 0, abort_flag, a.status, 0x3100);
      if (warp == 0) a.cyc[blockIdx.x] = clock64() - t0;
    }
  } else if (warp < a.issuers) {
    // the whole warp runs the loop and one elected lane issues: the operands of the instruction are
    // the same in every lane, so that they can be kept in uniform registers
    const long long t0 = clock64();
    const uint32_t base = tmem + (uint32_t)(warp * a.n_acc * a.n);
    uint32_t acc = 0;
#pragma unroll 1
    for (int it = 0; it < a.iters; ++it) {
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const uint32_t d_col = base + acc * (uint32_t)a.n;
        acc = acc + 1 == (uint32_t)a.n_acc ? 0u : acc + 1;
        if (elect_one()) {
          if (a.a_from_tmem) mma_ts(d_col, a_tmem + kk * 8, db + (uint64_t)(kk * 2), idesc, 1u);
          else mma_ss(d_col, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, 1u);
        }
      }
    }
    if (elect_one()) tc_commit(&bar[warp]);
    __syncwarp();
    mbar_wait(&bar[warp], 0, abort_flag, a.status, 0x3100);
    if (threadIdx.x == 0) a.cyc[blockIdx.x] = clock64() - t0;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
}

// TMA tile loads (box_rows x 128 B) of an L2-resident buffer, `stages` loads in flight per CTA.
struct TmaArgs { int iters, stages, box_rows, n_tiles; uint32_t* status; long long* cyc; };

__global__ void __launch_bounds__(32) mb_tma_kernel(const __grid_constant__ CUtensorMap tm, TmaArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int box_bytes = a.box_rows * 128;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + a.stages * box_bytes);
  volatile uint32_t* abort_flag = reinterpret_cast<uint32_t*>(bars + a.stages);
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) mbar_init(&bars[s], 1);
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tm);
    uint32_t tile = ((uint32_t)blockIdx.x * 7919u) & (uint32_t)(a.n_tiles - 1);
    const long long t0 = clock64();
#pragma unroll 1
    for (int i = 0; i < a.iters; ++i) {
      const int s = i % a.stages;
      if (i >= a.stages) mbar_wait(&bars[s], ((i / a.stages) - 1) & 1, abort_flag, a.status, 0x3200);
      mbar_expect_tx(&bars[s], (uint32_t)box_bytes);
      tile = (tile + 104729u) & (uint32_t)(a.n_tiles - 1);          // n_tiles is a power of two
      tma_load_2d(smem + s * box_bytes, &tm, &bars[s], 0, (int)tile * a.box_rows);
    }
    // drain: every stage's last load
    for (int i = a.iters; i < a.iters + a.stages; ++i) {
      const int s = i % a.stages;
      if (i >= a.stages) mbar_wait(&bars[s], ((i / a.stages) - 1) & 1, abort_flag, a.status, 0x3300);
    }
    a.cyc[blockIdx.x] = clock64() - t0;
  }
}

}  // namespace

extern "C" int32_t spv_microbench(spv_ctx* ctx, const spv_microbench_desc* d, void* buffer, size_t buffer_bytes,
                                  void* stream_, spv_microbench_result* out) {
  if (!ctx || !d || !out || !buffer) return SPV_ERR_INVALID_ARG;
  if (spv_on_device(ctx) != SPV_OK) return SPV_ERR_INVALID_ARG;
  if (d->iters < 1 || d->iters > (1 << 22) || d->ctas_per_sm < 1 || d->ctas_per_sm > 4) return SPV_ERR_INVALID_ARG;
  if ((uintptr_t)buffer & 255u) return SPV_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)stream_;
  const int grid = ctx->sm_count * d->ctas_per_sm;
  const size_t cyc_bytes = spv_align_up((size_t)grid * sizeof(long long), 256);
  if (buffer_bytes < cyc_bytes + 256) return SPV_ERR_WORKSPACE;
  long long* cyc = (long long*)buffer;
  void* rest = (char*)buffer + cyc_bytes;
  const size_t rest_bytes = buffer_bytes - cyc_bytes;
  double units = 0.0;
  cudaEvent_t e0, e1;
  SPV_CUDA_OK(cudaEventCreate(&e0));
  SPV_CUDA_OK(cudaEventCreate(&e1));
  int32_t st = SPV_OK;
  // each probe runs twice; the second run is timed
  for (int rep = 0; rep < 2 && st == SPV_OK; ++rep) {
    if (rep == 1) cudaEventRecord(e0, stream);
    switch (d->kind) {
      case SPV_MB_EX2: {
        if (d->threads < 32 || d->threads > 1024 || d->threads % 32) { st = SPV_ERR_INVALID_ARG; break; }
        mb_ex2_kernel<<<grid, d->threads, 0, stream>>>(d->iters, 0.7f, (float*)rest, cyc);
        units = (double)grid * d->threads * 8.0 * d->iters;
        break;
      }
      case SPV_MB_SOFTMAX_BODY: {
        if (d->threads < 32 || d->threads > 512 || d->threads % 32) { st = SPV_ERR_INVALID_ARG; break; }
        switch (d->poly_per_8) {
          case 0: mb_softmax_body_kernel<0><<<grid, d->threads, 0, stream>>>(d->iters, 1e-3f, (uint32_t*)rest, cyc); break;
          case 2: mb_softmax_body_kernel<2><<<grid, d->threads, 0, stream>>>(d->iters, 1e-3f, (uint32_t*)rest, cyc); break;
          case 4: mb_softmax_body_kernel<4><<<grid, d->threads, 0, stream>>>(d->iters, 1e-3f, (uint32_t*)rest, cyc); break;
          case 8: mb_softmax_body_kernel<8><<<grid, d->threads, 0, stream>>>(d->iters, 1e-3f, (uint32_t*)rest, cyc); break;
          default: st = SPV_ERR_INVALID_ARG;
        }
        units = (double)grid * d->threads * 64.0 * d->iters;
        break;
      }
      case SPV_MB_MMA_SS:
      case SPV_MB_MMA_TS: {
        if ((d->m != 64 && d->m != 128) || d->n < 16 || d->n > 256 || d->n % 16) { st = SPV_ERR_INVALID_ARG; break; }
        MmaArgs a;
        a.m = d->m; a.n = d->n; a.iters = d->iters; a.a_from_tmem = d->kind == SPV_MB_MMA_TS;
        a.tmem_cols = 512 / (d->ctas_per_sm == 3 ? 4 : d->ctas_per_sm);
        a.n_acc = d->accumulators < 1 ? 1 : d->accumulators;
        a.issue_mode = d->issue_mode != 0;
        a.issuers = d->issuers < 1 ? 1 : d->issuers;
        if (a.issuers > 4 || a.tmem_cols < a.issuers * a.n_acc * d->n + 32) { st = SPV_ERR_INVALID_ARG; break; }
        if (a.n_acc > 8 || a.tmem_cols < a.n_acc * d->n + 32) { st = SPV_ERR_INVALID_ARG; break; }
        a.status = ctx->d_status; a.cyc = cyc;
        const int smem = 16384 + 32768 + 1024 + 64;
        if (cudaFuncSetAttribute(mb_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) { st = SPV_ERR_CUDA; break; }
        mb_mma_kernel<<<grid, 128, smem, stream>>>(a);
        units = (double)grid * a.issuers * d->iters * 4.0 * 2.0 * d->m * d->n * 16.0;
        break;
      }
      case SPV_MB_L2_TMA: {
        if (d->box_rows < 8 || d->box_rows > 256 || d->box_rows % 8 || d->stages < 1 || d->stages > 8) { st = SPV_ERR_INVALID_ARG; break; }
        const int box_bytes = d->box_rows * 128;
        const int smem = d->stages * box_bytes + 1024 + 128;
        if (smem > 200 * 1024) { st = SPV_ERR_INVALID_ARG; break; }
        // the buffer the loads walk over: at most 32 MB, so that it stays in L2
        size_t span = rest_bytes > ((size_t)32 << 20) ? ((size_t)32 << 20) : rest_bytes;
        int n_tiles = 1;
        while ((size_t)(2 * n_tiles) * (size_t)box_bytes <= span) n_tiles *= 2;    // a power of two of tiles
        if (n_tiles < 64) { st = SPV_ERR_WORKSPACE; break; }
        CUtensorMap tm;
        const uint64_t dims[2] = {64, (uint64_t)n_tiles * d->box_rows};
        const uint64_t str[1] = {128};
        const uint32_t box[2] = {64, (uint32_t)d->box_rows};
        if ((st = spv_make_tmap_bf16(ctx, &tm, rest, 2, dims, str, box)) != SPV_OK) break;
        if (cudaFuncSetAttribute(mb_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) { st = SPV_ERR_CUDA; break; }
        TmaArgs a;
        a.iters = d->iters; a.stages = d->stages; a.box_rows = d->box_rows; a.n_tiles = n_tiles;
        a.status = ctx->d_status; a.cyc = cyc;
        mb_tma_kernel<<<grid, 32, smem, stream>>>(tm, a);
        units = (double)grid * d->iters * box_bytes;
        break;
      }
      default: st = SPV_ERR_INVALID_ARG;
    }
    if (st == SPV_OK) st = spv_launch_ok(ctx);
  }
  if (st == SPV_OK) {
    cudaEventRecord(e1, stream);
    if (cudaEventSynchronize(e1) != cudaSuccess) st = SPV_ERR_CUDA;
  }
  if (st == SPV_OK) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e0, e1);
    long long* h = new long long[grid];
    if (cudaMemcpy(h, cyc, (size_t)grid * sizeof(long long), cudaMemcpyDeviceToHost) != cudaSuccess) st = SPV_ERR_CUDA;
    long long mx = 0;
    for (int i = 0; i < grid; ++i) mx = h[i] > mx ? h[i] : mx;
    delete[] h;
    out->ms = ms;
    out->cycles = (double)mx;
    out->units = units;
    out->sm_count = ctx->sm_count;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  return st;
}
