// bf16 GEMM with fused epilogues for the ViT block (QKV / out-proj / MLP / patch embedding):
//   C[M, N] = A[M, K] * W[N, K]^T, fp32 accumulation in TMEM.
//
// Persistent kernel, one CTA per SM, K in slices of 64.  Two forms of the same body:
//   pair form   (M > 256) two CTAs of a cluster share one tcgen05.mma.cta_group::2 of shape
//               256 x 256 x 16: each CTA loads 128 rows of A and 128 of the 256 rows of W, the
//               even CTA issues the MMAs, each CTA's TMEM gets its 128 x 256 half of the tile and
//               each CTA runs its own epilogue.  A W slice crosses L2 -> shared memory once per
//               256 output rows instead of once per 128, and a stage is 32 KB (6-stage ring).
//   single form 128 x 256 tiles, 48 KB stages (4-stage ring), for small M.
//   warp 0      TMA producer (A and W slices, 128-byte swizzle)
//   warp 1      tcgen05.mma issuer (one thread), owns the TMEM allocation (2 x 256 columns, so
//               the epilogue of tile i overlaps the main loop of tile i+1)
//   warp 18     hands staged chunks to TMA (tile store or fp32 add-reduce) and returns the buffers
//   warps 2..17 epilogue, four threads per output row: TMEM -> registers -> bias / activation /
//               scale -> swizzled staging buffer -> TMA tile store (bf16 outputs, fp32 rows) or
//               fp32 TMA add-reduce into the residual stream
// Rows beyond M and columns beyond N are zero-filled by TMA on load and clipped by TMA on store.
#include "common.cuh"

namespace {

using namespace spv;

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int A_BYTES = BM * BK * 2;
template <bool PAIR> struct Ring {
  static constexpr int STAGES = PAIR ? 6 : 4;
  static constexpr int B_ROWS = PAIR ? BN / 2 : BN;       // rows of W one CTA loads per slice
  static constexpr int B_BYTES = B_ROWS * BK * 2;
};
constexpr int GEMM_THREADS = 608;      // warp 0 TMA, warp 1 MMA, warps 2-17 epilogue (four per TMEM lane quadrant),
                                       // warp 18 hands the staged chunks to TMA
constexpr int EPI_THREADS = 512;
constexpr int STORE_WARP = 18;
// named barriers (0 is __syncthreads): staging buffer b is FULL (written) / EMPTY (read by TMA); the 512
// epilogue threads and the 32 threads of the store warp take part in each
constexpr int BAR_FULL = 1, BAR_EMPTY = 3, BAR_EPI = 5, BAR_HANDOFF_THREADS = EPI_THREADS + 32;
constexpr int EPI_BYTES = 128 * 128;    // one staging buffer: 128 rows x 128 bytes (32 fp32 or 64 bf16 columns)
constexpr int GEMM_SMEM = 4 * (A_BYTES + BN * BK * 2) + 2 * EPI_BYTES + 1024 /*align*/ + 256 /*barriers*/ + BN * 4 /*bias*/;   // both forms: 192 KB of ring

struct EpiParams {
  void* out;
  int64_t ldo;
  const float* bias;
  const void* aux;
  int64_t ldaux;
  const float* scale;
  const float* addrow;
  int64_t ldadd;
  int32_t rows_per_image;
};

// Exact (erf) GELU.  erf by the rational/exponential form of Abramowitz & Stegun 7.1.26
// (|error| <= 1.5e-7, branch-free: one reciprocal, one exponential, five multiply-adds), which keeps
// the epilogue of the MLP GEMM shorter than its main loop; the absolute error of the GELU value is
// below |x| * 1e-7, far inside the bf16 rounding of the stored activation.
// Two values at a time: the multiply-adds run as packed fp32x2 instructions.  Written for the fewest
// instructions (the epilogue warps of the first MLP GEMM are bound by their issue slots):
//   gelu(x) = 0.5 x + |x| h,  h = 0.5 erf(|x| / sqrt 2) = 0.5 + q(t) e,
//   t = 1 / (1 + (p / sqrt 2) |x|),  e = exp(-x^2 / 2) = 2^(-(log2 e / 2) x^2),
//   q(t) = -0.5 (a1 t + a2 t^2 + a3 t^3 + a4 t^4 + a5 t^5)   (the factor folded into the coefficients).
__device__ __forceinline__ float2 gelu_erf2(float2 x) {
  const float2 ax = make_float2(fabsf(x.x), fabsf(x.y));
  const float2 den = __ffma2_rn(ax, make_float2(0.3275911f * 0.70710678118654752f, 0.3275911f * 0.70710678118654752f),
                                make_float2(1.0f, 1.0f));
  // one reciprocal for the pair: 1/a = b / (a b), 1/b = a / (a b)  (a, b in [1, 1 + 0.23 |x|])
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(den.x * den.y));
  const float2 t = __fmul2_rn(make_float2(den.y, den.x), make_float2(r, r));
  float2 q = __ffma2_rn(make_float2(-0.5f * 1.061405429f, -0.5f * 1.061405429f), t,
                        make_float2(0.5f * 1.453152027f, 0.5f * 1.453152027f));
  q = __ffma2_rn(q, t, make_float2(-0.5f * 1.421413741f, -0.5f * 1.421413741f));
  q = __ffma2_rn(q, t, make_float2(0.5f * 0.284496736f, 0.5f * 0.284496736f));
  q = __ffma2_rn(q, t, make_float2(-0.5f * 0.254829592f, -0.5f * 0.254829592f));
  q = __fmul2_rn(q, t);
  const float2 arg = __fmul2_rn(__fmul2_rn(x, x), make_float2(-0.72134752044448170f, -0.72134752044448170f));
  float2 e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.x) : "f"(arg.x));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.y) : "f"(arg.y));
  const float2 h = __ffma2_rn(q, e, make_float2(0.5f, 0.5f));                    // 0.5 erf(|x| / sqrt 2)
  return __ffma2_rn(ax, h, __fmul2_rn(x, make_float2(0.5f, 0.5f)));             // 0.5 x + |x| h
}
// x * sigmoid(x) with the hardware exponential and reciprocal (relative error about 1e-6, far
// inside the bf16 rounding of the stored value); exp(-x) = inf for x < -88 gives 1/inf = 0, so x * 0 = -0
__device__ __forceinline__ float silu(float x) {
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * -1.4426950408889634f));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
  return x * r;
}

__host__ __device__ constexpr bool epi_is_f32(int epi) { return epi == SPV_EPI_BIAS_SCALE_RESID || epi == SPV_EPI_BIAS_ADDROW; }

// Eight consecutive outputs of row m, columns n .. n+7 (accumulators in acc), with the epilogue
// arithmetic applied; the result stays fp32.
template <int EPI>
__device__ __forceinline__ void epilogue_math(const EpiParams& p, const float* tile_bias, int n_base, int m, int n,
                                              const uint32_t* acc, float* v) {
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(acc[i]);
  if (p.bias) {
    // the tile's 256 bias values sit in shared memory (tile_bias[0] belongs to column n_base)
    const float4 b0 = *reinterpret_cast<const float4*>(tile_bias + (n - n_base));
    const float4 b1 = *reinterpret_cast<const float4*>(tile_bias + (n - n_base) + 4);
    v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w;
    v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
  }
  if constexpr (EPI == SPV_EPI_BIAS_GELU) {
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      const float2 g = gelu_erf2(make_float2(v[i], v[i + 1]));
      v[i] = g.x;
      v[i + 1] = g.y;
    }
  } else if constexpr (EPI == SPV_EPI_BIAS_SILU) {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = silu(v[i]);
  } else if constexpr (EPI == SPV_EPI_BIAS_MUL) {
    const uint4 a = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.aux) +
                                                    (int64_t)m * p.ldaux + n);
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = *reinterpret_cast<const __nv_bfloat162*>(&aw[i]);
      v[2 * i] *= __low2float(h);
      v[2 * i + 1] *= __high2float(h);
    }
  } else if constexpr (EPI == SPV_EPI_BIAS_SCALE_RESID) {
    if (p.scale) {
      const float4 s0 = __ldg(reinterpret_cast<const float4*>(p.scale + n));
      const float4 s1 = __ldg(reinterpret_cast<const float4*>(p.scale + n + 4));
      v[0] *= s0.x; v[1] *= s0.y; v[2] *= s0.z; v[3] *= s0.w;
      v[4] *= s1.x; v[5] *= s1.y; v[6] *= s1.z; v[7] *= s1.w;
    }
  } else if constexpr (EPI == SPV_EPI_BIAS_ADDROW) {
    const float* ar = p.addrow + (int64_t)(m % p.rows_per_image) * p.ldadd + n;
    const float4 a0 = __ldg(reinterpret_cast<const float4*>(ar));
    const float4 a1 = __ldg(reinterpret_cast<const float4*>(ar + 4));
    v[0] += a0.x; v[1] += a0.y; v[2] += a0.z; v[3] += a0.w;
    v[4] += a1.x; v[5] += a1.y; v[6] += a1.z; v[7] += a1.w;
  }
}

__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void named_bar_arrive(int id, int threads) {
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <int EPI, bool PAIR>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
                 const __grid_constant__ CUtensorMap tm_out, int M, int N, int K, EpiParams ep, uint32_t* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int STAGES = Ring<PAIR>::STAGES, B_BYTES = Ring<PAIR>::B_BYTES;
  uint8_t* sA = smem;
  uint8_t* sB = smem + STAGES * A_BYTES;
  uint8_t* sE = smem + STAGES * (A_BYTES + B_BYTES);     // [2] epilogue staging, 128-byte swizzle
  uint64_t* bars = reinterpret_cast<uint64_t*>(sE + 2 * EPI_BYTES);
  uint64_t* full = bars;                 // [STAGES]  TMA -> MMA
  uint64_t* empty = bars + STAGES;       // [STAGES]  MMA -> TMA
  uint64_t* acc_full = bars + 2 * STAGES;       // [2] MMA -> epilogue
  uint64_t* acc_empty = bars + 2 * STAGES + 2;  // [2] epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* s_bias = reinterpret_cast<float*>(bars + 32);     // [BN] bias of the tile in the epilogue

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // pair form: a tile is 256 rows, CTA `rank` of the pair owns rows [128 rank, 128 rank + 128) of it
  // and loads rows [128 rank, 128 rank + 128) of the tile's 256 rows of W; the workers are the pairs
  constexpr int TILE_M = PAIR ? 2 * BM : BM;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int m_tiles = (M + TILE_M - 1) / TILE_M, n_tiles = (N + BN - 1) / BN;
  const int tiles = m_tiles * n_tiles;
  const int kblocks = (K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    // pair form: the even CTA's MMA thread waits for the epilogues of both CTAs
    for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], PAIR ? 2 * EPI_THREADS : EPI_THREADS); }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if constexpr (PAIR) cluster_sync_all();      // both CTAs' barriers exist before anything remote touches them
  if (warp == 1) {
    if constexpr (PAIR) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
    else { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&tm_a);
      tma_prefetch_desc(&tm_w);
      uint32_t it = 0;
      for (int tile = worker; tile < tiles; tile += n_workers) {
        // column tile fastest: the CTAs running together share a few row tiles of A and all of W in L2,
        // so A crosses HBM once instead of once per column tile
        const int m0 = (tile / n_tiles) * TILE_M + (int)rank * BM, n0 = (tile % n_tiles) * BN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % STAGES;
          mbar_wait(&empty[s], ((it / STAGES) & 1) ^ 1, abort_flag, status, 0x100 + s);
          if constexpr (PAIR) {
            // the bytes of both CTAs are counted on the even CTA's barrier, which its producer arms
            if (rank == 0) mbar_expect_tx(&full[s], 2 * (A_BYTES + B_BYTES));
            const uint32_t bar = mapa_shared(smem_u32(&full[s]), 0);
            tma_load_2d_pair(sA + s * A_BYTES, &tm_a, bar, kb * BK, m0);
            tma_load_2d_pair(sB + s * B_BYTES, &tm_w, bar, kb * BK, n0 + (int)rank * (BN / 2));
          } else {
            mbar_expect_tx(&full[s], A_BYTES + B_BYTES);
            tma_load_2d(sA + s * A_BYTES, &tm_a, &full[s], kb * BK, m0);
            tma_load_2d(sB + s * B_BYTES, &tm_w, &full[s], kb * BK, n0);
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = idesc_bf16(TILE_M, BN, false);
      uint32_t it = 0, tcount = 0;
      for (int tile = worker; tile < tiles; tile += n_workers, ++tcount) {
        const int a = tcount & 1;
        mbar_wait(&acc_empty[a], ((tcount >> 1) & 1) ^ 1, abort_flag, status, 0x200 + a);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * BN;
        for (int kb = 0; kb < kblocks; ++kb, ++it) {
          const int s = it % STAGES;
          mbar_wait(&full[s], (it / STAGES) & 1, abort_flag, status, 0x300 + s);
          tc_fence_after();
          const uint64_t da = smem_desc_sw128(smem_u32(sA + s * A_BYTES));
          const uint64_t db = smem_desc_sw128(smem_u32(sB + s * B_BYTES));
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            if constexpr (PAIR) mma_ss_pair(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) != 0);
            else mma_ss(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (kb | k) != 0);
          }
          if constexpr (PAIR) tc_commit_pair(&empty[s], 3);      // frees the stage in both CTAs
          else tc_commit(&empty[s]);
        }
        if constexpr (PAIR) tc_commit_pair(&acc_full[a], 3);     // both CTAs' epilogues may read their half
        else tc_commit(&acc_full[a]);
      }
    }
  } else if (warp == STORE_WARP) {
    // Store warp: waits until the epilogue threads have written a staging buffer, hands it to TMA
    // (a plain tile store, or an fp32 add into the residual stream, so that the residual is never
    // read here and every global access is a whole 128-byte row segment), and gives the buffer
    // back once TMA has read it.  The epilogue threads never wait for one another, only for a buffer.
    constexpr int CW = epi_is_f32(EPI) ? 32 : 64;
    uint32_t ec = 0;
    for (int tile = worker; tile < tiles; tile += n_workers) {
      const int m_base = (tile / n_tiles) * TILE_M + (int)rank * BM, n_base = (tile % n_tiles) * BN;
#pragma unroll 1
      for (int c = 0; c < BN / CW; ++c, ++ec) {
        const int n0 = n_base + c * CW;
        if (n0 >= N) break;
        const int bsel = ec & 1;
        named_bar_sync(BAR_FULL + bsel, BAR_HANDOFF_THREADS);
        if (lane == 0) {
          if (m_base < M) {                  // (the odd CTA's half of the last row tile may lie past M)
            uint8_t* buf = sE + bsel * EPI_BYTES;
            if constexpr (EPI == SPV_EPI_BIAS_SCALE_RESID) tma_reduce_add_2d(&tm_out, buf, n0, m_base);
            else tma_store_2d(&tm_out, buf, n0, m_base);
            bulk_commit();
            bulk_wait_read<0>();
          }
        }
        __syncwarp();
        named_bar_arrive(BAR_EMPTY + bsel, BAR_HANDOFF_THREADS);
      }
    }
    if (lane == 0) bulk_wait<0>();
  } else {
    // Epilogue: thread = output row.  A chunk of columns (32 fp32 or 64 bf16 = 128 bytes per row)
    // goes TMEM -> registers -> arithmetic -> swizzled staging buffer.
    constexpr bool F32 = epi_is_f32(EPI);
    constexpr int CW = F32 ? 32 : 64;            // columns per chunk
    constexpr int TW = CW / 4;                   // columns per thread: four threads share a row
    const int q = warp & 3;                      // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;            // which quarter of the chunk's columns
    const int row = q * 32 + lane;
    uint32_t tcount = 0, ec = 0;
    const uint32_t acc_empty_remote = PAIR ? mapa_shared(smem_u32(&acc_empty[0]), 0) : 0u;
    for (int tile = worker; tile < tiles; tile += n_workers, ++tcount) {
      const int a = tcount & 1;
      const int m_base = (tile / n_tiles) * TILE_M + (int)rank * BM, n_base = (tile % n_tiles) * BN;
      const int m = m_base + row;
      // the tile's bias goes to shared memory while the main loop still runs: a global load per
      // chunk would sit (with its L2 latency) on the epilogue's critical path.  The barrier before
      // the fill waits for the slowest thread's last read of the previous tile's values, the one
      // after it publishes the new ones.
      if (ep.bias) {
        named_bar_sync(BAR_EPI, EPI_THREADS);
        const int tcol = threadIdx.x - 64;
        if (tcol < BN) s_bias[tcol] = n_base + tcol < N ? __ldg(ep.bias + n_base + tcol) : 0.f;
        named_bar_sync(BAR_EPI, EPI_THREADS);
      }
      mbar_wait(&acc_full[a], (tcount >> 1) & 1, abort_flag, status, 0x400 + a);
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN;
#pragma unroll 1
      for (int c = 0; c < BN / CW; ++c, ++ec) {
        const int n0 = n_base + c * CW;
        if (n0 >= N) break;
        uint8_t* buf = sE + (ec & 1) * EPI_BYTES;
        uint32_t acc[TW];
        if constexpr (F32) tmem_ld8(taddr + c * CW + half * TW, acc);
        else tmem_ld16(taddr + c * CW + half * TW, acc);
        tc_wait_ld();
        uint4 o[TW / (F32 ? 4 : 8)];             // this thread's share of the staged row
#pragma unroll
        for (int g = 0; g < TW / 8; ++g) {
          float v[8];
          const int n = n0 + half * TW + 8 * g;
          // rows past M hold zeros (TMA fills them on load) and are clipped by TMA on store, so only
          // the epilogue that addresses global memory by row needs the per-lane row guard; without
          // it the groups are straight-line code and their dependency chains interleave
          if ((EPI != SPV_EPI_BIAS_MUL || m < M) && n < N) {
            epilogue_math<EPI>(ep, s_bias, n_base, m, n, acc + 8 * g, v);
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = 0.f;
          }
          if constexpr (F32) {
            o[2 * g] = make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
            o[2 * g + 1] = make_uint4(__float_as_uint(v[4]), __float_as_uint(v[5]), __float_as_uint(v[6]), __float_as_uint(v[7]));
          } else {
            o[g] = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
          }
        }
        // the arithmetic is done before the buffer is needed: TMA has read its previous contents
        if (ec >= 2) named_bar_sync(BAR_EMPTY + (ec & 1), BAR_HANDOFF_THREADS);
#pragma unroll
        for (int j = 0; j < 2; ++j)
          *reinterpret_cast<uint4*>(buf + row * 128 + (((2 * half + j) ^ (row & 7)) << 4)) = o[j];
        fence_async_smem();
        named_bar_arrive(BAR_FULL + (ec & 1), BAR_HANDOFF_THREADS);
      }
      tc_fence_before();
      if constexpr (PAIR) mbar_arrive_cluster(acc_empty_remote + 8u * (uint32_t)a);
      else mbar_arrive(&acc_empty[a]);
    }
    // take the store warp's last hand-backs, so that no barrier is left half way at exit
    if (ec >= 2) named_bar_sync(BAR_EMPTY + (ec & 1), BAR_HANDOFF_THREADS);
    if (ec >= 1) named_bar_sync(BAR_EMPTY + ((ec - 1) & 1), BAR_HANDOFF_THREADS);
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();      // neither CTA frees TMEM or leaves while the other may still signal it
  tc_fence_after();
  if (warp == 1) {
    if constexpr (PAIR) tmem_dealloc_pair(tmem_base, 512);
    else tmem_dealloc(tmem_base, 512);
  }
}

// the pair form pays off once a problem has more than one 256-row tile
inline bool use_pair(const spv_gemm_desc* d) { return d->m > 2 * BM; }

template <int EPI>
int32_t launch(spv_ctx* ctx, const CUtensorMap& ta, const CUtensorMap& tw, const spv_gemm_desc* d, const EpiParams& ep,
               cudaStream_t stream) {
  CUtensorMap tout;
  {
    const uint64_t dims[2] = {(uint64_t)d->n, (uint64_t)d->m};
    int32_t st;
    if (epi_is_f32(EPI)) {
      const uint64_t str[1] = {(uint64_t)d->ldo * 4};
      const uint32_t box[2] = {32, BM};
      st = spv_make_tmap_f32(ctx, &tout, ep.out, 2, dims, str, box);
    } else {
      const uint64_t str[1] = {(uint64_t)d->ldo * 2};
      const uint32_t box[2] = {64, BM};
      st = spv_make_tmap_bf16(ctx, &tout, ep.out, 2, dims, str, box);
    }
    if (st != SPV_OK) return st;
  }
  SpvProfScope prof(ctx, SPV_K_GEMM, stream, 2.0 * (double)d->m * (double)d->n * (double)d->k);
  const int n_tiles = (d->n + BN - 1) / BN;
  if (use_pair(d)) {
    // pair form: clusters of two CTAs, as many as can be resident at once
    static_assert(EPI >= 0 && EPI < 8, "per-context launch state is indexed by the epilogue variant");
    int& max_pairs = ctx->gemm_max_pairs[EPI];
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = GEMM_SMEM;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (max_pairs == 0) {
      SPV_CUDA_OK(cudaFuncSetAttribute(gemm_bf16_kernel<EPI, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM));
      cfg.gridDim = dim3(2 * (ctx->sm_count / 2));
      int n = 0;
      SPV_CUDA_OK(cudaOccupancyMaxActiveClusters(&n, gemm_bf16_kernel<EPI, true>, &cfg));
      if (n < 1) return SPV_ERR_CUDA;
      max_pairs = n < ctx->sm_count / 2 ? n : ctx->sm_count / 2;
    }
    const int tiles = ((d->m + 2 * BM - 1) / (2 * BM)) * n_tiles;
    cfg.gridDim = dim3(2 * (tiles < max_pairs ? tiles : max_pairs));
    SPV_CUDA_OK(cudaLaunchKernelEx(&cfg, gemm_bf16_kernel<EPI, true>, ta, tw, tout, d->m, d->n, d->k, ep, ctx->d_status));
    return spv_launch_ok(ctx);
  }
  if (!ctx->gemm_single_configured[EPI]) {
    SPV_CUDA_OK(cudaFuncSetAttribute(gemm_bf16_kernel<EPI, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM));
    ctx->gemm_single_configured[EPI] = 1;
  }
  const int tiles = ((d->m + BM - 1) / BM) * n_tiles;
  const int grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
  gemm_bf16_kernel<EPI, false><<<grid, GEMM_THREADS, GEMM_SMEM, stream>>>(ta, tw, tout, d->m, d->n, d->k, ep, ctx->d_status);
  return spv_launch_ok(ctx);
}

}  // namespace

extern "C" int32_t spv_gemm_bf16(spv_ctx* ctx, const spv_gemm_desc* d, const void* a, const void* w, void* out,
                                 void* stream_) {
  if (!ctx || !d || !a || !w || !out) return SPV_ERR_INVALID_ARG;
  if (spv_on_device(ctx) != SPV_OK) return SPV_ERR_INVALID_ARG;
  if (d->m < 1 || d->n < 1 || d->k < 1) return SPV_ERR_INVALID_ARG;
  if (d->k % 8 || d->n % 8 || d->lda % 8 || d->ldw % 8 || d->ldo % 8) return SPV_ERR_ALIGNMENT;
  if (d->lda < d->k || d->ldw < d->k || d->ldo < d->n) return SPV_ERR_INVALID_ARG;
  if (((uintptr_t)out & 15u) || ((uintptr_t)d->bias & 15u)) return SPV_ERR_ALIGNMENT;
  EpiParams ep;
  ep.out = out; ep.ldo = d->ldo; ep.bias = d->bias; ep.aux = d->aux; ep.ldaux = d->ldaux;
  ep.scale = d->scale; ep.addrow = d->addrow; ep.ldadd = d->ldadd; ep.rows_per_image = d->rows_per_image;
  if (d->epilogue == SPV_EPI_BIAS_MUL && (!d->aux || d->ldaux % 8 || ((uintptr_t)d->aux & 15u)))
    return SPV_ERR_INVALID_ARG;
  if (d->epilogue == SPV_EPI_BIAS_ADDROW && (!d->addrow || d->rows_per_image < 1 || d->ldadd % 4))
    return SPV_ERR_INVALID_ARG;
  CUtensorMap ta, tw;
  {
    const uint64_t dims[2] = {(uint64_t)d->k, (uint64_t)d->m};
    const uint64_t str[1] = {(uint64_t)d->lda * 2};
    const uint32_t box[2] = {BK, BM};
    int32_t st = spv_make_tmap_bf16(ctx, &ta, a, 2, dims, str, box);
    if (st != SPV_OK) return st;
  }
  {
    const uint64_t dims[2] = {(uint64_t)d->k, (uint64_t)d->n};
    const uint64_t str[1] = {(uint64_t)d->ldw * 2};
    const uint32_t box[2] = {BK, (uint32_t)(use_pair(d) ? BN / 2 : BN)};
    int32_t st = spv_make_tmap_bf16(ctx, &tw, w, 2, dims, str, box);
    if (st != SPV_OK) return st;
  }
  cudaStream_t stream = (cudaStream_t)stream_;
  switch (d->epilogue) {
    case SPV_EPI_BIAS: return launch<SPV_EPI_BIAS>(ctx, ta, tw, d, ep, stream);
    case SPV_EPI_BIAS_GELU: return launch<SPV_EPI_BIAS_GELU>(ctx, ta, tw, d, ep, stream);
    case SPV_EPI_BIAS_SILU: return launch<SPV_EPI_BIAS_SILU>(ctx, ta, tw, d, ep, stream);
    case SPV_EPI_BIAS_MUL: return launch<SPV_EPI_BIAS_MUL>(ctx, ta, tw, d, ep, stream);
    case SPV_EPI_BIAS_SCALE_RESID: return launch<SPV_EPI_BIAS_SCALE_RESID>(ctx, ta, tw, d, ep, stream);
    case SPV_EPI_BIAS_ADDROW: return launch<SPV_EPI_BIAS_ADDROW>(ctx, ta, tw, d, ep, stream);
    default: return SPV_ERR_INVALID_ARG;
  }
}
