// LayerNorm over fp32 residual rows, bf16 output (pre-LN of every ViT block and the final norm).
// One warp per row, 128-bit loads, the row kept in registers between the statistics and the
// normalisation, so each element crosses HBM once in (4 B) and once out (2 B).  The grid is
// persistent (as many CTAs as are resident at once) and every warp issues the loads of its next
// row before it reduces, normalises and stores the current one, so loads stay in flight the
// whole time.
#include "common.cuh"

namespace {

// kMaxVec float4 per lane are held in registers for the current row and as many for the next one
// (dim <= 128 * kMaxVec); the instantiation that just covers the row keeps the register count low,
// so that two CTAs fit an SM up to dim 1024.
template <int kMaxVec>
__global__ void __launch_bounds__(256, (kMaxVec <= 8 ? 2 : 1)) layernorm_kernel(const float* __restrict__ x, int64_t rows, int dim,
                                                        const float* __restrict__ gamma,
                                                        const float* __restrict__ beta, float eps,
                                                        __nv_bfloat16* __restrict__ y,
                                                        const int32_t* __restrict__ out_row) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
  const int nvec = dim >> 2;
  const float inv_dim = 1.0f / (float)dim;
  float4 nxt[kMaxVec];          // the row after the current one, in flight
  if (warp < rows) {
    const float4* xr0 = reinterpret_cast<const float4*>(x + warp * dim);
#pragma unroll
    for (int i = 0; i < kMaxVec; ++i) {
      const int c = lane + 32 * i;
      if (c < nvec) nxt[i] = __ldcs(xr0 + c);
    }
  }
  for (int64_t r = warp; r < rows; r += nwarps) {
    const float4* xr = reinterpret_cast<const float4*>(x + r * dim);
    float4 v[kMaxVec];
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < kMaxVec; ++i) {
      const int c = lane + 32 * i;
      if (c < nvec) {
        v[i] = nxt[i];
        sum += (v[i].x + v[i].y) + (v[i].z + v[i].w);
      }
    }
    if (r + nwarps < rows) {
      const float4* xn = reinterpret_cast<const float4*>(x + (r + nwarps) * dim);
#pragma unroll
      for (int i = 0; i < kMaxVec; ++i) {
        const int c = lane + 32 * i;
        if (c < nvec) nxt[i] = __ldcs(xn + c);
      }
    }
    for (int c = lane + 32 * kMaxVec; c < nvec; c += 32) {
      const float4 t = xr[c];
      sum += (t.x + t.y) + (t.z + t.w);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float mean = sum * inv_dim;
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < kMaxVec; ++i) {
      const int c = lane + 32 * i;
      if (c < nvec) {
        const float a = v[i].x - mean, b = v[i].y - mean, cc = v[i].z - mean, d = v[i].w - mean;
        sq += (a * a + b * b) + (cc * cc + d * d);
      }
    }
    for (int c = lane + 32 * kMaxVec; c < nvec; c += 32) {
      const float4 t = xr[c];
      const float a = t.x - mean, b = t.y - mean, cc = t.z - mean, d = t.w - mean;
      sq += (a * a + b * b) + (cc * cc + d * d);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    const float rstd = rsqrtf(sq * inv_dim + eps);
    const int64_t orow = out_row ? (int64_t)__ldg(out_row + r) : r;
    uint2* yr = reinterpret_cast<uint2*>(y + orow * dim);
    const float4* g4 = reinterpret_cast<const float4*>(gamma);
    const float4* b4 = reinterpret_cast<const float4*>(beta);
#pragma unroll
    for (int i = 0; i < kMaxVec; ++i) {
      const int c = lane + 32 * i;
      if (c < nvec) {
        const float4 g = __ldg(g4 + c), b = __ldg(b4 + c);
        uint2 o;
        o.x = spv::pack_bf16((v[i].x - mean) * rstd * g.x + b.x, (v[i].y - mean) * rstd * g.y + b.y);
        o.y = spv::pack_bf16((v[i].z - mean) * rstd * g.z + b.z, (v[i].w - mean) * rstd * g.w + b.w);
        yr[c] = o;
      }
    }
    for (int c = lane + 32 * kMaxVec; c < nvec; c += 32) {
      const float4 t = xr[c];
      const float4 g = __ldg(g4 + c), b = __ldg(b4 + c);
      uint2 o;
      o.x = spv::pack_bf16((t.x - mean) * rstd * g.x + b.x, (t.y - mean) * rstd * g.y + b.y);
      o.y = spv::pack_bf16((t.z - mean) * rstd * g.z + b.z, (t.w - mean) * rstd * g.w + b.w);
      yr[c] = o;
    }
  }
}

}  // namespace

extern "C" int32_t spv_layernorm(spv_ctx* ctx, const float* x, int64_t rows, int32_t dim, const float* gamma,
                                 const float* beta, float eps, void* y, const int32_t* out_row, void* stream) {
  if (!ctx || !x || !gamma || !beta || !y || rows < 1 || dim < 8) return SPV_ERR_INVALID_ARG;
  if (spv_on_device(ctx) != SPV_OK) return SPV_ERR_INVALID_ARG;
  if (dim % 8) return SPV_ERR_ALIGNMENT;
  if (((uintptr_t)x & 15u) || ((uintptr_t)y & 15u) || ((uintptr_t)gamma & 15u) || ((uintptr_t)beta & 15u))
    return SPV_ERR_ALIGNMENT;
  int64_t blocks = (rows + 7) / 8;
  const int64_t cap = (int64_t)ctx->sm_count * (dim <= 1024 ? 2 : 1);     // resident CTAs (see __launch_bounds__)
  if (blocks > cap) blocks = cap;
  SpvProfScope prof(ctx, SPV_K_LAYERNORM, (cudaStream_t)stream, (double)rows * dim * 6.0);
  const unsigned g = (unsigned)blocks;
  cudaStream_t st = (cudaStream_t)stream;
  __nv_bfloat16* yo = (__nv_bfloat16*)y;
  if (dim <= 512) layernorm_kernel<4><<<g, 256, 0, st>>>(x, rows, dim, gamma, beta, eps, yo, out_row);
  else if (dim <= 1024) layernorm_kernel<8><<<g, 256, 0, st>>>(x, rows, dim, gamma, beta, eps, yo, out_row);
  else if (dim <= 1536) layernorm_kernel<12><<<g, 256, 0, st>>>(x, rows, dim, gamma, beta, eps, yo, out_row);
  else layernorm_kernel<16><<<g, 256, 0, st>>>(x, rows, dim, gamma, beta, eps, yo, out_row);
  return spv_launch_ok(ctx);
}
