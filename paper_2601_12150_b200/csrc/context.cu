// Context, status codes and tensor-map construction (host side of libspatvit).
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "common.cuh"

extern "C" int32_t spv_create(spv_ctx** out, int32_t device) {
  if (!out || device < 0) return SPV_ERR_INVALID_ARG;
  *out = nullptr;
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || device >= n) return SPV_ERR_CUDA;
  SPV_CUDA_OK(cudaSetDevice(device));
  cudaDeviceProp prop;
  SPV_CUDA_OK(cudaGetDeviceProperties(&prop, device));
  if (prop.major != 10) return SPV_ERR_UNSUPPORTED;   // sm_100a code only
  spv_ctx* c = (spv_ctx*)calloc(1, sizeof(spv_ctx));
  if (!c) return SPV_ERR_CUDA;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  if (cudaMalloc((void**)&c->d_status, 256) != cudaSuccess) { free(c); return SPV_ERR_CUDA; }
  if (cudaMemset(c->d_status, 0, 256) != cudaSuccess) { cudaFree(c->d_status); free(c); return SPV_ERR_CUDA; }
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    cudaFree(c->d_status);
    free(c);
    return SPV_ERR_CUDA;
  }
  c->encode_tiled = (spv_encode_tiled_fn)fn;
  *out = c;
  return SPV_OK;
}

// ---- per-class event timing ------------------------------------------------------------------
struct SpvProfRec { cudaEvent_t e0, e1; int32_t cls; double work; };
struct SpvProf {
  std::vector<SpvProfRec> recs;        // event pairs, reused after every read
  size_t used = 0;
};

int32_t spv_prof_begin(spv_ctx* ctx, int32_t cls, cudaStream_t stream) {
  SpvProf* p = ctx->prof;
  if (!p) return -1;
  if (p->used == p->recs.size()) {
    SpvProfRec r{};
    if (cudaEventCreate(&r.e0) != cudaSuccess || cudaEventCreate(&r.e1) != cudaSuccess) return -1;
    p->recs.push_back(r);
  }
  SpvProfRec& r = p->recs[p->used];
  r.cls = cls;
  r.work = 0.0;
  if (cudaEventRecord(r.e0, stream) != cudaSuccess) return -1;
  return (int32_t)p->used++;
}

void spv_prof_end(spv_ctx* ctx, int32_t token, cudaStream_t stream, double work) {
  SpvProfRec& r = ctx->prof->recs[(size_t)token];
  r.work = work;
  cudaEventRecord(r.e1, stream);
}

extern "C" int32_t spv_profile_enable(spv_ctx* ctx, int32_t enable) {
  if (!ctx) return SPV_ERR_INVALID_ARG;
  if (enable && !ctx->prof) ctx->prof = new SpvProf();
  if (ctx->prof) ctx->prof->used = 0;
  ctx->prof_on = enable ? 1 : 0;
  return SPV_OK;
}

extern "C" int32_t spv_profile_read(spv_ctx* ctx, spv_kernel_stat* out) {
  if (!ctx || !out) return SPV_ERR_INVALID_ARG;
  SpvProf* p = ctx->prof;
  if (!p) return SPV_OK;
  for (size_t i = 0; i < p->used; ++i) {
    SpvProfRec& r = p->recs[i];
    SPV_CUDA_OK(cudaEventSynchronize(r.e1));
    float ms = 0.f;
    SPV_CUDA_OK(cudaEventElapsedTime(&ms, r.e0, r.e1));
    if (r.cls >= 0 && r.cls < SPV_K_COUNT) {
      out[r.cls].launches += 1;
      out[r.cls].ms += (double)ms;
      out[r.cls].work += r.work;
    }
  }
  p->used = 0;
  return SPV_OK;
}

extern "C" int32_t spv_destroy(spv_ctx* ctx) {
  if (!ctx) return SPV_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  if (ctx->prof) {
    for (SpvProfRec& r : ctx->prof->recs) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
    delete ctx->prof;
  }
  cudaFree(ctx->d_status);
  free(ctx);
  return SPV_OK;
}

extern "C" const char* spv_status_string(int32_t s) {
  switch (s) {
    case SPV_OK: return "ok";
    case SPV_ERR_INVALID_ARG: return "invalid argument";
    case SPV_ERR_UNSUPPORTED: return "unsupported configuration or device";
    case SPV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case SPV_ERR_CUDA: return "CUDA call failed";
    case SPV_ERR_TIMEOUT: return "bounded device-side wait expired";
    case SPV_ERR_ALIGNMENT: return "tensor base or stride not 16-byte aligned";
    case SPV_ERR_STATIC_LIMIT: return "request exceeds the built-in static scratch array";
    default: return "unknown status";
  }
}

extern "C" int32_t spv_check(spv_ctx* ctx, void* stream) {
  if (!ctx) return SPV_ERR_INVALID_ARG;
  SPV_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  uint32_t st[2] = {0, 0};
  SPV_CUDA_OK(cudaMemcpy(st, ctx->d_status, sizeof(st), cudaMemcpyDeviceToHost));
  if (st[0] != 0 || st[1] != 0) {
    ctx->last_site = st[0] != 0 ? st[0] : st[1];
    cudaMemset(ctx->d_status, 0, sizeof(st));
    return st[0] != 0 ? SPV_ERR_TIMEOUT : SPV_ERR_INVALID_ARG;
  }
  return SPV_OK;
}

// One thread waits on a barrier that gets no arrival, for at most limit_ns: the same parked try_wait and the
// same latch as the kernels' bounded waits, with the limit as an argument.
__global__ void selftest_wait_kernel(uint32_t limit_ns, uint32_t* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    spv::mbar_init(&bar, 1);
    spv::mbar_fence_init();
    uint32_t t0, t;
    asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t0));
    bool done = false;
    do {
      done = spv::mbar_try_wait_parked(&bar, 0, 1000u);
      asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t));
    } while (!done && t - t0 <= limit_ns);
    if (!done) atomicCAS(status, 0u, 0x5E1Fu);
  }
}

extern "C" int32_t spv_selftest_wait(spv_ctx* ctx, uint32_t limit_ns, void* stream) {
  if (!ctx) return SPV_ERR_INVALID_ARG;
  if (spv_on_device(ctx) != SPV_OK) return SPV_ERR_INVALID_ARG;
  if (limit_ns > 1000000u) limit_ns = 1000000u;
  selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(limit_ns, ctx->d_status);
  return spv_launch_ok(ctx);
}

extern "C" uint32_t spv_last_wait_site(const spv_ctx* ctx) { return ctx ? ctx->last_site : 0u; }

extern "C" int64_t spv_launch_count(const spv_ctx* ctx) { return ctx ? ctx->launches : 0; }

static int32_t make_tmap(spv_ctx* ctx, CUtensorMap* map, CUtensorMapDataType dtype, const void* base, int rank,
                         const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box) {
  if (((uintptr_t)base & 15u) != 0) return SPV_ERR_ALIGNMENT;
  cuuint64_t gdim[5];
  cuuint64_t gstr[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) {
    gdim[i] = dims[i];
    bx[i] = box[i];
    es[i] = 1;
    if (i > 0) {
      if (strides_bytes[i - 1] % 16 != 0) return SPV_ERR_ALIGNMENT;
      gstr[i - 1] = strides_bytes[i - 1];
    }
  }
  CUresult r = ctx->encode_tiled(map, dtype, (cuuint32_t)rank, (void*)base, gdim, gstr, bx, es,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SPV_OK : SPV_ERR_CUDA;
}

int32_t spv_make_tmap_bf16(spv_ctx* ctx, CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                           const uint64_t* strides_bytes, const uint32_t* box) {
  return make_tmap(ctx, map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, base, rank, dims, strides_bytes, box);
}

int32_t spv_make_tmap_f32(spv_ctx* ctx, CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                          const uint64_t* strides_bytes, const uint32_t* box) {
  return make_tmap(ctx, map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, base, rank, dims, strides_bytes, box);
}
