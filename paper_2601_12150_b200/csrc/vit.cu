#include "common.cuh"
extern "C" int32_t spv_vit_workspace_size(const spv_vit_config*, int32_t, int32_t, int32_t, size_t*) { return SPV_ERR_UNSUPPORTED; }
extern "C" int32_t vit_forward(spv_ctx*, const spv_vit_config*, const spv_vit_weights*, const float*, int32_t, int32_t,
                               int32_t, void*, int32_t*, const int32_t*, void*, size_t, void*) { return SPV_ERR_UNSUPPORTED; }
