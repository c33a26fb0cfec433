#include "common.cuh"
extern "C" int32_t spv_attn_workspace_size(const spv_attn_desc*, size_t*) { return SPV_ERR_UNSUPPORTED; }
extern "C" int32_t spatial_block_attention(spv_ctx*, const spv_attn_desc*, const void*, const void*, const void*,
                                           void*, float*, void*, size_t, void*) { return SPV_ERR_UNSUPPORTED; }
