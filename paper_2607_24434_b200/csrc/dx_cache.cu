// Accelerator expert cache (Sec. 3.5, Algorithm 1: cache C, in-flight set P).
#include "dx_internal.cuh"

const void** dx_cache_table(dx_cache*, int) { return nullptr; }
void dx_cache_note_use(dx_cache*, int, cudaStream_t) {}

extern "C" dx_status dx_layer_attach_cache(dx_layer*, dx_cache*, int32_t) { return DX_ERR_UNSUPPORTED; }
extern "C" dx_status expert_cache_create(dx_ctx*, int32_t, int32_t, int32_t, size_t, dx_cache**) { return DX_ERR_UNSUPPORTED; }
extern "C" dx_status expert_cache_destroy(dx_cache*) { return DX_ERR_UNSUPPORTED; }
extern "C" dx_status expert_cache_register(dx_cache*, int32_t, int32_t, const void*) { return DX_ERR_UNSUPPORTED; }
extern "C" dx_status expert_cache_prefetch(dx_cache*, int32_t, const int32_t*, int32_t) { return DX_ERR_UNSUPPORTED; }
extern "C" dx_status expert_cache_stage(dx_cache*, int32_t, const int32_t*, int32_t, void*) { return DX_ERR_UNSUPPORTED; }
extern "C" dx_status expert_cache_wait(dx_cache*, int32_t, const int32_t*, int32_t, void*, double) { return DX_ERR_UNSUPPORTED; }
extern "C" dx_status expert_cache_stats(dx_cache*, dx_cache_stats*) { return DX_ERR_UNSUPPORTED; }
extern "C" dx_status expert_cache_query(dx_cache*, int32_t, int32_t, int32_t*, int32_t*) { return DX_ERR_UNSUPPORTED; }
