// Head-similarity profiling (Algorithm 1, step 1).  Placeholder translation unit: the entry
// points exist so that the ABI is complete; the kernel is added separately.
#include <cuda_runtime.h>

#include "baklava.h"
#include "common.h"

extern "C" __attribute__((visibility("default"))) size_t baklava_profile_workspace_size(const baklava_shape* shape, int32_t P, int32_t T) {
    if (!shape || P <= 0 || T <= 0) return 0;
    return 256;
}

extern "C" __attribute__((visibility("default"))) int baklava_profile_heads(const baklava_shape* shape, const void* q, const void* k, const void* v,
                                     const int32_t* prompt_len, int32_t P, int32_t T,
                                     float* head_cos, float* token_cos, void* ws, size_t ws_bytes, void* stream) {
    (void)q; (void)k; (void)v; (void)prompt_len; (void)P; (void)T; (void)head_cos; (void)token_cos;
    (void)ws; (void)ws_bytes; (void)stream;
    int rc = baklava_check_shape(shape);
    if (rc) return rc;
    return BAKLAVA_ERR_UNSUPPORTED;
}
