// Tensor-core path (placeholder until the kernels land): reports "unsupported" so that
// dispatch uses the generic kernel.
#include "harp_internal.h"

harp_status_t harp_fast_build(harp_plan *plan) { (void)plan; return HARP_ERR_UNSUPPORTED; }
void harp_fast_destroy(harp_plan *plan) { (void)plan; }
harp_status_t harp_fast_apply(const harp_plan *, void *, int64_t, harp_dtype_t, int, cudaStream_t) {
    return HARP_ERR_UNSUPPORTED;
}
