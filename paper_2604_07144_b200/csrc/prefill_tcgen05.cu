// Prefill-chunk attention (placeholder until the tcgen05 kernel lands).
#include "internal.h"

namespace ap {

cudaError_t launch_prefill(const ap_kv_pool *, const ap_plan *, const void *, void *, float *, cudaStream_t) {
    return cudaErrorNotSupported;
}

}  // namespace ap
