// Chunked prefill against the paged cache (Eq. 1 with causal K_{<=t}); placeholder launcher
// until the tensor-core tile kernel lands.
#include "coopt_common.cuh"

namespace coopt {

int launch_paged_prefill(const coopt_cache*, const void*, void*, const int32_t*, const int32_t*, int32_t,
                         const int32_t*, int32_t, int32_t, int32_t, int32_t, float, void*, cudaStream_t) {
  return COOPT_ERR_UNSUPPORTED;
}

}  // namespace coopt
