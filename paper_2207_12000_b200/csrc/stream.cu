// Streaming pipeline for operands that live in host memory.
#include "gnnpre_internal.cuh"

namespace gnnpre {

int propagate_streamed(gnnpre_plan*, const float*, int64_t, int32_t, int32_t, float* const*, int64_t, int32_t,
                       cudaStream_t, gnnpre_stats_t*) {
    return GNNPRE_ERR_INVALID_ARG;
}

}  // namespace gnnpre
