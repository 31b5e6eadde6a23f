// Large-M tcgen05 / TMEM GEMM (placeholder translation unit until the kernel lands).
#include "cq_common.cuh"
#include "cq_internal.h"

namespace cq {

int gemm_tc_available() { return 0; }

cudaError_t launch_gemm_tc(const void *, const Dims &, const uint16_t *, uint16_t *, int64_t, int, uint8_t *,
                           const Workspace &, cudaStream_t) {
    return cudaErrorNotSupported;
}

}  // namespace cq
