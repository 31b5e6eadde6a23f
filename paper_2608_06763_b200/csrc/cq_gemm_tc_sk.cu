// Stream-K instantiations of the model-dtype tcgen05 GEMM (Section 5.3 dense path): the kernels that also run
// tiles shared by several CTAs.  See cq_gemm_tc_impl.cuh.
#include "cq_gemm_tc_impl.cuh"

namespace cq {

cudaError_t launch_gemm_tc_streamk(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int *status,
                                   float *partial, int *counters, bool act_f16, cudaStream_t st) {
    return launch_tc_variant<true>(layout, d, x, y, M, status, partial, counters, act_f16, st);
}

}  // namespace cq
