// Routed execution (Section 5.5): the routes are compacted and grouped by matrix so that every decoded weight
// tile serves all routes of its matrix.  This file holds the one kernel that is specific to it: the gather of
// the routed token rows into matrix-major order.  The products themselves are the ordinary kernels, one dispatch
// per matrix that has routes (cq_gemm_routed in cq_api.cu).
#include "cq_common.cuh"
#include "cq_internal.h"

namespace cq {

// xg[r][:] = x[route_token[r]][:] for r < R; 16-byte chunks when K is a multiple of 8, else element by element.
// A route whose token index lies outside [0, T) gets a zero row (the caller owns the map; nothing is read out of range).
__global__ void __launch_bounds__(256) gather_rows_kernel(const uint16_t *__restrict__ x, const int32_t *__restrict__ route_token,
                                                         uint16_t *__restrict__ xg, int64_t R, int64_t T, int64_t K, bool wide) {
    const int64_t r = blockIdx.x;
    if (r >= R) return;
    const int64_t t = route_token[r];
    const bool ok = t >= 0 && t < T;
    if (wide) {
        const uint4 *src = reinterpret_cast<const uint4 *>(x + (ok ? t : 0) * K);
        uint4 *dst = reinterpret_cast<uint4 *>(xg + r * K);
        for (int64_t c = threadIdx.x; c < (K >> 3); c += blockDim.x) dst[c] = ok ? src[c] : make_uint4(0, 0, 0, 0);
    } else {
        for (int64_t c = threadIdx.x; c < K; c += blockDim.x) xg[r * K + c] = ok ? x[t * K + c] : (uint16_t)0;
    }
}

cudaError_t launch_gather_rows(const uint16_t *x, const int32_t *route_token, uint16_t *xg, int64_t R, int64_t T, int64_t K,
                               cudaStream_t st) {
    const bool wide = K % 8 == 0 && ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(xg)) & 15u) == 0;
    gather_rows_kernel<<<(unsigned)R, 256, 0, st>>>(x, route_token, xg, R, T, K, wide);
    return cudaGetLastError();
}

}  // namespace cq
