// cq_gemv_static: the small-M product for callers that may not allocate device memory.
//
// The split-K GEMV needs a little scratch (arrival counters and partial sums).  cq_gemm takes it
// from a caller-provided workspace; this entry point takes it from a fixed array that is part of
// the library image instead, so the caller passes only inputs and outputs.
#include "../../include/cubicquant.h"

#include <cuda_runtime.h>

#include "cq_common.cuh"
#include "cq_internal.h"

namespace {

constexpr size_t STATIC_SCRATCH_BYTES = CQ_STATIC_SCRATCH_BYTES;
constexpr int MAX_DEVICES = 64;

// Lives in every GPU's memory from the moment the library is loaded there until the process exits.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

// device address of g_static_scratch on each device, filled in by the first call on that device
unsigned char *g_scratch_ptr[MAX_DEVICES] = {};

}  // namespace

#pragma GCC visibility push(default)
extern "C" int cq_gemv_static(const void *layout, int B, int G, const uint16_t *x, uint16_t *y, int64_t M, int64_t N,
                              int64_t K, void *stream) {
    using namespace cq;
    if (!layout || !x || !y || M <= 0 || N <= 0 || K <= 0 || B < 1 || B > 8) return CQ_ERR_INVALID_ARG;
    if ((G != 32 && G != 64 && G != 128 && G != 256 && G != 512) || K % G != 0 || M > 16) return CQ_ERR_UNSUPPORTED;
    if (((uintptr_t)layout | (uintptr_t)x | (uintptr_t)y) & 15u) return CQ_ERR_ALIGNMENT;
    const Dims d = make_dims(B, G, N, K);
    const Workspace plan = plan_workspace(d, M, CQ_MODEL_DTYPE);
    if (plan.total > STATIC_SCRATCH_BYTES) return CQ_ERR_WORKSPACE;  // problem too large for the built-in scratch

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return CQ_ERR_CUDA;
    if (dev < 0 || dev >= MAX_DEVICES) return CQ_ERR_UNSUPPORTED;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return CQ_ERR_CUDA;
    if (major != 10) return CQ_ERR_ARCH;
    if (!g_scratch_ptr[dev]) {
        // one-time set-up for this device (it is the current device): resolve the array's device address
        unsigned char *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_static_scratch) != cudaSuccess || !p) return CQ_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    unsigned char *ws = g_scratch_ptr[dev];
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the arrival counters must start at zero
    if (cudaMemsetAsync(ws + plan.counters_off, 0, plan.counters_bytes, st) != cudaSuccess) return CQ_ERR_CUDA;
    return launch_gemv(layout, d, x, y, M, CQ_MODEL_DTYPE, ws, plan, st) == cudaSuccess ? CQ_OK : CQ_ERR_CUDA;
}
#pragma GCC visibility pop
