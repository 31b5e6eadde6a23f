// cq_gemv_static: the small-M product for callers that may not allocate device memory.
//
// The split-K GEMV needs a little scratch (arrival counters and partial sums).  cq_gemm takes it
// from a caller-provided workspace; this entry point takes it from a fixed array that is part of
// the library image instead, so the caller passes only inputs and outputs.
#include "../../include/cubicquant.h"

#include <cuda_runtime.h>

#include <atomic>

#include "cq_common.cuh"
#include "cq_internal.h"

namespace {

constexpr size_t STATIC_SCRATCH_BYTES = CQ_STATIC_SCRATCH_BYTES;
constexpr int MAX_DEVICES = 64;

// Lives in every GPU's memory from the moment the library is loaded there until the process exits.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

// device address of g_static_scratch on each device, filled in by the first call on that device
// (atomic: host threads may make their first calls at the same time; they all store the same address)
std::atomic<unsigned char *> g_scratch_ptr[MAX_DEVICES];

// a failed CUDA call: remember its code for cq_last_cuda_error() and report CQ_ERR_CUDA
int cuda_failed(cudaError_t e) {
    cq::set_last_cuda_error(e);
    return CQ_ERR_CUDA;
}

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
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_failed(e);
    if (dev < 0 || dev >= MAX_DEVICES) return CQ_ERR_UNSUPPORTED;
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_failed(e);
    if (major != 10) return CQ_ERR_ARCH;
    unsigned char *ws = g_scratch_ptr[dev].load(std::memory_order_acquire);
    if (!ws) {
        // one-time set-up for this device (it is the current device): resolve the array's device address
        e = cudaGetSymbolAddress((void **)&ws, g_static_scratch);
        if (e != cudaSuccess) return cuda_failed(e);
        if (!ws) return cuda_failed(cudaErrorInvalidSymbol);
        g_scratch_ptr[dev].store(ws, std::memory_order_release);
    }
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the arrival counters and the status word must start at zero
    e = cudaMemsetAsync(ws + plan.status_off, 0, 256, st);
    if (e != cudaSuccess) return cuda_failed(e);
    e = cudaMemsetAsync(ws + plan.counters_off, 0, plan.counters_bytes, st);
    if (e != cudaSuccess) return cuda_failed(e);
    e = launch_gemv(layout, d, x, y, M, CQ_MODEL_DTYPE, false, ws, plan, st);
    return e == cudaSuccess ? CQ_OK : cuda_failed(e);
}
#pragma GCC visibility pop
