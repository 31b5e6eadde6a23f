// Internal launcher declarations shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "cq_common.cuh"

namespace cq {

cudaError_t launch_pack_codes(const int8_t *k, int B, int64_t N, int64_t K, uint8_t *codes, cudaStream_t st);
cudaError_t launch_repack(const uint8_t *codes, const float *scale, const uint16_t *a, const uint16_t *b, const Dims &d,
                          void *layout, cudaStream_t st);
cudaError_t launch_unpack(const void *layout, const Dims &d, uint8_t *codes, float *scale, uint16_t *a, uint16_t *b,
                          cudaStream_t st);
cudaError_t launch_decode_levels(const void *layout, const Dims &d, float *levels, cudaStream_t st);
cudaError_t launch_decode_carriers(const void *layout, const Dims &d, int8_t *carriers, cudaStream_t st);
cudaError_t launch_decode_weights(const void *layout, const Dims &d, float *What, cudaStream_t st);
cudaError_t launch_a8_partials(const void *layout, const Dims &d, const int8_t *x8, int64_t M, int32_t *P, cudaStream_t st);
// act_f16 (here and below): the 16-bit activation / output patterns are binary16 instead of bfloat16
cudaError_t launch_quantize_a8(const uint16_t *x, int64_t M, int64_t K, int8_t *x8, int64_t x8_pitch, float *dx,
                               bool operand_order, bool act_f16, cudaStream_t st);

// h[M][2 I] (gate | up, model dtype) -> INT8 carrier of silu(gate) * up in the MMA operand order, and its row scales
cudaError_t launch_swiglu_quantize_a8(const uint16_t *h, int64_t M, int64_t I, int8_t *x8, int64_t x8_pitch, float *dx,
                                      bool act_f16, cudaStream_t st);
// routed execution: xg[r] = x[route_token[r]] (zero row for an index outside [0, T))
cudaError_t launch_gather_rows(const uint16_t *x, const int32_t *route_token, uint16_t *xg, int64_t R, int64_t T, int64_t K,
                               cudaStream_t st);
cudaError_t launch_wait_timeout(int *status, long long limit_cycles, cudaStream_t st);

// Workspace carving (all offsets 256-byte aligned).
struct Workspace {
    size_t counters_off, counters_bytes;   // int32 arrival counters, one per 128-row block
    size_t partial_off, partial_bytes;     // fp32 split-K partial sums: small M [CTA][2][M][128]; model-dtype GEMM [CTA][2][BNT][128]; A8 GEMM [shared tile][slice][BN][128]
    size_t x8_off, x8_bytes;               // Dynamic A8: int8 activation carrier [M][Kp]
    size_t dx_off, dx_bytes;               // Dynamic A8: row scales [M]
    size_t status_off;                     // int32 device status word (bounded waits report here)
    size_t total;
};
Workspace plan_workspace(const Dims &d, int64_t M, int mode);

// Streaming multiprocessors of the current device (148 when no device can be asked).
int sm_count();

// cudaFuncSetAttribute is a per-DEVICE setting: `done` (one per kernel instantiation) remembers, as a bit
// mask, the devices on which it has been made, so a process that uses several GPUs sets it on each.
// Thread safe; devices beyond 63 simply set the attribute on every launch.
template <class Kern>
cudaError_t ensure_func_attr(Kern kern, std::atomic<uint64_t> &done, cudaFuncAttribute attr, int value) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool tracked = dev >= 0 && dev < 64;
    const uint64_t bit = tracked ? (1ull << dev) : 0;
    if (tracked && (done.load(std::memory_order_acquire) & bit)) return cudaSuccess;
    e = cudaFuncSetAttribute(kern, attr, value);
    if (e == cudaSuccess && tracked) done.fetch_or(bit, std::memory_order_release);
    return e;
}
// the thread's record of the last failed CUDA call (what cq_last_cuda_error returns)
void set_last_cuda_error(cudaError_t e);

// Decomposition of the small-M path: number of CTAs (one contiguous run of tiles each) and the
// largest number of CTAs that contribute to one 128-row block.
struct GemvPlan { int ctas, max_run, overhead; };
GemvPlan gemv_plan(const Dims &d, int64_t M, int mode);

// Small-M (M <= 16) split-K tensor-core GEMV, both activation modes.
// prequantized (Dynamic A8 only): the workspace already holds the INT8 carrier and the row scales of x (x is not read)
cudaError_t launch_gemv(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int mode,
                        bool act_f16, uint8_t *ws, const Workspace &plan, cudaStream_t st, bool prequantized = false);
int gemm_tc_token_tile(int64_t M);
struct TcPlan { int bnt, token_tiles, ctas, stream_k, p2, crossing; int64_t t_full; };
TcPlan gemm_tc_plan(const Dims &d, int64_t M);
int gemm_a8_token_tile(const Dims &d, int64_t M);
struct A8Plan { int bn, token_tiles, slices, ctas; int64_t t_full; };
A8Plan gemm_a8_plan(const Dims &d, int64_t M);

// offline encoder steps (cq_encode.cu)
cudaError_t launch_encode_assign(const float *W, int B, int G, int64_t N, int64_t K, const float *scale, const uint16_t *a,
                                 const uint16_t *b, int joint, int8_t *k, cudaStream_t st);
cudaError_t launch_encode_scale(const float *W, const int8_t *k, int B, int G, int64_t N, int64_t K, const uint16_t *a,
                                const uint16_t *b, int joint, float *scale, cudaStream_t st);
cudaError_t launch_encode_losses(const float *W, const int8_t *k, int B, int G, int64_t N, int64_t K, const float *scale,
                                 const uint16_t *a, const uint16_t *b, double *LC, double *LA8, cudaStream_t st);
cudaError_t launch_encode_search(const float *W, int B, int G, int64_t N, int64_t K, int joint, int effort, int8_t *k,
                                 float *scale, uint16_t *a, uint16_t *b, cudaStream_t st);
// Large-M tcgen05 / TMEM GEMM, both activation modes.
cudaError_t launch_gemm_tc(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int mode,
                           bool act_f16, uint8_t *ws, const Workspace &plan, cudaStream_t st);

// Large-M Dynamic-A8 GEMM: activation quantiser, then tcgen05 kind::i8 with per-group int32 partials.
cudaError_t launch_gemm_a8_tc(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, bool act_f16,
                              uint8_t *ws, const Workspace &plan, cudaStream_t st, bool prequantized = false);

}  // namespace cq
