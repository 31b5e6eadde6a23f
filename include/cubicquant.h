/*
 * cubicquant.h -- C ABI of the B200 (sm_100a) CubicQuant packed-weight GEMV / GEMM library.
 *
 * The library computes   y[M,N] = x[M,K] * What[N,K]^T   directly from packed B-bit
 * (1..8) weight codes whose per-group reconstruction levels follow the paper's monotone
 * cubic (Section 2.2, Eq. cubic), in two activation modes (Section 5.3 model dtype,
 * Section 5.4 Dynamic A8).
 *
 * Conventions common to every call
 *   - All pointers are DEVICE pointers unless the name says "host".  The caller owns every
 *     buffer; the library allocates no device memory and never synchronises the device
 *     (except cq_gemm_host, which waits for its own copies).
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *   - Return value: CQ_OK or a negative CQ_ERR_* code.  Argument errors are found on the
 *     host before anything is launched.
 *   - Logical weight matrix: N output channels x K input channels; groups are runs of G
 *     consecutive input channels inside one output row (Section 2.3).
 *   - Canonical (interchange) format, the paper's packed checkpoint view:
 *       codes  uint8 [N][ceil(K*B/8)]  continuous LSB-first bitstream per row, field j at bit
 *                                      j*B (Eq. gpu-packed-extraction); B-bit two's complement,
 *                                      pattern -2^(B-1) reserved and decoding to 0 (Eq. codes);
 *                                      W1: bit 1 = +1, bit 0 = -1.
 *       scale  float  [N][K/G]         s >= 0 (FP32, Appendix A item 3)
 *       a, b   fp16   [N][K/G]         shape coefficients as IEEE binary16 bit patterns
 *   - Device layout: private, tiled and interleaved for 128-bit coalesced loads with the
 *     group parameters stored beside the codes of their tile; produced by cq_repack and
 *     inverted bit-exactly by cq_unpack.
 *   - Supported: B in 1..8; G in {32, 64, 128, 256, 512}; K % G == 0; M, N, K >= 1.  K and N need
 *     not be multiples of the 128 x 128 tile (the layout pads).  For G = 256 / 512 the device layout
 *     repeats a group's parameter record in each of its 128-wide tiles, so it is 8 (G/128 - 1) bytes
 *     per group larger than the canonical format.
 */
#ifndef CUBICQUANT_H_
#define CUBICQUANT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    CQ_OK = 0,
    CQ_ERR_INVALID_ARG = -1, /* null pointer, M/N/K <= 0, B outside 1..8, unknown mode */
    CQ_ERR_UNSUPPORTED = -2, /* K % G != 0, G not in {32,64,128,256,512} */
    CQ_ERR_ALIGNMENT = -3,   /* a pointer is not 16-byte aligned */
    CQ_ERR_WORKSPACE = -4,   /* workspace_bytes smaller than cq_workspace_bytes() */
    CQ_ERR_ARCH = -5,        /* current device is not compute capability 10.x */
    CQ_ERR_CUDA = -6,        /* a CUDA runtime call or launch failed; see cq_last_cuda_error() */
    CQ_ERR_TIMEOUT = -7      /* a bounded device-side wait gave up (reported by cq_gemm_status) */
};

enum { CQ_MODEL_DTYPE = 0, CQ_DYN_A8 = 1 };

/* Human-readable name of a status code (static string). */
const char *cq_status_string(int status);
/* cudaError_t value of the last failed CUDA call made by this library on this thread (0 if none). */
int cq_last_cuda_error(void);

/* Bytes of the canonical code tensor: N * ceil(K*B/8). */
size_t cq_canonical_code_bytes(int B, int64_t N, int64_t K);
/* Effective stored bits per weight of the canonical format, B + 64/G (Eq. effective-bits). */
double cq_effective_bits(int B, int G);
/* Bytes of the device layout for an N x K matrix (codes + co-located parameters, including the
 * padding of N and K up to multiples of 128).  0 if the arguments are unsupported. */
size_t cq_layout_bytes(int B, int G, int64_t N, int64_t K);
/* Bytes of scratch cq_gemm needs for this problem (split-K partial sums and arrival counters;
 * Dynamic A8 adds the INT8 activation carrier and its row scales).  Never 0 for valid input.  The split-K
 * schedule, and with it this size, depends on the number of multiprocessors of the current device (148 are
 * assumed when no device can be asked): ask with the device current on which cq_gemm will run; cq_gemm
 * checks workspace_bytes against the device it runs on and returns CQ_ERR_WORKSPACE if it is too small. */
size_t cq_workspace_bytes(int B, int G, int64_t M, int64_t N, int64_t K, int mode);
/* Zero the arrival counters of a workspace.  Call once after allocating it (and after any
 * cq_gemm that returned an error); cq_gemm leaves the counters zero when it completes. */
int cq_workspace_init(void *workspace, size_t workspace_bytes, void *stream);

/* Signed logical codes k[N][K] (int8; W1: +-1) -> canonical packed bitstream (Section 2.1,
 * Eq. gpu-packed-extraction read backwards).  `codes` must hold cq_canonical_code_bytes(). */
int cq_pack_codes(const int8_t *k, int B, int64_t N, int64_t K, uint8_t *codes, void *stream);

/* Canonical format -> device layout (Section 2.1/2.3 data, re-tiled; a bijection). */
int cq_repack(const uint8_t *codes, const float *scale, const uint16_t *a, const uint16_t *b, int B, int G, int64_t N,
              int64_t K, void *layout, void *stream);
/* Device layout -> canonical format; returns exactly the bytes given to cq_repack. */
int cq_unpack(const void *layout, int B, int G, int64_t N, int64_t K, uint8_t *codes, float *scale, uint16_t *a,
              uint16_t *b, void *stream);

/* The hot path.  y[M][N] (bf16 bits, row-major) = x[M][K] (bf16 bits, row-major) * What^T.
 *   mode CQ_MODEL_DTYPE: continuous reconstruction of Eq. cubic; fp32 accumulation (Section 5.3).
 *   mode CQ_DYN_A8:      per-row absmax INT8 activations (Eq. a8-activation-scale/-quantization),
 *                        INT8 weight carriers (Eq. carrier), int32 group partials, fp32 rescale
 *                        (Eq. a8-output).
 * M <= 16 runs the split-K tensor-core GEMV; larger M the tcgen05/TMEM GEMM.
 * x, y, layout and workspace must be 16-byte aligned; x and y must not alias. */
int cq_gemm(const void *layout, int B, int G, const uint16_t *x, uint16_t *y, int64_t M, int64_t N, int64_t K,
            int mode, void *workspace, size_t workspace_bytes, void *stream);

/* The same product for a model whose dtype is IEEE binary16: x[M][K] and y[M][N] are binary16 bit patterns
 * (Section 5.3: the model-dtype path accepts FP16 or BF16 activations).  Everything else -- arguments,
 * modes, dispatch, workspace, errors -- is as for cq_gemm; in model-dtype mode the large-M kernel rounds its
 * decoded weight tiles to binary16 instead of bfloat16, and both modes write y in binary16. */
int cq_gemm_f16(const void *layout, int B, int G, const uint16_t *x, uint16_t *y, int64_t M, int64_t N, int64_t K,
                int mode, void *workspace, size_t workspace_bytes, void *stream);

/* A SwiGLU MLP block with the boundary in front of the down projection fused (Section 5.4, last paragraph:
 * activation and quantisation combined adjacent to the down projection; Section 6.4 says where the boundary must
 * not sit: the intermediate only changes its global-memory dtype if it is written out as a carrier by the
 * producing GEMM).  Three launches:
 *     h   = gate_up(x)                          [M][2 I], model dtype; gate = h[:, :I], up = h[:, I:]
 *     act = silu(gate) * up, rounded to the model dtype, and at once its Dynamic-A8 carrier and row scales
 *           (one kernel; the activation itself never reaches memory)
 *     y   = down(act) in Dynamic A8             [M][N], model dtype
 * so the result equals cq_gemm(gate_up) -> an elementwise activation operator -> cq_gemm(down, CQ_DYN_A8).
 * layout_gate_up: device layout of the 2 I x K matrix; layout_down: of the N x I matrix; x [M][K], y [M][N];
 * mode_gate_up: CQ_MODEL_DTYPE or CQ_DYN_A8; act_f16: 0 = bfloat16, 1 = binary16 activations and output.
 * workspace: cq_mlp_workspace_bytes() bytes, zeroed once with cq_workspace_init; cq_gemm_status(workspace) reports a
 * bounded wait of either projection that gave up.  Errors as cq_gemm; I must be a multiple of 8. */
size_t cq_mlp_workspace_bytes(int B_gate_up, int G_gate_up, int B_down, int G_down, int64_t M, int64_t K, int64_t I, int64_t N,
                              int mode_gate_up);
int cq_mlp_swiglu(const void *layout_gate_up, int B_gate_up, int G_gate_up, const void *layout_down, int B_down, int G_down,
                  const uint16_t *x, uint16_t *y, int64_t M, int64_t K, int64_t I, int64_t N, int mode_gate_up, int act_f16,
                  void *workspace, size_t workspace_bytes, void *stream);

/* Routed execution (Section 5.5): R token-matrix routes over E matrices of one shape and format, compacted and
 * grouped by matrix so that every decoded weight tile serves all routes of its matrix.  The caller supplies the route map
 * (routing probabilities, selection and route weights stay outside, as the paper leaves them):
 *     layouts_host        HOST array of E device pointers (device layouts of the E matrices, each N x K)
 *     route_token         DEVICE int32 [R]: the token (row of x) of each route, routes of matrix e at
 *                         [expert_offset[e], expert_offset[e+1])
 *     expert_offset_host  HOST int64 [E + 1], non-decreasing, [0] = 0, [E] = R
 *     x [T][K], y_routes [R][N] (route-major output, model dtype); act_f16 as for cq_mlp_swiglu
 * One gather kernel, then one ordinary cq_gemm dispatch per matrix that has routes, on `stream`.  A token index outside
 * [0, T) yields a zero input row.  workspace: cq_routed_workspace_bytes() bytes, zeroed once with cq_workspace_init.
 * Errors as cq_gemm; CQ_ERR_INVALID_ARG for an inconsistent offset array; N and K must be multiples of 8. */
size_t cq_routed_workspace_bytes(int B, int G, int E, const int64_t *expert_offset_host, int64_t N, int64_t K, int mode);
int cq_gemm_routed(const void *const *layouts_host, int E, int B, int G, const uint16_t *x, const int32_t *route_token,
                   const int64_t *expert_offset_host, uint16_t *y_routes, int64_t T, int64_t N, int64_t K, int mode, int act_f16,
                   void *workspace, size_t workspace_bytes, void *stream);

/* Reads back the device status word of a workspace (waits for `stream` first).  CQ_OK, or
 * CQ_ERR_TIMEOUT when a bounded device-side wait of an earlier cq_gemm on this workspace gave up
 * (its output is then undefined; re-initialise the workspace before reusing it). */
int cq_gemm_status(const void *workspace, size_t workspace_bytes, void *stream);

/* Same product with HOST activations and HOST output: copies x_host to the device, runs cq_gemm
 * and copies y back, all on `stream`, then waits for the stream.  x_dev (M*K bf16) and y_dev
 * (M*N bf16) are caller-provided device staging buffers.  Pinned host memory makes the copies
 * asynchronous; pageable memory also works. */
int cq_gemm_host(const void *layout, int B, int G, const uint16_t *x_host, uint16_t *y_host, uint16_t *x_dev,
                 uint16_t *y_dev, int64_t M, int64_t N, int64_t K, int mode, void *workspace, size_t workspace_bytes,
                 void *stream);

/* Small-M product (M <= 16, model dtype) for callers that cannot hand the library any scratch
 * memory.  (The paper has no counterpart to this call; it exists for integration reasons only.)
 *
 * Who needs it: code that runs where device allocation is off limits, for example an operator
 * plug-in on the request path of an inference server.  Such a plug-in is given its input and output
 * tensors and nothing else; it may not call cudaMalloc (it synchronises the whole device and can
 * fail under the server's fixed memory budget) and has no hook into the host framework's allocator
 * to ask for a workspace.  For those callers the split-K scratch (arrival counters and partial
 * sums) comes from an array of CQ_STATIC_SCRATCH_BYTES that is compiled into the library and
 * occupies that much memory on every GPU that loads it, until the process exits.
 *
 *   - Same arguments and result as cq_gemm(..., CQ_MODEL_DTYPE, ...) without the workspace; all
 *     pointers are device pointers owned by the caller, 16-byte aligned; enqueues on `stream`.
 *   - No allocation of any kind is made, neither by this call nor by anything it calls.
 *   - CQ_ERR_WORKSPACE when the problem needs more scratch than the built-in array holds
 *     (cq_workspace_bytes(B, G, M, N, K, CQ_MODEL_DTYPE) > CQ_STATIC_SCRATCH_BYTES);
 *     CQ_ERR_UNSUPPORTED for M > 16 or an unsupported format.
 *   - The first call on each device looks up the array's device address (with that device current);
 *     where the CUDA runtime loads modules lazily, that is also the moment the array's memory is
 *     committed on that device.  Make that first call during start-up, before any stream capture begins.
 *   - Every call on a device shares the one array and finds in it what the previous call left; the
 *     call clears the counters it relies on before launching.  Two calls whose kernels may overlap
 *     on the GPU (different streams, or host threads) race on the array: serialise them. */
#define CQ_STATIC_SCRATCH_BYTES (8u << 20)
int cq_gemv_static(const void *layout, int B, int G, const uint16_t *x, uint16_t *y, int64_t M, int64_t N, int64_t K,
                   void *stream);

/* Pieces of the path exposed for parity tests. */

/* Dynamic-A8 activation quantiser (Eq. a8-activation-scale, Eq. a8-activation-quantization):
 * x8[M][K] int8 and dx[M] float from x[M][K] bf16.  fp32 arithmetic: xbar = max(max|x|, 1e-10f),
 * dx = xbar / 127 (IEEE division), x8 = clip(round-half-away(x / dx), -127, 127). */
int cq_quantize_a8(const uint16_t *x, int64_t M, int64_t K, int8_t *x8, float *dx, void *stream);
/* The same quantiser for binary16 activations. */
int cq_quantize_a8_f16(const uint16_t *x, int64_t M, int64_t K, int8_t *x8, float *dx, void *stream);
/* Non-negative reconstruction levels of every group (Appendix B): levels[N][K/G][L] float,
 * L = 2^(B-1) (W1: L = 1, the scale). */
int cq_decode_levels(const void *layout, int B, int G, int64_t N, int64_t K, float *levels, void *stream);
/* Non-negative INT8 carriers of every group (Eq. carrier): carriers[N][K/G][L] int8. */
int cq_decode_carriers(const void *layout, int B, int G, int64_t N, int64_t K, int8_t *carriers, void *stream);
/* Dense reconstruction What[N][K] float (sign * level of every code; reserved pattern -> 0). */
int cq_decode_weights(const void *layout, int B, int G, int64_t N, int64_t K, float *What, void *stream);
/* Integer group partials of Eq. a8-output: P[M][N][K/G] int32 from x8[M][K]. */
int cq_debug_a8_partials(const void *layout, int B, int G, const int8_t *x8, int64_t M, int64_t N, int64_t K,
                         int32_t *P, void *stream);

/* The bounded device-side wait on its own (the pipelined kernels give every wait on a barrier a limit;
 * the paper has no counterpart, it is this library's failure reporting).  Launches one thread that
 * waits on a barrier nobody arrives on, with nothing in flight, gives up after `limit_cycles` SM clock
 * cycles (1 .. 2e9) and records that in the workspace's status word; the kernel then ends normally.
 * Afterwards cq_gemm_status(workspace) returns CQ_ERR_TIMEOUT until the workspace is re-initialised.
 * workspace: device pointer, 16-byte aligned, at least 512 bytes. */
int cq_debug_wait_timeout(void *workspace, size_t workspace_bytes, int64_t limit_cycles, void *stream);

/* How cq_gemm(..., mode, ...) with M > 16 spreads this problem over the current device (host-side query, launches
 * nothing; the paper has no counterpart).  plan must hold five values: plan[0] = tokens per output tile, plan[1] =
 * CTAs that compute one whole 128-channel x plan[0]-token tile each, plan[2] = CTAs that share the remaining tiles,
 * each taking a contiguous run of (tile, K) units (0 when every tile is computed whole), plan[3] = those remaining
 * tiles, plan[4] = 1 when a run may cross from one tile into the next, 0 when every shared tile is cut into the same
 * number of runs (always 0 in CQ_DYN_A8).  CQ_ERR_INVALID_ARG for M <= 16, an unknown mode or a null pointer. */
int cq_debug_gemm_plan(int B, int G, int64_t M, int64_t N, int64_t K, int mode, int64_t *plan);

/* ---- Offline encoder (the step before the hot path; Sections 4.1 and 4.3) --------------------------
 * W[N][K] float, logical signed codes k[N][K] int8 (what cq_pack_codes takes), scale[N][K/G] float,
 * a / b [N][K/G] binary16 bit patterns; all device pointers owned by the caller; nothing is allocated
 * and nothing synchronises.  objective: CQ_FIT_CONTINUOUS minimises L_C = sum (w - s q)^2
 * (Eq. offline-objective), CQ_FIT_JOINT minimises L_C + L_A8 with L_A8 taken against the INT8 carrier
 * (s / 127) r(k) (Eq. carrier-aware-objective); for B <= 2 the two coincide.  Decisions are taken in
 * fp64.  Errors: CQ_ERR_INVALID_ARG (null pointer, sizes <= 0, B outside 1..8, unknown objective or
 * effort), CQ_ERR_UNSUPPORTED (K % G != 0 or G > 512), CQ_ERR_CUDA. */
#define CQ_FIT_CONTINUOUS 0
#define CQ_FIT_JOINT 1
/* Codes for fixed stored parameters: nearest reconstruction level (Section 4.1), or the minimiser of
 * (u - s q)^2 + (u - s qtilde)^2 (Eq. carrier-aware-assignment); ties go to the smaller magnitude; the
 * reserved pattern is never produced; W1: the sign of w (w >= 0 -> +1). */
int cq_encode_assign(const float *W, int B, int G, int64_t N, int64_t K, const float *scale, const uint16_t *a,
                     const uint16_t *b, int objective, int8_t *k, void *stream);
/* Scale for fixed codes and shape: sum u z / sum z^2, or Eq. carrier-aware-scale; 0 for an all-zero group. */
int cq_encode_scale(const float *W, const int8_t *k, int B, int G, int64_t N, int64_t K, const uint16_t *a,
                    const uint16_t *b, int objective, float *scale, void *stream);
/* The two groupwise squared errors of Eq. continuous-and-carrier-loss: LC[N][K/G], LA8[N][K/G] double. */
int cq_encode_losses(const float *W, const int8_t *k, int B, int G, int64_t N, int64_t K, const float *scale,
                     const uint16_t *a, const uint16_t *b, double *LC, double *LA8, void *stream);
/* The whole groupwise encoder: a deterministic search over monotone shape candidates and soft clips
 * with alternating assignment / scale updates and a refinement of (s, a, b) by normal equations
 * (Eq. affine-cubic-level), scored on what is stored (a, b in binary16, s in binary32, assignment
 * repeated).  effort: 0 symmetric absmax integer grid, 1 clipped integer grid, 2 fast, 3 reference. */
int cq_encode(const float *W, int B, int G, int64_t N, int64_t K, int objective, int effort, int8_t *k, float *scale,
              uint16_t *a, uint16_t *b, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* CUBICQUANT_H_ */
