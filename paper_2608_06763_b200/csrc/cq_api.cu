// C ABI of the library (include/cubicquant.h): argument validation on the host, then launches.
#include "../../include/cubicquant.h"

#include <cuda_runtime.h>

#include "cq_common.cuh"
#include "cq_internal.h"

namespace cq {

static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }

int gemm_tc_available();

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

Workspace plan_workspace(const Dims &d, int64_t M, int mode) {
    Workspace w{};
    const int64_t Kp = (int64_t)d.KT * TILE;
    const int64_t Mc = M < 16 ? M : 16;  // rows handled by one small-M launch
    const GemvPlan gp = gemv_plan(d, Mc, mode);
    size_t off = 0;
    w.status_off = off; off += 256;  // first, so cq_gemm_status finds it without knowing the problem
    // arrival counters: one per 128-row block (small M) or per output tile (split-K GEMM)
    const int64_t bnt = mode == CQ_MODEL_DTYPE ? gemm_tc_token_tile(M) : gemm_a8_token_tile(d, M);
    const size_t n_ctr = (size_t)d.NB * (M > 16 ? (size_t)((M + bnt - 1) / bnt) : 1);
    w.counters_off = off; w.counters_bytes = align_up(n_ctr * 4, 256); off += w.counters_bytes;
    size_t part = (size_t)gp.ctas * 2 * Mc * TILE * 4;   // two partial slots per CTA
    if (M > 16 && mode == CQ_DYN_A8) {        // tiles of the last round cut into slices: one partial tile per slice
        const A8Plan ap = gemm_a8_plan(d, M);
        const size_t p2 = ap.slices > 1 ? (size_t)((int64_t)d.NB * ap.token_tiles - ap.t_full) * ap.slices * ap.bn * TILE * 4 : 0;
        if (p2 > part) part = p2;
    }
    if (M > 16 && mode == CQ_MODEL_DTYPE) {   // stream-K: two partial tiles per run
        const TcPlan tp = gemm_tc_plan(d, M);
        const size_t p2 = (size_t)tp.p2 * 2 * tp.bnt * TILE * 4;
        if (p2 > part) part = p2;
    }
    w.partial_off = off; w.partial_bytes = align_up(part, 256); off += w.partial_bytes;
    if (mode == CQ_DYN_A8) {
        w.x8_off = off; w.x8_bytes = align_up((size_t)(M + 127) / 128 * 128 * Kp, 256); off += w.x8_bytes;
        w.dx_off = off; w.dx_bytes = align_up((size_t)M * 4, 256); off += w.dx_bytes;
    }
    w.total = off;
    return w;
}

static int check_format(int B, int G, int64_t N, int64_t K) {
    if (B < 1 || B > 8 || N <= 0 || K <= 0 || G <= 0) return CQ_ERR_INVALID_ARG;
    if (G != 32 && G != 64 && G != 128 && G != 256 && G != 512) return CQ_ERR_UNSUPPORTED;
    if (K % G != 0) return CQ_ERR_UNSUPPORTED;
    return CQ_OK;
}
static bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

static int check_arch() {
    static thread_local int cached_dev = -1, cached_ok = 0;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; return CQ_ERR_CUDA; }
    if (dev != cached_dev) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) { g_last_cuda_error = (int)e; return CQ_ERR_CUDA; }
        cached_dev = dev;
        cached_ok = (major == 10);
    }
    return cached_ok ? CQ_OK : CQ_ERR_ARCH;
}

static int wrap(cudaError_t e) {
    if (e == cudaSuccess) return CQ_OK;
    g_last_cuda_error = (int)e;
    return CQ_ERR_CUDA;
}

}  // namespace cq

using namespace cq;

#pragma GCC visibility push(default)
extern "C" {

const char *cq_status_string(int status) {
    switch (status) {
        case CQ_OK: return "CQ_OK";
        case CQ_ERR_INVALID_ARG: return "CQ_ERR_INVALID_ARG";
        case CQ_ERR_UNSUPPORTED: return "CQ_ERR_UNSUPPORTED";
        case CQ_ERR_ALIGNMENT: return "CQ_ERR_ALIGNMENT";
        case CQ_ERR_WORKSPACE: return "CQ_ERR_WORKSPACE";
        case CQ_ERR_ARCH: return "CQ_ERR_ARCH";
        case CQ_ERR_CUDA: return "CQ_ERR_CUDA";
        case CQ_ERR_TIMEOUT: return "CQ_ERR_TIMEOUT";
        default: return "CQ_ERR_UNKNOWN";
    }
}

int cq_last_cuda_error(void) { return g_last_cuda_error; }

size_t cq_canonical_code_bytes(int B, int64_t N, int64_t K) {
    if (B < 1 || B > 8 || N <= 0 || K <= 0) return 0;
    return (size_t)N * (size_t)((K * B + 7) / 8);
}

double cq_effective_bits(int B, int G) { return (double)B + 64.0 / (double)G; }

size_t cq_layout_bytes(int B, int G, int64_t N, int64_t K) {
    if (check_format(B, G, N, K) != CQ_OK) return 0;
    const Dims d = make_dims(B, G, N, K);
    return (size_t)d.NB * d.KT * (size_t)d.tile_bytes;
}

size_t cq_workspace_bytes(int B, int G, int64_t M, int64_t N, int64_t K, int mode) {
    if (check_format(B, G, N, K) != CQ_OK || M <= 0 || (mode != CQ_MODEL_DTYPE && mode != CQ_DYN_A8)) return 0;
    return plan_workspace(make_dims(B, G, N, K), M, mode).total;
}

int cq_workspace_init(void *workspace, size_t workspace_bytes, void *stream) {
    if (!workspace || workspace_bytes == 0) return CQ_ERR_INVALID_ARG;
    // counters and the status word sit at the front of the workspace; zeroing everything is simplest
    return wrap(cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream));
}

int cq_pack_codes(const int8_t *k, int B, int64_t N, int64_t K, uint8_t *codes, void *stream) {
    if (!k || !codes || B < 1 || B > 8 || N <= 0 || K <= 0) return CQ_ERR_INVALID_ARG;
    return wrap(launch_pack_codes(k, B, N, K, codes, (cudaStream_t)stream));
}

int cq_repack(const uint8_t *codes, const float *scale, const uint16_t *a, const uint16_t *b, int B, int G, int64_t N,
              int64_t K, void *layout, void *stream) {
    if (!codes || !scale || !a || !b || !layout) return CQ_ERR_INVALID_ARG;
    int st = check_format(B, G, N, K);
    if (st != CQ_OK) return st;
    if (misaligned(layout)) return CQ_ERR_ALIGNMENT;
    return wrap(launch_repack(codes, scale, a, b, make_dims(B, G, N, K), layout, (cudaStream_t)stream));
}

int cq_unpack(const void *layout, int B, int G, int64_t N, int64_t K, uint8_t *codes, float *scale, uint16_t *a,
              uint16_t *b, void *stream) {
    if (!codes || !scale || !a || !b || !layout) return CQ_ERR_INVALID_ARG;
    int st = check_format(B, G, N, K);
    if (st != CQ_OK) return st;
    if (misaligned(layout)) return CQ_ERR_ALIGNMENT;
    return wrap(launch_unpack(layout, make_dims(B, G, N, K), codes, scale, a, b, (cudaStream_t)stream));
}

static int gemm_any(const void *layout, int B, int G, const uint16_t *x, uint16_t *y, int64_t M, int64_t N, int64_t K,
                    int mode, bool act_f16, void *workspace, size_t workspace_bytes, void *stream) {
    if (!layout || !x || !y || !workspace || M <= 0) return CQ_ERR_INVALID_ARG;
    if (mode != CQ_MODEL_DTYPE && mode != CQ_DYN_A8) return CQ_ERR_INVALID_ARG;
    int st = check_format(B, G, N, K);
    if (st != CQ_OK) return st;
    if (misaligned(layout) || misaligned(x) || misaligned(y) || misaligned(workspace)) return CQ_ERR_ALIGNMENT;
    const Dims d = make_dims(B, G, N, K);
    const Workspace plan = plan_workspace(d, M, mode);
    if (workspace_bytes < plan.total) return CQ_ERR_WORKSPACE;
    st = check_arch();
    if (st != CQ_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t *ws = (uint8_t *)workspace;
    if (M <= 16) return wrap(launch_gemv(layout, d, x, y, M, mode, act_f16, ws, plan, s));
    if (mode == CQ_MODEL_DTYPE) return wrap(launch_gemm_tc(layout, d, x, y, M, mode, act_f16, ws, plan, s));
    return wrap(launch_gemm_a8_tc(layout, d, x, y, M, act_f16, ws, plan, s));
}

int cq_gemm(const void *layout, int B, int G, const uint16_t *x, uint16_t *y, int64_t M, int64_t N, int64_t K,
            int mode, void *workspace, size_t workspace_bytes, void *stream) {
    return gemm_any(layout, B, G, x, y, M, N, K, mode, false, workspace, workspace_bytes, stream);
}

int cq_gemm_f16(const void *layout, int B, int G, const uint16_t *x, uint16_t *y, int64_t M, int64_t N, int64_t K,
                int mode, void *workspace, size_t workspace_bytes, void *stream) {
    return gemm_any(layout, B, G, x, y, M, N, K, mode, true, workspace, workspace_bytes, stream);
}

// Workspace of the fused MLP: [gate_up operator's workspace][h: M x 2 I model-dtype values][down operator's
// Dynamic-A8 workspace].  The down operator's plan is shifted so that both operators report into the one status
// word at the front.
struct MlpPlan { Workspace gu, dn; size_t h_off, total; };
static MlpPlan plan_mlp(const Dims &dgu, const Dims &ddn, int64_t M, int mode_gu) {
    MlpPlan p;
    p.gu = plan_workspace(dgu, M, mode_gu);
    p.h_off = align_up(p.gu.total, 256);
    const size_t dn_off = align_up(p.h_off + (size_t)M * (size_t)dgu.N * 2, 256);
    p.dn = plan_workspace(ddn, M, CQ_DYN_A8);
    p.dn.counters_off += dn_off; p.dn.partial_off += dn_off; p.dn.x8_off += dn_off; p.dn.dx_off += dn_off;
    p.dn.status_off = 0;
    p.total = dn_off + p.dn.total;
    return p;
}

size_t cq_mlp_workspace_bytes(int B_gu, int G_gu, int B_dn, int G_dn, int64_t M, int64_t K, int64_t I, int64_t N, int mode_gate_up) {
    if (check_format(B_gu, G_gu, 2 * I, K) != CQ_OK || check_format(B_dn, G_dn, N, I) != CQ_OK || M <= 0) return 0;
    if (mode_gate_up != CQ_MODEL_DTYPE && mode_gate_up != CQ_DYN_A8) return 0;
    return plan_mlp(make_dims(B_gu, G_gu, 2 * I, K), make_dims(B_dn, G_dn, N, I), M, mode_gate_up).total;
}

int cq_mlp_swiglu(const void *layout_gate_up, int B_gu, int G_gu, const void *layout_down, int B_dn, int G_dn, const uint16_t *x,
                  uint16_t *y, int64_t M, int64_t K, int64_t I, int64_t N, int mode_gate_up, int act_f16, void *workspace,
                  size_t workspace_bytes, void *stream) {
    if (!layout_gate_up || !layout_down || !x || !y || !workspace || M <= 0 || I <= 0) return CQ_ERR_INVALID_ARG;
    if (mode_gate_up != CQ_MODEL_DTYPE && mode_gate_up != CQ_DYN_A8) return CQ_ERR_INVALID_ARG;
    int st = check_format(B_gu, G_gu, 2 * I, K);
    if (st == CQ_OK) st = check_format(B_dn, G_dn, N, I);
    if (st != CQ_OK) return st;
    if (I % 8 != 0) return CQ_ERR_UNSUPPORTED;
    if (misaligned(layout_gate_up) || misaligned(layout_down) || misaligned(x) || misaligned(y) || misaligned(workspace))
        return CQ_ERR_ALIGNMENT;
    const Dims dgu = make_dims(B_gu, G_gu, 2 * I, K), ddn = make_dims(B_dn, G_dn, N, I);
    const MlpPlan plan = plan_mlp(dgu, ddn, M, mode_gate_up);
    if (workspace_bytes < plan.total) return CQ_ERR_WORKSPACE;
    st = check_arch();
    if (st != CQ_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t *ws = (uint8_t *)workspace;
    uint16_t *h = reinterpret_cast<uint16_t *>(ws + plan.h_off);
    const bool f16 = act_f16 != 0;
    // 1. gate_up, an ordinary operator: model-dtype output
    cudaError_t e;
    if (M <= 16) e = launch_gemv(layout_gate_up, dgu, x, h, M, mode_gate_up, f16, ws, plan.gu, s);
    else if (mode_gate_up == CQ_MODEL_DTYPE) e = launch_gemm_tc(layout_gate_up, dgu, x, h, M, mode_gate_up, f16, ws, plan.gu, s);
    else e = launch_gemm_a8_tc(layout_gate_up, dgu, x, h, M, f16, ws, plan.gu, s);
    if (e != cudaSuccess) return wrap(e);
    // 2. gated activation and the down projection's activation quantiser in one kernel
    e = launch_swiglu_quantize_a8(h, M, I, reinterpret_cast<int8_t *>(ws + plan.dn.x8_off), (int64_t)ddn.KT * TILE,
                                  reinterpret_cast<float *>(ws + plan.dn.dx_off), f16, s);
    if (e != cudaSuccess) return wrap(e);
    // 3. the down projection on the carrier that is already in its workspace
    if (M <= 16) e = launch_gemv(layout_down, ddn, nullptr, y, M, CQ_DYN_A8, f16, ws, plan.dn, s, true);
    else e = launch_gemm_a8_tc(layout_down, ddn, nullptr, y, M, f16, ws, plan.dn, s, true);
    return wrap(e);
}

// Workspace of the routed product: [gathered rows: R x K model-dtype values][the largest per-matrix cq_gemm workspace].
static bool routed_offsets_ok(const int64_t *off, int E, int64_t R) {
    if (!off || off[0] != 0 || off[E] != R) return false;
    for (int e = 0; e < E; ++e) if (off[e + 1] < off[e]) return false;
    return true;
}
static size_t routed_sub_bytes(const Dims &d, const int64_t *off, int E, int mode) {
    size_t need = 0;
    for (int e = 0; e < E; ++e) {
        const int64_t m = off[e + 1] - off[e];
        if (m > 0) { const size_t t = plan_workspace(d, m, mode).total; if (t > need) need = t; }
    }
    return need;
}

size_t cq_routed_workspace_bytes(int B, int G, int E, const int64_t *expert_offset_host, int64_t N, int64_t K, int mode) {
    if (check_format(B, G, N, K) != CQ_OK || E <= 0 || !expert_offset_host || (mode != CQ_MODEL_DTYPE && mode != CQ_DYN_A8)) return 0;
    const int64_t R = expert_offset_host[E];
    if (R <= 0 || !routed_offsets_ok(expert_offset_host, E, R)) return 0;
    return align_up((size_t)R * K * 2, 256) + routed_sub_bytes(make_dims(B, G, N, K), expert_offset_host, E, mode);
}

int cq_gemm_routed(const void *const *layouts_host, int E, int B, int G, const uint16_t *x, const int32_t *route_token,
                   const int64_t *expert_offset_host, uint16_t *y_routes, int64_t T, int64_t N, int64_t K, int mode, int act_f16,
                   void *workspace, size_t workspace_bytes, void *stream) {
    if (!layouts_host || !x || !route_token || !expert_offset_host || !y_routes || !workspace || E <= 0 || T <= 0)
        return CQ_ERR_INVALID_ARG;
    if (mode != CQ_MODEL_DTYPE && mode != CQ_DYN_A8) return CQ_ERR_INVALID_ARG;
    int st = check_format(B, G, N, K);
    if (st != CQ_OK) return st;
    const int64_t R = expert_offset_host[E];
    if (R <= 0 || !routed_offsets_ok(expert_offset_host, E, R)) return CQ_ERR_INVALID_ARG;
    for (int e = 0; e < E; ++e) {
        if (!layouts_host[e]) return CQ_ERR_INVALID_ARG;
        if (misaligned(layouts_host[e])) return CQ_ERR_ALIGNMENT;
    }
    if (misaligned(x) || misaligned(y_routes) || misaligned(workspace) || (K * 2) % 16 != 0 || (N * 2) % 16 != 0) return CQ_ERR_ALIGNMENT;
    const Dims d = make_dims(B, G, N, K);
    const size_t xg_bytes = align_up((size_t)R * K * 2, 256), sub = routed_sub_bytes(d, expert_offset_host, E, mode);
    if (workspace_bytes < xg_bytes + sub) return CQ_ERR_WORKSPACE;
    st = check_arch();
    if (st != CQ_OK) return st;
    uint16_t *xg = reinterpret_cast<uint16_t *>(workspace);
    cudaError_t e0 = launch_gather_rows(x, route_token, xg, R, T, K, (cudaStream_t)stream);
    if (e0 != cudaSuccess) return wrap(e0);
    uint8_t *sub_ws = (uint8_t *)workspace + xg_bytes;
    for (int e = 0; e < E; ++e) {   // one dispatch per matrix that has routes: its decoded tiles serve all of them
        const int64_t r0 = expert_offset_host[e], m = expert_offset_host[e + 1] - r0;
        if (m == 0) continue;
        st = gemm_any(layouts_host[e], B, G, xg + r0 * K, y_routes + r0 * N, m, N, K, mode, act_f16 != 0, sub_ws, sub, stream);
        if (st != CQ_OK) return st;
    }
    return CQ_OK;
}

int cq_gemm_status(const void *workspace, size_t workspace_bytes, void *stream) {
    if (!workspace || workspace_bytes < 512) return CQ_ERR_INVALID_ARG;
    // the status word is the first word of every workspace (plan_workspace)
    int host = 0;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return wrap(e);
    e = cudaMemcpy(&host, (const uint8_t *)workspace, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return wrap(e);
    return host == 0 ? CQ_OK : CQ_ERR_TIMEOUT;
}

int cq_gemm_host(const void *layout, int B, int G, const uint16_t *x_host, uint16_t *y_host, uint16_t *x_dev,
                 uint16_t *y_dev, int64_t M, int64_t N, int64_t K, int mode, void *workspace, size_t workspace_bytes,
                 void *stream) {
    if (!x_host || !y_host || !x_dev || !y_dev || M <= 0 || N <= 0 || K <= 0) return CQ_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyAsync(x_dev, x_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return wrap(e);
    int st = cq_gemm(layout, B, G, x_dev, y_dev, M, N, K, mode, workspace, workspace_bytes, stream);
    if (st != CQ_OK) return st;
    e = cudaMemcpyAsync(y_host, y_dev, (size_t)M * N * 2, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return wrap(e);
    return wrap(cudaStreamSynchronize(s));
}

static int check_encode(int B, int G, int64_t N, int64_t K, int objective) {
    if (B < 1 || B > 8 || N <= 0 || K <= 0 || G <= 0) return CQ_ERR_INVALID_ARG;
    if (objective != CQ_FIT_CONTINUOUS && objective != CQ_FIT_JOINT) return CQ_ERR_INVALID_ARG;
    if (K % G != 0 || G > 512) return CQ_ERR_UNSUPPORTED;
    return CQ_OK;
}

int cq_encode_assign(const float *W, int B, int G, int64_t N, int64_t K, const float *scale, const uint16_t *a,
                     const uint16_t *b, int objective, int8_t *k, void *stream) {
    if (!W || !scale || !a || !b || !k) return CQ_ERR_INVALID_ARG;
    const int st = check_encode(B, G, N, K, objective);
    if (st != CQ_OK) return st;
    return wrap(launch_encode_assign(W, B, G, N, K, scale, a, b, objective, k, (cudaStream_t)stream));
}

int cq_encode_scale(const float *W, const int8_t *k, int B, int G, int64_t N, int64_t K, const uint16_t *a,
                    const uint16_t *b, int objective, float *scale, void *stream) {
    if (!W || !scale || !a || !b || !k) return CQ_ERR_INVALID_ARG;
    const int st = check_encode(B, G, N, K, objective);
    if (st != CQ_OK) return st;
    return wrap(launch_encode_scale(W, k, B, G, N, K, a, b, objective, scale, (cudaStream_t)stream));
}

int cq_encode_losses(const float *W, const int8_t *k, int B, int G, int64_t N, int64_t K, const float *scale,
                     const uint16_t *a, const uint16_t *b, double *LC, double *LA8, void *stream) {
    if (!W || !scale || !a || !b || !k || !LC || !LA8) return CQ_ERR_INVALID_ARG;
    const int st = check_encode(B, G, N, K, CQ_FIT_JOINT);
    if (st != CQ_OK) return st;
    return wrap(launch_encode_losses(W, k, B, G, N, K, scale, a, b, LC, LA8, (cudaStream_t)stream));
}

int cq_encode(const float *W, int B, int G, int64_t N, int64_t K, int objective, int effort, int8_t *k, float *scale,
              uint16_t *a, uint16_t *b, void *stream) {
    if (!W || !scale || !a || !b || !k || effort < 0 || effort > 3) return CQ_ERR_INVALID_ARG;
    const int st = check_encode(B, G, N, K, objective);
    if (st != CQ_OK) return st;
    return wrap(launch_encode_search(W, B, G, N, K, objective, effort, k, scale, a, b, (cudaStream_t)stream));
}

int cq_quantize_a8(const uint16_t *x, int64_t M, int64_t K, int8_t *x8, float *dx, void *stream) {
    if (!x || !x8 || !dx || M <= 0 || K <= 0) return CQ_ERR_INVALID_ARG;
    return wrap(launch_quantize_a8(x, M, K, x8, K, dx, false, false, (cudaStream_t)stream));
}

int cq_quantize_a8_f16(const uint16_t *x, int64_t M, int64_t K, int8_t *x8, float *dx, void *stream) {
    if (!x || !x8 || !dx || M <= 0 || K <= 0) return CQ_ERR_INVALID_ARG;
    return wrap(launch_quantize_a8(x, M, K, x8, K, dx, false, true, (cudaStream_t)stream));
}

#define CQ_DEBUG_PROLOGUE()                                   \
    if (!layout) return CQ_ERR_INVALID_ARG;                   \
    {                                                         \
        int st_ = check_format(B, G, N, K);                   \
        if (st_ != CQ_OK) return st_;                         \
    }                                                         \
    if (misaligned(layout)) return CQ_ERR_ALIGNMENT;          \
    const Dims d = make_dims(B, G, N, K);

int cq_decode_levels(const void *layout, int B, int G, int64_t N, int64_t K, float *levels, void *stream) {
    if (!levels) return CQ_ERR_INVALID_ARG;
    CQ_DEBUG_PROLOGUE();
    return wrap(launch_decode_levels(layout, d, levels, (cudaStream_t)stream));
}

int cq_decode_carriers(const void *layout, int B, int G, int64_t N, int64_t K, int8_t *carriers, void *stream) {
    if (!carriers) return CQ_ERR_INVALID_ARG;
    CQ_DEBUG_PROLOGUE();
    return wrap(launch_decode_carriers(layout, d, carriers, (cudaStream_t)stream));
}

int cq_decode_weights(const void *layout, int B, int G, int64_t N, int64_t K, float *What, void *stream) {
    if (!What) return CQ_ERR_INVALID_ARG;
    CQ_DEBUG_PROLOGUE();
    return wrap(launch_decode_weights(layout, d, What, (cudaStream_t)stream));
}

int cq_debug_gemm_plan(int B, int G, int64_t M, int64_t N, int64_t K, int mode, int64_t *plan) {
    if (!plan || M <= 16 || (mode != CQ_MODEL_DTYPE && mode != CQ_DYN_A8)) return CQ_ERR_INVALID_ARG;
    const int st = check_format(B, G, N, K);
    if (st != CQ_OK) return st;
    const Dims d = make_dims(B, G, N, K);
    if (mode == CQ_MODEL_DTYPE) {
        const TcPlan tp = gemm_tc_plan(d, M);
        plan[0] = tp.bnt; plan[1] = tp.t_full; plan[2] = tp.p2; plan[3] = (int64_t)d.NB * tp.token_tiles - tp.t_full;
        plan[4] = tp.crossing;
    } else {
        const A8Plan ap = gemm_a8_plan(d, M);
        const int64_t shared = (int64_t)d.NB * ap.token_tiles - ap.t_full;
        plan[0] = ap.bn; plan[1] = ap.t_full; plan[2] = shared * ap.slices; plan[3] = shared; plan[4] = 0;
    }
    return CQ_OK;
}

int cq_debug_wait_timeout(void *workspace, size_t workspace_bytes, int64_t limit_cycles, void *stream) {
    if (!workspace || workspace_bytes < 512 || limit_cycles <= 0 || limit_cycles > 2000000000ll) return CQ_ERR_INVALID_ARG;
    if (misaligned(workspace)) return CQ_ERR_ALIGNMENT;
    const int st = check_arch();
    if (st != CQ_OK) return st;
    // the status word is the first word of every workspace (plan_workspace)
    return wrap(launch_wait_timeout((int *)workspace, (long long)limit_cycles, (cudaStream_t)stream));
}

int cq_debug_a8_partials(const void *layout, int B, int G, const int8_t *x8, int64_t M, int64_t N, int64_t K,
                         int32_t *P, void *stream) {
    if (!x8 || !P || M <= 0) return CQ_ERR_INVALID_ARG;
    CQ_DEBUG_PROLOGUE();
    return wrap(launch_a8_partials(layout, d, x8, M, P, (cudaStream_t)stream));
}

}  // extern "C"
#pragma GCC visibility pop
