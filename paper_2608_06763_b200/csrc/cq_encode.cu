// Offline encoder steps on the GPU (the step before the hot path): groupwise code assignment,
// closed-form scale, the two reconstruction losses, and the deterministic candidate search, under
// the continuous objective of Section 4.1 or the dual-path objective L_C + L_A8 of Section 4.3.
//
// Decisions (which code, which candidate) are taken in fp64, the precision the method is stated in;
// the carrier grid uses the pinned fp32 sequence of Eq. carrier.  This file is compiled without
// floating-point contraction so that a product followed by a sum rounds twice, as written.
//
// One thread owns one group in the search kernel (groups are independent and the search is
// branchy); the assignment / scale / loss kernels use one block per group.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/cubicquant.h"
#include "cq_internal.h"

namespace cq {
namespace {

constexpr int MAXG = 512;      // largest group (Section 5.4: G <= 512)
constexpr int MAXL = 128;      // most non-negative levels (W8)

__device__ __forceinline__ int top_code(int B) { return (1 << (B - 1)) - 1; }   // M of Eq. codes
__device__ __forceinline__ double half_bits_to_double(uint16_t h) { return (double)__half2float(__ushort_as_half(h)); }
__device__ __forceinline__ uint16_t double_to_half_bits(double v) { return __half_as_ushort(__double2half(v)); }

// q(t) = t [a + t (b + c t)], c = 1 - a - b (Eq. cubic)
__device__ __forceinline__ double level_curve(double t, double a, double b) {
    const double c = 1.0 - a - b;
    return t * (a + t * (b + t * c));
}

// m(a, b) = min over [0, 1] of q'(t) (Eq. shape-domain): the end points, and the vertex of the
// quadratic when it lies inside the interval and opens upwards
__device__ __noinline__ double shape_margin(double a, double b) {
    const double c = 1.0 - a - b;
    double m = fmin(a, 3.0 - 2.0 * a - b);
    if (c > 0.0 && b < 0.0 && b > -3.0 * c) m = fmin(m, a - b * b / (3.0 * c));
    return m;
}

// carrier-grid levels round(127 q) / 127 of a shape given in fp32 (Eq. carrier-grid), the rounding by
// the pinned fp32 sequence t = i / M, c = (1 - a) - b, q = t fma(t, fma(t, c, b), a), RNE(127 q)
__device__ __noinline__ void carrier_grid(int B, float a, float b, double *zt) {
    const int M = top_code(B);
    if (B == 2) { zt[0] = 0.0; zt[1] = 1.0; return; }
    const float c = __fsub_rn(__fsub_rn(1.0f, a), b);
    for (int i = 0; i <= M; ++i) {
        const float t = __fdiv_rn((float)i, (float)M);
        const float q = __fmul_rn(t, fmaf(t, fmaf(t, c, b), a));
        int r = __float2int_rn(__fmul_rn(127.0f, q));
        r = min(max(r, 0), 127);
        zt[i] = (double)r / 127.0;
    }
}

// nearest level among increasing y_0 .. y_M, ties to the lower index, saturating at M
__device__ __forceinline__ int nearest_level(double u, const double *y, int M) {
    int lo = 0, hi = M;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (u <= 0.5 * (y[mid] + y[mid + 1])) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// minimiser of (u - s z_i)^2 + (u - s zt_i)^2 (Eq. carrier-aware-assignment), first minimum wins
__device__ __forceinline__ int joint_level(double u, double s, const double *z, const double *zt, int M) {
    int best = 0;
    double bc = INFINITY;
    for (int i = 0; i <= M; ++i) {
        const double d1 = u - s * z[i], d2 = u - s * zt[i];
        const double cst = d1 * d1 + d2 * d2;
        if (cst < bc) { bc = cst; best = i; }
    }
    return best;
}

// ------------------------------------------------------------------ per-group kernels (one block per group)
__global__ void __launch_bounds__(128) assign_kernel(const float *__restrict__ W, int B, int G, int64_t K, int64_t ng,
                                                     const float *__restrict__ scale, const uint16_t *__restrict__ a,
                                                     const uint16_t *__restrict__ b, int joint, int8_t *__restrict__ k) {
    __shared__ double z[MAXL], zt[MAXL], y[MAXL];
    const int64_t gi = blockIdx.x, n = gi / ng, g = gi % ng;
    const float *w = W + n * K + g * G;
    int8_t *ko = k + n * K + g * G;
    if (B == 1) {
        for (int j = threadIdx.x; j < G; j += blockDim.x) ko[j] = (int8_t)(w[j] >= 0.0f ? 1 : -1);
        return;
    }
    const int M = top_code(B);
    const double s = (double)scale[gi], av = half_bits_to_double(a[gi]), bv = half_bits_to_double(b[gi]);
    for (int i = threadIdx.x; i <= M; i += blockDim.x) {
        z[i] = level_curve((double)i / (double)M, av, bv);
        y[i] = s * z[i];
    }
    if (joint && threadIdx.x == 0) carrier_grid(B, (float)av, (float)bv, zt);
    __syncthreads();
    for (int j = threadIdx.x; j < G; j += blockDim.x) {
        const double u = fabs((double)w[j]);
        const int i = joint ? joint_level(u, s, z, zt, M) : nearest_level(u, y, M);
        ko[j] = (int8_t)(w[j] < 0.0f ? -i : i);
    }
}

// sums of a block in a fixed order: each thread adds its strided elements, then thread 0 adds the
// per-thread sums in thread order
__device__ double block_sum(double v, double *sh) {
    sh[threadIdx.x] = v;
    __syncthreads();
    double tot = 0.0;
    if (threadIdx.x == 0) for (int i = 0; i < (int)blockDim.x; ++i) tot += sh[i];
    __syncthreads();
    return tot;   // valid in thread 0
}

// scale[g] = sum u (z + zt) / sum (z^2 + zt^2) (Eq. carrier-aware-scale), or the continuous analogue
__global__ void __launch_bounds__(128) scale_kernel(const float *__restrict__ W, const int8_t *__restrict__ k, int B, int G,
                                                    int64_t K, int64_t ng, const uint16_t *__restrict__ a,
                                                    const uint16_t *__restrict__ b, int joint, float *__restrict__ scale) {
    __shared__ double z[MAXL], zt[MAXL], sh[128];
    const int64_t gi = blockIdx.x, n = gi / ng, g = gi % ng;
    const float *w = W + n * K + g * G;
    const int8_t *kk = k + n * K + g * G;
    const int M = B == 1 ? 1 : top_code(B);
    if (B > 1) {
        const double av = half_bits_to_double(a[gi]), bv = half_bits_to_double(b[gi]);
        for (int i = threadIdx.x; i <= M; i += blockDim.x) z[i] = level_curve((double)i / (double)M, av, bv);
        if (threadIdx.x == 0) {
            if (joint) carrier_grid(B, (float)av, (float)bv, zt);
            else for (int i = 0; i <= M; ++i) zt[i] = 0.0;
        }
    }
    __syncthreads();
    double num = 0.0, den = 0.0;
    for (int j = threadIdx.x; j < G; j += blockDim.x) {
        const double u = fabs((double)w[j]);
        if (B == 1) { num += u; den += 1.0; continue; }
        const int c = kk[j];
        const int i = (c == -(1 << (B - 1))) ? 0 : abs(c);
        if (joint) { num += u * (z[i] + zt[i]); den += z[i] * z[i] + zt[i] * zt[i]; }
        else { num += u * z[i]; den += z[i] * z[i]; }
    }
    const double tn = block_sum(num, sh), td = block_sum(den, sh);
    if (threadIdx.x == 0) scale[gi] = td > 0.0 ? (float)(tn / td) : 0.0f;
}

// L_C = sum (w - s q)^2 and L_A8 = sum (w - (s / 127) r)^2 per group (Eq. continuous-and-carrier-loss)
__global__ void __launch_bounds__(128) losses_kernel(const float *__restrict__ W, const int8_t *__restrict__ k, int B, int G,
                                                     int64_t K, int64_t ng, const float *__restrict__ scale,
                                                     const uint16_t *__restrict__ a, const uint16_t *__restrict__ b,
                                                     double *__restrict__ LC, double *__restrict__ LA8) {
    __shared__ double z[MAXL], zt[MAXL], sh[128];
    const int64_t gi = blockIdx.x, n = gi / ng, g = gi % ng;
    const float *w = W + n * K + g * G;
    const int8_t *kk = k + n * K + g * G;
    const double s = (double)scale[gi];
    const int M = B == 1 ? 1 : top_code(B);
    if (B > 1) {
        const double av = half_bits_to_double(a[gi]), bv = half_bits_to_double(b[gi]);
        for (int i = threadIdx.x; i <= M; i += blockDim.x) z[i] = level_curve((double)i / (double)M, av, bv);
        if (threadIdx.x == 0) carrier_grid(B, (float)av, (float)bv, zt);
    }
    __syncthreads();
    double lc = 0.0, la = 0.0;
    for (int j = threadIdx.x; j < G; j += blockDim.x) {
        const int c = kk[j];
        const double wv = (double)w[j];
        if (B == 1) { const double d = wv - (c > 0 ? 1.0 : -1.0) * s; lc += d * d; la += d * d; continue; }
        const int i = (c == -(1 << (B - 1))) ? 0 : abs(c);
        const double sg = c < 0 ? -1.0 : 1.0;
        const double d1 = wv - sg * s * z[i], d2 = wv - sg * s * zt[i];
        lc += d1 * d1; la += d2 * d2;
    }
    const double tc = block_sum(lc, sh), ta = block_sum(la, sh);
    if (threadIdx.x == 0) { LC[gi] = tc; LA8[gi] = ta; }
}

// ------------------------------------------------------------------ the candidate search (one thread per group)
struct Fit { double loss; float s; uint16_t a16, b16; bool valid; };

struct GroupWork {
    const float *w;      // the group's weights
    int G, B, M, joint;
    double u[MAXG];      // |w|
    int idx[MAXG];       // magnitude indices of the candidate at hand
    int8_t cand[MAXG];   // its signed codes
    int8_t *out;         // best codes so far (global memory)
    Fit best;
};

__device__ __noinline__ double fitted_scale(const GroupWork &gw, const double *z, const double *zt, double fallback) {
    double num = 0.0, den = 0.0;
    for (int j = 0; j < gw.G; ++j) {
        const int i = gw.idx[j];
        if (gw.joint) { num += gw.u[j] * (z[i] + zt[i]); den += z[i] * z[i] + zt[i] * zt[i]; }
        else { num += gw.u[j] * z[i]; den += z[i] * z[i]; }
    }
    return den > 0.0 ? num / den : fallback;
}

__device__ __noinline__ void assign_all(GroupWork &gw, double s, const double *z, const double *zt, const double *y) {
    if (gw.joint) for (int j = 0; j < gw.G; ++j) gw.idx[j] = joint_level(gw.u[j], s, z, zt, gw.M);
    else for (int j = 0; j < gw.G; ++j) gw.idx[j] = nearest_level(gw.u[j], y, gw.M);
}

// Score what would be stored (Section 4.1, end; Section 4.3 for the joint objective): a, b to binary16,
// s to binary32, strictly monotone curve required, assignment repeated under the rounded parameters,
// the scale re-fitted and re-rounded once, assignment repeated, loss of the stored representation.
__device__ __noinline__ Fit score_serialised(GroupWork &gw, double s, double a, double b, bool joint) {
    Fit f; f.valid = false; f.loss = INFINITY; f.s = 0.0f; f.a16 = 0; f.b16 = 0;
    const int M = gw.M;
    const uint16_t a16 = double_to_half_bits(a), b16 = double_to_half_bits(b);
    const double ar = half_bits_to_double(a16), br = half_bits_to_double(b16);
    if (!(s > 0.0) || !isfinite(s)) return f;
    if (!(shape_margin(ar, br) > 0.0)) return f;
    double z[MAXL], zt[MAXL], y[MAXL];
    for (int i = 0; i <= M; ++i) z[i] = level_curve((double)i / (double)M, ar, br);
    for (int i = 0; i < M; ++i) if (!(z[i + 1] > z[i])) return f;
    if (joint) carrier_grid(gw.B, (float)ar, (float)br, zt);
    float s32 = (float)s;
    const int keep = gw.joint;
    gw.joint = joint ? 1 : 0;
    for (int pass = 0; pass < 2; ++pass) {
        for (int i = 0; i <= M; ++i) y[i] = (double)s32 * z[i];
        assign_all(gw, (double)s32, z, zt, y);
        if (pass == 0) {
            const double s2 = fitted_scale(gw, z, zt, (double)s32);
            if (s2 > 0.0 && isfinite(s2)) s32 = (float)s2;
        }
    }
    gw.joint = keep;
    if (!(s32 > 0.0f)) return f;
    double loss = 0.0;
    for (int j = 0; j < gw.G; ++j) {
        const double d = gw.u[j] - y[gw.idx[j]];
        loss += d * d;
        if (joint) { const double d2 = gw.u[j] - (double)s32 * zt[gw.idx[j]]; loss += d2 * d2; }
        gw.cand[j] = (int8_t)(gw.w[j] < 0.0f ? -gw.idx[j] : gw.idx[j]);
    }
    f.valid = true; f.loss = loss; f.s = s32; f.a16 = a16; f.b16 = b16;
    return f;
}

__device__ __noinline__ void keep_if_better(GroupWork &gw, const Fit &f) {
    if (f.valid && f.loss < gw.best.loss) {   // strict: ties keep the earlier candidate
        gw.best = f;
        for (int j = 0; j < gw.G; ++j) gw.out[j] = gw.cand[j];
    }
}

// 3 x 3 linear system by Gaussian elimination with partial pivoting (row permutation kept in perm)
__device__ __noinline__ bool solve_3x3(double A[3][3], double r[3], double p[3]) {
    int perm[3] = {0, 1, 2};
    for (int c = 0; c < 3; ++c) {
        int piv = c;
        for (int i = c + 1; i < 3; ++i) if (fabs(A[perm[i]][c]) > fabs(A[perm[piv]][c])) piv = i;
        const int t = perm[c]; perm[c] = perm[piv]; perm[piv] = t;
        const double dd = A[perm[c]][c];
        if (fabs(dd) < 1e-300) return false;
        for (int i = c + 1; i < 3; ++i) {
            const double f = A[perm[i]][c] / dd;
            for (int j = c; j < 3; ++j) A[perm[i]][j] -= f * A[perm[c]][j];
            r[perm[i]] -= f * r[perm[c]];
        }
    }
    for (int c = 2; c >= 0; --c) {
        double acc = r[perm[c]];
        for (int j = c + 1; j < 3; ++j) acc -= A[perm[c]][j] * p[j];
        p[c] = acc / A[perm[c]][c];
    }
    return true;
}

// One candidate: from shape (a, b) and scale s0 alternate assignment and fitted scale `iters` times,
// then `refine` rounds in which, with the assignment held, the levels s (t^3 + a (t - t^3) + b (t^2 - t^3))
// (Eq. affine-cubic-level) are fitted by the 3 x 3 normal equations in (s, s a, s b); a step is kept
// only while the curve stays strictly monotone with some margin.
__device__ __noinline__ void try_candidate(GroupWork &gw, double a, double b, double s0, int iters, int refine) {
    const int M = gw.M;
    double z[MAXL], zt[MAXL], y[MAXL];
    double s = s0;
    for (int it = 0; it < iters; ++it) {
        for (int i = 0; i <= M; ++i) { z[i] = level_curve((double)i / (double)M, a, b); y[i] = s * z[i]; }
        if (gw.joint) carrier_grid(gw.B, (float)a, (float)b, zt);
        assign_all(gw, s, z, zt, y);
        s = fitted_scale(gw, z, zt, s);
    }
    for (int rf = 0; rf < refine; ++rf) {
        for (int i = 0; i <= M; ++i) { z[i] = level_curve((double)i / (double)M, a, b); y[i] = s * z[i]; }
        if (gw.joint) carrier_grid(gw.B, (float)a, (float)b, zt);
        assign_all(gw, s, z, zt, y);
        double A[3][3] = {{0.0, 0.0, 0.0}, {0.0, 0.0, 0.0}, {0.0, 0.0, 0.0}}, r[3] = {0.0, 0.0, 0.0}, p[3];
        for (int j = 0; j < gw.G; ++j) {
            const double t = (double)gw.idx[j] / (double)M, t2 = t * t, t3 = t2 * t;
            const double phi[3] = {t3, t - t3, t2 - t3};
            for (int x = 0; x < 3; ++x) {
                r[x] += phi[x] * gw.u[j];
                for (int yy = 0; yy < 3; ++yy) A[x][yy] += phi[x] * phi[yy];
            }
        }
        if (!solve_3x3(A, r, p)) break;
        if (!(p[0] > 0.0) || !isfinite(p[0])) break;
        const double an = p[1] / p[0], bn = p[2] / p[0];
        if (!isfinite(an) || !isfinite(bn) || !(shape_margin(an, bn) > 1e-3)) break;
        if (fabs(an) > 8.0 || fabs(bn) > 8.0) break;
        s = p[0]; a = an; b = bn;
    }
    keep_if_better(gw, score_serialised(gw, s, a, b, gw.joint != 0));
}

// Candidate lists of the search (a deterministic set of monotone shapes and soft clips; the
// uniform-integer point (1, 0) first).  effort 1: (1, 0) with 15 clips; 2: 11 shapes x 3 clips;
// 3: a dense shape grid x 6 clips.
__device__ __noinline__ int shape_list(int effort, double (*out)[2]) {
    int n = 0;
    out[n][0] = 1.0; out[n][1] = 0.0; ++n;
    if (effort < 2) return n;
    if (effort == 2) {
        const double as[4] = {0.4, 0.6, 0.8, 1.0}, bs[3] = {-0.6, -0.3, 0.0};
        for (int i = 0; i < 4; ++i) for (int j = 0; j < 3; ++j) {
            if (as[i] == 1.0 && bs[j] == 0.0) continue;
            if (shape_margin(as[i], bs[j]) > 0.02) { out[n][0] = as[i]; out[n][1] = bs[j]; ++n; }
        }
        return n;
    }
    for (int i = 2; i <= 12; ++i) for (int j = -10; j <= 2; ++j) {
        const double a = 0.1 * i, b = 0.1 * j;
        if (i == 10 && j == 0) continue;
        if (shape_margin(a, b) > 0.02) { out[n][0] = a; out[n][1] = b; ++n; }
    }
    return n;
}

__device__ __noinline__ void search_group(GroupWork &gw, int effort, float *s_out, uint16_t *a_out, uint16_t *b_out) {
    const uint16_t ONE16 = 0x3C00;
    const int G = gw.G, B = gw.B;
    double umax = 0.0, usum = 0.0;
    for (int j = 0; j < G; ++j) { gw.u[j] = fabs((double)gw.w[j]); usum += gw.u[j]; if (gw.u[j] > umax) umax = gw.u[j]; }
    *a_out = ONE16; *b_out = 0;
    if (umax == 0.0) {   // all-zero group: s = 0, codes 0 (W1: +1)
        *s_out = 0.0f;
        for (int j = 0; j < G; ++j) gw.out[j] = (int8_t)(B == 1 ? 1 : 0);
        return;
    }
    if (B == 1) {        // sign codes; s = mean |w| minimises sum (w - k s)^2
        *s_out = (float)(usum / G);
        for (int j = 0; j < G; ++j) gw.out[j] = (int8_t)(gw.w[j] >= 0.0f ? 1 : -1);
        return;
    }
    gw.best.valid = false; gw.best.loss = INFINITY; gw.best.s = 0.0f; gw.best.a16 = ONE16; gw.best.b16 = 0;
    const float s_abs = (float)umax;
    if (effort == 0) {   // symmetric absmax integer quantisation
        double y[MAXL];
        for (int i = 0; i <= gw.M; ++i) y[i] = (double)s_abs * level_curve((double)i / (double)gw.M, 1.0, 0.0);
        for (int j = 0; j < G; ++j) {
            const int i = nearest_level(gw.u[j], y, gw.M);
            gw.out[j] = (int8_t)(gw.w[j] < 0.0f ? -i : i);
        }
        *s_out = s_abs;
        return;
    }
    double shapes[200][2];
    int ns = (B == 2) ? 1 : shape_list(effort, shapes);   // W2: the shape is not identifiable
    if (B == 2) { shapes[0][0] = 1.0; shapes[0][1] = 0.0; }
    const double clips_fast[3] = {1.0, 0.85, 0.7};
    const double clips_ref[6] = {1.0, 0.9, 0.8, 0.7, 0.6, 0.5};
    const double clips_int[15] = {1.0, 0.95, 0.9, 0.85, 0.8, 0.75, 0.7, 0.65, 0.6, 0.55, 0.5, 0.45, 0.4, 0.35, 0.3};
    const double *clips; int nc, iters, refine;
    if (effort == 1) { clips = clips_int; nc = 15; iters = 6; refine = 0; }
    else if (effort == 2) { clips = clips_fast; nc = 3; iters = 3; refine = 8; }
    else { clips = clips_ref; nc = 6; iters = 4; refine = 12; }
    if (B == 2) refine = 0;
    // the clipped uniform-integer candidates always compete first: never worse than clipped INT
    if (effort >= 2)
        for (int ci = 0; ci < 15; ++ci) try_candidate(gw, 1.0, 0.0, clips_int[ci] * umax, 6, 0);
    for (int si = 0; si < ns; ++si)
        for (int ci = 0; ci < nc; ++ci) try_candidate(gw, shapes[si][0], shapes[si][1], clips[ci] * umax, iters, refine);
    if (!gw.best.valid) {
        double y[MAXL];
        for (int i = 0; i <= gw.M; ++i) y[i] = (double)s_abs * level_curve((double)i / (double)gw.M, 1.0, 0.0);
        for (int j = 0; j < G; ++j) {
            const int i = nearest_level(gw.u[j], y, gw.M);
            gw.out[j] = (int8_t)(gw.w[j] < 0.0f ? -i : i);
        }
        *s_out = s_abs;
        return;
    }
    *s_out = gw.best.s; *a_out = gw.best.a16; *b_out = gw.best.b16;
}

__global__ void __launch_bounds__(32) search_kernel(const float *__restrict__ W, int B, int G, int64_t N, int64_t K, int joint,
                                                    int effort, int8_t *__restrict__ k, float *__restrict__ scale,
                                                    uint16_t *__restrict__ a, uint16_t *__restrict__ b) {
    const int64_t ng = K / G, gi = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (gi >= N * ng) return;
    const int64_t n = gi / ng, g = gi % ng;
    GroupWork gw;
    gw.w = W + n * K + g * G;
    gw.G = G; gw.B = B; gw.M = B == 1 ? 1 : top_code(B);
    gw.out = k + n * K + g * G;
    const bool dual = joint && B > 2;   // W1 / W2 levels lie on the carrier grid: the objectives coincide
    gw.joint = 0;
    float s0; uint16_t a0, b0;
    if (!dual) {
        search_group(gw, effort, &s0, &a0, &b0);
    } else {
        // The continuous fitter's answer competes too, re-scored under the joint objective, so the dual-path
        // result is never worse (jointly) than the continuous-only one.  It is found first (it uses the
        // output codes as scratch), then the joint search runs, then the two are compared.
        float sc; uint16_t ac, bc;
        search_group(gw, effort, &sc, &ac, &bc);
        const bool have_c = effort >= 1 && gw.best.valid;
        gw.joint = 1;
        search_group(gw, effort, &s0, &a0, &b0);
        if (have_c && effort >= 1) {
            const Fit f = score_serialised(gw, (double)sc, half_bits_to_double(ac), half_bits_to_double(bc), true);
            if (f.valid && f.loss < gw.best.loss) {
                gw.best = f;
                for (int j = 0; j < G; ++j) gw.out[j] = gw.cand[j];
                s0 = f.s; a0 = f.a16; b0 = f.b16;
            }
        }
    }
    scale[gi] = s0; a[gi] = a0; b[gi] = b0;
}

}  // namespace

cudaError_t launch_encode_assign(const float *W, int B, int G, int64_t N, int64_t K, const float *scale, const uint16_t *a,
                                 const uint16_t *b, int joint, int8_t *k, cudaStream_t st) {
    const int64_t ng = K / G;
    assign_kernel<<<(unsigned)(N * ng), 128, 0, st>>>(W, B, G, K, ng, scale, a, b, joint && B > 2, k);
    return cudaGetLastError();
}
cudaError_t launch_encode_scale(const float *W, const int8_t *k, int B, int G, int64_t N, int64_t K, const uint16_t *a,
                                const uint16_t *b, int joint, float *scale, cudaStream_t st) {
    const int64_t ng = K / G;
    scale_kernel<<<(unsigned)(N * ng), 128, 0, st>>>(W, k, B, G, K, ng, a, b, joint && B > 2, scale);
    return cudaGetLastError();
}
cudaError_t launch_encode_losses(const float *W, const int8_t *k, int B, int G, int64_t N, int64_t K, const float *scale,
                                 const uint16_t *a, const uint16_t *b, double *LC, double *LA8, cudaStream_t st) {
    const int64_t ng = K / G;
    losses_kernel<<<(unsigned)(N * ng), 128, 0, st>>>(W, k, B, G, K, ng, scale, a, b, LC, LA8);
    return cudaGetLastError();
}
cudaError_t launch_encode_search(const float *W, int B, int G, int64_t N, int64_t K, int joint, int effort, int8_t *k,
                                 float *scale, uint16_t *a, uint16_t *b, cudaStream_t st) {
    const int64_t groups = N * (K / G);
    static std::atomic<uint64_t> attr_done{0};   // the per-thread work arrays live in local memory: prefer L1 over shared memory
    (void)ensure_func_attr(search_kernel, attr_done, cudaFuncAttributePreferredSharedMemoryCarveout, 0);
    search_kernel<<<(unsigned)((groups + 31) / 32), 32, 0, st>>>(W, B, G, N, K, joint, effort, k, scale, a, b);
    return cudaGetLastError();
}

}  // namespace cq
