/*
 * CubicQuant CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, step-by-step restatement of what the packed GEMV/GEMM path
 * computes, written from the paper's definitions.  It shares no code with the
 * CUDA library and is only ever used by tests, by the smoke check and by the
 * CPU-baseline leg of the benchmark.
 *
 * Arithmetic is fp64 unless a bit-exact contract pins an fp32 sequence
 * (Dynamic-A8 weight carriers and activation quantiser; compile with
 * -ffp-contract=off so the sequence below is what runs).
 *
 * Every function names the passage of the paper it follows.
 *
 * Pins (tests/test_oracle_*.py): uniform-INT special case, endpoint
 * identities, m(a,b) against a brute-force minimum, population distortion
 * tables and closed forms (python side), brute-force nearest level and
 * least-squares scale on tiny groups, storage size, A8 identities; for the
 * carrier-aware objective of Section 4.3: enumeration of every code vector, the
 * joint decision boundaries, stationarity of the joint loss in s, the W1 / W2 and
 * integer-grid cases where the carrier projection is the identity.
 * Parity unpinned: the *search* inside cqo_encode / cqo_encode_joint (candidate list, clip list,
 * iteration counts are this file's reading; several (codes, params) outputs are
 * valid for one input).  Its building blocks (assignment, scale) are pinned, and
 * its result is checked against invariants (never worse than clipped INT, never
 * emits the reserved pattern, serialised curves strictly monotone).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define CQO_API __attribute__((visibility("default")))

/* ------------------------------------------------------------------ number formats */

/* IEEE binary16 bits -> double (exact). */
static double half_to_double(uint16_t h) {
    int sign = (h >> 15) & 1, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(m + 1024), e - 25);
    return sign ? -v : v;
}

/* double -> IEEE binary16 bits, round to nearest even. */
static uint16_t double_to_half(double d) {
    uint16_t sign = signbit(d) ? 0x8000u : 0;
    double a = fabs(d);
    if (isnan(a)) return (uint16_t)(sign | 0x7E00u);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7C00u);
    if (a < ldexp(1.0, -25)) return sign; /* below half of the smallest subnormal (ties to even -> 0) */
    int e;
    (void)frexp(a, &e); /* a = f * 2^e, f in [0.5,1) */
    int ue = e - 1;     /* a in [2^ue, 2^(ue+1)) */
    if (ue < -14) ue = -14;
    double scaled = ldexp(a, 10 - ue); /* mantissa units */
    double r = nearbyint(scaled);      /* default rounding mode: to nearest even */
    int mant = (int)r;
    int be = ue + 15;
    if (ue == -14 && mant < 1024) return (uint16_t)(sign | mant); /* subnormal */
    if (mant == 2048) { mant = 1024; be += 1; }
    if (be >= 31) return (uint16_t)(sign | 0x7C00u);
    return (uint16_t)(sign | (be << 10) | (mant - 1024));
}

static double bf16_to_double(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* An activation's value from its 16-bit pattern: the model dtype is bfloat16 or binary16 (Section 5.3:
 * the model-dtype path accepts FP16 or BF16 activations); both promote to double exactly. */
static double act_to_double(uint16_t bits, int act_f16) { return act_f16 ? half_to_double(bits) : bf16_to_double(bits); }

CQO_API double cqo_half_to_double(uint16_t h) { return half_to_double(h); }
CQO_API uint16_t cqo_double_to_half(double d) { return double_to_half(d); }

CQO_API int cqo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ format (Section 2) */

/* Largest magnitude code M = 2^(B-1) - 1 (Eq. codes).  B = 1 is the binary case. */
static int max_code(int B) { return (1 << (B - 1)) - 1; }

/* Number of stored non-negative levels: M + 1 = 2^(B-1) for B > 1; one (the scale) for W1. */
CQO_API int cqo_num_levels(int B) { return B == 1 ? 1 : (1 << (B - 1)); }

/* Packed bytes of the whole matrix, T_W = N K (B/8 + 8/G) (Eq. cubic-weight-bytes). */
CQO_API double cqo_storage_bytes(int64_t N, int64_t K, int B, int G) {
    return (double)N * (double)K * ((double)B / 8.0 + 8.0 / (double)G);
}

/* Bytes of one packed row: rows start byte aligned, ceil(K B / 8) bytes each. */
CQO_API int64_t cqo_row_bytes(int64_t K, int B) { return (K * B + 7) / 8; }

/* Monotonicity margin m(a,b) = min over [0,1] of q'(t) = a + 2 b t + 3 c t^2 (Eq. shape-domain). */
CQO_API double cqo_shape_margin(double a, double b) {
    double c = 1.0 - a - b;
    double m = fmin(a, 3.0 - 2.0 * a - b);
    if (c > 0.0 && b < 0.0 && b > -3.0 * c) m = fmin(m, a - b * b / (3.0 * c));
    return m;
}

/* Normalised level curve q(t) = t [a + t (b + c t)], c = 1 - a - b (Eq. cubic). */
static double curve(double t, double a, double b) {
    double c = 1.0 - a - b;
    return t * (a + t * (b + t * c));
}

/* Non-negative reconstruction levels of one group (Appendix B):
 * B = 1 -> {s};  B > 1 -> level_i = s q(i/M), i = 0..M.  a and b are binary16 bit patterns. */
CQO_API void cqo_levels(int B, float s, uint16_t a16, uint16_t b16, double *levels) {
    if (B == 1) { levels[0] = (double)s; return; }
    int M = max_code(B);
    double a = half_to_double(a16), b = half_to_double(b16);
    for (int i = 0; i <= M; ++i) {
        double t = (double)i / (double)M;
        levels[i] = (double)s * curve(t, a, b);
    }
}

/* Dynamic-A8 weight carriers r = RNE(127 q(i/M)) for the non-negative magnitudes
 * (Eq. carrier, Appendix A item 7).  The paper leaves the precision of 127 q open; the
 * reading pinned here is this fp32 sequence (Horner as in Eq. gpu-horner):
 *   t = (float)i / (float)M;  c = (1 - a) - b;  q = t * fma(t, fma(t, c, b), a);
 *   r = rint(127 * q) clamped to [0, 127].
 * W1 and W2 have only the levels {0, 1} on the normalised axis, which sit on the
 * carrier grid (Section 4.3, last paragraph): r in {0, 127} whatever (a, b). */
CQO_API void cqo_carriers(int B, uint16_t a16, uint16_t b16, int8_t *r) {
    if (B == 1) { r[0] = 127; return; }
    if (B == 2) { r[0] = 0; r[1] = 127; return; }
    int M = max_code(B);
    float a = (float)half_to_double(a16), b = (float)half_to_double(b16);
    float c = (1.0f - a) - b;
    for (int i = 0; i <= M; ++i) {
        float t = (float)i / (float)M;
        float inner = fmaf(t, c, b);
        float mid = fmaf(t, inner, a);
        float q = t * mid;
        float v = rintf(127.0f * q);
        int iv = (int)v;
        if (iv < 0) iv = 0;
        if (iv > 127) iv = 127;
        r[i] = (int8_t)iv;
    }
}

/* Signed codes -> packed bytes.  Continuous bitstream in row-major order, field j of a row
 * at bit offset j B, least significant bit first inside and across bytes (the order that
 * Eq. gpu-packed-extraction reads back); B-bit two's complement for B > 1; W1 stores one
 * bit, 1 for +1 and 0 for -1.  Rows start on a byte; pad bits of the last byte are zero. */
CQO_API void cqo_pack(const int8_t *k, int64_t N, int64_t K, int B, uint8_t *out) {
    int64_t rb = cqo_row_bytes(K, B);
    memset(out, 0, (size_t)(N * rb));
    for (int64_t n = 0; n < N; ++n) {
        uint8_t *row = out + n * rb;
        for (int64_t j = 0; j < K; ++j) {
            int code = k[n * K + j];
            unsigned field = (B == 1) ? (code > 0 ? 1u : 0u) : ((unsigned)code & ((1u << B) - 1u));
            for (int bit = 0; bit < B; ++bit) {
                int64_t pos = j * B + bit;
                if ((field >> bit) & 1u) row[pos >> 3] |= (uint8_t)(1u << (pos & 7));
            }
        }
    }
}

/* Packed bytes -> signed codes, by Eq. gpu-packed-extraction:
 *   p = floor(j B / 8), d = (j B) mod 8, u = ((byte[p] >> d) | (byte[p+1] << (8 - d))) & (2^B - 1),
 * then sign extension.  The reserved pattern comes back as -2^(B-1); W1 bits as +-1. */
CQO_API void cqo_unpack(const uint8_t *codes, int64_t N, int64_t K, int B, int8_t *k) {
    int64_t rb = cqo_row_bytes(K, B);
    for (int64_t n = 0; n < N; ++n) {
        const uint8_t *row = codes + n * rb;
        for (int64_t j = 0; j < K; ++j) {
            int64_t p = (j * B) >> 3;
            int d = (int)((j * B) & 7);
            unsigned lo = row[p];
            unsigned hi = (d + B > 8) ? row[p + 1] : 0u;
            unsigned u = ((lo >> d) | (hi << (8 - d))) & ((1u << B) - 1u);
            int v;
            if (B == 1) v = u ? 1 : -1;
            else v = (u & (1u << (B - 1))) ? (int)u - (1 << B) : (int)u;
            k[n * K + j] = (int8_t)v;
        }
    }
}

/* Reconstruction of one signed code from its group's levels (Appendix B `decode`;
 * Section 2.1: the reserved most-negative pattern decodes to zero). */
static double decode_code(int B, int code, const double *levels) {
    if (B == 1) return code > 0 ? levels[0] : -levels[0];
    if (code == -(1 << (B - 1))) return 0.0;
    int mag = code < 0 ? -code : code;
    double v = levels[mag];
    return code < 0 ? -v : v;
}

/* Dense reconstruction  What[n][k]  (fp64) of a packed matrix. */
CQO_API void cqo_decode_dense(const uint8_t *codes, const float *s, const uint16_t *a, const uint16_t *b,
                              int B, int G, int64_t N, int64_t K, double *What) {
    int64_t ng = K / G;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        int8_t *kk = (int8_t *)malloc((size_t)K);
        double lev[128];
        cqo_unpack(codes + n * cqo_row_bytes(K, B), 1, K, B, kk);
        for (int64_t g = 0; g < ng; ++g) {
            cqo_levels(B, s[n * ng + g], a[n * ng + g], b[n * ng + g], lev);
            for (int j = 0; j < G; ++j) What[n * K + g * G + j] = decode_code(B, kk[g * G + j], lev);
        }
        free(kk);
    }
}

/* ------------------------------------------------------------------ encoder (Section 4.1) */

/* Nearest-level magnitude index for u >= 0 among increasing levels y_0..y_M, values beyond
 * y_M saturating at M (Section 4.1).  Ties go to the lower index (this file's reading). */
static int nearest_index(double u, const double *y, int M) {
    int lo = 0, hi = M; /* smallest i with u <= (y_i + y_{i+1})/2, else M */
    while (lo < hi) {
        int mid = (lo + hi) >> 1;
        if (u <= 0.5 * (y[mid] + y[mid + 1])) hi = mid; else lo = mid + 1;
    }
    return lo;
}

/* Codes of one group for fixed serialised parameters: nearest reconstruction of each weight.
 * Never produces the reserved pattern; a magnitude index 0 is code 0; W1: sign only (w >= 0 -> +1). */
CQO_API void cqo_assign_group(const float *w, int G, int B, float s, uint16_t a16, uint16_t b16, int8_t *k) {
    if (B == 1) { for (int j = 0; j < G; ++j) k[j] = (int8_t)(w[j] >= 0.0f ? 1 : -1); return; }
    int M = max_code(B);
    double lev[128];
    cqo_levels(B, s, a16, b16, lev);
    for (int j = 0; j < G; ++j) {
        double u = fabs((double)w[j]);
        int i = nearest_index(u, lev, M);
        k[j] = (int8_t)(w[j] < 0.0f ? -i : i);
    }
}

/* Squared reconstruction error of one group, the summand of Eq. offline-objective. */
CQO_API double cqo_group_sse(const float *w, int G, int B, float s, uint16_t a16, uint16_t b16, const int8_t *k) {
    double lev[128], sse = 0.0;
    cqo_levels(B, s, a16, b16, lev);
    for (int j = 0; j < G; ++j) {
        double d = (double)w[j] - decode_code(B, k[j], lev);
        sse += d * d;
    }
    return sse;
}

/* ------------------------------------------------------------------ carrier-aware fitting (Section 4.3) */

/* Carrier-grid levels of a shape given in fp32: ztilde_i = r_i / 127 with r_i by the pinned
 * sequence of cqo_carriers (Eq. carrier-grid).  W2: {0, 1}. */
static void carrier_grid(int B, float a, float b, double *zt) {
    int M = max_code(B);
    if (B == 2) { zt[0] = 0.0; zt[1] = 1.0; return; }
    float c = (1.0f - a) - b;
    for (int i = 0; i <= M; ++i) {
        float t = (float)i / (float)M;
        float q = t * fmaf(t, fmaf(t, c, b), a);
        int iv = (int)rintf(127.0f * q);
        if (iv < 0) iv = 0;
        if (iv > 127) iv = 127;
        zt[i] = (double)iv / 127.0;
    }
}

/* Normalised continuous levels z_i = q(i/M) and carrier-grid levels ztilde_i = round(127 z_i)/127
 * of a serialised shape (Eq. carrier-grid; z in fp64, the rounding by the pinned carrier sequence). */
CQO_API void cqo_joint_levels(int B, uint16_t a16, uint16_t b16, double *z, double *zt) {
    int M = max_code(B);
    double a = half_to_double(a16), b = half_to_double(b16);
    for (int i = 0; i <= M; ++i) z[i] = curve((double)i / (double)M, a, b);
    carrier_grid(B, (float)a, (float)b, zt);
}

/* Magnitude index minimising (u - s z_i)^2 + (u - s ztilde_i)^2 over i = 0..M
 * (Eq. carrier-aware-assignment), by plain scan; ties go to the lower index. */
static int joint_index(double u, double s, const double *z, const double *zt, int M) {
    int best = 0;
    double bc = INFINITY;
    for (int i = 0; i <= M; ++i) {
        double d1 = u - s * z[i], d2 = u - s * zt[i];
        double cst = d1 * d1 + d2 * d2;
        if (cst < bc) { bc = cst; best = i; }
    }
    return best;
}

/* Codes of one group for fixed serialised parameters under the joint objective
 * (Eq. carrier-aware-assignment).  W1: sign only. */
CQO_API void cqo_assign_group_joint(const float *w, int G, int B, float s, uint16_t a16, uint16_t b16, int8_t *k) {
    if (B == 1) { for (int j = 0; j < G; ++j) k[j] = (int8_t)(w[j] >= 0.0f ? 1 : -1); return; }
    int M = max_code(B);
    double z[128], zt[128];
    cqo_joint_levels(B, a16, b16, z, zt);
    for (int j = 0; j < G; ++j) {
        int i = joint_index(fabs((double)w[j]), (double)s, z, zt, M);
        k[j] = (int8_t)(w[j] < 0.0f ? -i : i);
    }
}

/* The two groupwise squared errors of Eq. continuous-and-carrier-loss for stored codes:
 * L_C against s q(t_k) and L_A8 against (s / 127) r(k). */
CQO_API void cqo_group_losses(const float *w, int G, int B, float s, uint16_t a16, uint16_t b16, const int8_t *k,
                              double *LC, double *LA8) {
    double lc = 0.0, la = 0.0;
    if (B == 1) {
        for (int j = 0; j < G; ++j) { double d = (double)w[j] - (k[j] > 0 ? 1.0 : -1.0) * (double)s; lc += d * d; }
        *LC = lc; *LA8 = lc; return;
    }
    double z[128], zt[128];
    cqo_joint_levels(B, a16, b16, z, zt);
    for (int j = 0; j < G; ++j) {
        int kk = k[j], i = kk < 0 ? -kk : kk;
        double sg = kk < 0 ? -1.0 : 1.0;
        if (kk == -(1 << (B - 1))) { i = 0; } /* reserved pattern decodes to zero */
        double d1 = (double)w[j] - sg * (double)s * z[i], d2 = (double)w[j] - sg * (double)s * zt[i];
        lc += d1 * d1; la += d2 * d2;
    }
    *LC = lc; *LA8 = la;
}

/* Shared scale minimising L_C + L_A8 for fixed codes and shape (Eq. carrier-aware-scale):
 * s* = sum u_j (z_j + ztilde_j) / sum (z_j^2 + ztilde_j^2); 0 when the denominator vanishes. */
CQO_API double cqo_joint_scale(const float *w, const int8_t *k, int G, int B, uint16_t a16, uint16_t b16) {
    if (B == 1) { double su = 0.0; for (int j = 0; j < G; ++j) su += fabs((double)w[j]); return su / G; }
    double z[128], zt[128], num = 0.0, den = 0.0;
    cqo_joint_levels(B, a16, b16, z, zt);
    for (int j = 0; j < G; ++j) {
        int kk = k[j], i = kk < 0 ? -kk : kk;
        if (kk == -(1 << (B - 1))) i = 0;
        double u = fabs((double)w[j]);
        num += u * (z[i] + zt[i]);
        den += z[i] * z[i] + zt[i] * zt[i];
    }
    return den > 0.0 ? num / den : 0.0;
}

static double joint_ls_scale(const double *u, const int *idx, int G, const double *z, const double *zt, double fallback) {
    double num = 0.0, den = 0.0;
    for (int j = 0; j < G; ++j) { int i = idx[j]; num += u[j] * (z[i] + zt[i]); den += z[i] * z[i] + zt[i] * zt[i]; }
    return den > 0.0 ? num / den : fallback;
}

/* Least-squares scale for fixed magnitude indices and shape:  s = sum u_j z_j / sum z_j^2
 * with z_j = q(t_{i_j})  (the continuous-only analogue of Eq. carrier-aware-scale). */
static double ls_scale(const double *u, const int *idx, int G, const double *z, double fallback) {
    double num = 0.0, den = 0.0;
    for (int j = 0; j < G; ++j) { double zz = z[idx[j]]; num += u[j] * zz; den += zz * zz; }
    return den > 0.0 ? num / den : fallback;
}

/* Solve the 3x3 system A p = r by Gaussian elimination with partial pivoting; 0 on success. */
static int solve3(double A[3][3], double r[3], double p[3]) {
    int perm[3] = {0, 1, 2};
    for (int c = 0; c < 3; ++c) {
        int piv = c;
        for (int i = c + 1; i < 3; ++i) if (fabs(A[perm[i]][c]) > fabs(A[perm[piv]][c])) piv = i;
        int t = perm[c]; perm[c] = perm[piv]; perm[piv] = t;
        double d = A[perm[c]][c];
        if (fabs(d) < 1e-300) return 1;
        for (int i = c + 1; i < 3; ++i) {
            double f = A[perm[i]][c] / d;
            for (int j = c; j < 3; ++j) A[perm[i]][j] -= f * A[perm[c]][j];
            r[perm[i]] -= f * r[perm[c]];
        }
    }
    for (int c = 2; c >= 0; --c) {
        double acc = r[perm[c]];
        for (int j = c + 1; j < 3; ++j) acc -= A[perm[c]][j] * p[j];
        p[c] = acc / A[perm[c]][c];
    }
    return 0;
}

typedef struct {
    double sse;
    float s;
    uint16_t a16, b16;
    int valid;
} fit_t;

/* Evaluate a serialised candidate (Section 4.1, last sentences): map a, b to binary16 and
 * s to binary32, require a strictly monotone curve (Eq. monotonicity, and strictly
 * increasing discrete levels), repeat the assignment under the rounded parameters,
 * re-fit and re-round the scale once, and return the squared error of what is stored. */
static fit_t serialise_and_score(const float *w, const double *u, int G, int B, double s, double a, double b,
                                 int8_t *kbuf, int joint) {
    fit_t f; f.valid = 0; f.sse = INFINITY; f.s = 0; f.a16 = 0; f.b16 = 0;
    int M = max_code(B);
    uint16_t a16 = double_to_half(a), b16 = double_to_half(b);
    double ar = half_to_double(a16), br = half_to_double(b16);
    if (!(s > 0.0) || !isfinite(s)) return f;
    if (!(cqo_shape_margin(ar, br) > 0.0)) return f;
    double z[128], zt[128];
    for (int i = 0; i <= M; ++i) z[i] = curve((double)i / (double)M, ar, br);
    for (int i = 0; i < M; ++i) if (!(z[i + 1] > z[i])) return f;
    if (joint) carrier_grid(B, (float)ar, (float)br, zt);
    int idx[512];
    double y[128];
    float s32 = (float)s;
    for (int pass = 0; pass < 2; ++pass) {
        for (int i = 0; i <= M; ++i) y[i] = (double)s32 * z[i];
        if (joint) for (int j = 0; j < G; ++j) idx[j] = joint_index(u[j], (double)s32, z, zt, M);
        else for (int j = 0; j < G; ++j) idx[j] = nearest_index(u[j], y, M);
        if (pass == 0) {
            double s2 = joint ? joint_ls_scale(u, idx, G, z, zt, (double)s32) : ls_scale(u, idx, G, z, (double)s32);
            if (s2 > 0.0 && isfinite(s2)) s32 = (float)s2;
        }
    }
    if (!(s32 > 0.0f)) return f;
    double sse = 0.0;
    for (int j = 0; j < G; ++j) {
        double d = u[j] - y[idx[j]];
        sse += d * d;
        if (joint) { double d2 = u[j] - (double)s32 * zt[idx[j]]; sse += d2 * d2; }  /* L_C + L_A8 */
        kbuf[j] = (int8_t)(w[j] < 0.0f ? -idx[j] : idx[j]);
    }
    f.valid = 1; f.sse = sse; f.s = s32; f.a16 = a16; f.b16 = b16;
    return f;
}

/* One candidate of the search: start from shape (a, b) and scale s0, alternate nearest-level
 * assignment and least-squares scale `iters` times, then `refine` rounds of the joint
 * refinement.  The refinement uses Eq. affine-cubic-level: with the assignment held fixed the
 * levels s (r_i + a u_i + b v_i), r_i = t^3, u_i = t - t^3, v_i = t^2 - t^3, are linear in
 * (s, s a, s b), so the squared error is minimised by 3x3 normal equations; a step is kept
 * only while the curve stays strictly monotone (m(a, b) > margin). */
static void run_candidate(const float *w, const double *u, int G, int B, double a, double b, double s0,
                          int iters, int refine, fit_t *best, int8_t *kbest, int8_t *kbuf, int joint) {
    int M = max_code(B);
    double z[128], y[128], zt[128];
    int idx[512];
    double s = s0;
    /* joint objective (Section 4.3): the same candidates and the same refinement proposals, but the
     * assignment is Eq. carrier-aware-assignment, the scale Eq. carrier-aware-scale, and the score
     * L_C + L_A8; the carrier grid of an unserialised shape is taken from its fp32 value */
    for (int it = 0; it < iters; ++it) {
        for (int i = 0; i <= M; ++i) { z[i] = curve((double)i / (double)M, a, b); y[i] = s * z[i]; }
        if (joint) {
            carrier_grid(B, (float)a, (float)b, zt);
            for (int j = 0; j < G; ++j) idx[j] = joint_index(u[j], s, z, zt, M);
            s = joint_ls_scale(u, idx, G, z, zt, s);
        } else {
            for (int j = 0; j < G; ++j) idx[j] = nearest_index(u[j], y, M);
            s = ls_scale(u, idx, G, z, s);
        }
    }
    for (int rf = 0; rf < refine; ++rf) {
        for (int i = 0; i <= M; ++i) { z[i] = curve((double)i / (double)M, a, b); y[i] = s * z[i]; }
        if (joint) {
            carrier_grid(B, (float)a, (float)b, zt);
            for (int j = 0; j < G; ++j) idx[j] = joint_index(u[j], s, z, zt, M);
        } else {
            for (int j = 0; j < G; ++j) idx[j] = nearest_index(u[j], y, M);
        }
        double A[3][3] = {{0}}, r[3] = {0}, p[3];
        for (int j = 0; j < G; ++j) {
            double t = (double)idx[j] / (double)M, t2 = t * t, t3 = t2 * t;
            double phi[3] = {t3, t - t3, t2 - t3};
            for (int x = 0; x < 3; ++x) {
                r[x] += phi[x] * u[j];
                for (int yy = 0; yy < 3; ++yy) A[x][yy] += phi[x] * phi[yy];
            }
        }
        if (solve3(A, r, p)) break;
        if (!(p[0] > 0.0) || !isfinite(p[0])) break;
        double an = p[1] / p[0], bn = p[2] / p[0];
        if (!isfinite(an) || !isfinite(bn) || !(cqo_shape_margin(an, bn) > 1e-3)) break;
        if (fabs(an) > 8.0 || fabs(bn) > 8.0) break;
        s = p[0]; a = an; b = bn;
    }
    fit_t f = serialise_and_score(w, u, G, B, s, a, b, kbuf, joint);
    if (f.valid && f.sse < best->sse) { /* strict: ties keep the earlier candidate */
        *best = f;
        memcpy(kbest, kbuf, (size_t)G);
    }
}

/* Candidate lists (this file's reading of "a deterministic set of monotonic (a,b) candidates"
 * and "jointly refines scale and clipping").  The uniform-integer point (1, 0) is always first. */
static int build_shapes(int effort, double (*out)[2]) {
    int n = 0;
    out[n][0] = 1.0; out[n][1] = 0.0; ++n;
    if (effort < 2) return n;
    if (effort == 2) {
        const double as[] = {0.4, 0.6, 0.8, 1.0}, bs[] = {-0.6, -0.3, 0.0};
        for (int i = 0; i < 4; ++i) for (int j = 0; j < 3; ++j) {
            if (as[i] == 1.0 && bs[j] == 0.0) continue;
            if (cqo_shape_margin(as[i], bs[j]) > 0.02) { out[n][0] = as[i]; out[n][1] = bs[j]; ++n; }
        }
        return n;
    }
    for (int i = 2; i <= 12; ++i) for (int j = -10; j <= 2; ++j) { /* a = 0.2..1.2, b = -1.0..0.2 */
        double a = 0.1 * i, b = 0.1 * j;
        if (i == 10 && j == 0) continue;
        if (cqo_shape_margin(a, b) > 0.02) { out[n][0] = a; out[n][1] = b; ++n; }
    }
    return n;
}

/* Encoder effort levels:
 *   0  uniform-integer point only, scale = max|w| (textbook symmetric absmax INT; a pin)
 *   1  uniform-integer point only, clipping scale optimised (the "clipped INT" baseline)
 *   2  fast: the candidates of 1, then 12 shapes x 3 clips, 3 assignment/scale rounds, 8 refinement rounds
 *   3  reference: the candidates of 1, then a dense shape grid x 6 clips, 4 assignment/scale rounds,
 *      12 refinement rounds */
static void encode_group(const float *w, int G, int B, int effort, int joint, int8_t *k, float *s_out, uint16_t *a_out,
                         uint16_t *b_out) {
    const uint16_t ONE16 = 0x3C00;
    double u[512], umax = 0.0, usum = 0.0;
    for (int j = 0; j < G; ++j) { u[j] = fabs((double)w[j]); usum += u[j]; if (u[j] > umax) umax = u[j]; }
    *a_out = ONE16; *b_out = 0;
    if (umax == 0.0) { /* all-zero group: s = 0, codes 0 (W1: +1) */
        *s_out = 0.0f;
        for (int j = 0; j < G; ++j) k[j] = (int8_t)(B == 1 ? 1 : 0);
        return;
    }
    if (B == 1) { /* W1: sign codes; s = mean |w| minimises sum (w - k s)^2 */
        *s_out = (float)(usum / G);
        for (int j = 0; j < G; ++j) k[j] = (int8_t)(w[j] >= 0.0f ? 1 : -1);
        return;
    }
    int8_t kbuf[512];
    fit_t best; best.valid = 0; best.sse = INFINITY; best.s = 0; best.a16 = ONE16; best.b16 = 0;
    if (effort == 0) { /* textbook symmetric absmax INT: s = max|w|, nearest level on the linear grid */
        float s32 = (float)umax;
        cqo_assign_group(w, G, B, s32, ONE16, 0, k);
        *s_out = s32;
        return;
    }
    double shapes[200][2];
    int ns = (B == 2) ? 1 : build_shapes(effort, shapes); /* W2: shape not identifiable -> (1, 0) only */
    if (B == 2) { shapes[0][0] = 1.0; shapes[0][1] = 0.0; }
    const double clips_fast[] = {1.0, 0.85, 0.7};
    const double clips_ref[] = {1.0, 0.9, 0.8, 0.7, 0.6, 0.5};
    const double clips_int[] = {1.0, 0.95, 0.9, 0.85, 0.8, 0.75, 0.7, 0.65, 0.6, 0.55, 0.5, 0.45, 0.4, 0.35, 0.3};
    const double *clips; int nc, iters, refine;
    if (effort == 1) { clips = clips_int; nc = 15; iters = 6; refine = 0; }
    else if (effort == 2) { clips = clips_fast; nc = 3; iters = 3; refine = 8; }
    else { clips = clips_ref; nc = 6; iters = 4; refine = 12; }
    if (B == 2) refine = 0;
    /* the optimally clipped uniform-integer candidates always compete first, so the result is never
     * worse than clipped INT under the same objective (Section 2.2, after Eq. int-special-case) */
    if (effort >= 2)
        for (int ci = 0; ci < 15; ++ci)
            run_candidate(w, u, G, B, 1.0, 0.0, clips_int[ci] * umax, 6, 0, &best, k, kbuf, joint);
    for (int si = 0; si < ns; ++si)
        for (int ci = 0; ci < nc; ++ci)
            run_candidate(w, u, G, B, shapes[si][0], shapes[si][1], clips[ci] * umax, iters, refine, &best, k, kbuf, joint);
    if (joint && effort >= 1 && B > 2) {
        /* the continuous fitter's own answer also competes, re-scored under the joint objective, so the
         * carrier-aware result is never worse (jointly) than the continuous-only one */
        int8_t kc[512]; float sc; uint16_t ac, bc;
        encode_group(w, G, B, effort, 0, kc, &sc, &ac, &bc);
        fit_t f = serialise_and_score(w, u, G, B, (double)sc, half_to_double(ac), half_to_double(bc), kbuf, 1);
        if (f.valid && f.sse < best.sse) { best = f; memcpy(k, kbuf, (size_t)G); }
    }
    if (!best.valid) { /* cannot happen for finite input; keep absmax INT */
        float s32 = (float)umax;
        cqo_assign_group(w, G, B, s32, ONE16, 0, k);
        *s_out = s32;
        return;
    }
    *s_out = best.s; *a_out = best.a16; *b_out = best.b16;
}

/* Groupwise encoder of a whole matrix (Eq. offline-objective): signed codes k[N][K] and
 * per-group (s, a, b) of shape [N][K/G]. */
CQO_API void cqo_encode(const float *W, int64_t N, int64_t K, int B, int G, int effort, int8_t *k, float *s,
                        uint16_t *a, uint16_t *b) {
    int64_t ng = K / G;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t gi = 0; gi < N * ng; ++gi) {
        int64_t n = gi / ng, g = gi % ng;
        encode_group(W + n * K + g * G, G, B, effort, 0, k + n * K + g * G, &s[gi], &a[gi], &b[gi]);
    }
}

/* The same search under the dual-path objective L_C + L_A8 of Section 4.3 (effort 0, the absmax INT
 * pin, is objective-free).  For W1 / W2 the levels lie on the carrier grid, so the result equals cqo_encode's. */
CQO_API void cqo_encode_joint(const float *W, int64_t N, int64_t K, int B, int G, int effort, int8_t *k, float *s,
                              uint16_t *a, uint16_t *b) {
    int64_t ng = K / G;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t gi = 0; gi < N * ng; ++gi) {
        int64_t n = gi / ng, g = gi % ng;
        encode_group(W + n * K + g * G, G, B, effort, B > 2 ? 1 : 0, k + n * K + g * G, &s[gi], &a[gi], &b[gi]);
    }
}

/* ------------------------------------------------------------------ model-dtype product (Section 5.3) */

/* y[m][n] = sum_k x[m][k] What[n][k]: the continuous reconstruction of Eq. cubic is the
 * semantic reference of this mode.  x holds bfloat16 bit patterns (promoted exactly);
 * accumulation in fp64.  rows / cols select the activation rows m and output channels n to
 * evaluate (NULL = all); y is [nrows][ncols]. */
CQO_API void cqo_gemm_model_act(const uint8_t *codes, const float *s, const uint16_t *a, const uint16_t *b, int B, int G,
                                int64_t N, int64_t K, const uint16_t *x, int act_f16, int64_t M, const int64_t *rows,
                                int64_t nrows, const int64_t *cols, int64_t ncols, double *y) {
    int64_t ng = K / G;
    (void)N; (void)M;
#pragma omp parallel
    {
        int8_t *kk = (int8_t *)malloc((size_t)K);
        double *wrow = (double *)malloc(sizeof(double) * (size_t)K);
        double lev[128];
#pragma omp for schedule(dynamic, 8)
        for (int64_t ci = 0; ci < ncols; ++ci) {
            int64_t n = cols ? cols[ci] : ci;
            cqo_unpack(codes + n * cqo_row_bytes(K, B), 1, K, B, kk);
            for (int64_t g = 0; g < ng; ++g) {
                cqo_levels(B, s[n * ng + g], a[n * ng + g], b[n * ng + g], lev);
                for (int j = 0; j < G; ++j) wrow[g * G + j] = decode_code(B, kk[g * G + j], lev);
            }
            for (int64_t ri = 0; ri < nrows; ++ri) {
                int64_t m = rows ? rows[ri] : ri;
                const uint16_t *xr = x + m * K;
                double acc = 0.0;
                for (int64_t j = 0; j < K; ++j) acc += act_to_double(xr[j], act_f16) * wrow[j];
                y[ri * ncols + ci] = acc;
            }
        }
        free(kk); free(wrow);
    }
}

CQO_API void cqo_gemm_model(const uint8_t *codes, const float *s, const uint16_t *a, const uint16_t *b, int B, int G,
                            int64_t N, int64_t K, const uint16_t *x, int64_t M, const int64_t *rows, int64_t nrows,
                            const int64_t *cols, int64_t ncols, double *y) {
    cqo_gemm_model_act(codes, s, a, b, B, G, N, K, x, 0, M, rows, nrows, cols, ncols, y);   /* bfloat16 activations */
}

/* ------------------------------------------------------------------ Dynamic A8 (Section 5.4) */

/* Per-row activation quantiser (Eq. a8-activation-scale, Eq. a8-activation-quantization):
 *   xbar = max(max_j |x_j|, eps),  d_x = xbar / 127,  x8_j = clip(round_away(x_j / d_x), -127, 127).
 * Bit-exact contract, so the arithmetic is pinned to fp32: eps = 1e-10f, both divisions are
 * IEEE fp32 divisions, roundf rounds halves away from zero. */
CQO_API void cqo_quantize_a8_act(const uint16_t *x, int act_f16, int64_t M, int64_t K, int8_t *x8, float *dx) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        float xbar = 0.0f;
        for (int64_t j = 0; j < K; ++j) {
            float v = fabsf((float)act_to_double(x[m * K + j], act_f16));
            if (v > xbar) xbar = v;
        }
        if (!(xbar > 1e-10f)) xbar = 1e-10f;
        float d = xbar / 127.0f;
        dx[m] = d;
        for (int64_t j = 0; j < K; ++j) {
            float v = (float)act_to_double(x[m * K + j], act_f16) / d;
            float r = roundf(v);
            if (r > 127.0f) r = 127.0f;
            if (r < -127.0f) r = -127.0f;
            x8[m * K + j] = (int8_t)r;
        }
    }
}

CQO_API void cqo_quantize_a8(const uint16_t *x, int64_t M, int64_t K, int8_t *x8, float *dx) {
    cqo_quantize_a8_act(x, 0, M, K, x8, dx);   /* bfloat16 activations */
}

/* Integer partials and output of the Dynamic-A8 product (Eq. a8-output):
 *   P_g = sum_{j in g} x8_j r_g(k_j)  (exact integers),   y = sum_g (d_x s_g / 127) P_g,
 * the latter evaluated in fp64 from the fp32 d_x and s_g.  P (optional) is
 * [nrows][ncols][K/G] int32; |P_g| <= G 127^2 (Eq. a8-int32-bound) is asserted by
 * returning the number of violations. */
CQO_API int64_t cqo_gemm_a8(const uint8_t *codes, const float *s, const uint16_t *a, const uint16_t *b, int B, int G,
                            int64_t N, int64_t K, const int8_t *x8, const float *dx, int64_t M, const int64_t *rows,
                            int64_t nrows, const int64_t *cols, int64_t ncols, double *y, int32_t *P) {
    int64_t ng = K / G;
    int64_t violations = 0;
    (void)N; (void)M;
#pragma omp parallel reduction(+ : violations)
    {
        int8_t *kk = (int8_t *)malloc((size_t)K);
        int8_t *rrow = (int8_t *)malloc((size_t)K);
        int8_t car[128];
#pragma omp for schedule(dynamic, 8)
        for (int64_t ci = 0; ci < ncols; ++ci) {
            int64_t n = cols ? cols[ci] : ci;
            cqo_unpack(codes + n * cqo_row_bytes(K, B), 1, K, B, kk);
            for (int64_t g = 0; g < ng; ++g) {
                cqo_carriers(B, a[n * ng + g], b[n * ng + g], car);
                for (int j = 0; j < G; ++j) {
                    int code = kk[g * G + j], r;
                    if (B == 1) r = code > 0 ? car[0] : -car[0];
                    else if (code == -(1 << (B - 1))) r = 0;
                    else r = code < 0 ? -car[-code] : car[code];
                    rrow[g * G + j] = (int8_t)r;
                }
            }
            for (int64_t ri = 0; ri < nrows; ++ri) {
                int64_t m = rows ? rows[ri] : ri;
                const int8_t *xr = x8 + m * K;
                double acc = 0.0;
                for (int64_t g = 0; g < ng; ++g) {
                    int64_t pg = 0;
                    for (int j = 0; j < G; ++j) pg += (int64_t)xr[g * G + j] * (int64_t)rrow[g * G + j];
                    if (llabs(pg) > (int64_t)G * 127 * 127) ++violations;
                    if (P) P[(ri * ncols + ci) * ng + g] = (int32_t)pg;
                    acc += ((double)dx[m] * (double)s[n * ng + g] / 127.0) * (double)pg;
                }
                y[ri * ncols + ci] = acc;
            }
        }
        free(kk); free(rrow);
    }
    return violations;
}
