// Small-M (M <= 16) packed GEMV: split-K, weights streamed exactly once, warp-level tensor-core
// MMAs doing the multiply and the k reduction (Section 5.3 narrow-row path; Section 5.4 for A8).
//
// Work decomposition: CTA = one 128-row block x one K slice; its 8 warps own the 8 row blocks of
// 16 rows.  A lane's 128-bit loads land directly in its MMA A-fragment positions (see
// cq_common.cuh), so decode is: mask two codes out of a word, turn them into fp16 by the
// exponent-bias trick, evaluate the group's cubic in half2 Horner form (Eq. gpu-horner) on the
// power-of-two-normalised code, and feed the MMA.  The group scale s_g is applied to the fp32
// group reduction, as the paper's narrow path does.  Activations are converted bf16 -> fp16 with
// a per-token power-of-two scale chosen per CTA so that nothing overflows or loses bits.
//
// Dynamic A8 uses the INT8 m16n8k32 MMA on signed carriers looked up in a per-warp table of the
// group's non-negative carriers (Eq. carrier), int32 group partials, fp32 rescale (Eq. a8-output).
#include "cq_common.cuh"
#include "cq_internal.h"

namespace cq {

namespace {

constexpr int GEMV_THREADS = 256;
constexpr int XS_PAD = 16;          // halves of padding per staged activation row (bank spread)
constexpr int MAX_SLICE_TILES = 16; // K tiles per CTA at most (bounds shared memory)

__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_s8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ld_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ld_stream8(const void *p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

template <int B>
struct Rec { uint32_t w[2 * B]; };

template <int B>
__device__ __forceinline__ void load_rec(Rec<B> &r, const uint8_t *rbp, int lane) {
    constexpr int NFQ = (2 * B) / 4;
#pragma unroll
    for (int q = 0; q < NFQ; ++q) {
        const uint4 v = ld_stream16(rbp + (q * 32 + lane) * 16);
        r.w[4 * q + 0] = v.x; r.w[4 * q + 1] = v.y; r.w[4 * q + 2] = v.z; r.w[4 * q + 3] = v.w;
    }
    if constexpr ((2 * B) % 4 != 0) {
        const uint2 v = ld_stream8(rbp + NFQ * 512 + lane * 8);
        r.w[4 * NFQ + 0] = v.x; r.w[4 * NFQ + 1] = v.y;
    }
}

// Two stored codes of pair p as packed 16-bit integers (u_lo | u_hi << 16).  Generic form.
template <int B>
__device__ __forceinline__ uint32_t pair_codes(const uint32_t (&w)[2 * B], int p) {
    uint32_t u2 = 0;
#pragma unroll
    for (int i = 0; i < plane_count(B); ++i) {
        const int pw = plane_width(B, i), ppw = 16 / pw;
        const int W = plane_word_base(B, i) + p / ppw, pos = (p % ppw) * pw;
        const uint32_t m = ((1u << pw) - 1u) * 0x00010001u;
        u2 |= ((w[W] >> pos) & m) << plane_bit_offset(B, i);
    }
    return u2;
}

// Pair p as half2 of the normalised signed code:  B >= 3: k / 2^(B-1);  B = 2: k;  B = 1: k (+-1).
// The stored code lands in the fp16 mantissa under exponent bits 0x6400 (value 1024 + u * 2^pos);
// one exact FMA removes the offset and the position scale.
template <int B>
__device__ __forceinline__ __half2 pair_T(const uint32_t (&w)[2 * B], int p) {
    if constexpr (plane_count(B) == 1) {
        constexpr int PPW = 16 / B;
        const int W = p / PPW;
        int pos = (p % PPW) * B;
        uint32_t word = w[W];
        if constexpr (B == 1) {  // keep the field off mantissa bit 0 so the offset constant stays representable
            if (pos <= 6) { word <<= 1; pos += 1; } else { word >>= 6; pos -= 6; }
        } else {
            if (pos + B > 10) { word >>= 8; pos -= 8; }
        }
        const uint32_t m = (((1u << B) - 1u) << pos) * 0x00010001u;
        const uint32_t hbits = (word & m) | 0x64006400u;
        float sc, off;
        if constexpr (B == 1) { sc = exp2f((float)(1 - pos)); off = -(exp2f((float)(11 - pos)) + 1.0f); }
        else if constexpr (B == 2) { sc = exp2f((float)(-pos)); off = -(exp2f((float)(10 - pos)) + 2.0f); }
        else { sc = exp2f((float)(-(pos + B - 1))); off = -(exp2f((float)(10 - pos - (B - 1))) + 1.0f); }
        return __hfma2(*reinterpret_cast<const __half2 *>(&hbits), __float2half2_rn(sc), __float2half2_rn(off));
    } else {
        const uint32_t hbits = pair_codes<B>(w, p) | 0x64006400u;
        const float sc = exp2f((float)(-(B - 1))), off = -(exp2f((float)(10 - (B - 1))) + 1.0f);
        return __hfma2(*reinterpret_cast<const __half2 *>(&hbits), __float2half2_rn(sc), __float2half2_rn(off));
    }
}

struct RowCoef { __half2 a2, b2, c2; float s; };

// Coefficients of q as a polynomial in T = k / 2^(B-1):  t = |T| rho, rho = 2^(B-1) / M, so
// q = |T| (a rho + |T| (b rho^2 + |T| c rho^3)).
template <int B>
__device__ __forceinline__ RowCoef make_coef(const GroupParams &p) {
    RowCoef c;
    c.s = fabsf(p.s);
    if constexpr (B >= 3) {
        constexpr float rho = (float)(1 << (B - 1)) / (float)((1 << (B - 1)) - 1);
        const float a = __half2float(p.a), b = __half2float(p.b), cc = (1.0f - a) - b;
        c.a2 = __float2half2_rn(a * rho);
        c.b2 = __float2half2_rn(b * rho * rho);
        c.c2 = __float2half2_rn(cc * rho * rho * rho);
    }
    return c;
}

template <int B, bool FIX>
__device__ __forceinline__ uint32_t level_pair(__half2 T, const RowCoef &c) {
    if constexpr (FIX) {  // reserved pattern: T = -1 (B >= 3) or k = -2 (B = 2) decodes to zero
        const __half2 bad = __float2half2_rn(B == 2 ? -2.0f : -1.0f);
        T = __hmul2(T, __hne2(T, bad));
    }
    __half2 v;
    if constexpr (B >= 3) {
        const __half2 at = __habs2(T);
        v = __hmul2(T, __hfma2(at, __hfma2(at, c.c2, c.b2), c.a2));
    } else {
        v = T;
    }
    return *reinterpret_cast<uint32_t *>(&v);
}

// ------------------------------------------------------------------------------------------
// MODE 0: model dtype.  MODE 1: Dynamic A8 (xq = int8 carrier [M][x8_pitch], dxs = row scales).
template <int B, int G, int NT, int MODE>
__global__ void __launch_bounds__(GEMV_THREADS)
gemv_kernel(const uint8_t *__restrict__ layout, Dims d, const uint16_t *__restrict__ x, const int8_t *__restrict__ xq,
            int64_t x8_pitch, const float *__restrict__ dxs, uint16_t *__restrict__ y, int M, int S,
            float *__restrict__ partial, int *__restrict__ counters) {
    constexpr int GPT = TILE / G;      // groups per tile
    constexpr int CPG = G / 16;        // 16-wide k chunks per group
    constexpr int L = B == 1 ? 1 : (1 << (B - 1));
    extern __shared__ __align__(16) uint8_t smem[];
    __shared__ float s_inv[16];
    __shared__ unsigned s_max[16];
    __shared__ int s_last;

    const int nb = blockIdx.x / S, sk = blockIdx.x % S;
    const int kb0 = (int)(((int64_t)sk * d.KT) / S), kb1 = (int)(((int64_t)(sk + 1) * d.KT) / S);
    const int slice_k = (kb1 - kb0) * TILE;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int64_t k_base = (int64_t)kb0 * TILE;

    const uint8_t *tile0 = layout + ((size_t)nb * d.KT + kb0) * (size_t)d.tile_bytes;
    const uint8_t *rbp0 = tile0 + warp * 256 * B;
    const uint8_t *prm0 = tile0 + d.code_bytes + ((warp * 16 + g) * GPT) * 8;  // row g of this row block

    // issue the first weight loads before touching the activations
    constexpr int PF = (B <= 4) ? 2 : 1;
    Rec<B> rec[PF + 1];
    GroupParams prm[PF + 1][2][GPT];
#pragma unroll
    for (int i = 0; i < PF; ++i)
        if (kb0 + i < kb1) {
            load_rec<B>(rec[i], rbp0 + (size_t)i * d.tile_bytes, lane);
#pragma unroll
            for (int gi = 0; gi < GPT; ++gi) {
                prm[i][0][gi] = *(const GroupParams *)(prm0 + (size_t)i * d.tile_bytes + gi * 8);
                prm[i][1][gi] = *(const GroupParams *)(prm0 + (size_t)i * d.tile_bytes + (8 * GPT + gi) * 8);
            }
        }

    // ---- stage the activation slice
    const int XS = slice_k + XS_PAD;  // elements per staged row
    if constexpr (MODE == 0) {
        __half *xs = reinterpret_cast<__half *>(smem);
        if (threadIdx.x < 16) s_max[threadIdx.x] = 0;
        __syncthreads();
        const int cpr = slice_k / 8;  // 16-byte chunks per row
        const bool vec = (d.K % 8) == 0;
        for (int idx = threadIdx.x; idx < M * cpr; idx += GEMV_THREADS) {
            const int m = idx / cpr, c = idx % cpr;
            const int64_t k = k_base + (int64_t)c * 8;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (vec) {
                if (k < d.K) v = *(const uint4 *)(x + (int64_t)m * d.K + k);
            } else {
                uint16_t e[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) e[q] = (k + q < d.K) ? x[(int64_t)m * d.K + k + q] : (uint16_t)0;
                v.x = e[0] | (e[1] << 16); v.y = e[2] | (e[3] << 16); v.z = e[4] | (e[5] << 16); v.w = e[6] | (e[7] << 16);
            }
            *(uint4 *)(xs + m * XS + c * 8) = v;  // raw bf16 for now
            unsigned mx = 0;  // largest |bf16| bit pattern of the chunk
            const uint32_t ws[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) { mx = max(mx, ws[q] & 0x7FFFu); mx = max(mx, (ws[q] >> 16) & 0x7FFFu); }
            atomicMax(&s_max[m], mx);
        }
        __syncthreads();
        if (threadIdx.x < 16) {
            // power-of-two scale putting the row maximum in [2^14, 2^15)
            const float mxf = __uint_as_float(s_max[threadIdx.x] << 16);
            int sh = 0;
            if (mxf > 0.0f && mxf < 3.0e38f) sh = 14 - (int)((s_max[threadIdx.x] >> 7) & 0xFF) + 127;
            sh = max(min(sh, 100), -100);
            s_inv[threadIdx.x] = exp2f((float)(-sh));
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < M * cpr; idx += GEMV_THREADS) {
            const int m = idx / cpr, c = idx % cpr;
            const float sc = 1.0f / s_inv[m];
            uint4 v = *(uint4 *)(xs + m * XS + c * 8);
            uint32_t ws[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float lo = __uint_as_float(ws[q] << 16) * sc, hi = __uint_as_float(ws[q] & 0xFFFF0000u) * sc;
                const __half2 h = __floats2half2_rn(lo, hi);
                ws[q] = *reinterpret_cast<const uint32_t *>(&h);
            }
            *(uint4 *)(xs + m * XS + c * 8) = make_uint4(ws[0], ws[1], ws[2], ws[3]);
        }
    } else {
        int8_t *xs = reinterpret_cast<int8_t *>(smem);
        const int cpr = slice_k / 16;
        for (int idx = threadIdx.x; idx < M * cpr; idx += GEMV_THREADS) {
            const int m = idx / cpr, c = idx % cpr;
            // the carrier is written with a pitch that is a multiple of 128, zero beyond K
            *(uint4 *)(xs + m * XS + c * 16) = *(const uint4 *)(xq + (int64_t)m * x8_pitch + k_base + c * 16);
        }
        if (threadIdx.x < 16) s_inv[threadIdx.x] = threadIdx.x < M ? dxs[threadIdx.x] * (1.0f / 127.0f) : 0.0f;
    }
    __syncthreads();

    // per-warp carrier table (A8): [16 rows][L] int8 after the activation rows
    int8_t *ctab = nullptr;
    if constexpr (MODE == 1 && B >= 3) ctab = reinterpret_cast<int8_t *>(smem) + 16 * XS + warp * 16 * L;

    float acc[NT][4];
#pragma unroll
    for (int tb = 0; tb < NT; ++tb)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[tb][i] = 0.0f;

    for (int kb = kb0; kb < kb1; ++kb) {
        // prefetch PF tiles ahead
        if (kb + PF < kb1) {
            const size_t off = (size_t)(kb + PF - kb0) * d.tile_bytes;
            load_rec<B>(rec[PF], rbp0 + off, lane);
#pragma unroll
            for (int gi = 0; gi < GPT; ++gi) {
                prm[PF][0][gi] = *(const GroupParams *)(prm0 + off + gi * 8);
                prm[PF][1][gi] = *(const GroupParams *)(prm0 + off + (8 * GPT + gi) * 8);
            }
        }
        const int kl = (kb - kb0) * TILE;  // k offset inside the staged slice
#pragma unroll
        for (int gi = 0; gi < GPT; ++gi) {
            const GroupParams p_lo = prm[0][0][gi], p_hi = prm[0][1][gi];
            const bool fix = B > 1 && __any_sync(0xffffffffu, (__float_as_uint(p_lo.s) | __float_as_uint(p_hi.s)) >> 31);
            if constexpr (MODE == 0) {
                const RowCoef c_lo = make_coef<B>(p_lo), c_hi = make_coef<B>(p_hi);
                float D[NT][4];
#pragma unroll
                for (int tb = 0; tb < NT; ++tb)
#pragma unroll
                    for (int i = 0; i < 4; ++i) D[tb][i] = 0.0f;
                const __half *xs = reinterpret_cast<const __half *>(smem);
#pragma unroll
                for (int jj = 0; jj < CPG; ++jj) {
                    const int j = gi * CPG + jj;
                    uint32_t A[4];
                    if (!fix) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) A[i] = level_pair<B, false>(pair_T<B>(rec[0].w, 4 * j + i), (i & 1) ? c_hi : c_lo);
                    } else {
#pragma unroll
                        for (int i = 0; i < 4; ++i) A[i] = level_pair<B, true>(pair_T<B>(rec[0].w, 4 * j + i), (i & 1) ? c_hi : c_lo);
                    }
#pragma unroll
                    for (int tb = 0; tb < NT; ++tb) {
                        const int tok = tb * 8 + g;
                        uint2 bf = make_uint2(0, 0);
                        if (tok < M) bf = *(const uint2 *)(xs + tok * XS + kl + 16 * j + 4 * t);
                        mma_f16(D[tb], A, bf.x, bf.y);
                    }
                }
#pragma unroll
                for (int tb = 0; tb < NT; ++tb) {
                    acc[tb][0] = fmaf(c_lo.s, D[tb][0], acc[tb][0]);
                    acc[tb][1] = fmaf(c_lo.s, D[tb][1], acc[tb][1]);
                    acc[tb][2] = fmaf(c_hi.s, D[tb][2], acc[tb][2]);
                    acc[tb][3] = fmaf(c_hi.s, D[tb][3], acc[tb][3]);
                }
            } else {
                // carrier table of this group for the warp's 16 rows: lane (g, t) fills entries i = t mod 4
                if constexpr (B >= 3) {
                    __syncwarp();
                    const float a_lo = __half2float(p_lo.a), b_lo = __half2float(p_lo.b);
                    const float a_hi = __half2float(p_hi.a), b_hi = __half2float(p_hi.b);
                    for (int i = t; i < L; i += 4) {
                        ctab[g * L + i] = (int8_t)carrier_of(B, i, a_lo, b_lo);
                        ctab[(g + 8) * L + i] = (int8_t)carrier_of(B, i, a_hi, b_hi);
                    }
                    __syncwarp();
                }
                int D[NT][4];
#pragma unroll
                for (int tb = 0; tb < NT; ++tb)
#pragma unroll
                    for (int i = 0; i < 4; ++i) D[tb][i] = 0;
                const int8_t *xs = reinterpret_cast<const int8_t *>(smem);
#pragma unroll
                for (int jj = 0; jj < CPG; jj += 2) {
                    const int j = gi * CPG + jj;
                    uint32_t A[4];
                    // a0: row g chunk j; a1: row g+8 chunk j; a2: row g chunk j+1; a3: row g+8 chunk j+1
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        const int jc = j + (r >> 1), hi_row = r & 1;
                        uint32_t packed = 0;
#pragma unroll
                        for (int e = 0; e < 2; ++e) {  // registers (hi_row) and (2 + hi_row) hold k+0,1 and k+2,3
                            const uint32_t u2 = pair_codes<B>(rec[0].w, 4 * jc + 2 * e + hi_row);
#pragma unroll
                            for (int hh = 0; hh < 2; ++hh) {
                                const unsigned u = (u2 >> (16 * hh)) & 0xFFFFu;
                                const int code = signed_code(B, u);
                                int rv;
                                if constexpr (B <= 2) rv = 127 * code;
                                else { rv = ctab[(g + 8 * hi_row) * L + abs(code)]; rv = code < 0 ? -rv : rv; }
                                packed |= ((uint32_t)rv & 0xFFu) << (8 * (2 * e + hh));
                            }
                        }
                        A[r] = packed;
                    }
#pragma unroll
                    for (int tb = 0; tb < NT; ++tb) {
                        const int tok = tb * 8 + g;
                        uint32_t b0 = 0, b1 = 0;
                        if (tok < M) {
                            b0 = *(const uint32_t *)(xs + tok * XS + kl + 16 * j + 4 * t);
                            b1 = *(const uint32_t *)(xs + tok * XS + kl + 16 * (j + 1) + 4 * t);
                        }
                        mma_s8(D[tb], A, b0, b1);
                    }
                }
                const float s_lo = fabsf(p_lo.s), s_hi = fabsf(p_hi.s);
#pragma unroll
                for (int tb = 0; tb < NT; ++tb) {
                    acc[tb][0] = fmaf(s_lo, (float)D[tb][0], acc[tb][0]);
                    acc[tb][1] = fmaf(s_lo, (float)D[tb][1], acc[tb][1]);
                    acc[tb][2] = fmaf(s_hi, (float)D[tb][2], acc[tb][2]);
                    acc[tb][3] = fmaf(s_hi, (float)D[tb][3], acc[tb][3]);
                }
            }
        }
        // rotate the prefetch registers
#pragma unroll
        for (int i = 0; i < PF; ++i) {
            rec[i] = rec[i + 1];
#pragma unroll
            for (int gi = 0; gi < GPT; ++gi) { prm[i][0][gi] = prm[i + 1][0][gi]; prm[i][1][gi] = prm[i + 1][1][gi]; }
        }
    }

    // ---- epilogue: lane (g, t) holds rows g, g+8 x tokens 2t, 2t+1 of each token block
    const int64_t Np = (int64_t)d.NB * TILE;
    const int64_t n_lo = (int64_t)nb * TILE + warp * 16 + g;
#pragma unroll
    for (int tb = 0; tb < NT; ++tb)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int tok = tb * 8 + 2 * t + (i & 1);
            const int64_t n = n_lo + ((i >> 1) ? 8 : 0);
            if (tok >= M) continue;
            const float v = acc[tb][i] * s_inv[tok];
            if (S == 1) {
                if (n < d.N) y[(int64_t)tok * d.N + n] = __bfloat16_as_ushort(__float2bfloat16_rn(v));
            } else {
                partial[((int64_t)sk * M + tok) * Np + n] = v;
            }
        }
    if (S == 1) return;

    // ---- split-K combine: the last CTA of this row block to arrive sums the slices in index order
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int old = atomicAdd(&counters[nb], 1);
        s_last = (old == S - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int idx = threadIdx.x; idx < M * TILE; idx += GEMV_THREADS) {
        const int m = idx / TILE, r = idx % TILE;
        const int64_t n = (int64_t)nb * TILE + r;
        float sum = 0.0f;
        for (int q = 0; q < S; ++q) sum += __ldcg(&partial[((int64_t)q * M + m) * Np + n]);
        if (n < d.N) y[(int64_t)m * d.N + n] = __bfloat16_as_ushort(__float2bfloat16_rn(sum));
    }
    if (threadIdx.x == 0) counters[nb] = 0;  // leave the workspace ready for the next call
}

template <int B, int G, int NT, int MODE>
cudaError_t launch_one(const void *layout, const Dims &d, const uint16_t *x, const int8_t *xq, int64_t x8_pitch,
                       const float *dxs, uint16_t *y, int M, int S, float *partial, int *counters, cudaStream_t st) {
    const int slice_tiles = (d.KT + S - 1) / S;
    const int XS = slice_tiles * TILE + XS_PAD;
    size_t smem = MODE == 0 ? (size_t)M * XS * 2 : (size_t)16 * XS + 8 * 16 * (B == 1 ? 1 : (1 << (B - 1)));
    auto kern = gemv_kernel<B, G, NT, MODE>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    kern<<<d.NB * S, GEMV_THREADS, smem, st>>>((const uint8_t *)layout, d, x, xq, x8_pitch, dxs, y, M, S, partial, counters);
    return cudaGetLastError();
}

template <int B, int G>
cudaError_t dispatch_nt_mode(const void *layout, const Dims &d, const uint16_t *x, const int8_t *xq, int64_t x8_pitch,
                             const float *dxs, uint16_t *y, int M, int mode, int S, float *partial, int *counters,
                             cudaStream_t st) {
    if (mode == 0) {
        if (M <= 8) return launch_one<B, G, 1, 0>(layout, d, x, xq, x8_pitch, dxs, y, M, S, partial, counters, st);
        return launch_one<B, G, 2, 0>(layout, d, x, xq, x8_pitch, dxs, y, M, S, partial, counters, st);
    }
    if (M <= 8) return launch_one<B, G, 1, 1>(layout, d, x, xq, x8_pitch, dxs, y, M, S, partial, counters, st);
    return launch_one<B, G, 2, 1>(layout, d, x, xq, x8_pitch, dxs, y, M, S, partial, counters, st);
}

template <int B>
cudaError_t dispatch_g(const void *layout, const Dims &d, const uint16_t *x, const int8_t *xq, int64_t x8_pitch,
                       const float *dxs, uint16_t *y, int M, int mode, int S, float *partial, int *counters,
                       cudaStream_t st) {
    switch (d.G) {
        case 32: return dispatch_nt_mode<B, 32>(layout, d, x, xq, x8_pitch, dxs, y, M, mode, S, partial, counters, st);
        case 64: return dispatch_nt_mode<B, 64>(layout, d, x, xq, x8_pitch, dxs, y, M, mode, S, partial, counters, st);
        default: return dispatch_nt_mode<B, 128>(layout, d, x, xq, x8_pitch, dxs, y, M, mode, S, partial, counters, st);
    }
}

}  // namespace

// Split-K factor of the small-M path: enough CTAs to fill 148 SMs about three times over, at
// most MAX_SLICE_TILES K tiles per CTA, at least one.
int gemv_split_k(const Dims &d) {
    int S = (444 + d.NB - 1) / d.NB;
    if (S > d.KT) S = d.KT;
    const int min_s = (d.KT + MAX_SLICE_TILES - 1) / MAX_SLICE_TILES;
    if (S < min_s) S = min_s;
    if (S < 1) S = 1;
    return S;
}

cudaError_t launch_gemv(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int mode,
                        uint8_t *ws, const Workspace &plan, cudaStream_t st) {
    const int S = plan.split_k;
    float *partial = reinterpret_cast<float *>(ws + plan.partial_off);
    int *counters = reinterpret_cast<int *>(ws + plan.counters_off);
    int8_t *xq = reinterpret_cast<int8_t *>(ws + plan.x8_off);
    float *dxs = reinterpret_cast<float *>(ws + plan.dx_off);
    const int64_t pitch = (int64_t)d.KT * TILE;
    if (mode == 1) {
        cudaError_t e = launch_quantize_a8(x, M, d.K, xq, pitch, dxs, st);
        if (e != cudaSuccess) return e;
    }
    switch (d.B) {
        case 1: return dispatch_g<1>(layout, d, x, xq, pitch, dxs, y, (int)M, mode, S, partial, counters, st);
        case 2: return dispatch_g<2>(layout, d, x, xq, pitch, dxs, y, (int)M, mode, S, partial, counters, st);
        case 3: return dispatch_g<3>(layout, d, x, xq, pitch, dxs, y, (int)M, mode, S, partial, counters, st);
        case 4: return dispatch_g<4>(layout, d, x, xq, pitch, dxs, y, (int)M, mode, S, partial, counters, st);
        case 5: return dispatch_g<5>(layout, d, x, xq, pitch, dxs, y, (int)M, mode, S, partial, counters, st);
        case 6: return dispatch_g<6>(layout, d, x, xq, pitch, dxs, y, (int)M, mode, S, partial, counters, st);
        case 7: return dispatch_g<7>(layout, d, x, xq, pitch, dxs, y, (int)M, mode, S, partial, counters, st);
        default: return dispatch_g<8>(layout, d, x, xq, pitch, dxs, y, (int)M, mode, S, partial, counters, st);
    }
}

}  // namespace cq
