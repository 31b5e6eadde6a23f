// Small-M (M <= 16) packed GEMV: weights streamed exactly once, warp-level tensor-core MMAs doing
// the multiply and the k reduction (Section 5.3 narrow-row path; Section 5.4 for Dynamic A8).
//
// Work decomposition (balanced, persistent): the NB x KT grid of 128 x 128 weight tiles is cut
// into P equal contiguous runs (P = resident CTAs of the whole GPU), one per CTA, in row-block
// major order.  A run covers one or more row blocks; for each it streams its K range, and either
// writes y (it covered the whole K range) or a partial sum into one of its two slots; the CTA that completes
// a row block adds the partials in K order (deterministic) and writes y.
//
// Streaming: a run is one contiguous byte range of the layout.  One thread moves it tile by tile
// into a shared-memory ring with bulk asynchronous copies (cp.async.bulk, completion on an mbarrier
// per stage), so the bytes in flight do not depend on the registers of the warps; the 8 warps own
// the 8 groups of 16 rows of a tile, read their slice of a stage with 128-bit shared loads that
// land directly in their MMA A-fragment positions (cq_common.cuh) and hand the stage back through
// a second mbarrier.  Weights never depend on the previous kernel of the stream, so the first
// round of copies is issued before the programmatic-dependency wait.
//
// Decode (model dtype): two codes are masked out of a word straight into fp16 mantissas
// (exponent-bias trick) and one exact packed-half add leaves the signed code; the group's cubic is
// evaluated in half2 Horner form (Eq. gpu-horner) as T (ca + |T| (cb + |T| cc)) and the group scale s_g
// multiplies the fp32 group sum, as in the paper's narrow path.  W3 reads its eight levels from a
// register table with byte permutes instead; W1 / W2 have no shape.  Activations go bf16 -> fp16 with
// a per-token power-of-two scale so that nothing overflows or loses bits.
//
// Multiply: one or two tokens use a packed-half FMA per pair of weights into half2 accumulators that
// are promoted to fp32 once per group (a warp-level MMA holds the scheduler's issue port for about a
// dozen cycles and wastes seven of its eight token columns there); three to sixteen tokens use the
// m16n8k16 MMA (fp16 in, fp32 accumulate), the weights' loads landing directly in its A fragment.
//
// Dynamic A8 uses the INT8 m16n8k32 MMA on signed carriers (Eq. carrier) taken from a per-(row, group)
// table indexed by the stored code -- in registers and read with byte permutes for B <= 4, in shared
// memory otherwise (a8_row_regs in cq_decode.cuh) -- int32 group partials, fp32 rescale (Eq. a8-output).
#include <cstdlib>

#include "cq_common.cuh"
#include "cq_decode.cuh"
#include "cq_internal.h"
#include "cq_tc_ptx.cuh"

namespace cq {

namespace {

#ifndef CQ_GEMV_CTAS_PER_SM
#define CQ_GEMV_CTAS_PER_SM 3
#endif
constexpr int GEMV_WARPS = 8;                        // one warp per group of 16 rows of a tile
constexpr int GEMV_THREADS = GEMV_WARPS * 32;
constexpr int XS_PAD = 16;     // elements of padding per staged fp16 activation row (bank spread: 32 bytes)
constexpr int XS_PAD8 = 32;    // the same for an INT8 row
constexpr int MAX_SUB = 16;    // K tiles staged at a time (bounds shared memory)
// Kernel variants: MODE 0 model dtype with MMA (NT blocks of 8 tokens), MODE 1 Dynamic A8 (the same blocks),
// MODE 2 model dtype without MMA (NT = tokens, 1 or 2).
__host__ __device__ constexpr int gemv_rows(int NT, int MODE) { return MODE == 2 ? NT : 8 * NT; }
// most shared memory the staged activations (and the Dynamic-A8 carrier tables) of a variant can take
__host__ __device__ constexpr int gemv_x_bytes_max(int B, int NT, int MODE) {
    return MODE == 1 ? gemv_rows(NT, MODE) * (MAX_SUB * TILE + XS_PAD8) + (B >= 3 ? 8 * 16 * carrier_table_stride(B) : 0)
                     : gemv_rows(NT, MODE) * (MAX_SUB * TILE + 2 * XS_PAD) * 2;
}
__host__ __device__ constexpr int gemv_smem_budget(int ctas) { return (227 * 1024) / ctas - 2048; }   // dynamic shared memory of a CTA
// How a CTA's tiles reach the registers.  Straight from global memory into a two- or three-deep register
// prefetch where that fits the registers (it measured a little faster there); through a shared-memory ring
// filled by bulk copies where it does not: G = 32 (four parameter records per tile row), the widths made of
// several bit planes, and the two-token variant.
__host__ __device__ constexpr bool gemv_uses_ring(int B, int G, int NT, int MODE) {
    return G == 32 || (B >= 5 && B <= 7) || (MODE == 2 && NT == 2);
}
// Resident CTAs per SM: three where the registers (80 per thread: one token block) and a ring of at least
// four stages allow it, otherwise two.
__host__ __device__ constexpr int gemv_occ(int B, int G, int NT, int MODE) {
    if (MODE != 2 && NT == 2) return 2;
    if (!gemv_uses_ring(B, G, NT, MODE)) return CQ_GEMV_CTAS_PER_SM;
    const int tb = 2048 * B + 1024 * (TILE / G);
    return (gemv_smem_budget(CQ_GEMV_CTAS_PER_SM) - (gemv_x_bytes_max(B, NT, MODE) + 127) / 128 * 128) / tb >= 4 ? CQ_GEMV_CTAS_PER_SM : 2;
}
// the variant that serves M rows in an activation mode
__host__ __device__ constexpr int gemv_variant_mode(int64_t M, int mode) { return mode == 1 ? 1 : (M <= 2 ? 2 : 0); }
__host__ __device__ constexpr int gemv_variant_nt(int64_t M, int mode) { return (mode == 0 && M <= 2) ? (int)M : (M <= 8 ? 1 : 2); }
constexpr int MAX_STAGES = 16;                       // ring stages (bounded by the mbarrier arrays)
constexpr int ERR_GEMV_FULL = 31, ERR_GEMV_EMPTY = 32;   // status codes of the two ring waits

__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_s8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// the same MMAs with a zero C operand (the first MMA of a group: no accumulator registers to clear)
__device__ __forceinline__ void mma_f16_z(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.0f));
}
__device__ __forceinline__ void mma_s8_z(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "r"(0));
}

__device__ __forceinline__ void compute_barrier() { __syncthreads(); }

template <int B, int GPT>
struct TileRegs {
    uint32_t w[2 * B];
    uint2 prm[2][GPT];  // {s bits, a | b << 16} of rows g and g + 8
};

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
template <int B, int GPT, class T>
__device__ __forceinline__ void load_tile_g(T &r, const uint8_t *wl, const uint8_t *pl, int lane) {
    constexpr int NFQ = (2 * B) / 4;
#pragma unroll
    for (int q = 0; q < NFQ; ++q) {
        const uint4 v = ld_stream16(wl + q * 512);
        r.w[4 * q + 0] = v.x; r.w[4 * q + 1] = v.y; r.w[4 * q + 2] = v.z; r.w[4 * q + 3] = v.w;
    }
    if constexpr ((2 * B) % 4 != 0) {
        const uint2 v = ld_stream8(wl + NFQ * 512 - lane * 8);
        r.w[4 * NFQ + 0] = v.x; r.w[4 * NFQ + 1] = v.y;
    }
#pragma unroll
    for (int gi = 0; gi < GPT; ++gi) {
        r.prm[0][gi] = ld_stream8(pl + gi * 8);
        r.prm[1][gi] = ld_stream8(pl + (8 * GPT + gi) * 8);
    }
}
// A warp's slice of a ring stage -> registers.  wl = stage + row-block base + lane * 16 (codes);
// pl = parameter record of row g of the row block.
template <int B, int GPT>
__device__ __forceinline__ void load_tile(TileRegs<B, GPT> &r, const uint8_t *wl, const uint8_t *pl, int lane) {
    constexpr int NFQ = (2 * B) / 4;
#pragma unroll
    for (int q = 0; q < NFQ; ++q) {
        const uint4 v = *reinterpret_cast<const uint4 *>(wl + q * 512);
        r.w[4 * q + 0] = v.x; r.w[4 * q + 1] = v.y; r.w[4 * q + 2] = v.z; r.w[4 * q + 3] = v.w;
    }
    if constexpr ((2 * B) % 4 != 0) {
        const uint2 v = *reinterpret_cast<const uint2 *>(wl + NFQ * 512 - lane * 8);  // the tail is indexed lane * 8, not lane * 16
        r.w[4 * NFQ + 0] = v.x; r.w[4 * NFQ + 1] = v.y;
    }
#pragma unroll
    for (int gi = 0; gi < GPT; ++gi) {
        r.prm[0][gi] = *reinterpret_cast<const uint2 *>(pl + gi * 8);
        r.prm[1][gi] = *reinterpret_cast<const uint2 *>(pl + (8 * GPT + gi) * 8);
    }
}

// Per-row coefficients of the level polynomial in code units: pair_K returns the signed code T in units of
// rho = code_unit<B>() (the integer k for B <= 6, k / 2^(B-1) above), the normalised position is t = |T| rho,
// so level / s = sign(k) (a t + b t^2 + c t^3) = T (ca + |T| (cb + |T| cc)) with ca = a rho, cb = b rho^2,
// cc = c rho^3, c = 1 - a - b (Eq. gpu-horner).  Formed in fp32 from the stored fp16 a and b, then rounded to
// fp16 once.
struct RowPoly { __half2 ca, cb, cc; float s; };
template <int B>
__device__ __forceinline__ RowPoly make_poly(uint2 p) {
    RowPoly r;
    r.s = __uint_as_float(p.x & 0x7FFFFFFFu);
    if constexpr (B >= 3) {
        constexpr float rho = code_unit<B>();
        const __half2 ab = as_h2(p.y);
        const float a = __low2float(ab), b = __high2float(ab), c = (1.0f - a) - b;
        r.ca = __float2half2_rn(a * rho);
        r.cb = __float2half2_rn(b * (rho * rho));
        r.cc = __float2half2_rn(c * (rho * rho * rho));
    }
    return r;
}
// signed level / s of a pair of codes (reserved pattern -> 0 when FIX)
template <int B, int P, bool FIX>
__device__ __forceinline__ __half2 level_of_pair(const uint32_t (&w)[2 * B], const DecodeRegs &dr, const RowPoly &c) {
    __half2 T = pair_K<B, P>(w, dr);
    if constexpr (FIX) T = __hmul2(T, __hne2(T, __float2half2_rn(B == 2 ? -2.0f : B <= 6 ? -(float)(1 << (B - 1)) : -1.0f)));
    if constexpr (B >= 3) {
        const __half2 aT = __habs2(T);
        return __hmul2(T, __hfma2(aT, __hfma2(aT, c.cc, c.cb), c.ca));
    } else {
        return T;
    }
}

// One group of a tile, model dtype, M > 2 (MODE 0).  xs = staged activations (fp16), xo[tb] = element offset of
// this lane's token row of token block tb (row g of the block, clamped to the last real row) plus 4 t.
// CPG MMAs per token block into D, then acc += s * D.
template <int B, int G, int NT, int GI, bool FIX>
__device__ __forceinline__ void group_model(const TileRegs<B, TILE / G> &r, const DecodeRegs &dr, const __half *xs, const int (&xo)[NT],
                                            float (&acc)[NT][4]) {
    constexpr int CPG = G / 16;
    const RowPoly c_lo = make_poly<B>(r.prm[0][GI]), c_hi = make_poly<B>(r.prm[1][GI]);
    float D[2][NT][4];   // two accumulator sets so consecutive MMAs do not wait on each other
    static_for<CPG>([&](auto jc) {
        constexpr int jj = decltype(jc)::value, j = GI * CPG + jj;
        uint32_t A[4];
        A[0] = as_u32(level_of_pair<B, 4 * j + 0, FIX>(r.w, dr, c_lo));
        A[1] = as_u32(level_of_pair<B, 4 * j + 1, FIX>(r.w, dr, c_hi));
        A[2] = as_u32(level_of_pair<B, 4 * j + 2, FIX>(r.w, dr, c_lo));
        A[3] = as_u32(level_of_pair<B, 4 * j + 3, FIX>(r.w, dr, c_hi));
#pragma unroll
        for (int tb = 0; tb < NT; ++tb) {
            const uint2 bf = *reinterpret_cast<const uint2 *>(xs + xo[tb] + 16 * j);
            if constexpr (jj < 2) mma_f16_z(D[j & 1][tb], A, bf.x, bf.y);
            else mma_f16(D[j & 1][tb], A, bf.x, bf.y);
        }
    });
#pragma unroll
    for (int tb = 0; tb < NT; ++tb) {
        acc[tb][0] = fmaf(c_lo.s, D[0][tb][0] + D[1][tb][0], acc[tb][0]);
        acc[tb][1] = fmaf(c_lo.s, D[0][tb][1] + D[1][tb][1], acc[tb][1]);
        acc[tb][2] = fmaf(c_hi.s, D[0][tb][2] + D[1][tb][2], acc[tb][2]);
        acc[tb][3] = fmaf(c_hi.s, D[0][tb][3] + D[1][tb][3], acc[tb][3]);
    }
}

// One group of a tile, Dynamic A8: INT8 MMAs into int32 partials P_g, then acc += s * P_g.
// xs = staged INT8 activations in operand order, xo[tb] = byte offset of this lane's token row plus 8 t;
// ctab = this warp's table space.
template <int B, int G, int NT, int GI>
__device__ __forceinline__ void group_a8(const TileRegs<B, TILE / G> &r, const int8_t *xs, const int (&xo)[NT], int8_t *ctab,
                                         const float *tt, int g, int t, float (&acc)[NT][4]) {
    constexpr int MPG = G / 32;                  // MMAs per group
    constexpr int L = B == 1 ? 1 : (1 << (B - 1));
    constexpr int NE = carrier_table_stride(B);   // bytes from one row's table to the next
    const uint2 p_lo = r.prm[0][GI], p_hi = r.prm[1][GI];
    uint4 tab_lo = make_uint4(0, 0, 0, 0), tab_hi = make_uint4(0, 0, 0, 0);
    const int8_t *trow_lo = ctab + g * NE, *trow_hi = ctab + (g + 8) * NE;
    if constexpr (B >= 3) {  // lane (g, t) fills magnitudes i = t mod 4 of rows g and g + 8: u = L + i and u = L - i
        __syncwarp();
        const __half2 ab_lo = as_h2(p_lo.y), ab_hi = as_h2(p_hi.y);
        const float a_lo = __low2float(ab_lo), b_lo = __high2float(ab_lo);
        const float a_hi = __low2float(ab_hi), b_hi = __high2float(ab_hi);
        for (int i = t; i < L; i += 4) {
            const float ti = tt[i];   // i / M, divided once per CTA
            const int c_lo = carrier_at(ti, a_lo, b_lo), c_hi = carrier_at(ti, a_hi, b_hi);
            ctab[g * NE + L + i] = (int8_t)c_lo;
            ctab[g * NE + L - i] = (int8_t)(-c_lo);
            ctab[(g + 8) * NE + L + i] = (int8_t)c_hi;
            ctab[(g + 8) * NE + L - i] = (int8_t)(-c_hi);
        }
        if (t == 0) { ctab[g * NE] = 0; ctab[(g + 8) * NE] = 0; }   // the reserved pattern
        __syncwarp();
        if constexpr (B == 4) {
            tab_lo = *reinterpret_cast<const uint4 *>(trow_lo);
            tab_hi = *reinterpret_cast<const uint4 *>(trow_hi);
        } else if constexpr (B == 3) {
            const uint2 v0 = *reinterpret_cast<const uint2 *>(trow_lo), v1 = *reinterpret_cast<const uint2 *>(trow_hi);
            tab_lo.x = v0.x; tab_lo.y = v0.y; tab_hi.x = v1.x; tab_hi.y = v1.y;
        }
    }
    int D[NT][4];
    static_for<MPG>([&](auto mc) {
        constexpr int mi = decltype(mc)::value, MI = GI * MPG + mi;
        uint32_t A[4];
        a8_row_regs<B, 0, MI>(r.w, tab_lo, trow_lo, A[0], A[2]);
        a8_row_regs<B, 1, MI>(r.w, tab_hi, trow_hi, A[1], A[3]);
#pragma unroll
        for (int tb = 0; tb < NT; ++tb) {
            const uint2 bf = *reinterpret_cast<const uint2 *>(xs + xo[tb] + 32 * MI);
            if constexpr (mi == 0) mma_s8_z(D[tb], A, bf.x, bf.y);
            else mma_s8(D[tb], A, bf.x, bf.y);
        }
    });
    const float s_lo = __uint_as_float(p_lo.x & 0x7FFFFFFFu), s_hi = __uint_as_float(p_hi.x & 0x7FFFFFFFu);
#pragma unroll
    for (int tb = 0; tb < NT; ++tb) {
        acc[tb][0] = fmaf(s_lo, (float)D[tb][0], acc[tb][0]);
        acc[tb][1] = fmaf(s_lo, (float)D[tb][1], acc[tb][1]);
        acc[tb][2] = fmaf(s_hi, (float)D[tb][2], acc[tb][2]);
        acc[tb][3] = fmaf(s_hi, (float)D[tb][3], acc[tb][3]);
    }
}

// One group of a tile, model dtype, W3: with only eight stored codes the group's levels are kept as a
// signed fp16 table per row -- q(1/3) and q(2/3) by the fp32 Horner form of Eq. gpu-horner, the other
// entries are 0 and +-1 (u = 0, the reserved pattern, reads 0) -- split into a low-byte and a high-byte
// register pair.  A half-word of four codes (the selector assembled from the 2-bit and the 1-bit plane,
// as in a8_row_regs) fetches four levels with two byte permutes, two more interleave the bytes into
// half2 MMA operands.  K order inside a 32-wide block is the operand order of cq_decode.cuh, which
// the staged activations follow: k = 16 a + 4 t + 2 h + e at half position 8 t + 4 e + 2 a + h.
// xo[tb] = element offset of this lane's token row plus 8 t.
template <int G, int NT, int GI>
__device__ __forceinline__ void group_model_w3(const TileRegs<3, TILE / G> &r, const __half *xs, const int (&xo)[NT], float (&acc)[NT][4]) {
    constexpr int MPG = G / 32;   // 32-wide k blocks per group, two k = 16 MMAs each
    uint32_t tlo[2][2], thi[2][2];
    float sc[2];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
        const uint2 p = r.prm[rr][GI];
        sc[rr] = __uint_as_float(p.x & 0x7FFFFFFFu);
        const __half2 ab = as_h2(p.y);
        const float a = __low2float(ab), b = __high2float(ab), c = (1.0f - a) - b;
        constexpr float t1 = 1.0f / 3.0f, t2 = 2.0f / 3.0f;
        const float q1 = t1 * fmaf(t1, fmaf(t1, c, b), a), q2 = t2 * fmaf(t2, fmaf(t2, c, b), a);
        const uint32_t q12 = as_u32(__floats2half2_rn(q1, q2)), nq = q12 | 0x80008000u;
        constexpr uint32_t K = 0x003CBC00u;            // bytes 4..7 of a permute: 0x00, 0xBC (-1), 0x3C (+1), 0x00
        tlo[rr][0] = prmt(q12, 0u, 0x0244u);           // low bytes of  0, -1, -q2, -q1
        tlo[rr][1] = prmt(q12, 0u, 0x4204u);           //               0, q1, q2, 1
        thi[rr][0] = prmt(nq, K, 0x1354u);             // high bytes of 0, -1, -q2, -q1
        thi[rr][1] = prmt(q12, K, 0x6314u);            //               0, q1, q2, 1
    }
    float D[NT][4];
    static_for<MPG>([&](auto mc) {
        constexpr int mi = decltype(mc)::value, MI = GI * MPG + mi;
        uint32_t A[2][4];   // [e][a0 a1 a2 a3]
        static_for<2>([&](auto rc) {
            constexpr int RR = decltype(rc)::value;
            constexpr int rho = (2 + 2 * (MI & 1) + RR) & 3;   // where the 1-bit plane keeps this selector's bits
            const uint32_t x0 = RR ? (r.w[MI] >> 2) : r.w[MI];
            const uint32_t w1 = r.w[4 + (MI >> 1)];
            const uint32_t y = rho == 2 ? w1 : rho == 3 ? (w1 >> 1) : rho == 0 ? (w1 << 2) : (w1 << 1);
            const uint32_t sel = (x0 & 0x33333333u) | (y & 0x44444444u);
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const uint32_t se = e ? (sel >> 16) : sel;
                const uint32_t lo4 = prmt(tlo[RR][0], tlo[RR][1], se), hi4 = prmt(thi[RR][0], thi[RR][1], se);
                A[e][RR] = prmt(lo4, hi4, 0x5140u);        // levels of n = 0, 1
                A[e][2 + RR] = prmt(lo4, hi4, 0x7362u);    // levels of n = 2, 3
            }
        });
#pragma unroll
        for (int tb = 0; tb < NT; ++tb) {
            const uint4 bf = *reinterpret_cast<const uint4 *>(xs + xo[tb] + 32 * MI);
            if constexpr (mi == 0) mma_f16_z(D[tb], A[0], bf.x, bf.y);
            else mma_f16(D[tb], A[0], bf.x, bf.y);
            mma_f16(D[tb], A[1], bf.z, bf.w);
        }
    });
#pragma unroll
    for (int tb = 0; tb < NT; ++tb) {
        acc[tb][0] = fmaf(sc[0], D[tb][0], acc[tb][0]);
        acc[tb][1] = fmaf(sc[0], D[tb][1], acc[tb][1]);
        acc[tb][2] = fmaf(sc[1], D[tb][2], acc[tb][2]);
        acc[tb][3] = fmaf(sc[1], D[tb][3], acc[tb][3]);
    }
}


// ---- the one- and two-token path (MODE 2): no MMA.  A warp-level MMA occupies the issue port of its
// scheduler for about as long as a dozen ordinary instructions, and with one token seven eighths of its
// columns are wasted; a packed-half FMA per pair of weights and token is cheaper.  Lane (g, t) keeps,
// per token, a half2 accumulator for each of its two rows (the even and the odd k of its pairs); it is
// promoted to fp32 and scaled by s once per group, and the four lanes that share a row add their
// partial sums when the row block is finished.  NT is the number of tokens; xo[tok] is the element offset
// of the token's staged row plus 4 t (W3: 8 t, operand order).  The staged activations are scaled so that
// the row maximum lies in [2^10, 2^11): sixteen products of a normalised level cannot leave the fp16 range.
__device__ __forceinline__ float h2sum(__half2 v) { return __low2float(v) + __high2float(v); }

template <int B, int G, int NT, int GI, bool FIX>
__device__ __forceinline__ void group_dot(const TileRegs<B, TILE / G> &r, const DecodeRegs &dr, const __half *xs, const int (&xo)[NT],
                                          float (&acc)[NT][4]) {
    constexpr int CPG = G / 16;
    const RowPoly c[2] = {make_poly<B>(r.prm[0][GI]), make_poly<B>(r.prm[1][GI])};
    __half2 h[NT][2];
#pragma unroll
    for (int tk = 0; tk < NT; ++tk) { h[tk][0] = __float2half2_rn(0.0f); h[tk][1] = h[tk][0]; }
    static_for<CPG>([&](auto jc) {
        constexpr int jj = decltype(jc)::value, j = GI * CPG + jj;
        uint2 xv[NT];
#pragma unroll
        for (int tk = 0; tk < NT; ++tk) xv[tk] = *reinterpret_cast<const uint2 *>(xs + xo[tk] + 16 * j);
        static_for<4>([&](auto ic) {
            constexpr int i = decltype(ic)::value, rr = i & 1;
            const __half2 lv = level_of_pair<B, 4 * j + i, FIX>(r.w, dr, c[rr]);
#pragma unroll
            for (int tk = 0; tk < NT; ++tk) h[tk][rr] = __hfma2(lv, as_h2(i < 2 ? xv[tk].x : xv[tk].y), h[tk][rr]);
        });
    });
#pragma unroll
    for (int tk = 0; tk < NT; ++tk) {
        acc[tk][0] = fmaf(c[0].s, h2sum(h[tk][0]), acc[tk][0]);
        acc[tk][2] = fmaf(c[1].s, h2sum(h[tk][1]), acc[tk][2]);
    }
}

// W3 on the dot path: the register table of group_model_w3, the levels multiplied into half2 accumulators.
template <int G, int NT, int GI>
__device__ __forceinline__ void group_dot_w3(const TileRegs<3, TILE / G> &r, const __half *xs, const int (&xo)[NT], float (&acc)[NT][4]) {
    constexpr int MPG = G / 32;
    uint32_t tlo[2][2], thi[2][2];
    float sc[2];
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
        const uint2 p = r.prm[rr][GI];
        sc[rr] = __uint_as_float(p.x & 0x7FFFFFFFu);
        const __half2 ab = as_h2(p.y);
        const float a = __low2float(ab), b = __high2float(ab), c = (1.0f - a) - b;
        constexpr float t1 = 1.0f / 3.0f, t2 = 2.0f / 3.0f;
        const float q1 = t1 * fmaf(t1, fmaf(t1, c, b), a), q2 = t2 * fmaf(t2, fmaf(t2, c, b), a);
        const uint32_t q12 = as_u32(__floats2half2_rn(q1, q2)), nq = q12 | 0x80008000u;
        constexpr uint32_t K = 0x003CBC00u;
        tlo[rr][0] = prmt(q12, 0u, 0x0244u);
        tlo[rr][1] = prmt(q12, 0u, 0x4204u);
        thi[rr][0] = prmt(nq, K, 0x1354u);
        thi[rr][1] = prmt(q12, K, 0x6314u);
    }
    __half2 h[NT][2];
#pragma unroll
    for (int tk = 0; tk < NT; ++tk) { h[tk][0] = __float2half2_rn(0.0f); h[tk][1] = h[tk][0]; }
    static_for<MPG>([&](auto mc) {
        constexpr int mi = decltype(mc)::value, MI = GI * MPG + mi;
        uint4 xv[NT];
#pragma unroll
        for (int tk = 0; tk < NT; ++tk) xv[tk] = *reinterpret_cast<const uint4 *>(xs + xo[tk] + 32 * MI);
        static_for<2>([&](auto rc) {
            constexpr int RR = decltype(rc)::value;
            constexpr int rho = (2 + 2 * (MI & 1) + RR) & 3;
            const uint32_t x0 = RR ? (r.w[MI] >> 2) : r.w[MI];
            const uint32_t w1 = r.w[4 + (MI >> 1)];
            const uint32_t y = rho == 2 ? w1 : rho == 3 ? (w1 >> 1) : rho == 0 ? (w1 << 2) : (w1 << 1);
            const uint32_t sel = (x0 & 0x33333333u) | (y & 0x44444444u);
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const uint32_t se = e ? (sel >> 16) : sel;
                const uint32_t lo4 = prmt(tlo[RR][0], tlo[RR][1], se), hi4 = prmt(thi[RR][0], thi[RR][1], se);
                const __half2 l01 = as_h2(prmt(lo4, hi4, 0x5140u)), l23 = as_h2(prmt(lo4, hi4, 0x7362u));
#pragma unroll
                for (int tk = 0; tk < NT; ++tk) {
                    h[tk][RR] = __hfma2(l01, as_h2(e ? xv[tk].z : xv[tk].x), h[tk][RR]);
                    h[tk][RR] = __hfma2(l23, as_h2(e ? xv[tk].w : xv[tk].y), h[tk][RR]);
                }
            }
        });
    });
#pragma unroll
    for (int tk = 0; tk < NT; ++tk) {
        acc[tk][0] = fmaf(sc[0], h2sum(h[tk][0]), acc[tk][0]);
        acc[tk][2] = fmaf(sc[1], h2sum(h[tk][1]), acc[tk][2]);
    }
}

template <int B, int G, int NT, int MODE>
__device__ __forceinline__ void compute_tile(const TileRegs<B, TILE / G> &r, const DecodeRegs &dr, const uint8_t *xs, const int (&xo)[NT],
                                             int8_t *ctab, const float *tt, int g, int t, float (&acc)[NT][4]) {
    constexpr int GPT = TILE / G;
    static_for<GPT>([&](auto gc) {
        constexpr int GI = decltype(gc)::value;
        if constexpr (MODE == 2 && B == 3) {
            group_dot_w3<G, NT, GI>(r, reinterpret_cast<const __half *>(xs), xo, acc);
        } else if constexpr (MODE == 2) {
            const bool fix = B > 1 && __any_sync(0xffffffffu, (r.prm[0][GI].x | r.prm[1][GI].x) >> 31);
            if (!fix) group_dot<B, G, NT, GI, false>(r, dr, reinterpret_cast<const __half *>(xs), xo, acc);
            else group_dot<B, G, NT, GI, true>(r, dr, reinterpret_cast<const __half *>(xs), xo, acc);
        } else if constexpr (MODE == 0 && B == 3) {
            group_model_w3<G, NT, GI>(r, reinterpret_cast<const __half *>(xs), xo, acc);
        } else if constexpr (MODE == 0) {
            const bool fix = B > 1 && __any_sync(0xffffffffu, (r.prm[0][GI].x | r.prm[1][GI].x) >> 31);
            if (!fix) group_model<B, G, NT, GI, false>(r, dr, reinterpret_cast<const __half *>(xs), xo, acc);
            else group_model<B, G, NT, GI, true>(r, dr, reinterpret_cast<const __half *>(xs), xo, acc);
        } else {
            group_a8<B, G, NT, GI>(r, reinterpret_cast<const int8_t *>(xs), xo, ctab, tt, g, t, acc);
        }
    });
}

// How the NB x KT tiles are cut into one contiguous run per CTA.  Runs are cut on a "virtual" line
// in which every row block is KT tiles preceded by E overhead units: a CTA whose run crosses into
// a new row block pays a second prologue and a second combine, worth about E tiles, so it is given
// that many tiles fewer.  With V units and P CTAs, CTA c owns the units [floor(V c / P), floor(V (c + 1) / P)).
__host__ __device__ inline int64_t cut_start(int64_t c, int64_t V, int64_t P) { return (V * c) / P; }
// The CTA whose run holds tile (nb, kb): the largest c with floor(V c / P) <= v, i.e. V c < (v + 1) P.
__host__ __device__ inline int owner_of(int nb, int kb, int KT, int E, int64_t V, int64_t P) {
    const int64_t v = (int64_t)nb * (KT + E) + E + kb;
    return (int)(((v + 1) * P - 1) / V);
}

// A wait on a ring barrier.  Every wait is bounded; a wait that gives up records its code in the
// status word and marks the CTA, after which the CTA no longer waits (its output is then undefined,
// cq_gemm_status reports CQ_ERR_TIMEOUT) but still runs to its end.
__device__ __forceinline__ void ring_wait(uint64_t *bar, uint32_t parity, volatile int *dead, int *status, int code) {
    if (tc::mbar_try_wait(bar, parity)) return;
    if (*dead) return;
    if (!tc::mbar_wait(bar, parity, status, code)) *dead = 1;
}

// ------------------------------------------------------------------------------------------
// MODE 0: model dtype (MMA, NT blocks of 8 tokens).  MODE 1: Dynamic A8 (xq = int8 carrier [M][x8_pitch],
// dxs = row scales).  MODE 2: model dtype without MMA for NT = M <= 2 tokens.
template <int B, int G, int NT, int MODE>
__global__ void __launch_bounds__(GEMV_THREADS, gemv_occ(B, G, NT, MODE))
gemv_kernel(const uint8_t *__restrict__ layout, Dims d, const uint16_t *__restrict__ x, const int8_t *__restrict__ xq,
            int64_t x8_pitch, const float *__restrict__ dxs, uint16_t *__restrict__ y, int M, int E,
            float *__restrict__ partial, int *__restrict__ counters, int nstage, uint32_t ring_off, int *__restrict__ status, bool xf16) {
    constexpr int GPT = TILE / G;
    constexpr int L = B == 1 ? 1 : (1 << (B - 1));
    constexpr bool RING = gemv_uses_ring(B, G, NT, MODE);
    constexpr bool F16 = MODE != 1;        // activations staged as fp16 (model dtype) or as the INT8 carrier
    constexpr int ES = F16 ? 2 : 1;        // bytes per staged activation element
    constexpr int CB = 2048 * B, TB = CB + 1024 * GPT;   // bytes of a tile's code part and of a whole tile
    constexpr int XPAD = F16 ? (B == 3 ? 2 * XS_PAD : XS_PAD) : XS_PAD8;   // W3 reads 16 bytes per lane: rows 64 bytes apart in the banks
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ __align__(8) uint64_t s_full[MAX_STAGES], s_empty[MAX_STAGES];
    __shared__ float s_inv[16];
    __shared__ unsigned s_max[16];
    __shared__ int s_last, s_dead;
    __shared__ float s_t[MODE == 1 && B >= 3 ? 128 : 1];   // Dynamic A8: t_i = i / M of the carrier tables

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int VT = d.KT + E;                       // virtual units per row block
    const int64_t V = (int64_t)d.NB * VT, P = gridDim.x;
    int64_t v_begin, v_end;
    const bool small = V * (P + 1) < (1ll << 31);   // the usual case: 32-bit divisions
    auto row_block_of = [&](int64_t v) { return small ? (int)((uint32_t)v / (uint32_t)VT) : (int)(v / VT); };
    if (small) {
        v_begin = ((uint32_t)V * blockIdx.x) / (uint32_t)P;
        v_end = ((uint32_t)V * (blockIdx.x + 1u)) / (uint32_t)P;
    } else {
        v_begin = cut_start(blockIdx.x, V, P);
        v_end = cut_start((int64_t)blockIdx.x + 1, V, P);
    }
    if (threadIdx.x < nstage) { tc::mbar_init(&s_full[threadIdx.x], 1); tc::mbar_init(&s_empty[threadIdx.x], GEMV_WARPS); }
    if (threadIdx.x < 32) tc::fence_barrier_init();
    if (threadIdx.x == 0) s_dead = 0;
    if (threadIdx.x < 16) { s_max[threadIdx.x] = 0; s_inv[threadIdx.x] = 1.0f; }
    if constexpr (MODE == 1 && B >= 3) {
        if (threadIdx.x < L) s_t[threadIdx.x] = __fdiv_rn((float)threadIdx.x, (float)(L - 1));
    }
    __syncthreads();
    uint8_t *ring = smem + ring_off;

    // ---- the ring's producer is lane 0 of warp 0.  The run's tiles are one contiguous byte range: it is
    // copied stage by stage, the first round right away (weights do not depend on the previous kernel of
    // the stream), later tiles into the stage of the tile consumed one step earlier.
    // Every thread walks its CTA's run once (a few iterations): where it starts in the layout and how many
    // tiles it holds.  The first round of copies is started by the lanes of warp 0, one stage each.
    const uint8_t *src = layout;
    int n_tiles = 0;
    {
        int64_t first = -1;
        for (int64_t v = v_begin; v < v_end;) {
            const int nb = row_block_of(v);
            const int64_t ve = min(v_end, (int64_t)(nb + 1) * VT);
            const int kb_begin = max(0, (int)(v - (int64_t)nb * VT) - E), kb_end = max(0, (int)(ve - (int64_t)nb * VT) - E);
            v = ve;
            if (kb_end > kb_begin) {
                if (first < 0) first = (int64_t)nb * d.KT + kb_begin;
                n_tiles += kb_end - kb_begin;
            }
        }
        src += (size_t)(first < 0 ? 0 : first) * (size_t)TB;
    }
    if (RING && warp == 0 && lane < n_tiles && lane < nstage) {
        tc::mbar_arrive_expect_tx(&s_full[lane], (uint32_t)TB);
        tc::bulk_load(ring + (size_t)lane * TB, src + (size_t)lane * TB, (uint32_t)TB, &s_full[lane]);
    }
    DecodeRegs dr = {};
    if constexpr (F16 && B != 3) dr = load_decode_regs();

    int8_t *ctab = nullptr;
    if constexpr (MODE == 1 && B >= 3) ctab = reinterpret_cast<int8_t *>(smem) + M * (MAX_SUB * TILE + XS_PAD8) + warp * 16 * carrier_table_stride(B);

    int st = 0, prev_st = 0;            // ring stage of the next tile (and of the one before it)
    uint32_t ph = 0, prev_ph = 0;       // and the parity its "full" barrier completes with
    int it = 0;                         // tiles consumed so far
    bool first_slice = true;
    for (int64_t v = v_begin; v < v_end;) {
        const int nb = row_block_of(v);
        const int64_t ve = min(v_end, (int64_t)(nb + 1) * VT);        // end of this CTA's units in row block nb
        const int kb_begin = max(0, (int)(v - (int64_t)nb * VT) - E);
        const int kb_end = max(0, (int)(ve - (int64_t)nb * VT) - E);
        v = ve;
        if (kb_end <= kb_begin) continue;                              // only overhead units of this row block
        float total[NT][4];
#pragma unroll
        for (int tb = 0; tb < NT; ++tb)
#pragma unroll
            for (int i = 0; i < 4; ++i) total[tb][i] = 0.0f;

        for (int ks = kb_begin; ks < kb_end; ks += MAX_SUB) {
            const int ke = min(kb_end, ks + MAX_SUB);
            const int slice_k = (ke - ks) * TILE, XS = slice_k + XPAD;
            const int64_t k_base = (int64_t)ks * TILE;

            // The activations, the workspace and y may be produced or still used by the kernel launched
            // before this one: wait for it (a no-op unless the launch allowed programmatic overlap), then
            // let the next kernel's CTAs start as soon as there is room for them.
            if (first_slice) {
                asm volatile("griddepcontrol.wait;" ::: "memory");
                asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
                first_slice = false;
            }
            // direct variant: the first tiles of the slice are requested before the activations are staged
            constexpr int NBUF = RING ? 1 : (B <= 4 ? 3 : 2);
            const uint8_t *tile0 = layout + ((size_t)nb * d.KT + ks) * (size_t)TB;
            const uint8_t *wl = tile0 + warp * 256 * B + lane * 16;              // next tile to load (codes)
            const uint8_t *pl = tile0 + CB + ((warp * 16 + g) * GPT) * 8;        // next tile to load (params)
            TileRegs<B, GPT> buf0, buf1, buf2;   // separate objects (an array of them ends up in local memory)
            auto buf_at = [&](auto ic) -> TileRegs<B, GPT> & {
                constexpr int i = decltype(ic)::value;
                if constexpr (i == 0) return buf0;
                else if constexpr (i == 1) return buf1;
                else return buf2;
            };
            if constexpr (!RING) {
                static_for<NBUF>([&](auto ic) {
                    constexpr int i = decltype(ic)::value;
                    if (ks + i < ke) load_tile_g<B, GPT>(buf_at(ic), wl + i * TB, pl + i * TB, lane);
                });
                wl += NBUF * TB; pl += NBUF * TB;   // tile offsets inside a round of NBUF loads are immediates
            }
            compute_barrier();  // previous slice fully consumed

            // ---- the activation slice: asynchronous copies straight into shared memory.  Thread c owns
            // the 16-byte chunk c of every token row (a slice has at most 256 chunks per row).
            const int cpr = F16 ? slice_k / 8 : slice_k / 16;
            const int c = threadIdx.x;
            if (c < cpr) {
                for (int m = 0; m < M; ++m) {
                    uint8_t *dst = smem + ((size_t)m * XS) * ES + (size_t)c * 16;
                    const void *src = nullptr;
                    if constexpr (F16) {
                        const int64_t k = k_base + (int64_t)c * 8;
                        if (k < d.K) src = x + (int64_t)m * d.K + k;   // K % 8 == 0 always
                    } else {
                        src = xq + (int64_t)m * x8_pitch + k_base + c * 16;  // already in MMA operand order; pitch multiple of 128, zero beyond K
                    }
                    if (src) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
                    else *(uint4 *)dst = make_uint4(0, 0, 0, 0);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            if constexpr (F16) {
                __half *xs = reinterpret_cast<__half *>(smem);
                // pass 1: row maxima of |x| (as bf16 bit patterns) from the chunks this thread copied
                auto thread_max = [&](int m) -> unsigned {
                    unsigned mx = 0;
                    if (c < cpr) {
                        const uint4 v4 = *(const uint4 *)(xs + m * XS + c * 8);
                        const uint32_t ws[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
                        for (int q = 0; q < 4; ++q) { mx = max(mx, ws[q] & 0x7FFFu); mx = max(mx, (ws[q] >> 16) & 0x7FFFu); }
                    }
                    return mx;
                };
                // pass 2: every thread derives the power-of-two scale that puts the row maximum in
                // [2^14, 2^15) (MODE 2: [2^10, 2^11), its sums stay in fp16) and converts the chunks it owns
                auto convert_row = [&](int m) {
                    const unsigned mb = s_max[m];
                    bool usable;
                    const int e_max = act_max_exponent(mb, xf16, usable);   // the row maximum lies in [2^e_max, 2^(e_max+1))
                    int sh = usable ? (MODE == 2 ? 10 : 14) - e_max : 0;
                    sh = max(min(sh, 100), -100);
                    const float sc = __uint_as_float((uint32_t)(127 + sh) << 23);   // 2^sh
                    if (threadIdx.x == m) s_inv[m] = __uint_as_float((uint32_t)(127 - sh) << 23);
                    uint32_t ws[4] = {0u, 0u, 0u, 0u};
                    if (c < cpr) {
                        const uint4 v4 = *(const uint4 *)(xs + m * XS + c * 8);
                        ws[0] = v4.x; ws[1] = v4.y; ws[2] = v4.z; ws[3] = v4.w;
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float lo = act_to_float(ws[q] & 0xFFFFu, xf16) * sc, hi = act_to_float(ws[q] >> 16, xf16) * sc;
                            ws[q] = as_u32(__floats2half2_rn(lo, hi));
                        }
                    }
                    if constexpr (B != 3) {
                        if (c < cpr) *(uint4 *)(xs + m * XS + c * 8) = make_uint4(ws[0], ws[1], ws[2], ws[3]);
                    } else {
                        // W3 reads its activations in the operand order of cq_decode.cuh: the four chunks of a
                        // 32-wide block (four neighbouring lanes) are all read before any of them is rewritten
                        __syncwarp();
                        if (c < cpr) {
                            __half *blk = xs + m * XS + (c >> 2) * 32 + 16 * (c & 1) + 2 * ((c >> 1) & 1);   // t = 2 (c & 1), a = (c >> 1) & 1
#pragma unroll
                            for (int tt = 0; tt < 2; ++tt) {   // values k+0, k+2 (e = 0) | k+1, k+3 (e = 1) of t = 2 (c & 1) + tt
                                *reinterpret_cast<uint32_t *>(blk + 8 * tt) = prmt(ws[2 * tt], ws[2 * tt + 1], 0x5410u);
                                *reinterpret_cast<uint32_t *>(blk + 8 * tt + 4) = prmt(ws[2 * tt], ws[2 * tt + 1], 0x7632u);
                            }
                        }
                    }
                };
                if (M <= 2) {   // the common decode case: short plain loops
                    for (int m = 0; m < M; ++m) {
                        const unsigned mx = __reduce_max_sync(0xffffffffu, thread_max(m));
                        if (lane == 0 && mx) atomicMax(&s_max[m], mx);
                    }
                    compute_barrier();
                    for (int m = 0; m < M; ++m) convert_row(m);
                } else {        // more rows: they are independent, so their loads, reductions and atomics overlap
                    unsigned mxs[8 * NT];
#pragma unroll
                    for (int m = 0; m < 8 * NT; ++m) mxs[m] = m < M ? thread_max(m) : 0u;
#pragma unroll
                    for (int m = 0; m < 8 * NT; ++m) {
                        if (m < M) {
                            const unsigned mx = __reduce_max_sync(0xffffffffu, mxs[m]);
                            if (lane == 0 && mx) atomicMax(&s_max[m], mx);
                        }
                    }
                    compute_barrier();
#pragma unroll 4
                    for (int m = 0; m < 8 * NT; ++m)
                        if (m < M) convert_row(m);
                }
            } else {
                if (threadIdx.x < 16) s_inv[threadIdx.x] = threadIdx.x < M ? dxs[threadIdx.x] * (1.0f / 127.0f) : 0.0f;
            }
            compute_barrier();
            if (F16 && threadIdx.x < 16) s_max[threadIdx.x] = 0;  // next slice's maxima start from zero

            // ---- consume the tiles of this slice from the ring
            float acc[NT][4];
#pragma unroll
            for (int tb = 0; tb < NT; ++tb)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[tb][i] = 0.0f;
            // this lane's B-fragment base per token block: row g of the block (token columns beyond M read
            // the last real row; their results are never stored), k offset 4 t or 8 t, in elements
            int xo[NT];
#pragma unroll
            for (int tb = 0; tb < NT; ++tb)
                xo[tb] = (MODE == 2 ? min(tb, M - 1) : min(tb * 8 + g, M - 1)) * XS + ((F16 && B != 3) ? 4 : 8) * t;
            const uint8_t *xcur = smem;
            if constexpr (!RING) {
                int to_load = (ke - ks) - NBUF;                              // tiles not yet requested
                for (int left = ke - ks; left > 0; left -= NBUF) {
                    static_for<NBUF>([&](auto ic) {
                        constexpr int i = decltype(ic)::value;
                        if (i < left) {
                            compute_tile<B, G, NT, MODE>(buf_at(ic), dr, xcur, xo, ctab, s_t, g, t, acc);
                            xcur += TILE * ES;
                            if (to_load > 0) { load_tile_g<B, GPT>(buf_at(ic), wl + i * TB, pl + i * TB, lane); --to_load; }
                        }
                    });
                    wl += NBUF * TB; pl += NBUF * TB;
                }
            } else {
#pragma unroll 1
            for (int kb = ks; kb < ke; ++kb) {
                // Refill the stage every warp has copied out of by now (that of the previous tile) with the tile
                // nstage - 1 ahead; the warps take turns so that no warp carries the producer's instructions alone.
                if (lane == 0 && it > 0 && ((it - 1) & (GEMV_WARPS - 1)) == warp && it - 1 + nstage < n_tiles) {
                    ring_wait(&s_empty[prev_st], prev_ph, &s_dead, status, ERR_GEMV_EMPTY);
                    tc::mbar_arrive_expect_tx(&s_full[prev_st], (uint32_t)TB);
                    tc::bulk_load(ring + (size_t)prev_st * TB, src + (size_t)(it - 1 + nstage) * TB, (uint32_t)TB, &s_full[prev_st]);
                }
                ring_wait(&s_full[st], ph, &s_dead, status, ERR_GEMV_FULL);
                const uint8_t *stage = ring + (size_t)st * TB;
                TileRegs<B, GPT> regs;
                load_tile<B, GPT>(regs, stage + warp * 256 * B + lane * 16, stage + CB + ((warp * 16 + g) * GPT) * 8, lane);
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&s_empty[st]);   // this warp's slice of the stage is in registers
                prev_st = st; prev_ph = ph; ++it;
                if (++st == nstage) { st = 0; ph ^= 1u; }
                compute_tile<B, G, NT, MODE>(regs, dr, xcur, xo, ctab, s_t, g, t, acc);
                xcur += TILE * ES;
            }
            }
            // fold the slice in true units: lane (g, t) holds rows g, g+8 x tokens 2t, 2t+1 (MODE 2: token tb)
#pragma unroll
            for (int tb = 0; tb < NT; ++tb)
#pragma unroll
                for (int i = 0; i < 4; ++i) total[tb][i] = fmaf(acc[tb][i], s_inv[MODE == 2 ? tb : tb * 8 + 2 * t + (i & 1)], total[tb][i]);
        }

        // ---- finish this row block
        const bool whole = (kb_begin == 0 && kb_end == d.KT);
        // A run has at most two partial segments: one that starts inside a row block (its first) and
        // one that starts a row block without finishing it (its last); each CTA owns two partial slots.
        const int64_t n_lo = (int64_t)nb * TILE + warp * 16 + g;
        float *pslot = partial + ((size_t)blockIdx.x * 2 + (kb_begin > 0 ? 1 : 0)) * (size_t)(M * TILE);
        if constexpr (MODE == 2) {   // the four lanes of a row add their partial sums; lane t = 0 keeps the result
#pragma unroll
            for (int tb = 0; tb < NT; ++tb)
#pragma unroll
                for (int i = 0; i < 4; i += 2) {
                    total[tb][i] += __shfl_xor_sync(0xffffffffu, total[tb][i], 1);
                    total[tb][i] += __shfl_xor_sync(0xffffffffu, total[tb][i], 2);
                }
        }
#pragma unroll
        for (int tb = 0; tb < NT; ++tb)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (MODE == 2 && ((i & 1) || t != 0)) continue;
                const int tok = MODE == 2 ? tb : tb * 8 + 2 * t + (i & 1);
                const int r = warp * 16 + g + ((i >> 1) ? 8 : 0);
                if (tok >= M) continue;
                if (whole) {
                    const int64_t n = n_lo + ((i >> 1) ? 8 : 0);
                    if (n < d.N) y[(int64_t)tok * d.N + n] = float_to_act(total[tb][i], xf16);
                } else {
                    pslot[tok * TILE + r] = total[tb][i];
                }
            }
        if (!whole) {
            // The counter of a row block collects the tiles done; the CTA that completes it adds the
            // partials in K order.  The barrier orders the CTA's partial stores before thread 0's release;
            // its acquire plus the second barrier make the other CTAs' partials visible to every thread.
            compute_barrier();
            if (threadIdx.x == 0) {
                int old;
                asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(counters + nb), "r"(kb_end - kb_begin) : "memory");
                s_last = (old + (kb_end - kb_begin) == d.KT);
            }
            compute_barrier();
            if (s_last) {
                const int c_first = owner_of(nb, 0, d.KT, E, V, P);   // its segment starts the row block: slot 0
                const int n_contrib = owner_of(nb, d.KT - 1, d.KT, E, V, P) - c_first + 1;
                const float *pb = partial + ((size_t)c_first * 2 + 1) * (size_t)(M * TILE);   // slot 1 of CTA c_first + q
                if (M <= 2) {
                    for (int idx = threadIdx.x; idx < M * TILE; idx += GEMV_THREADS) {
                        const int m = idx / TILE, r = idx % TILE;
                        const int64_t n = (int64_t)nb * TILE + r;
                        float sum = 0.0f;
                        for (int q0 = 0; q0 < n_contrib; q0 += 8) {  // eight independent loads in flight, added in K order
                            float vv[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const size_t off = (size_t)(q0 + i) * 2 * (M * TILE) - (q0 + i == 0 ? (size_t)(M * TILE) : 0);
                                vv[i] = (q0 + i < n_contrib) ? __ldcg(pb + off + idx) : 0.0f;
                            }
#pragma unroll
                            for (int i = 0; i < 8; ++i) sum += vv[i];
                        }
                        if (n < d.N) y[(int64_t)m * d.N + n] = float_to_act(sum, xf16);
                    }
                } else {
                    // four consecutive channels of one token per thread and step (128-bit loads), up to eight
                    // slots in flight, added in K order
                    for (int idx = threadIdx.x; idx < M * (TILE / 4); idx += GEMV_THREADS) {
                        const int m = idx / (TILE / 4), r = (idx % (TILE / 4)) * 4;
                        const int64_t n = (int64_t)nb * TILE + r;
                        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (int q0 = 0; q0 < n_contrib; q0 += 8) {
                            float4 vv[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const size_t off = (size_t)(q0 + i) * 2 * (M * TILE) - (q0 + i == 0 ? (size_t)(M * TILE) : 0);
                                vv[i] = (q0 + i < n_contrib) ? __ldcg(reinterpret_cast<const float4 *>(pb + off + m * TILE + r))
                                                             : make_float4(0.f, 0.f, 0.f, 0.f);
                            }
#pragma unroll
                            for (int i = 0; i < 8; ++i) { sum.x += vv[i].x; sum.y += vv[i].y; sum.z += vv[i].z; sum.w += vv[i].w; }
                        }
                        const float o[4] = {sum.x, sum.y, sum.z, sum.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (n + e < d.N) y[(int64_t)m * d.N + n + e] = float_to_act(o[e], xf16);
                    }
                }
                if (threadIdx.x == 0) counters[nb] = 0;  // leave the workspace ready for the next call
            }
        }
    }
    // A CTA that gave up on a wait may still have copies in flight into its shared memory: give them time to land.
    if (s_dead) {
#pragma unroll 1
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
}

template <int B, int G, int NT, int MODE>
cudaError_t launch_one(const void *layout, const Dims &d, const uint16_t *x, const int8_t *xq, int64_t x8_pitch,
                       const float *dxs, uint16_t *y, int M, int P, int max_run, int E, float *partial, int *counters,
                       int *status, bool act_f16, cudaStream_t st) {
    constexpr int GPT = TILE / G;
    constexpr int TB = 2048 * B + 1024 * GPT;
    int64_t sub64 = max_run;   // the longest run bounds the activation slice a CTA stages
    if (sub64 > d.KT) sub64 = d.KT;
    if (sub64 > MAX_SUB) sub64 = MAX_SUB;
    const int sub_tiles = (int)sub64;
    const int XS = sub_tiles * TILE + (B == 3 ? 2 * XS_PAD : XS_PAD);
    size_t xbytes = MODE != 1 ? (size_t)M * XS * 2 : (size_t)M * (MAX_SUB * TILE + XS_PAD8) + (B >= 3 ? 8 * 16 * carrier_table_stride(B) : 0);
    const uint32_t ring_off = (uint32_t)((xbytes + 127) / 128 * 128);
    constexpr int OCC = gemv_occ(B, G, NT, MODE);
    int nstage = 0;
    if (gemv_uses_ring(B, G, NT, MODE)) {
        nstage = (int)((gemv_smem_budget(OCC) - (int64_t)ring_off) / TB);
        if (nstage > MAX_STAGES) nstage = MAX_STAGES;
        if (nstage > max_run) nstage = max_run < 2 ? 2 : max_run;   // a run never holds more tiles than this
        if (nstage < 2) return cudaErrorInvalidConfiguration;
    }
    const size_t smem = ring_off + (size_t)nstage * TB;
    auto kern = gemv_kernel<B, G, NT, MODE>;
    static std::atomic<uint64_t> attr_done{0};
    cudaError_t e = ensure_func_attr(kern, attr_done, cudaFuncAttributeMaxDynamicSharedMemorySize, gemv_smem_budget(OCC));
    if (e != cudaSuccess) return e;
    // Programmatic dependent launch: this kernel may begin (and prefetch weights) while the previous
    // kernel of the stream drains; it waits for that kernel before touching anything but the weights.
    static const bool use_pdl = getenv("CQ_NO_PDL") == nullptr;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)P);
    cfg.blockDim = dim3(GEMV_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = use_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, (const uint8_t *)layout, d, x, xq, x8_pitch, dxs, y, M, E, partial, counters, nstage,
                              ring_off, status, act_f16);
}

template <int B, int G>
cudaError_t dispatch_nt_mode(const void *layout, const Dims &d, const uint16_t *x, const int8_t *xq, int64_t x8_pitch,
                             const float *dxs, uint16_t *y, int M, int mode, int P, int max_run, int E, float *partial,
                             int *counters, int *status, bool act_f16, cudaStream_t st) {
    if (mode == 0) {
        if (M == 1) return launch_one<B, G, 1, 2>(layout, d, x, xq, x8_pitch, dxs, y, M, P, max_run, E, partial, counters, status, act_f16, st);
        if (M == 2) return launch_one<B, G, 2, 2>(layout, d, x, xq, x8_pitch, dxs, y, M, P, max_run, E, partial, counters, status, act_f16, st);
        if (M <= 8) return launch_one<B, G, 1, 0>(layout, d, x, xq, x8_pitch, dxs, y, M, P, max_run, E, partial, counters, status, act_f16, st);
        return launch_one<B, G, 2, 0>(layout, d, x, xq, x8_pitch, dxs, y, M, P, max_run, E, partial, counters, status, act_f16, st);
    }
    if (M <= 8) return launch_one<B, G, 1, 1>(layout, d, x, xq, x8_pitch, dxs, y, M, P, max_run, E, partial, counters, status, act_f16, st);
    return launch_one<B, G, 2, 1>(layout, d, x, xq, x8_pitch, dxs, y, M, P, max_run, E, partial, counters, status, act_f16, st);
}

template <int B>
cudaError_t dispatch_g(const void *layout, const Dims &d, const uint16_t *x, const int8_t *xq, int64_t x8_pitch,
                       const float *dxs, uint16_t *y, int M, int mode, int P, int max_run, int E, float *partial,
                       int *counters, int *status, bool act_f16, cudaStream_t st) {
    switch (d.G) {
        case 32: return dispatch_nt_mode<B, 32>(layout, d, x, xq, x8_pitch, dxs, y, M, mode, P, max_run, E, partial, counters, status, act_f16, st);
        case 64: return dispatch_nt_mode<B, 64>(layout, d, x, xq, x8_pitch, dxs, y, M, mode, P, max_run, E, partial, counters, status, act_f16, st);
        default: return dispatch_nt_mode<B, 128>(layout, d, x, xq, x8_pitch, dxs, y, M, mode, P, max_run, E, partial, counters, status, act_f16, st);
    }
}

}  // namespace

// Streaming multiprocessors of the current device (148 on a B200; that figure also stands in when no
// device can be asked, so that size queries work on a machine without a GPU).
int sm_count() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return 148; }
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { (void)cudaGetLastError(); return 148; }
    cached[dev].store(n, std::memory_order_relaxed);
    return n;
}

// Number of CTAs of the small-M path (one run of tiles each; as many as are resident at once, matching
// the __launch_bounds__ of the kernel) and the length of the longest run.
GemvPlan gemv_plan(const Dims &d, int64_t M, int mode) {
    GemvPlan p;
    const int64_t T = (int64_t)d.NB * d.KT;
    const int G = d.G > TILE ? TILE : d.G;   // wide groups run the G = 128 code
    int64_t P = (int64_t)sm_count() * gemv_occ(d.B, G, gemv_variant_nt(M, mode), gemv_variant_mode(M, mode));
    if (P > T) P = T;
    p.ctas = (int)P;
    p.overhead = (T / P >= 6) ? 3 : 0;   // a second prologue + combine costs about three tiles of work
    p.max_run = (int)(((int64_t)d.NB * (d.KT + p.overhead)) / P + 1);   // units, an upper bound of the tiles in a run
    return p;
}

cudaError_t launch_gemv(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int mode,
                        bool act_f16, uint8_t *ws, const Workspace &plan, cudaStream_t st, bool prequantized) {
    const GemvPlan gp = gemv_plan(d, M, mode);
    float *partial = reinterpret_cast<float *>(ws + plan.partial_off);
    int *counters = reinterpret_cast<int *>(ws + plan.counters_off);
    int *status = reinterpret_cast<int *>(ws + plan.status_off);
    int8_t *xq = reinterpret_cast<int8_t *>(ws + plan.x8_off);
    float *dxs = reinterpret_cast<float *>(ws + plan.dx_off);
    const int64_t pitch = (int64_t)d.KT * TILE;
    if (mode == 1 && !prequantized) {
        cudaError_t e = launch_quantize_a8(x, M, d.K, xq, pitch, dxs, true, act_f16, st);
        if (e != cudaSuccess) return e;
    }
    const int Mi = (int)M, P = gp.ctas, ms = gp.max_run;
    const int E = gp.overhead;
#ifdef CQ_GEMV_SUBSET   // development builds: only the widths under study
    switch (d.B) {
        case 1: return dispatch_g<1>(layout, d, x, xq, pitch, dxs, y, Mi, mode, P, ms, E, partial, counters, status, act_f16, st);
        case 4: return dispatch_g<4>(layout, d, x, xq, pitch, dxs, y, Mi, mode, P, ms, E, partial, counters, status, act_f16, st);
        default: return cudaErrorNotSupported;
    }
#else
    switch (d.B) {
        case 1: return dispatch_g<1>(layout, d, x, xq, pitch, dxs, y, Mi, mode, P, ms, E, partial, counters, status, act_f16, st);
        case 2: return dispatch_g<2>(layout, d, x, xq, pitch, dxs, y, Mi, mode, P, ms, E, partial, counters, status, act_f16, st);
        case 3: return dispatch_g<3>(layout, d, x, xq, pitch, dxs, y, Mi, mode, P, ms, E, partial, counters, status, act_f16, st);
        case 4: return dispatch_g<4>(layout, d, x, xq, pitch, dxs, y, Mi, mode, P, ms, E, partial, counters, status, act_f16, st);
        case 5: return dispatch_g<5>(layout, d, x, xq, pitch, dxs, y, Mi, mode, P, ms, E, partial, counters, status, act_f16, st);
        case 6: return dispatch_g<6>(layout, d, x, xq, pitch, dxs, y, Mi, mode, P, ms, E, partial, counters, status, act_f16, st);
        case 7: return dispatch_g<7>(layout, d, x, xq, pitch, dxs, y, Mi, mode, P, ms, E, partial, counters, status, act_f16, st);
        default: return dispatch_g<8>(layout, d, x, xq, pitch, dxs, y, Mi, mode, P, ms, E, partial, counters, status, act_f16, st);
    }
#endif
}

}  // namespace cq
