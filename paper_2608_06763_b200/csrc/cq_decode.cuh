// Code-pair extraction and the half2 level evaluation shared by the small-M and large-M kernels.
//
// A lane's record (cq_common.cuh) holds 32 pairs of stored codes; pair P sits in one 32-bit word per
// bit plane (pair_word / pair_pos) with its first code in the low and its second in the high 16 bits.  pair_T turns a
// pair into the normalised signed codes T = k / 2^(B-1) as half2 with one mask (the code lands in
// the fp16 mantissa under exponent bits 0x6400, value 1024 + u 2^pos) and one exact FMA; level_pair
// evaluates the group's cubic in Horner form (Eq. gpu-horner) on it.
#pragma once
#include <utility>

#include "cq_common.cuh"

namespace cq {

template <int... I, class F>
__device__ __forceinline__ void static_for_impl(F &&f, std::integer_sequence<int, I...>) {
    (f(std::integral_constant<int, I>{}), ...);
}
template <int N, class F>
__device__ __forceinline__ void static_for(F &&f) {
    static_for_impl(static_cast<F &&>(f), std::make_integer_sequence<int, N>{});
}

// fp16 bit patterns built with integer arithmetic only (so they are compile-time constants)
constexpr uint32_t h2dup(uint32_t h) { return h | (h << 16); }
constexpr uint32_t half_pow2(int e) { return (uint32_t)((e + 15) << 10); }                      // 2^e, -14 <= e <= 15
constexpr uint32_t half_neg_pow2_plus(int q, int c) {                                            // -(2^q + c), c < 2^q, q <= 10
    return 0x8000u | (uint32_t)((q + 15) << 10) | (uint32_t)(c << (10 - q));
}
__device__ __forceinline__ __half2 as_h2(uint32_t v) { return *reinterpret_cast<__half2 *>(&v); }
__device__ __forceinline__ uint32_t as_u32(__half2 v) { return *reinterpret_cast<uint32_t *>(&v); }

// Two stored codes of pair P as packed 16-bit integers (u_lo | u_hi << 16).
template <int B, int P>
__device__ __forceinline__ uint32_t pair_codes(const uint32_t (&w)[2 * B]) {
    uint32_t u2 = 0;
    static_for<plane_count(B)>([&](auto ic) {
        constexpr int i = decltype(ic)::value;
        constexpr int pw = plane_width(B, i);
        constexpr int W = plane_word_base(B, i) + pair_word(pw, P), pos = pair_pos(pw, P);
        constexpr uint32_t m = ((1u << pw) - 1u) * 0x00010001u;
        u2 |= ((w[W] >> pos) & m) << plane_bit_offset(B, i);
    });
    return u2;
}

// Pair P as half2 of the normalised signed code:  B >= 3: T = k / 2^(B-1);  B <= 2: k itself.
// The stored code lands in the fp16 mantissa under exponent bits 0x6400 (value 1024 + u 2^pos);
// one exact FMA removes the offset and the position scale.
template <int B, int P>
__device__ __forceinline__ __half2 pair_T(const uint32_t (&w)[2 * B]) {
    if constexpr (plane_count(B) == 1) {
        constexpr int W = pair_word(B, P), pos0 = pair_pos(B, P);
        // B = 1 keeps the field off mantissa bit 0 (the offset constant must stay representable);
        // other widths shift by 8 when the field would leave the 10 mantissa bits
        constexpr int shl = (B == 1 && pos0 <= 6) ? 1 : 0;
        constexpr int shr = (B == 1) ? (pos0 <= 6 ? 0 : 6) : (pos0 + B > 10 ? 8 : 0);
        constexpr int pos = pos0 + shl - shr;
        const uint32_t word = shl ? (w[W] << shl) : (shr ? (w[W] >> shr) : w[W]);
        constexpr uint32_t m = (((1u << B) - 1u) << pos) * 0x00010001u;
        const uint32_t hbits = (word & m) | 0x64006400u;
        constexpr uint32_t sc = (B == 1) ? half_pow2(1 - pos) : (B == 2) ? half_pow2(-pos) : half_pow2(-(pos + B - 1));
        constexpr uint32_t off = (B == 1) ? half_neg_pow2_plus(11 - pos, 1)
                               : (B == 2) ? half_neg_pow2_plus(10 - pos, 2)
                                          : half_neg_pow2_plus(10 - pos - (B - 1), 1);
        return __hfma2(as_h2(hbits), as_h2(h2dup(sc)), as_h2(h2dup(off)));
    } else {
        const uint32_t hbits = pair_codes<B, P>(w) | 0x64006400u;
        constexpr uint32_t sc = half_pow2(-(B - 1)), off = half_neg_pow2_plus(10 - (B - 1), 1);
        return __hfma2(as_h2(hbits), as_h2(h2dup(sc)), as_h2(h2dup(off)));
    }
}

// The small-M kernel's variant, arranged so that every instruction carries at most one literal: a
// logic or a packed-half instruction encodes a single immediate (and a packed-half FMA none in its
// addend), so any further constant costs a register move per use unless it lives in a register; the
// few that must are read once per kernel from constant memory (`DecodeRegs`), which keeps the
// compiler from folding them back into literals.  What comes out is the signed code in "code units":
//   B = 1:     +-1, the bit sent straight to the fp16 sign: 0xBC00 ^ (bit << 15)  (a shift and one logic op)
//   B = 2..6:  the integer k itself: the field is read as base + u under exponent bits chosen by
//              where the field sits (base = 2^(10 - pos)), and one add of the literal -(base + 2^(B-1))
//              leaves k, exactly;
//   B = 7, 8:  T = k / 2^(B-1) by one FMA (scale as the literal, offset from a register): k^3 would
//              leave the fp16 range.
// code_unit<B>() is the normalised position t of one unit: t = |T| code_unit.
template <int B>
__host__ __device__ constexpr float code_unit() {
    return B <= 2 ? 1.0f : B <= 6 ? 1.0f / (float)((1 << (B - 1)) - 1) : (float)(1 << (B - 1)) / (float)((1 << (B - 1)) - 1);
}
struct DecodeRegs { uint32_t one_neg; uint32_t off; uint32_t magic[4]; };
__constant__ uint32_t c_decode_consts[8] = {
    0xBC00BC00u,                                          // -1, -1
    0xC880C880u,                                          // -9, -9 = -(1024 + 128) / 128, the FMA addend of B = 8
    0x64006400u, 0x5C005C00u, 0x54005400u, 0x4C004C00u,   // exponent bits for a field at bit 0 / 2 / 4 / 6: base 1024 / 256 / 64 / 16
    0u, 0u};
__device__ __forceinline__ DecodeRegs load_decode_regs() {
    DecodeRegs r;
    r.one_neg = c_decode_consts[0];
    r.off = c_decode_consts[1];
#pragma unroll
    for (int i = 0; i < 4; ++i) r.magic[i] = c_decode_consts[2 + i];
    return r;
}
__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t b, uint32_t c) {   // (a & b) | c
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t lop3_and_xor(uint32_t a, uint32_t b, uint32_t c) {  // (a & b) ^ c
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
template <int B, int P>
__device__ __forceinline__ __half2 pair_K(const uint32_t (&w)[2 * B], const DecodeRegs &dr) {
    if constexpr (B == 1) {
        constexpr int W = pair_word(1, P), pos0 = pair_pos(1, P);
        const uint32_t word = pos0 == 15 ? w[W] : (w[W] << (15 - pos0));
        return as_h2(lop3_and_xor(word, 0x80008000u, dr.one_neg));
    } else if constexpr (B == 2 || B == 4) {
        constexpr int W = pair_word(B, P), pos0 = pair_pos(B, P);
        constexpr int shr = pos0 >= 8 ? 8 : 0, pos = pos0 - shr;
        const uint32_t word = shr ? (w[W] >> shr) : w[W];
        constexpr uint32_t m = (((1u << B) - 1u) << pos) * 0x00010001u;
        const uint32_t hbits = lop3_and_or(word, m, dr.magic[pos / 2]);     // base + u, base = 2^(10 - pos)
        constexpr uint32_t off = half_neg_pow2_plus(10 - pos, B == 2 ? 2 : 8);   // -(base + 2^(B-1))
        return __hadd2(as_h2(hbits), as_h2(h2dup(off)));
    } else if constexpr (B == 8) {
        constexpr int W = pair_word(8, P), pos0 = pair_pos(8, P);
        const uint32_t word = pos0 ? (w[W] >> 8) : w[W];
        const uint32_t hbits = lop3_and_or(word, 0x00FF00FFu, dr.magic[0]);
        return __hfma2(as_h2(hbits), as_h2(h2dup(half_pow2(-7))), as_h2(dr.off));   // (1024 + u) / 128 - 9
    } else if constexpr (B == 7) {
        const uint32_t hbits = pair_codes<7, P>(w) | 0x64006400u;
        // (1024 + u) / 64 - 17 has no register constant of its own: -17 = 2 * (-9) + 1 is not worth a second one
        return __hfma2(as_h2(hbits), as_h2(h2dup(half_pow2(-6))), as_h2(h2dup(half_neg_pow2_plus(4, 1))));
    } else {   // B = 3, 5, 6: planes assembled, then the same add
        const uint32_t hbits = pair_codes<B, P>(w) | 0x64006400u;
        return __hadd2(as_h2(hbits), as_h2(h2dup(half_neg_pow2_plus(10, 1 << (B - 1)))));
    }
}

struct RowCoef { __half2 a2, b2, c2; float s; };

// Coefficients of q as a polynomial in T = k / 2^(B-1):  t = |T| rho, rho = 2^(B-1) / M, so
// q = |T| (a rho + |T| (b rho^2 + |T| c rho^3)), c = 1 - a - b.  Built in half2 arithmetic from the
// stored fp16 a and b (each coefficient is rounded to fp16 anyway; c rho^3 takes two FMA roundings).
constexpr uint32_t half_bits_of(float v) {   // fp16 bit pattern of a positive normal v (round to nearest, ties up)
    int e = 0;
    float m = v;
    while (m >= 2.0f) { m *= 0.5f; ++e; }
    while (m < 1.0f) { m *= 2.0f; --e; }
    const uint32_t frac = (uint32_t)((m - 1.0f) * 1024.0f + 0.5f);
    return (uint32_t)((e + 15) << 10) + frac;   // a carry out of the fraction bumps the exponent
}
template <int B>
__device__ __forceinline__ RowCoef make_coef(uint2 p) {
    RowCoef c;
    c.s = __uint_as_float(p.x & 0x7FFFFFFFu);
    if constexpr (B >= 3) {
        constexpr float rho = (float)(1 << (B - 1)) / (float)((1 << (B - 1)) - 1);
        constexpr uint32_t r1 = h2dup(half_bits_of(rho)), r2 = h2dup(half_bits_of(rho * rho)), r3 = h2dup(half_bits_of(rho * rho * rho));
        const __half2 a2 = as_h2(__byte_perm(p.y, 0, 0x1010)), b2 = as_h2(__byte_perm(p.y, 0, 0x3232));
        c.a2 = __hmul2(a2, as_h2(r1));
        c.b2 = __hmul2(b2, as_h2(r2));
        const __half2 nr3 = as_h2(r3 | 0x80008000u);
        c.c2 = __hfma2(b2, nr3, __hfma2(a2, nr3, as_h2(r3)));   // rho^3 - rho^3 a - rho^3 b
    }
    return c;
}

template <int B, bool FIX>
__device__ __forceinline__ uint32_t level_pair(__half2 T, const RowCoef &c) {
    if constexpr (FIX) {  // reserved pattern: T = -1 (B >= 3) or k = -2 (B = 2) decodes to zero
        const __half2 bad = __float2half2_rn(B == 2 ? -2.0f : -1.0f);
        T = __hmul2(T, __hne2(T, bad));
    }
    if constexpr (B >= 3) {
        const __half2 at = __habs2(T);
        return as_u32(__hmul2(T, __hfma2(at, __hfma2(at, c.c2, c.b2), c.a2)));
    } else {
        return as_u32(T);
    }
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Dynamic A8 operand order (both INT8 kernels).  One k = 32 MMA step takes the 32-wide k block m of a
// tile.  Inside it
// k = 16 a + 4 t + 2 h + e is held by lane t at byte n = 2 a + h of A register a0 / a1 (rows g / g+8)
// for e = 0 and a2 / a3 for e = 1 (small-M kernel), i.e. at byte 8 t + 4 e + n of the block, which is
// where the layout's half-words put it.  The internal activation quantiser writes x8 in the same order.
//
// Carriers (Eq. carrier) come from a per-(row, group) table indexed by the stored code u, so the
// sign and the reserved pattern (u = 0 -> 0) are part of the table:
//   B = 4: the table's two 8-byte halves (u < 8, u >= 8) live in registers; a half-word of four
//          codes, masked to 3 bits each, is the selector of a byte permute into each half, and the
//          codes' top bits (expanded to byte masks by two sign-replicating permutes) pick between them;
//   B = 3: one 8-byte table, the selector assembled from the 2-bit and the 1-bit plane;
//   B <= 2: the carriers are 0 / +-127, a constant table;
//   B >= 5: the table stays in shared memory and is read per code.
template <int B, int RR, int MI>
__device__ __forceinline__ void a8_row_regs(const uint32_t (&w)[2 * B], const uint4 &tab, const int8_t *trow,
                                            uint32_t &lo, uint32_t &hi) {
    if constexpr (B == 4) {
        const uint32_t word = w[2 * MI + RR];
        const uint32_t ws = word & 0x77777777u, wh = ws >> 16, w4 = word << 4;
        const uint32_t m_lo = prmt(w4, word, 0xD9C8u), m_hi = prmt(w4, word, 0xFBEAu);   // 0xFF where u >= 8
        const uint32_t n_lo = prmt(tab.x, tab.y, ws), p_lo = prmt(tab.z, tab.w, ws);
        const uint32_t n_hi = prmt(tab.x, tab.y, wh), p_hi = prmt(tab.z, tab.w, wh);
        lo = (p_lo & m_lo) | (n_lo & ~m_lo);
        hi = (p_hi & m_hi) | (n_hi & ~m_hi);
    } else if constexpr (B == 3) {
        constexpr int rho = (2 + 2 * (MI & 1) + RR) & 3;   // where the 1-bit plane keeps this selector's bits
        const uint32_t x0 = RR ? (w[MI] >> 2) : w[MI];
        const uint32_t w1 = w[4 + (MI >> 1)];
        const uint32_t y = rho == 2 ? w1 : rho == 3 ? (w1 >> 1) : rho == 0 ? (w1 << 2) : (w1 << 1);
        const uint32_t sel = (x0 & 0x33333333u) | (y & 0x44444444u);
        lo = prmt(tab.x, tab.y, sel);
        hi = prmt(tab.x, tab.y, sel >> 16);
    } else if constexpr (B == 2) {
        const uint32_t sel = (RR ? (w[MI] >> 2) : w[MI]) & 0x33333333u;
        lo = prmt(0x7F008100u, 0u, sel);          // u = 0 reserved -> 0, 1 -> -127, 2 -> 0, 3 -> +127
        hi = prmt(0x7F008100u, 0u, sel >> 16);
    } else if constexpr (B == 1) {
        constexpr int rho = (2 + 2 * (MI & 1) + RR) & 3;
        const uint32_t sel = (w[MI >> 1] >> rho) & 0x11111111u;
        lo = prmt(0x00007F81u, 0u, sel);          // bit 0 -> -127, bit 1 -> +127
        hi = prmt(0x00007F81u, 0u, sel >> 16);
    } else {
        lo = 0; hi = 0;
        static_for<4>([&](auto nc) {
            constexpr int n = decltype(nc)::value, p = 4 * (2 * MI + (n >> 1)) + 2 * (n & 1) + RR;
            const uint32_t u2 = pair_codes<B, p>(w);
            lo |= (uint32_t)(uint8_t)trow[u2 & 0xFFFFu] << (8 * n);
            hi |= (uint32_t)(uint8_t)trow[u2 >> 16] << (8 * n);
        });
    }
}

}  // namespace cq
