// Shared definitions of the CubicQuant sm_100a library: the private device layout and the
// bit-field extraction every kernel uses.
//
// Device layout (what cq_repack writes; Section 2.1 / 2.3 data re-tiled, a bijection):
//
//   The N x K code matrix is padded to Np x Kp (multiples of 128) and cut into 128 x 128 tiles,
//   stored tile after tile with the K index fastest: tile (nb, kb) at (nb * KT + kb) * tile_bytes.
//   A tile is   [codes: 8 row blocks of 16 rows x 128 k][params: 128 rows x max(1, 128/G) records x 8 B];
//   for G = 256 / 512 each 128-wide tile of a group repeats the group's record, so every tile stays
//   self-contained (the layout is then larger than the canonical format by 8 (G/128 - 1) bytes per group).
//   The 8-byte parameter record of a (row, group) is {float s, half a, half b}; the sign bit of s
//   (s >= 0 in the format) flags a group that contains the reserved code pattern.
//
//   Inside a row block, lane l = 4*g + t of a warp owns rows {g, g+8} and, for each of the eight
//   16-wide k chunks j, the four k positions 16 j + 4 t + {0,1,2,3}: exactly the A fragment of a
//   warp-level m16n8k16 MMA (and, two chunks at a time, of the m16n8k32 INT8 MMA).  Its 64 codes
//   form 32 pairs p = 4 j + i, register i = {row g | k+0,1}, {row g+8 | k+0,1}, {row g | k+2,3},
//   {row g+8 | k+2,3}; a pair sits in one 32-bit word with its first code in the low and its
//   second code in the high 16 bits, so both are extracted by one mask.
//
//   Stored code u = k + 2^(B-1) (offset binary; u = 0 is the reserved pattern), W1: u = bit.
//   u is split into bit planes of power-of-two width (B = 3 -> 2+1, 5 -> 4+1, 6 -> 4+2,
//   7 -> 4+2+1) so every field is extracted with shifts and masks only.  A plane of width pw holds
//   16/pw pairs per word; pair_word / pair_pos below give the word and bit position of a pair.
//   Write p = 4 j + 2 h + r (chunk j = 2 w + a, k half h, row half r) and n = 2 a + h:
//     pw = 4: word 2 w + r, nibble n           -- a 16-bit half holds four codes of ONE row from one
//     pw = 2: word w, field 2 n + r               32-wide k block, 4 bits apart, so it serves directly as
//     pw = 1: word w / 2, bit 4 n + rho(w, r)     the selector of a byte-permute table lookup (Dynamic A8)
//     pw = 8: word p / 2, byte p % 2
//   A lane's 2B words are stored as 16-byte quads, quad Q of lane l at ((Q * 32) + l) * 16 inside
//   the row block (then an 8-byte tail when 2B is not a multiple of 4), so every warp load is one
//   contiguous 512- or 256-byte run.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace cq {

constexpr int TILE = 128;

struct Dims {
    int B, G;
    int64_t N, K;
    int NB, KT;       // tiles along N and K
    int gpt;          // parameter records per tile row = max(1, 128 / G)
    int code_bytes;   // bytes of the code part of a tile = 2048 * B
    int tile_bytes;   // code_bytes + 128 * gpt * 8
};

__host__ __device__ inline Dims make_dims(int B, int G, int64_t N, int64_t K) {
    Dims d;
    d.B = B; d.G = G; d.N = N; d.K = K;
    d.NB = (int)((N + TILE - 1) / TILE);
    d.KT = (int)((K + TILE - 1) / TILE);
    d.gpt = G >= TILE ? 1 : TILE / G;   // G = 256 / 512: every 128-wide tile of a group carries a copy of its record
    d.code_bytes = 2048 * B;
    d.tile_bytes = d.code_bytes + TILE * d.gpt * 8;
    return d;
}

// ---- bit planes of the stored code u -------------------------------------------------------
__host__ __device__ constexpr int plane_count(int B) { return (B == 3 || B == 5 || B == 6) ? 2 : (B == 7 ? 3 : 1); }
__host__ __device__ constexpr int plane_width(int B, int i) {
    return B == 1 ? 1 : B == 2 ? 2 : B == 3 ? (i == 0 ? 2 : 1) : B == 4 ? 4 : B == 5 ? (i == 0 ? 4 : 1)
         : B == 6 ? (i == 0 ? 4 : 2) : B == 7 ? (i == 0 ? 4 : (i == 1 ? 2 : 1)) : 8;
}
__host__ __device__ constexpr int plane_bit_offset(int B, int i) {  // position of the plane inside u
    return i == 0 ? 0 : (i == 1 ? plane_width(B, 0) : plane_width(B, 0) + plane_width(B, 1));
}
__host__ __device__ constexpr int plane_word_base(int B, int i) {   // first word of the plane in a lane record
    return 2 * plane_bit_offset(B, i);
}

// Word (inside its plane) and bit position (in the low 16-bit half; the pair's second code sits
// 16 bits higher) of logical pair p = 4 j + 2 h + r in a plane of width pw.
__host__ __device__ constexpr int pair_word(int pw, int p) {
    const int r = p & 1, w = p >> 3;
    return pw == 4 ? 2 * w + r : pw == 2 ? w : pw == 1 ? (w >> 1) : (p >> 1);
}
__host__ __device__ constexpr int pair_pos(int pw, int p) {
    const int r = p & 1, h = (p >> 1) & 1, a = (p >> 2) & 1, w = p >> 3, n = 2 * a + h;
    return pw == 4 ? 4 * n : pw == 2 ? 2 * (2 * n + r) : pw == 1 ? 4 * n + ((2 + 2 * (w & 1) + r) & 3) : 8 * (p & 1);
}

// inverse: the pair stored in slot q (0 .. 16/pw - 1, position q * pw) of word wi of a plane
__host__ __device__ constexpr int pair_at(int pw, int wi, int q) {
    if (pw == 8) return 2 * wi + q;
    if (pw == 4) return 8 * (wi >> 1) + 2 * q + (wi & 1);
    if (pw == 2) return 8 * wi + 2 * (q >> 1) + (q & 1);
    const int c = ((q & 3) - 2) & 3;   // pw == 1: bit 4 n + rho, rho = (2 + 2 (w & 1) + r) & 3
    return 8 * (2 * wi + (c >> 1)) + 2 * (q >> 2) + (c & 1);
}

// byte offset of word W (0 .. 2B-1) of lane `lane` inside a row block
__host__ __device__ inline int word_byte_offset(int B, int W, int lane) {
    const int nfq = (2 * B) / 4;
    if (W < 4 * nfq) return (((W >> 2) * 32) + lane) * 16 + (W & 3) * 4;
    return nfq * 512 + lane * 8 + (W - 4 * nfq) * 4;
}

// Where weight (r, kk) of a tile lives: lane, pair index and half (0 = low 16 bits).
struct Slot { int rb, lane, pair, half; };
__host__ __device__ inline Slot slot_of(int r, int kk) {
    Slot s;
    const int rr = r & 15, g = rr & 7, hi_row = rr >> 3;
    const int j = kk >> 4, kin = kk & 15, t = kin >> 2, sl = kin & 3;
    s.rb = r >> 4;
    s.lane = g * 4 + t;
    s.pair = 4 * j + ((sl >> 1) * 2 + hi_row);
    s.half = sl & 1;
    return s;
}
// inverse: (rb, lane, pair, half) -> (r, kk)
__host__ __device__ inline void weight_of(int rb, int lane, int pair, int half, int &r, int &kk) {
    const int g = lane >> 2, t = lane & 3, j = pair >> 2, i = pair & 3;
    r = rb * 16 + g + ((i & 1) ? 8 : 0);
    kk = 16 * j + 4 * t + (i >> 1) * 2 + half;
}

// ---- activations / outputs in the model dtype: bfloat16 or binary16 bit patterns (Section 5.3) ----------
// value of one 16-bit activation pattern
__device__ __forceinline__ float act_to_float(uint32_t bits16, bool f16) {
    return f16 ? __half2float(__ushort_as_half((unsigned short)bits16)) : __uint_as_float(bits16 << 16);
}
// fp32 -> the output dtype, round to nearest even
__device__ __forceinline__ uint16_t float_to_act(float v, bool f16) {
    return f16 ? __half_as_ushort(__float2half_rn(v)) : __bfloat16_as_ushort(__float2bfloat16_rn(v));
}
// Power-of-two exponent e with |x| < 2^(e+1) for the largest magnitude pattern of a row (sign cleared; for
// finite values the integer order of the patterns is the order of the magnitudes).  `usable` is false for
// an all-zero row and for Inf / NaN (no rescaling then).
__device__ __forceinline__ int act_max_exponent(unsigned max_bits, bool f16, bool &usable) {
    if (f16) {
        const int ef = (int)((max_bits >> 10) & 0x1F);
        usable = max_bits != 0 && ef != 31;
        return (ef == 0 ? 1 : ef) - 15;          // subnormals count as 2^-14
    }
    const int ef = (int)((max_bits >> 7) & 0xFF);
    usable = max_bits != 0 && ef != 255;
    return ef - 127;
}

struct __align__(8) GroupParams { float s; __half a; __half b; };

__device__ __forceinline__ const uint8_t *tile_ptr(const void *layout, const Dims &d, int nb, int kb) {
    return (const uint8_t *)layout + ((size_t)nb * d.KT + kb) * (size_t)d.tile_bytes;
}

// Slow generic accessor: stored code u of weight (n, k) (n < Np, k < Kp).
__device__ inline unsigned fetch_u(const void *layout, const Dims &d, int64_t n, int64_t k) {
    const int nb = (int)(n >> 7), kb = (int)(k >> 7);
    const Slot s = slot_of((int)(n & 127), (int)(k & 127));
    const uint8_t *rbp = tile_ptr(layout, d, nb, kb) + s.rb * 256 * d.B;
    unsigned u = 0;
    const int np = plane_count(d.B);
    for (int i = 0; i < np; ++i) {
        const int pw = plane_width(d.B, i);
        const int W = plane_word_base(d.B, i) + pair_word(pw, s.pair);
        const int pos = pair_pos(pw, s.pair) + 16 * s.half;
        const uint32_t w = *(const uint32_t *)(rbp + word_byte_offset(d.B, W, s.lane));
        u |= ((w >> pos) & ((1u << pw) - 1u)) << plane_bit_offset(d.B, i);
    }
    return u;
}

__device__ inline GroupParams fetch_params(const void *layout, const Dims &d, int64_t n, int64_t kgroup) {
    const int nb = (int)(n >> 7);
    const int kb = d.G > TILE ? (int)(kgroup * (d.G / TILE)) : (int)(kgroup / d.gpt);   // first tile of a wide group
    const int gi = d.G > TILE ? 0 : (int)(kgroup % d.gpt);
    const uint8_t *p = tile_ptr(layout, d, nb, kb) + d.code_bytes + (((int)(n & 127)) * d.gpt + gi) * 8;
    return *(const GroupParams *)p;
}

// Signed code k from the stored code u (reserved pattern -> 0; W1: bit -> +-1).
__host__ __device__ inline int signed_code(int B, unsigned u) {
    if (B == 1) return u ? 1 : -1;
    if (u == 0) return 0;
    return (int)u - (1 << (B - 1));
}

// Normalised level q(i/M) by the Horner form of Eq. gpu-horner in fp32:
//   t = i / M (IEEE division), c = (1 - a) - b, q = t * fma(t, fma(t, c, b), a).
__device__ __forceinline__ float level_q(int i, int M, float a, float b) {
    const float t = __fdiv_rn((float)i, (float)M);
    const float c = __fsub_rn(__fsub_rn(1.0f, a), b);
    return __fmul_rn(t, fmaf(t, fmaf(t, c, b), a));
}

// Row stride (bytes) of a shared-memory carrier table of 2^B entries per row: tables read per code
// (B >= 5) are padded by one word so that the same entry of different rows falls into different banks.
__host__ __device__ constexpr int carrier_table_stride(int B) { return (1 << B) + (B >= 5 ? 4 : 0); }

// INT8 carrier (Eq. carrier) at the normalised position t = i / M: RNE(127 q(t)), clamped to [0, 127],
// by the fp32 sequence c = (1 - a) - b, q = t fma(t, fma(t, c, b), a).
__device__ __forceinline__ int carrier_at(float t, float a, float b) {
    const float c = __fsub_rn(__fsub_rn(1.0f, a), b);
    const float q = __fmul_rn(t, fmaf(t, fmaf(t, c, b), a));
    const int r = __float2int_rn(__fmul_rn(127.0f, q));
    return min(max(r, 0), 127);
}
// INT8 carrier of magnitude index i; W1 / W2 have only the normalised levels {0, 1}, which sit on the carrier grid.
__device__ __forceinline__ int carrier_of(int B, int i, float a, float b) {
    if (B == 1) return 127;
    if (B == 2) return i ? 127 : 0;
    const int M = (1 << (B - 1)) - 1;
    return carrier_at(__fdiv_rn((float)i, (float)M), a, b);
}

}  // namespace cq
