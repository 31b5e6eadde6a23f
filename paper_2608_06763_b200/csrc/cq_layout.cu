// Format kernels: canonical <-> device layout, debug decoders, and the Dynamic-A8 activation
// quantiser.  All of them are one-time or test-side operations except cq::launch_quantize_a8.
#include "cq_common.cuh"
#include "cq_internal.h"
#include "cq_tc_ptx.cuh"

namespace cq {

// ---------------------------------------------------------------- canonical bitstream helpers
// B-bit field j of a canonical row (Eq. gpu-packed-extraction): p = floor(jB/8), d = jB mod 8,
// u = ((byte[p] >> d) | (byte[p+1] << (8-d))) & (2^B - 1).
__device__ __forceinline__ unsigned canonical_field(const uint8_t *row, int64_t j, int B, int64_t row_bytes) {
    const int64_t bit = j * B, p = bit >> 3;
    const int dlt = (int)(bit & 7);
    unsigned lo = row[p];
    unsigned hi = (dlt + B > 8 && p + 1 < row_bytes) ? row[p + 1] : 0u;
    return ((lo >> dlt) | (hi << (8 - dlt))) & ((1u << B) - 1u);
}

// canonical field -> stored code u (offset binary: the two's-complement sign bit flipped)
__device__ __forceinline__ unsigned stored_from_field(int B, unsigned f) { return B == 1 ? f : (f ^ (1u << (B - 1))); }
__device__ __forceinline__ unsigned field_from_stored(int B, unsigned u) { return B == 1 ? u : (u ^ (1u << (B - 1))); }

// ---------------------------------------------------------------- cq_pack_codes
// one thread per output byte: gathers the bits of the (up to 8) fields that touch it
__global__ void pack_codes_kernel(const int8_t *__restrict__ k, int B, int64_t N, int64_t K, int64_t row_bytes,
                                  uint8_t *__restrict__ codes) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * row_bytes) return;
    const int64_t n = idx / row_bytes, byte = idx % row_bytes;
    unsigned out = 0;
    for (int bit = 0; bit < 8; ++bit) {
        const int64_t bi = byte * 8 + bit, j = bi / B;
        if (j >= K) break;
        const int fb = (int)(bi % B);
        const int code = k[n * K + j];
        const unsigned field = (B == 1) ? (code > 0 ? 1u : 0u) : ((unsigned)code & ((1u << B) - 1u));
        out |= ((field >> fb) & 1u) << bit;
    }
    codes[idx] = (uint8_t)out;
}

// ---------------------------------------------------------------- cq_repack
// one thread per 32-bit code word of the layout
__global__ void repack_codes_kernel(const uint8_t *__restrict__ codes, Dims d, int64_t row_bytes, uint8_t *__restrict__ layout) {
    const int words_per_rb = 64 * d.B;   // 32 lanes * 2B words
    const int words_per_tile = 8 * words_per_rb;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t total = (int64_t)d.NB * d.KT * words_per_tile;
    if (idx >= total) return;
    const int64_t tile = idx / words_per_tile;
    int rem = (int)(idx % words_per_tile);
    const int rb = rem / words_per_rb; rem %= words_per_rb;
    const int lane = rem / (2 * d.B), W = rem % (2 * d.B);
    const int nb = (int)(tile / d.KT), kb = (int)(tile % d.KT);
    // which plane does word W belong to
    int pl = 0;
    for (int i = plane_count(d.B) - 1; i > 0; --i) if (W >= plane_word_base(d.B, i)) { pl = i; break; }
    const int pw = plane_width(d.B, pl), bo = plane_bit_offset(d.B, pl);
    const int wi = W - plane_word_base(d.B, pl);
    uint32_t word = 0;
    for (int q = 0; q < 16 / pw; ++q) {
        const int pair = pair_at(pw, wi, q);
        for (int half = 0; half < 2; ++half) {
            int r, kk;
            weight_of(rb, lane, pair, half, r, kk);
            const int64_t n = (int64_t)nb * TILE + r, k = (int64_t)kb * TILE + kk;
            unsigned u;
            if (n < d.N && k < d.K) u = stored_from_field(d.B, canonical_field(codes + n * row_bytes, k, d.B, row_bytes));
            else u = (d.B == 1) ? 1u : (1u << (d.B - 1));  // padding: code 0 (W1: +1), its scale is 0
            word |= ((u >> bo) & ((1u << pw) - 1u)) << (q * pw + 16 * half);
        }
    }
    uint8_t *dst = layout + (size_t)tile * d.tile_bytes + rb * 256 * d.B + word_byte_offset(d.B, W, lane);
    *(uint32_t *)dst = word;
}

// one thread per (tile, row, group-in-tile): parameter record, with the reserved-pattern flag
__global__ void repack_params_kernel(const uint8_t *__restrict__ codes, const float *__restrict__ scale,
                                     const uint16_t *__restrict__ a, const uint16_t *__restrict__ b, Dims d,
                                     int64_t row_bytes, uint8_t *__restrict__ layout) {
    const int per_tile = TILE * d.gpt;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)d.NB * d.KT * per_tile) return;
    const int64_t tile = idx / per_tile;
    const int rem = (int)(idx % per_tile), r = rem / d.gpt, gi = rem % d.gpt;
    const int nb = (int)(tile / d.KT), kb = (int)(tile % d.KT);
    const int64_t n = (int64_t)nb * TILE + r, ng = d.K / d.G;
    const int64_t kg = d.G > TILE ? ((int64_t)kb * TILE) / d.G : (int64_t)kb * d.gpt + gi;
    uint32_t sbits = 0;
    uint16_t ha = 0x3C00, hb = 0;  // (1, 0)
    if (n < d.N && kg < ng) {
        sbits = __float_as_uint(scale[n * ng + kg]) & 0x7FFFFFFFu;
        ha = a[n * ng + kg];
        hb = b[n * ng + kg];
        if (d.B > 1) {
            bool reserved = false;
            for (int j = 0; j < d.G; ++j)
                reserved |= canonical_field(codes + n * row_bytes, kg * d.G + j, d.B, row_bytes) == (1u << (d.B - 1));
            if (reserved) sbits |= 0x80000000u;
        }
    }
    uint32_t *dst = (uint32_t *)(layout + (size_t)tile * d.tile_bytes + d.code_bytes + (r * d.gpt + gi) * 8);
    dst[0] = sbits;
    dst[1] = (uint32_t)ha | ((uint32_t)hb << 16);
}

// ---------------------------------------------------------------- cq_unpack
// one thread per canonical byte
__global__ void unpack_codes_kernel(const void *__restrict__ layout, Dims d, int64_t row_bytes, uint8_t *__restrict__ codes) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= d.N * row_bytes) return;
    const int64_t n = idx / row_bytes, byte = idx % row_bytes;
    unsigned out = 0;
    int64_t last_j = -1;
    unsigned field = 0;
    for (int bit = 0; bit < 8; ++bit) {
        const int64_t bi = byte * 8 + bit, j = bi / d.B;
        if (j >= d.K) break;
        if (j != last_j) { field = field_from_stored(d.B, fetch_u(layout, d, n, j)); last_j = j; }
        out |= ((field >> (int)(bi % d.B)) & 1u) << bit;
    }
    codes[idx] = (uint8_t)out;
}

__global__ void unpack_params_kernel(const void *__restrict__ layout, Dims d, float *__restrict__ scale,
                                     uint16_t *__restrict__ a, uint16_t *__restrict__ b) {
    const int64_t ng = d.K / d.G;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= d.N * ng) return;
    const GroupParams p = fetch_params(layout, d, idx / ng, idx % ng);
    scale[idx] = fabsf(p.s);
    a[idx] = __half_as_ushort(p.a);
    b[idx] = __half_as_ushort(p.b);
}

// ---------------------------------------------------------------- debug decoders
// levels[N][K/G][L]: level_i = s * q(i/M) (Appendix B), fp32 Horner; W1: the scale
__global__ void decode_levels_kernel(const void *__restrict__ layout, Dims d, float *__restrict__ levels) {
    const int L = d.B == 1 ? 1 : (1 << (d.B - 1));
    const int64_t ng = d.K / d.G;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= d.N * ng * L) return;
    const int i = (int)(idx % L);
    const int64_t grp = idx / L;
    const GroupParams p = fetch_params(layout, d, grp / ng, grp % ng);
    const float s = fabsf(p.s);
    float v;
    if (d.B == 1) v = s;
    else v = __fmul_rn(s, level_q(i, L - 1, __half2float(p.a), __half2float(p.b)));
    levels[idx] = v;
}

__global__ void decode_carriers_kernel(const void *__restrict__ layout, Dims d, int8_t *__restrict__ carriers) {
    const int L = d.B == 1 ? 1 : (1 << (d.B - 1));
    const int64_t ng = d.K / d.G;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= d.N * ng * L) return;
    const int i = (int)(idx % L);
    const int64_t grp = idx / L;
    const GroupParams p = fetch_params(layout, d, grp / ng, grp % ng);
    carriers[idx] = (int8_t)carrier_of(d.B, i, __half2float(p.a), __half2float(p.b));
}

__global__ void decode_weights_kernel(const void *__restrict__ layout, Dims d, float *__restrict__ What) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= d.N * d.K) return;
    const int64_t n = idx / d.K, k = idx % d.K;
    const int code = signed_code(d.B, fetch_u(layout, d, n, k));
    const GroupParams p = fetch_params(layout, d, n, k / d.G);
    const float s = fabsf(p.s);
    float v;
    if (d.B == 1) v = s;
    else {
        const int M = (1 << (d.B - 1)) - 1;
        v = __fmul_rn(s, level_q(abs(code), M, __half2float(p.a), __half2float(p.b)));
    }
    What[idx] = code < 0 ? -v : (code == 0 ? 0.0f : v);
}

// P[M][N][K/G] = sum_{j in g} x8[m][j] * r(k_j)   (Eq. a8-output), one thread per partial
__global__ void a8_partials_kernel(const void *__restrict__ layout, Dims d, const int8_t *__restrict__ x8, int64_t M,
                                   int32_t *__restrict__ P) {
    const int64_t ng = d.K / d.G;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= M * d.N * ng) return;
    const int64_t g = idx % ng, n = (idx / ng) % d.N, m = idx / (ng * d.N);
    const GroupParams p = fetch_params(layout, d, n, g);
    const float a = __half2float(p.a), b = __half2float(p.b);
    int acc = 0;
    for (int j = 0; j < d.G; ++j) {
        const int64_t k = g * d.G + j;
        const int code = signed_code(d.B, fetch_u(layout, d, n, k));
        int r = code == 0 ? 0 : carrier_of(d.B, abs(code), a, b);
        if (code < 0) r = -r;
        acc += (int)x8[m * d.K + k] * r;
    }
    P[idx] = acc;
}

// ---------------------------------------------------------------- Dynamic-A8 activation quantiser
// One block per row (Eq. a8-activation-scale, Eq. a8-activation-quantization).  fp32 arithmetic:
// xbar = max(max|x|, 1e-10f); dx = xbar / 127 (IEEE); x8 = clip(round-half-away(x / dx), +-127).
// Written with a row pitch so the GEMM can ask for a padded carrier.
// plain version for rows whose length or addresses do not allow 16-byte accesses
__global__ void __launch_bounds__(256) quantize_a8_scalar_kernel(const uint16_t *__restrict__ x, int64_t M, int64_t K,
                                                         int8_t *__restrict__ x8, int64_t x8_pitch,
                                                         float *__restrict__ dx, bool f16) {
    __shared__ float red[8];
    __shared__ float s_d;
    const int64_t m = blockIdx.x;
    const uint16_t *row = x + m * K;
    float mx = 0.0f;
    for (int64_t j = threadIdx.x; j < K; j += blockDim.x)
        mx = fmaxf(mx, fabsf(act_to_float(row[j], f16)));
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
    __syncthreads();
    if (threadIdx.x == 0) {
        float v = red[0];
        for (int i = 1; i < (int)(blockDim.x >> 5); ++i) v = fmaxf(v, red[i]);
        v = fmaxf(v, 1e-10f);
        const float d = __fdiv_rn(v, 127.0f);
        s_d = d;
        dx[m] = d;
    }
    __syncthreads();
    const float d = s_d;
    int8_t *orow = x8 + m * x8_pitch;
    for (int64_t j = threadIdx.x; j < x8_pitch; j += blockDim.x) {
        int q = 0;
        if (j < K) {
            const float v = __fdiv_rn(act_to_float(row[j], f16), d);
            float r = roundf(v);  // halves away from zero
            r = fminf(fmaxf(r, -127.0f), 127.0f);
            q = (int)r;
        }
        orow[j] = (int8_t)q;
    }
}

// 16-byte loads, 8-byte stores: K and the pitch multiples of 8, x 16-byte and x8 8-byte aligned
template <bool OPERAND_ORDER>
__global__ void __launch_bounds__(1024) quantize_a8_kernel(const uint16_t *__restrict__ x, int64_t M, int64_t K,
                                                          int8_t *__restrict__ x8, int64_t x8_pitch,
                                                          float *__restrict__ dx, bool f16) {
    // the kernel launched next may start now (its first steps do not touch what this one writes)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ unsigned red[32];
    __shared__ float s_d;
    const int64_t m = blockIdx.x;
    const uint4 *row = reinterpret_cast<const uint4 *>(x + m * K);   // K % 8 == 0 and x is 16-byte aligned
    const int64_t chunks = K >> 3;                                    // 8 values per 16-byte chunk
    // pass 1: the row maximum of |x| as a bf16 bit pattern (for non-NaN values the integer order of
    // the patterns with the sign cleared is the order of the magnitudes); the first chunk stays in registers
    uint4 keep = make_uint4(0, 0, 0, 0);
    unsigned mx = 0;
    for (int64_t j = threadIdx.x; j < chunks; j += blockDim.x) {
        const uint4 v = row[j];
        if (j == threadIdx.x) keep = v;
        const uint32_t ws[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) { mx = max(mx, ws[q] & 0x7FFFu); mx = max(mx, (ws[q] >> 16) & 0x7FFFu); }
    }
    mx = __reduce_max_sync(0xffffffffu, mx);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
    __syncthreads();
    if (threadIdx.x < 32) {
        unsigned v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0u;
        v = __reduce_max_sync(0xffffffffu, v);
        if (threadIdx.x == 0) {
            const float xbar = fmaxf(act_to_float(v, f16), 1e-10f);
            const float d = __fdiv_rn(xbar, 127.0f);
            s_d = d;
            dx[m] = d;
        }
    }
    __syncthreads();
    const float d = s_d;
    // pass 2: x8 = clip(round_half_away(x / d)), 8 values per thread and step
    uint2 *orow = reinterpret_cast<uint2 *>(x8 + m * x8_pitch);
    const int64_t out_chunks = x8_pitch >> 3;
    for (int64_t j = threadIdx.x; j < out_chunks; j += blockDim.x) {
        uint32_t out[2] = {0u, 0u};
        if (j < chunks) {
            const uint4 v = (j == threadIdx.x) ? keep : row[j];
            const uint32_t ws[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const uint32_t bits16 = (q & 1) ? (ws[q >> 1] >> 16) : (ws[q >> 1] & 0xFFFFu);
                float r = roundf(__fdiv_rn(act_to_float(bits16, f16), d));  // halves away from zero
                r = fminf(fmaxf(r, -127.0f), 127.0f);
                out[q >> 2] |= ((uint32_t)(int)r & 0xFFu) << (8 * (q & 3));
            }
        }
        if constexpr (!OPERAND_ORDER) {
            orow[j] = make_uint2(out[0], out[1]);
        } else {
            // k = 32 m + 16 a + 4 t + 2 h + e goes to byte 32 m + 8 t + 4 e + 2 a + h (cq_decode.cuh); this
            // chunk holds t = 2 (j & 1) + {0, 1} of half a = (j >> 1) & 1
            uint8_t *blk = reinterpret_cast<uint8_t *>(x8 + m * x8_pitch) + (j >> 2) * 32 + 2 * ((j >> 1) & 1) + 16 * (j & 1);
#pragma unroll
            for (int tt = 0; tt < 2; ++tt) {
                const uint32_t pr = __byte_perm(out[tt], 0u, 0x3120);   // bytes (k+0, k+2 | k+1, k+3)
                *reinterpret_cast<uint16_t *>(blk + 8 * tt) = (uint16_t)pr;
                *reinterpret_cast<uint16_t *>(blk + 8 * tt + 4) = (uint16_t)(pr >> 16);
            }
        }
    }
}

// ---------------------------------------------------------------- fused gated activation + quantiser
// The boundary in front of an MLP's down projection (Section 5.4, last paragraph): the row of the gate_up
// output h[m] = (gate | up), 2 I values in the model dtype, goes to act = silu(gate) * up -- evaluated in fp32
// and rounded to the model dtype, which is what a separate activation operator would have written -- and
// straight on to that row's Dynamic-A8 carrier (Eq. a8-activation-scale, Eq. a8-activation-quantization) in the
// MMA operand order, without the activation ever reaching memory.  One CTA per row; I % 8 == 0.
__device__ __forceinline__ uint32_t gated_act_bits(uint32_t g16, uint32_t u16, bool f16) {
    const float g = act_to_float(g16, f16), u = act_to_float(u16, f16);
    const float sg = __fdiv_rn(g, __fadd_rn(1.0f, expf(-g)));
    return float_to_act(__fmul_rn(sg, u), f16);
}
__device__ __forceinline__ uint4 gated_act_chunk(const uint4 &g, const uint4 &u, bool f16) {
    const uint32_t gw[4] = {g.x, g.y, g.z, g.w}, uw[4] = {u.x, u.y, u.z, u.w};
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
        o[q] = gated_act_bits(gw[q] & 0xFFFFu, uw[q] & 0xFFFFu, f16) | (gated_act_bits(gw[q] >> 16, uw[q] >> 16, f16) << 16);
    return make_uint4(o[0], o[1], o[2], o[3]);
}
__global__ void __launch_bounds__(1024) swiglu_quantize_a8_kernel(const uint16_t *__restrict__ h, int64_t M, int64_t I,
                                                                 int8_t *__restrict__ x8, int64_t x8_pitch,
                                                                 float *__restrict__ dx, bool f16) {
    asm volatile("griddepcontrol.wait;" ::: "memory");               // h comes from the kernel launched before
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ unsigned red[32];
    __shared__ float s_d;
    const int64_t m = blockIdx.x;
    const uint4 *grow = reinterpret_cast<const uint4 *>(h + m * 2 * I), *urow = reinterpret_cast<const uint4 *>(h + m * 2 * I + I);
    const int64_t chunks = I >> 3;
    uint4 keep = make_uint4(0, 0, 0, 0);   // this thread's first chunk of the activation stays in registers
    unsigned mx = 0;
    for (int64_t j = threadIdx.x; j < chunks; j += blockDim.x) {
        const uint4 v = gated_act_chunk(grow[j], urow[j], f16);
        if (j == threadIdx.x) keep = v;
        const uint32_t ws[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) { mx = max(mx, ws[q] & 0x7FFFu); mx = max(mx, (ws[q] >> 16) & 0x7FFFu); }
    }
    mx = __reduce_max_sync(0xffffffffu, mx);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
    __syncthreads();
    if (threadIdx.x < 32) {
        unsigned v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0u;
        v = __reduce_max_sync(0xffffffffu, v);
        if (threadIdx.x == 0) {
            const float xbar = fmaxf(act_to_float(v, f16), 1e-10f);
            const float d = __fdiv_rn(xbar, 127.0f);
            s_d = d;
            dx[m] = d;
        }
    }
    __syncthreads();
    const float d = s_d;
    const int64_t out_chunks = x8_pitch >> 3;
    for (int64_t j = threadIdx.x; j < out_chunks; j += blockDim.x) {
        uint32_t out[2] = {0u, 0u};
        if (j < chunks) {
            const uint4 v = (j == threadIdx.x) ? keep : gated_act_chunk(grow[j], urow[j], f16);
            const uint32_t ws[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const uint32_t bits16 = (q & 1) ? (ws[q >> 1] >> 16) : (ws[q >> 1] & 0xFFFFu);
                float r = roundf(__fdiv_rn(act_to_float(bits16, f16), d));
                r = fminf(fmaxf(r, -127.0f), 127.0f);
                out[q >> 2] |= ((uint32_t)(int)r & 0xFFu) << (8 * (q & 3));
            }
        }
        // the operand order of quantize_a8_kernel<true>
        uint8_t *blk = reinterpret_cast<uint8_t *>(x8 + m * x8_pitch) + (j >> 2) * 32 + 2 * ((j >> 1) & 1) + 16 * (j & 1);
#pragma unroll
        for (int tt = 0; tt < 2; ++tt) {
            const uint32_t pr = __byte_perm(out[tt], 0u, 0x3120);
            *reinterpret_cast<uint16_t *>(blk + 8 * tt) = (uint16_t)pr;
            *reinterpret_cast<uint16_t *>(blk + 8 * tt + 4) = (uint16_t)(pr >> 16);
        }
    }
}

// ---------------------------------------------------------------- launchers
static inline unsigned blocks_for(int64_t n, int t) { return (unsigned)((n + t - 1) / t); }

cudaError_t launch_pack_codes(const int8_t *k, int B, int64_t N, int64_t K, uint8_t *codes, cudaStream_t st) {
    const int64_t rbts = (K * B + 7) / 8;
    pack_codes_kernel<<<blocks_for(N * rbts, 256), 256, 0, st>>>(k, B, N, K, rbts, codes);
    return cudaGetLastError();
}

cudaError_t launch_repack(const uint8_t *codes, const float *scale, const uint16_t *a, const uint16_t *b, const Dims &d,
                          void *layout, cudaStream_t st) {
    const int64_t rbts = (d.K * d.B + 7) / 8;
    const int64_t words = (int64_t)d.NB * d.KT * 8 * 64 * d.B;
    repack_codes_kernel<<<blocks_for(words, 256), 256, 0, st>>>(codes, d, rbts, (uint8_t *)layout);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int64_t recs = (int64_t)d.NB * d.KT * TILE * d.gpt;
    repack_params_kernel<<<blocks_for(recs, 256), 256, 0, st>>>(codes, scale, a, b, d, rbts, (uint8_t *)layout);
    return cudaGetLastError();
}

cudaError_t launch_unpack(const void *layout, const Dims &d, uint8_t *codes, float *scale, uint16_t *a, uint16_t *b,
                          cudaStream_t st) {
    const int64_t rbts = (d.K * d.B + 7) / 8;
    unpack_codes_kernel<<<blocks_for(d.N * rbts, 256), 256, 0, st>>>(layout, d, rbts, codes);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    unpack_params_kernel<<<blocks_for(d.N * (d.K / d.G), 256), 256, 0, st>>>(layout, d, scale, a, b);
    return cudaGetLastError();
}

cudaError_t launch_decode_levels(const void *layout, const Dims &d, float *levels, cudaStream_t st) {
    const int L = d.B == 1 ? 1 : (1 << (d.B - 1));
    decode_levels_kernel<<<blocks_for(d.N * (d.K / d.G) * L, 256), 256, 0, st>>>(layout, d, levels);
    return cudaGetLastError();
}
cudaError_t launch_decode_carriers(const void *layout, const Dims &d, int8_t *carriers, cudaStream_t st) {
    const int L = d.B == 1 ? 1 : (1 << (d.B - 1));
    decode_carriers_kernel<<<blocks_for(d.N * (d.K / d.G) * L, 256), 256, 0, st>>>(layout, d, carriers);
    return cudaGetLastError();
}
cudaError_t launch_decode_weights(const void *layout, const Dims &d, float *What, cudaStream_t st) {
    decode_weights_kernel<<<blocks_for(d.N * d.K, 256), 256, 0, st>>>(layout, d, What);
    return cudaGetLastError();
}
cudaError_t launch_a8_partials(const void *layout, const Dims &d, const int8_t *x8, int64_t M, int32_t *P, cudaStream_t st) {
    a8_partials_kernel<<<blocks_for(M * d.N * (d.K / d.G), 128), 128, 0, st>>>(layout, d, x8, M, P);
    return cudaGetLastError();
}
cudaError_t launch_quantize_a8(const uint16_t *x, int64_t M, int64_t K, int8_t *x8, int64_t x8_pitch, float *dx,
                               bool operand_order, bool act_f16, cudaStream_t st) {
    const bool wide = K % 8 == 0 && x8_pitch % 8 == 0 && (reinterpret_cast<uintptr_t>(x) & 15u) == 0 &&
                      (reinterpret_cast<uintptr_t>(x8) & 7u) == 0;
    if (operand_order && !(wide && x8_pitch % 32 == 0)) return cudaErrorInvalidValue;   // internal callers pad the pitch to 128
    if (!wide) {
        quantize_a8_scalar_kernel<<<(unsigned)M, 256, 0, st>>>(x, M, K, x8, x8_pitch, dx, act_f16);
        return cudaGetLastError();
    }
    int64_t threads = ((K >> 3) + 31) / 32 * 32;   // one 8-value chunk per thread when the row is short enough
    if (threads > 1024) threads = 1024;
    if (M > 64 && threads > 256) threads = 256;    // many rows: smaller CTAs fill the SMs better
    if (operand_order) quantize_a8_kernel<true><<<(unsigned)M, (unsigned)threads, 0, st>>>(x, M, K, x8, x8_pitch, dx, act_f16);
    else quantize_a8_kernel<false><<<(unsigned)M, (unsigned)threads, 0, st>>>(x, M, K, x8, x8_pitch, dx, act_f16);
    return cudaGetLastError();
}

cudaError_t launch_swiglu_quantize_a8(const uint16_t *h, int64_t M, int64_t I, int8_t *x8, int64_t x8_pitch, float *dx,
                                      bool act_f16, cudaStream_t st) {
    if (I % 8 != 0 || x8_pitch % 32 != 0 || (reinterpret_cast<uintptr_t>(h) & 15u) != 0) return cudaErrorInvalidValue;
    int64_t threads = ((I >> 3) + 31) / 32 * 32;
    if (threads > 1024) threads = 1024;
    if (M > 64 && threads > 256) threads = 256;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)M);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, swiglu_quantize_a8_kernel, h, M, I, x8, x8_pitch, dx, act_f16);
}

// ---------------------------------------------------------------- cq_debug_wait_timeout
// The bounded wait of the pipelined kernels, on its own: one thread waits on a barrier that nobody
// arrives on (nothing is in flight, nothing is copied), gives up after `limit` cycles and records the
// code in the status word, exactly as a stuck pipeline stage would.  The kernel then returns normally.
__global__ void wait_timeout_kernel(int *status, long long limit) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        tc::fence_barrier_init();
        (void)tc::mbar_wait(&bar, 0, status, 99, limit);
    }
}
cudaError_t launch_wait_timeout(int *status, long long limit_cycles, cudaStream_t st) {
    wait_timeout_kernel<<<1, 32, 0, st>>>(status, limit_cycles);
    return cudaGetLastError();
}

}  // namespace cq
