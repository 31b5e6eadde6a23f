// Large-M packed GEMM on the 5th-generation tensor cores (Section 5.3 dense path, re-done for
// sm_100a): weights stay packed in HBM and are decoded into bf16 shared-memory operand tiles
// right before tcgen05.mma consumes them; accumulators live in TMEM.
//
// Roles inside a CTA (one 128-row x BN-token output tile):
//   warp 0      producer: bulk-copies raw layout tiles (codes + co-located group parameters) and
//               TMA-loads activation tiles x[BN x 64] (128-byte swizzle) into a ring of stages
//   warp 1      allocates TMEM, issues tcgen05.mma (one elected lane), commits to mbarriers
//   warps 2..17 decode: raw tile -> s_g * q(|k|/M) * sign (Eq. cubic; q by the half2 Horner form of
//               Eq. gpu-horner on the power-of-two-normalised code, scale in fp32), rounded to bf16 and stored in
//               the K-major 128-byte-swizzled layout the MMA reads; then the epilogue
//               (tcgen05.ld -> bf16 -> y)
// Weights sit on the MMA's M side (TMEM lane = output channel), tokens on its N side, so any
// token count maps to a legal instruction shape and each epilogue thread owns one output channel.
//
// Every wait on an mbarrier is bounded: a wait that runs out sets a status word in global memory
// and makes the role leave its loop; the CTA still releases TMEM and exits.
#include "cq_common.cuh"
#include "cq_decode.cuh"
#include "cq_internal.h"
#include "cq_tc_ptx.cuh"

namespace cq {

int gemm_tc_available() { return 1; }

// Token tile of the model-dtype GEMM for M rows, and its split-K factor: when the output tiles
// alone would leave most of the 148 SMs idle, the K range is cut so that about one CTA per SM runs.
int gemm_tc_token_tile(int64_t M) { return M <= 32 ? 32 : M <= 64 ? 64 : M <= 128 ? 128 : M <= 256 ? 256 : 512; }
int gemm_tc_split_k(const Dims &d, int64_t M) {
    const int64_t bnt = gemm_tc_token_tile(M);
    const int64_t ctas = (int64_t)d.NB * ((M + bnt - 1) / bnt);
    if (ctas >= 100 || M > 1024) return 1;   // beyond that the output tiles alone fill the SMs, or the combine costs more than it saves
    int64_t sk = sm_count() / ctas;
    if (sk > 8) sk = 8;
    if (sk > d.KT / 4) sk = d.KT / 4;   // at least four layout tiles per slice
    return sk < 1 ? 1 : (int)sk;
}

namespace {

using namespace tc;

constexpr int DEC_WARPS = 16;                 // decoder / epilogue warps
constexpr int TC_THREADS = 64 + 32 * DEC_WARPS;
constexpr int A_STAGE_BYTES = 128 * 128;  // 128 rows x 64 bf16
constexpr int RAW_STAGES = 2;

// ---------------------------------------------------------------- decode helpers
// Two reconstructed weights s * sign(k) * q(|k| / M) of one pair, rounded to bf16 (the dense path
// of Section 5.3 rounds the temporary operand to the activation dtype).  q is evaluated in half2
// (11-bit significand, finer than the bf16 it is rounded to), the scale is applied in fp32.
template <int B, int P, bool FIX, bool F16>
__device__ __forceinline__ uint32_t weight_pair_bf16(const uint32_t (&w)[2 * B], const RowCoef &c) {
    const __half2 T = pair_T<B, P>(w);
    const uint32_t q = level_pair<B, FIX>(T, c);
    const float2 f = __half22float2(as_h2(q));
    if constexpr (F16) {   // binary16 activations: the temporary operand is rounded to binary16
        return as_u32(__floats2half2_rn(f.x * c.s, f.y * c.s));
    } else {
        const __nv_bfloat162 v = __floats2bfloat162_rn(f.x * c.s, f.y * c.s);
        return *reinterpret_cast<const uint32_t *>(&v);
    }
}

// W3: the eight stored codes of a (row, group) index a signed bf16 table of s * sign(k) * q(|k| / 3)
// (u = 0, the reserved pattern, and k = 0 read zero), kept as a low-byte and a high-byte register pair
// and read four codes at a time with byte permutes; q(1/3) and q(2/3) by the fp32 Horner form.
struct W3Table { uint32_t lo[2], hi[2]; };
__device__ __forceinline__ uint32_t pack_act2(float lo, float hi, bool f16) {   // two values in the activation dtype
    if (f16) return as_u32(__floats2half2_rn(lo, hi));
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}
__device__ __forceinline__ W3Table w3_table(uint2 p, bool f16) {
    const float s = __uint_as_float(p.x & 0x7FFFFFFFu);
    const __half2 ab = as_h2(p.y);
    const float a = __low2float(ab), b = __high2float(ab), c = (1.0f - a) - b;
    constexpr float t1 = 1.0f / 3.0f, t2 = 2.0f / 3.0f;
    const float q1 = t1 * fmaf(t1, fmaf(t1, c, b), a), q2 = t2 * fmaf(t2, fmaf(t2, c, b), a);
    const uint32_t q12 = pack_act2(s * q1, s * q2, f16), ss = pack_act2(s, 0.0f, f16);
    const uint32_t nq = q12 | 0x80008000u, ns = ss | 0x00008000u;
    W3Table t;                                  // entries u = 0 .. 7:  0, -s, -s q2, -s q1 | 0, s q1, s q2, s
    t.lo[0] = prmt(nq, ns, 0x0247u) & 0xFFFFFF00u;   // low bytes:  0, (-s).lo, (-s q2).lo, (-s q1).lo
    t.lo[1] = prmt(q12, ss, 0x4207u) & 0xFFFFFF00u;  //             0, (s q1).lo, (s q2).lo, s.lo
    t.hi[0] = prmt(nq, ns, 0x1357u) & 0xFFFFFF00u;   // high bytes: 0, (-s).hi, (-s q2).hi, (-s q1).hi
    t.hi[1] = prmt(q12, ss, 0x5317u) & 0xFFFFFF00u;  //             0, (s q1).hi, (s q2).hi, s.hi
    return t;
}
// the eight weights of row half RR in the 32-wide k block MI, as bf16 pairs in natural k order:
// out[0] = (k+0, k+1), out[1] = (k+2, k+3) of chunk 2 MI, out[2], out[3] the same of chunk 2 MI + 1
template <int RR, int MI>
__device__ __forceinline__ void w3_block(const uint32_t (&w)[6], const W3Table &t, uint32_t (&out)[4]) {
    constexpr int rho = (2 + 2 * (MI & 1) + RR) & 3;   // where the 1-bit plane keeps this selector's bits
    const uint32_t x0 = RR ? (w[MI] >> 2) : w[MI];
    const uint32_t w1 = w[4 + (MI >> 1)];
    const uint32_t y = rho == 2 ? w1 : rho == 3 ? (w1 >> 1) : rho == 0 ? (w1 << 2) : (w1 << 1);
    const uint32_t sel = (x0 & 0x33333333u) | (y & 0x44444444u), sel1 = sel >> 16;
    // selector nibble n = 2 a + h of half-word e holds k = 16 a + 4 t + 2 h + e
    const uint32_t l0 = prmt(t.lo[0], t.lo[1], sel), h0 = prmt(t.hi[0], t.hi[1], sel);
    const uint32_t l1 = prmt(t.lo[0], t.lo[1], sel1), h1 = prmt(t.hi[0], t.hi[1], sel1);
    const uint32_t e0a = prmt(l0, h0, 0x5140u), e0b = prmt(l0, h0, 0x7362u);   // (k+0, k+2) of chunks 2 MI, 2 MI + 1
    const uint32_t e1a = prmt(l1, h1, 0x5140u), e1b = prmt(l1, h1, 0x7362u);   // (k+1, k+3)
    out[0] = prmt(e0a, e1a, 0x5410u); out[1] = prmt(e0a, e1a, 0x7632u);
    out[2] = prmt(e0b, e1b, 0x5410u); out[3] = prmt(e0b, e1b, 0x7632u);
}

struct TcParams {
    const uint8_t *layout;
    uint16_t *y;
    int *status;
    Dims d;
    int M;
    int raw_stage_bytes;  // tile_bytes rounded up to 1024
    float *partial;       // split-K: fp32 partial sums [SK][M][Np]
    int *counters;        // split-K: arrival counters, one per (row block, token tile)
    bool f16;             // activations and output are binary16 instead of bfloat16 (the weights are decoded to match)
};

// ---------------------------------------------------------------- the kernel (model dtype)
constexpr int tc_stages(int BN, int NACC) { return BN * NACC >= 512 ? 2 : (BN == 256 ? 3 : 4); }

// One CTA computes 128 output channels x (NACC * BN) tokens: NACC accumulators of BN columns share
// every decoded weight tile, which halves the decode work per flop at NACC = 2.
template <int B, int G, int BN, int NACC>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap xmap, TcParams prm) {
    constexpr int GPT = TILE / G;
    constexpr int STAGES = tc_stages(BN, NACC);        // ring of 64-wide k blocks
    constexpr int B_TILE_BYTES = BN * 128;             // one TMA box: BN tokens x 64 k
    constexpr int B_STAGE_BYTES = NACC * B_TILE_BYTES;
    constexpr int BNT = BN * NACC;                     // tokens per CTA
    constexpr uint32_t TMEM_COLS = BNT < 32 ? 32 : BNT;
    extern __shared__ __align__(1024) uint8_t smem[];  // 1024-byte alignment is what the swizzled tiles need
    uint8_t *sA = smem;                                        // STAGES x 16 KB
    uint8_t *sB = sA + STAGES * A_STAGE_BYTES;                 // STAGES x BN x 128 B
    uint8_t *sRaw = sB + STAGES * B_STAGE_BYTES;               // RAW_STAGES x raw_stage_bytes
    uint64_t *bars = reinterpret_cast<uint64_t *>(sRaw + RAW_STAGES * prm.raw_stage_bytes);
    uint64_t *a_full = bars, *b_full = bars + STAGES, *st_empty = bars + 2 * STAGES;
    uint64_t *raw_full = bars + 3 * STAGES, *raw_empty = raw_full + RAW_STAGES, *acc_full = raw_empty + RAW_STAGES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);

    const Dims &d = prm.d;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nb = blockIdx.x, mt = blockIdx.y;
    // split-K: blockIdx.z takes the layout tiles [kt0, kt0 + KT) of the K range
    const int kt0 = (int)(((int64_t)d.KT * blockIdx.z) / gridDim.z);
    const int KT = (int)(((int64_t)d.KT * (blockIdx.z + 1)) / gridDim.z) - kt0;
    const int NKB = 2 * KT;         // 64-wide k blocks

    if ((smem_u32(smem) & 1023u) != 0) {  // cannot happen with the alignment attribute; never run misaligned
        if (threadIdx.x == 0) atomicCAS(prm.status, 0, 9);
        return;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&a_full[s], DEC_WARPS); mbar_init(&b_full[s], 1); mbar_init(&st_empty[s], 1); }
        for (int s = 0; s < RAW_STAGES; ++s) { mbar_init(&raw_full[s], 1); mbar_init(&raw_empty[s], DEC_WARPS); }
        mbar_init(acc_full, 1);
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ===== producer
        if (lane == 0) {
            const uint8_t *tiles = prm.layout + ((size_t)nb * d.KT + kt0) * (size_t)d.tile_bytes;
            bool ok = true;
            for (int kb = 0; kb < NKB && ok; ++kb) {
                if ((kb & 1) == 0) {
                    const int t = kb >> 1, rs = t % RAW_STAGES;
                    if (t >= RAW_STAGES) ok = mbar_wait(&raw_empty[rs], ((t / RAW_STAGES) - 1) & 1, prm.status, 1);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&raw_full[rs], (uint32_t)d.tile_bytes);
                    bulk_load(sRaw + rs * prm.raw_stage_bytes, tiles + (size_t)t * d.tile_bytes, (uint32_t)d.tile_bytes, &raw_full[rs]);
                }
                const int s = kb % STAGES;
                if (kb >= STAGES) ok = mbar_wait(&st_empty[s], ((kb / STAGES) - 1) & 1, prm.status, 2);
                if (!ok) break;
                mbar_arrive_expect_tx(&b_full[s], B_STAGE_BYTES);
#pragma unroll
                for (int a = 0; a < NACC; ++a)
                    tma_load_2d(sB + s * B_STAGE_BYTES + a * B_TILE_BYTES, &xmap, &b_full[s], (2 * kt0 + kb) * 64, mt * BNT + a * BN);
            }
        }
    } else if (warp == 1) {
        // ===== MMA issuer
        if (lane == 0) {
            const uint32_t idesc = prm.f16 ? idesc_f16(BN) : idesc_bf16(BN);
            bool ok = true;
            for (int kb = 0; kb < NKB && ok; ++kb) {
                const int s = kb % STAGES;
                const uint32_t ph = (kb / STAGES) & 1;
                ok = mbar_wait(&a_full[s], ph, prm.status, 3) && mbar_wait(&b_full[s], ph, prm.status, 4);
                if (!ok) break;
                tc_fence_after();
                const uint64_t adesc = smem_desc_sw128(smem_u32(sA + s * A_STAGE_BYTES));
#pragma unroll
                for (int a = 0; a < NACC; ++a) {
                    const uint64_t bdesc = smem_desc_sw128(smem_u32(sB + s * B_STAGE_BYTES + a * B_TILE_BYTES));
#pragma unroll
                    for (int k = 0; k < 4; ++k)  // four K = 16 steps, 32 bytes apart inside the swizzle atom
                        umma_bf16(tmem_base + a * BN, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
                }
                umma_commit(&st_empty[s]);  // frees the stage when these MMAs have read it
            }
            umma_commit(acc_full);
        }
    } else {
        // ===== decoders (warps 2..17), then epilogue.  Per 64-wide k block, decoder dw owns row block
        // dw / 2 and the two 16-wide chunks 2 (dw % 2), 2 (dw % 2) + 1 of the block.
        const int dw = warp - 2, g = lane >> 2, t = lane & 3;
        const int rb = dw >> 1, jh = dw & 1;
        bool ok = true;
        for (int tile = 0; tile < KT && ok; ++tile) {
            const int rs = tile % RAW_STAGES;
            ok = mbar_wait(&raw_full[rs], (tile / RAW_STAGES) & 1, prm.status, 5);
            if (!ok) break;
            const uint8_t *raw = sRaw + rs * prm.raw_stage_bytes;
            const uint8_t *rbp = raw + rb * 256 * B;
            uint32_t w[2 * B];
            {
                constexpr int NFQ = (2 * B) / 4;
#pragma unroll
                for (int q = 0; q < NFQ; ++q) {
                    const uint4 v = *(const uint4 *)(rbp + (q * 32 + lane) * 16);
                    w[4 * q + 0] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
                }
                if constexpr ((2 * B) % 4 != 0) {
                    const uint2 v = *(const uint2 *)(rbp + NFQ * 512 + lane * 8);
                    w[4 * NFQ + 0] = v.x; w[4 * NFQ + 1] = v.y;
                }
            }
            const uint8_t *prow = raw + d.code_bytes + ((rb * 16 + g) * GPT) * 8;
            W3Table w3_lo{}, w3_hi{};   // W3: level tables of rows g and g + 8; one per tile when the group spans it
            if constexpr (B == 3 && G == 128) {
                w3_lo = w3_table(*(const uint2 *)prow, prm.f16);
                w3_hi = w3_table(*(const uint2 *)(prow + 8 * GPT * 8), prm.f16);
            }
#pragma unroll 1
            for (int half_k = 0; half_k < 2 && ok; ++half_k) {
                const int kb = 2 * tile + half_k, s = kb % STAGES;
                if (kb >= STAGES) ok = mbar_wait(&st_empty[s], ((kb / STAGES) - 1) & 1, prm.status, 6);
                if (!ok) break;
                uint8_t *a_stage = sA + s * A_STAGE_BYTES;
                // rows g (low) and g + 8 (high) of the row block: their 128-byte rows in the stage
                uint8_t *row_lo = a_stage + (rb * 2 + 0) * 1024 + g * 128;
                uint8_t *row_hi = a_stage + (rb * 2 + 1) * 1024 + g * 128;
                auto do_unit = [&](auto jq) {
                    constexpr int JQ = decltype(jq)::value;        // pair of chunks 2 JQ, 2 JQ + 1 of the tile
                    constexpr int gi = (32 * JQ) / G;              // both chunks lie in this group
                    const uint2 p_lo = *(const uint2 *)(prow + gi * 8), p_hi = *(const uint2 *)(prow + (8 * GPT + gi) * 8);
                    if constexpr (B == 3) {
                        // table decode (w3_block): no per-weight arithmetic, the reserved pattern reads zero
                        if constexpr (G < 128) { w3_lo = w3_table(p_lo, prm.f16); w3_hi = w3_table(p_hi, prm.f16); }
                        uint32_t o_lo[4], o_hi[4];
                        w3_block<0, JQ>(w, w3_lo, o_lo);
                        w3_block<1, JQ>(w, w3_hi, o_hi);
                        static_for<2>([&](auto jc) {
                            constexpr int jcv = decltype(jc)::value, jl = (2 * JQ + jcv) & 3;
                            const int off = (((2 * jl + (t >> 1)) ^ g) * 16) + (t & 1) * 8;
                            *(uint2 *)(row_lo + off) = make_uint2(o_lo[2 * jcv], o_lo[2 * jcv + 1]);
                            *(uint2 *)(row_hi + off) = make_uint2(o_hi[2 * jcv], o_hi[2 * jcv + 1]);
                        });
                        return;
                    }
                    const RowCoef c_lo = make_coef<B>(p_lo), c_hi = make_coef<B>(p_hi);
                    const bool fix = B > 1 && __any_sync(0xffffffffu, (p_lo.x | p_hi.x) >> 31);  // reserved pattern present
                    auto emit = [&](auto fx, auto hx) {
                        constexpr bool FIX = decltype(fx)::value, F16 = decltype(hx)::value;
                        static_for<2>([&](auto jc) {
                            constexpr int j = 2 * JQ + decltype(jc)::value, jl = j & 3;
                            uint2 lo, hi;  // four consecutive k of one row = 8 bytes
                            lo.x = weight_pair_bf16<B, 4 * j + 0, FIX, F16>(w, c_lo);
                            hi.x = weight_pair_bf16<B, 4 * j + 1, FIX, F16>(w, c_hi);
                            lo.y = weight_pair_bf16<B, 4 * j + 2, FIX, F16>(w, c_lo);
                            hi.y = weight_pair_bf16<B, 4 * j + 3, FIX, F16>(w, c_hi);
                            // k offset inside the 64-wide block: 16 jl + 4 t -> 16-byte chunk 2 jl + t/2, swizzled by the row
                            const int chunk = (2 * jl + (t >> 1)) ^ g;
                            const int off = chunk * 16 + (t & 1) * 8;
                            *(uint2 *)(row_lo + off) = lo;
                            *(uint2 *)(row_hi + off) = hi;
                        });
                    };
                    if (!prm.f16) { if (!fix) emit(std::false_type{}, std::false_type{}); else emit(std::true_type{}, std::false_type{}); }
                    else { if (!fix) emit(std::false_type{}, std::true_type{}); else emit(std::true_type{}, std::true_type{}); }
                };
                switch (half_k * 2 + jh) {
                    case 0: do_unit(std::integral_constant<int, 0>{}); break;
                    case 1: do_unit(std::integral_constant<int, 1>{}); break;
                    case 2: do_unit(std::integral_constant<int, 2>{}); break;
                    default: do_unit(std::integral_constant<int, 3>{}); break;
                }
                fence_proxy_async();   // generic-proxy stores -> visible to the tensor core's async proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(&a_full[s]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&raw_empty[rs]);
        }
        // ----- epilogue: TMEM lane = output channel, column = token
        if (ok) ok = mbar_wait(acc_full, 0, prm.status, 7);
        tc_fence_after();
        if (ok) {
            const int q4 = warp & 3;                       // TMEM lane quarter this warp may access
            const int cp = dw >> 2;                        // which of four column parts
            const int64_t n = (int64_t)nb * TILE + q4 * 32 + lane;
#pragma unroll 1
            for (int c0 = cp * 32; c0 < BNT; c0 += 128) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)c0, r);
                tmem_ld_wait();
                if (n < d.N || gridDim.z > 1) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int64_t m = (int64_t)mt * BNT + c0 + i;
                        if (m < prm.M) {
                            if (gridDim.z == 1) prm.y[m * d.N + n] = float_to_act(__uint_as_float(r[i]), prm.f16);
                            else prm.partial[((size_t)blockIdx.z * prm.M + m) * ((size_t)d.NB * TILE) + n] = __uint_as_float(r[i]);
                        }
                    }
                }
            }
        }
    }
    if (*reinterpret_cast<volatile int *>(prm.status) != 0) {
        // a wait gave up: give copies that are still in flight time to land before shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
    if (gridDim.z > 1) {
        // split-K combine: the last CTA of this output tile to arrive adds the slices in slice order.
        // The barrier above ordered the CTA's partial stores before thread 0's release.
        volatile int *s_last_p = reinterpret_cast<volatile int *>(tmem_slot + 1);   // scratch word after the TMEM slot
        int *ctr = prm.counters + (nb * gridDim.y + mt);
        if (threadIdx.x == 0) {
            int old;
            asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(ctr) : "memory");
            *s_last_p = (old == (int)gridDim.z - 1);
        }
        __syncthreads();
        if (*s_last_p) {
            const size_t Np = (size_t)d.NB * TILE;
            // each thread takes four consecutive channels of one token at a time (128-bit loads), two such
            // quads per step, all loads issued before the sums
            constexpr int QUADS = BNT * TILE / 4;
            for (int base = threadIdx.x; base < QUADS; base += 2 * TC_THREADS) {
                float4 v[2][8];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int qd = base + u * TC_THREADS;
                    const int64_t m = (int64_t)mt * BNT + qd / (TILE / 4), n = (int64_t)nb * TILE + (qd % (TILE / 4)) * 4;
                    const bool live = qd < QUADS && m < prm.M;
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        v[u][q] = (live && q < (int)gridDim.z)
                                      ? __ldcg(reinterpret_cast<const float4 *>(prm.partial + ((size_t)q * prm.M + m) * Np + n))
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int qd = base + u * TC_THREADS;
                    const int64_t m = (int64_t)mt * BNT + qd / (TILE / 4), n = (int64_t)nb * TILE + (qd % (TILE / 4)) * 4;
                    if (qd >= QUADS || m >= prm.M) continue;
                    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int q = 0; q < 8; ++q) { sum.x += v[u][q].x; sum.y += v[u][q].y; sum.z += v[u][q].z; sum.w += v[u][q].w; }  // slice order
                    const float o[4] = {sum.x, sum.y, sum.z, sum.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (n + e < d.N) prm.y[m * d.N + n + e] = float_to_act(o[e], prm.f16);
                }
            }
            if (threadIdx.x == 0) *ctr = 0;  // leave the workspace ready for the next call
        }
    }
}

// ---------------------------------------------------------------- host side
template <int B, int G, int BN, int NACC>
cudaError_t launch_bn(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int *status,
                      float *partial, int *counters, bool act_f16, cudaStream_t st) {
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return cudaErrorNotSupported;
    CUtensorMap xmap;
    const cuuint64_t dims[2] = {(cuuint64_t)d.K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)d.K * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)BN};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&xmap, act_f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<uint16_t *>(x), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    constexpr int STAGES = tc_stages(BN, NACC);
    TcParams p;
    p.layout = (const uint8_t *)layout; p.y = y; p.status = status; p.d = d; p.M = (int)M;
    p.raw_stage_bytes = (d.tile_bytes + 1023) / 1024 * 1024;
    const size_t smem = (size_t)STAGES * (A_STAGE_BYTES + NACC * BN * 128) + (size_t)RAW_STAGES * p.raw_stage_bytes + 256;
    auto kern = gemm_tc_kernel<B, G, BN, NACC>;
    static std::atomic<uint64_t> attr_done{0};   // per kernel instantiation: the devices it has been set on
    cudaError_t ea = ensure_func_attr(kern, attr_done, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (ea != cudaSuccess) return ea;
    p.partial = partial; p.counters = counters; p.f16 = act_f16;
    dim3 grid((unsigned)d.NB, (unsigned)((M + BN * NACC - 1) / (BN * NACC)), (unsigned)gemm_tc_split_k(d, M));
    kern<<<grid, TC_THREADS, smem, st>>>(xmap, p);
    return cudaGetLastError();
}

template <int B, int G>
cudaError_t launch_g(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int *status,
                     float *partial, int *counters, bool act_f16, cudaStream_t st) {
    if (M <= 32) return launch_bn<B, G, 32, 1>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    if (M <= 64) return launch_bn<B, G, 64, 1>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    if (M <= 128) return launch_bn<B, G, 128, 1>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    if (M <= 256) return launch_bn<B, G, 256, 1>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    return launch_bn<B, G, 256, 2>(layout, d, x, y, M, status, partial, counters, act_f16, st);
}

template <int B>
cudaError_t launch_b(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int *status,
                     float *partial, int *counters, bool act_f16, cudaStream_t st) {
    switch (d.G) {
        case 32: return launch_g<B, 32>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 64: return launch_g<B, 64>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        default: return launch_g<B, 128>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    }
}

}  // namespace

cudaError_t launch_gemm_tc(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int mode,
                           bool act_f16, uint8_t *ws, const Workspace &plan, cudaStream_t st) {
    if (mode != 0) return cudaErrorNotSupported;
    int *status = reinterpret_cast<int *>(ws + plan.status_off);
    float *partial = reinterpret_cast<float *>(ws + plan.partial_off);
    int *counters = reinterpret_cast<int *>(ws + plan.counters_off);
    switch (d.B) {
        case 1: return launch_b<1>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 2: return launch_b<2>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 3: return launch_b<3>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 4: return launch_b<4>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 5: return launch_b<5>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 6: return launch_b<6>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 7: return launch_b<7>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        default: return launch_b<8>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    }
}

}  // namespace cq
