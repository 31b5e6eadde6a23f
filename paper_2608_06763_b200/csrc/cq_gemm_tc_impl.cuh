// The model-dtype GEMM kernel and its launchers, as templates on SK: SK = false computes one whole output tile
// per CTA; SK = true adds the stream-K runs (tiles shared by several CTAs, partial tiles, the addition by the
// last CTA to arrive).  Each of the two is instantiated in a translation unit of its own, which keeps the code
// of the common case free of the other's registers and lets the two compile side by side.
#pragma once
#include "cq_common.cuh"
#include "cq_decode.cuh"
#include "cq_internal.h"
#include "cq_tc_ptx.cuh"

namespace cq {
namespace {


using namespace tc;

constexpr int DEC_WARPS = 16;                 // decoder / epilogue warps
constexpr int TC_THREADS = 64 + 32 * DEC_WARPS + 32;   // producer of activations, MMA issuer, decoders, producer of raw tiles
constexpr int A_STAGE_BYTES = 128 * 128;  // 128 rows x 64 bf16

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
    float *partial;       // stream-K: fp32 partial tiles [CTA][2][BNT][128]
    int *counters;        // stream-K: layout tiles done, one per output tile
    int MT;               // token tiles
    int64_t t_full;       // tiles computed whole, one CTA each
    int p2;               // CTAs that share the units of the remaining tiles (stream-K)
    bool f16;             // activations and output are binary16 instead of bfloat16 (the weights are decoded to match)
};

// ---------------------------------------------------------------- the kernel (model dtype)
// Depth of the ring of activation tiles (64-wide k blocks) and of the ring of decoded weight tiles.  The 512-token
// tile has room for two activation stages only (64 KB each); its weight stages are 16 KB, so four of them let
// the decoders run two layout tiles ahead of the MMAs instead of in lockstep with them.
constexpr int tc_stages(int BN, int NACC) { return BN * NACC >= 512 ? 2 : (BN == 256 ? 3 : 4); }
constexpr int tc_raw_stage_bytes(int B, int G) { return (2048 * B + 1024 * (TILE / G) + 1023) / 1024 * 1024; }
// Weight stages: up to four, fewer where the activation ring and two raw tiles leave less room.
constexpr int tc_stages_a(int B, int G, int BN, int NACC) {
    const int left = 226 * 1024 - 512 - tc_stages(BN, NACC) * NACC * BN * 128 - 2 * tc_raw_stage_bytes(B, G);
    const int n = left / A_STAGE_BYTES;
    return n > 4 ? 4 : n < 2 ? 2 : n;
}
constexpr int tc_ring_bytes(int B, int G, int BN, int NACC) {
    return tc_stages_a(B, G, BN, NACC) * A_STAGE_BYTES + tc_stages(BN, NACC) * NACC * BN * 128;
}
// Raw layout tiles in flight per CTA: as many as the shared memory left by the operand rings holds, two to four.
constexpr int tc_raw_stages(int B, int G, int BN, int NACC) {
    const int left = 226 * 1024 - 512 - tc_ring_bytes(B, G, BN, NACC);
    const int n = left / tc_raw_stage_bytes(B, G);
    return n > 4 ? 4 : n < 2 ? 2 : n;
}

__device__ __forceinline__ void named_barrier_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// The work of one CTA.  The output is cut into tiles of 128 channels x BNT tokens (tile = mt * NB + nb, so
// that CTAs running side by side read the same activations), each tile into its KT layout tiles along K.
// CTAs 0 .. t_full - 1 compute one whole tile each; the hardware hands them to the SMs as these become free,
// and CTAs that start together sweep K in step, so the activations they share stay in L2.
// Stream-K: the units (tile, k) of the remaining tiles are dealt out as p2 contiguous runs, CTA t_full + c
// owning [floor(V2 c / p2), floor(V2 (c + 1) / p2)), never more than one tile long; a run may begin and end
// inside a tile, and a tile shared by several CTAs is finished by the last of them to arrive.
struct Seg { int nb, mt, k0, k1; int64_t tile; };
template <bool SK>
struct SegWalk {
    int64_t t_full, v, v_end, V2;
    int KT, NB, p2, c2;
    bool whole_left;
    __device__ SegWalk(const TcParams &prm) {
        if constexpr (!SK) {   // one whole tile per CTA, nothing else
            KT = prm.d.KT; NB = prm.d.NB; p2 = 0; c2 = 0; t_full = 0; v = v_end = V2 = 0; whole_left = true;
            return;
        }
        KT = prm.d.KT; NB = prm.d.NB; p2 = prm.p2; t_full = prm.t_full;
        whole_left = (int64_t)blockIdx.x < t_full;
        c2 = (int)((int64_t)blockIdx.x - t_full);   // index of the run
        V2 = ((int64_t)NB * prm.MT - t_full) * KT;
        if (!whole_left) { v = (V2 * c2) / p2; v_end = (V2 * (c2 + 1)) / p2; }
        else { v = 0; v_end = 0; }
    }
    __device__ bool next(Seg &s) {
        if (whole_left) {
            whole_left = false;
            s.tile = blockIdx.x; s.k0 = 0; s.k1 = KT;
        } else {
            if (v >= v_end) return false;
            const int64_t tl = v / KT;
            s.tile = t_full + tl;
            s.k0 = (int)(v - tl * KT);
            const int64_t ve = min(v_end, (tl + 1) * KT);
            s.k1 = s.k0 + (int)(ve - v);
            v = ve;
        }
        s.mt = (int)(s.tile / NB); s.nb = (int)(s.tile - (int64_t)s.mt * NB);
        return true;
    }
};

// One CTA computes tiles of 128 output channels x (NACC * BN) tokens: NACC accumulators of BN columns share
// every decoded weight tile, which halves the decode work per flop at NACC = 2.
template <int B, int G, int BN, int NACC, bool SK>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap xmap, TcParams prm) {
    constexpr int GPT = TILE / G;
    constexpr int STAGES = tc_stages(BN, NACC);        // ring of activation tiles (64-wide k blocks)
    constexpr int STAGES_A = tc_stages_a(B, G, BN, NACC);   // ring of decoded weight tiles
    constexpr int RAW_STAGES = tc_raw_stages(B, G, BN, NACC);
    constexpr int B_TILE_BYTES = BN * 128;             // one TMA box: BN tokens x 64 k
    constexpr int B_STAGE_BYTES = NACC * B_TILE_BYTES;
    constexpr int BNT = BN * NACC;                     // tokens per tile
    constexpr uint32_t TMEM_COLS = BNT < 32 ? 32 : BNT;
    extern __shared__ __align__(1024) uint8_t smem[];  // 1024-byte alignment is what the swizzled tiles need
    uint8_t *sA = smem;                                        // STAGES_A x 16 KB
    uint8_t *sB = sA + STAGES_A * A_STAGE_BYTES;               // STAGES x NACC x BN x 128 B
    uint8_t *sRaw = sB + STAGES * B_STAGE_BYTES;               // RAW_STAGES x raw_stage_bytes
    uint64_t *bars = reinterpret_cast<uint64_t *>(sRaw + RAW_STAGES * prm.raw_stage_bytes);
    uint64_t *a_full = bars, *a_empty = a_full + STAGES_A, *b_full = a_empty + STAGES_A, *b_empty = b_full + STAGES;
    uint64_t *raw_full = b_empty + STAGES, *raw_empty = raw_full + RAW_STAGES, *acc_full = raw_empty + RAW_STAGES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
    volatile int *s_last_p = reinterpret_cast<volatile int *>(tmem_slot + 1);    // "this CTA completes the tile"
    volatile int *gave_up = reinterpret_cast<volatile int *>(tmem_slot + 2);     // a bounded wait ran out somewhere in the CTA

    const Dims &d = prm.d;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if ((smem_u32(smem) & 1023u) != 0) {  // cannot happen with the alignment attribute; never run misaligned
        if (threadIdx.x == 0) atomicCAS(prm.status, 0, 9);
        return;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES_A; ++s) { mbar_init(&a_full[s], DEC_WARPS); mbar_init(&a_empty[s], 1); }
        for (int s = 0; s < STAGES; ++s) { mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1); }
        for (int s = 0; s < RAW_STAGES; ++s) { mbar_init(&raw_full[s], 1); mbar_init(&raw_empty[s], DEC_WARPS); }
        mbar_init(acc_full, 1);
        fence_barrier_init();
        *gave_up = 0;
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Every wait is bounded.  One that runs out records its code in the status word and raises the CTA's flag;
    // from then on no role waits any more, but each still walks its loops to the end (the decoders meet at
    // named barriers, so none of them may leave early): the output is then undefined and the status says so.
    auto wait = [&](uint64_t *bar, uint32_t parity, int code) {
        if (!mbar_wait(bar, parity, prm.status, code, WAIT_LIMIT_CYCLES, gave_up)) *gave_up = 1;
    };

    SegWalk<SK> walk(prm);
    Seg seg;
    if (warp == 0) {
        // ===== producer of the activation tiles.  Nothing but the wait for the stage stands between the MMAs
        // that free it and the TMA that refills it: with two stages that latency is on the critical path.
        if (lane == 0) {
            int kbc = 0;     // 64-wide k blocks issued so far (they index the ring)
            while (walk.next(seg)) {
                for (int t = seg.k0; t < seg.k1; ++t) {
                    for (int half_k = 0; half_k < 2; ++half_k, ++kbc) {
                        const int s = kbc % STAGES;
                        if (kbc >= STAGES) wait(&b_empty[s], ((kbc / STAGES) - 1) & 1, 2);
                        mbar_arrive_expect_tx(&b_full[s], B_STAGE_BYTES);
#pragma unroll
                        for (int a = 0; a < NACC; ++a)
                            tma_load_2d(sB + s * B_STAGE_BYTES + a * B_TILE_BYTES, &xmap, &b_full[s], (2 * t + half_k) * 64, seg.mt * BNT + a * BN);
                    }
                }
            }
        }
    } else if (warp == 2 + DEC_WARPS) {
        // ===== producer of the raw layout tiles (its own warp, so that a wait for the decoders never delays
        // an activation tile)
        if (lane == 0) {
            int tcnt = 0;    // layout tiles issued so far
            while (walk.next(seg)) {
                const uint8_t *tiles = prm.layout + (size_t)seg.nb * d.KT * (size_t)d.tile_bytes;
                for (int t = seg.k0; t < seg.k1; ++t, ++tcnt) {
                    const int rs = tcnt % RAW_STAGES;
                    if (tcnt >= RAW_STAGES) wait(&raw_empty[rs], ((tcnt / RAW_STAGES) - 1) & 1, 1);
                    mbar_arrive_expect_tx(&raw_full[rs], (uint32_t)d.tile_bytes);
                    bulk_load(sRaw + rs * prm.raw_stage_bytes, tiles + (size_t)t * d.tile_bytes, (uint32_t)d.tile_bytes, &raw_full[rs]);
                }
            }
        }
    } else if (warp == 1) {
        // ===== MMA issuer
        if (lane == 0) {
            const uint32_t idesc = prm.f16 ? idesc_f16(BN) : idesc_bf16(BN);
            int kbc = 0;
            while (walk.next(seg)) {
                const int nkb = 2 * (seg.k1 - seg.k0);
                for (int i = 0; i < nkb; ++i, ++kbc) {
                    const int s = kbc % STAGES, sa = kbc % STAGES_A;
                    wait(&a_full[sa], (kbc / STAGES_A) & 1, 3);
                    wait(&b_full[s], (kbc / STAGES) & 1, 4);
                    tc_fence_after();
                    const uint64_t adesc = smem_desc_sw128(smem_u32(sA + sa * A_STAGE_BYTES));
#pragma unroll
                    for (int a = 0; a < NACC; ++a) {
                        const uint64_t bdesc = smem_desc_sw128(smem_u32(sB + s * B_STAGE_BYTES + a * B_TILE_BYTES));
#pragma unroll
                        for (int k = 0; k < 4; ++k)  // four K = 16 steps, 32 bytes apart inside the swizzle atom
                            umma_bf16(tmem_base + a * BN, adesc + 2 * k, bdesc + 2 * k, idesc, (i | k) != 0);
                    }
                    umma_commit(&a_empty[sa]);  // frees the two stages when these MMAs have read them
                    umma_commit(&b_empty[s]);
                }
                // The accumulators of this segment are complete when these MMAs are.  The next segment's first MMA
                // overwrites them, but it waits for a decoded stage, and the decoders decode again only after
                // all of them have read the accumulators.
                umma_commit(acc_full);
            }
        }
    } else {
        // ===== decoders (warps 2..17), then epilogue.  Per 64-wide k block, decoder dw owns row block
        // dw / 2 and the two 16-wide chunks 2 (dw % 2), 2 (dw % 2) + 1 of the block.
        const int dw = warp - 2, g = lane >> 2, t = lane & 3;
        const int rb = dw >> 1, jh = dw & 1;
        const int dec_tid = threadIdx.x - 64;
        int kbc = 0, tcnt = 0, segc = 0;
#pragma unroll 1
        while (walk.next(seg)) {
#pragma unroll 1
        for (int tile = seg.k0; tile < seg.k1; ++tile, ++tcnt) {
            const int rs = tcnt % RAW_STAGES;
            wait(&raw_full[rs], (tcnt / RAW_STAGES) & 1, 5);
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
            // G = 128: one group spans the tile, so its coefficients are formed once per tile, not once per 64-wide block
            RowCoef tc_lo{}, tc_hi{};
            bool tfix = false;
            if constexpr (B != 3 && G == 128) {
                const uint2 q_lo = *(const uint2 *)prow, q_hi = *(const uint2 *)(prow + 8 * GPT * 8);
                tc_lo = make_coef<B>(q_lo); tc_hi = make_coef<B>(q_hi);
                tfix = B > 1 && __any_sync(0xffffffffu, (q_lo.x | q_hi.x) >> 31);
            }
            // one 64-wide block: this warp's unit JQ of the tile (unit = two 16-wide chunks of 16 rows)
            auto do_block = [&](auto jq_block) {
                const int kb = kbc++, s = kb % STAGES_A;
                if (kb >= STAGES_A) wait(&a_empty[s], ((kb / STAGES_A) - 1) & 1, 6);
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
                    RowCoef c_lo, c_hi;
                    bool fix;   // reserved pattern present
                    if constexpr (G == 128) { c_lo = tc_lo; c_hi = tc_hi; fix = tfix; }
                    else { c_lo = make_coef<B>(p_lo); c_hi = make_coef<B>(p_hi); fix = B > 1 && __any_sync(0xffffffffu, (p_lo.x | p_hi.x) >> 31); }
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
                do_unit(jq_block);
                fence_proxy_async();   // generic-proxy stores -> visible to the tensor core's async proxy
                __syncwarp();
                if (lane == 0) mbar_arrive(&a_full[s]);
            };
            // the first 64-wide block of the tile holds units 0 and 1, the second units 2 and 3; jh picks the warp's
            if (jh == 0) { do_block(std::integral_constant<int, 0>{}); do_block(std::integral_constant<int, 2>{}); }
            else { do_block(std::integral_constant<int, 1>{}); do_block(std::integral_constant<int, 3>{}); }
            __syncwarp();
            if (lane == 0) mbar_arrive(&raw_empty[rs]);
        }
        // ----- epilogue of the segment: TMEM lane = output channel, column = token
        wait(acc_full, segc & 1, 7);
        ++segc;
        tc_fence_after();
        const bool whole = !SK || (seg.k0 == 0 && seg.k1 == d.KT);
        {
            const int q4 = warp & 3;                       // TMEM lane quarter this warp may access
            const int cp = dw >> 2;                        // which of four column parts
            const int64_t n = (int64_t)seg.nb * TILE + q4 * 32 + lane;
            if ((d.N & 7) == 0 && (!SK || (int64_t)blockIdx.x < prm.t_full)) {
                // A CTA whose only work is this whole tile, and rows of y that start on 16-byte boundaries: the tile goes
                // through shared memory (the activation ring is idle by now: every MMA has completed and nothing more is
                // loaded; a CTA with a run of several segments may already be loading the next one) as
                // [token][128 channels] in the output dtype, and leaves it in 16-byte pieces, eight channels of one
                // token per thread, instead of one 2-byte store per output.
                uint16_t *stage = reinterpret_cast<uint16_t *>(sB);
#pragma unroll 1
                for (int c0 = cp * 32; c0 < BNT; c0 += 128) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)c0, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) stage[(c0 + i) * TILE + q4 * 32 + lane] = float_to_act(__uint_as_float(r[i]), prm.f16);
                }
                named_barrier_sync(1, 32 * DEC_WARPS);
                const int64_t m0 = (int64_t)seg.mt * BNT, n0 = (int64_t)seg.nb * TILE;
                for (int c = dec_tid; c < BNT * (TILE / 8); c += 32 * DEC_WARPS) {
                    const int tok = c / (TILE / 8), part = c % (TILE / 8);
                    if (m0 + tok < prm.M && n0 + part * 8 < d.N)   // N is a multiple of 8: a piece is inside or outside as a whole
                        *reinterpret_cast<uint4 *>(prm.y + (m0 + tok) * d.N + n0 + part * 8) = *reinterpret_cast<const uint4 *>(stage + tok * TILE + part * 8);
                }
            } else if (whole) {
#pragma unroll 1
                for (int c0 = cp * 32; c0 < BNT; c0 += 128) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)c0, r);
                    tmem_ld_wait();
                    if (n < d.N) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const int64_t m = (int64_t)seg.mt * BNT + c0 + i;
                            if (m < prm.M) prm.y[m * d.N + n] = float_to_act(__uint_as_float(r[i]), prm.f16);
                        }
                    }
                }
            } else {
                // A run has at most two partial segments: its first (which begins inside a tile) and its last
                // (which begins a tile without finishing it); each run owns two partial slots [BNT][128].
                float *slot = prm.partial + ((size_t)walk.c2 * 2 + (seg.k0 > 0 ? 1 : 0)) * (size_t)(BNT * TILE) + q4 * 32 + lane;
#pragma unroll 1
                for (int c0 = cp * 32; c0 < BNT; c0 += 128) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)c0, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) slot[(c0 + i) * TILE] = __uint_as_float(r[i]);
                }
            }
        }
        tc_fence_before();   // the accumulators have been read before this warp's next arrival lets the MMAs go on
        if (SK && !whole) {
            // The tile's counter collects the layout tiles done; the CTA that completes it adds the partial tiles
            // in K order.  The first barrier orders the decoders' partial stores before the release; the acquire
            // plus the second barrier make the other CTAs' partials visible to every decoder.
            named_barrier_sync(1, 32 * DEC_WARPS);
            if (dec_tid == 0) {
                int old;
                asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(prm.counters + seg.tile), "r"(seg.k1 - seg.k0) : "memory");
                *s_last_p = (old + (seg.k1 - seg.k0) == d.KT);
            }
            named_barrier_sync(1, 32 * DEC_WARPS);
            if (*s_last_p) {
                const int64_t v0 = (seg.tile - walk.t_full) * d.KT;
                const int c_first = (int)(((v0 + 1) * walk.p2 - 1) / walk.V2);                     // run that owns the tile's first unit
                const int n_contrib = (int)(((v0 + d.KT) * walk.p2 - 1) / walk.V2) - c_first + 1;   // ... up to the owner of its last
                // Four consecutive channels of one token per load; every thread keeps four such quads of up to four
                // contributors in flight (the partial tiles come from L2: it is the loads in flight that set the pace),
                // and adds the contributors in K order.
                constexpr int QUADS = BNT * TILE / 4, NTHR = 32 * DEC_WARPS;
                const size_t slot_elems = (size_t)(BNT * TILE);
                for (int base = dec_tid; base < QUADS; base += 4 * NTHR) {
                    float4 sum[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) sum[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int q0 = 0; q0 < n_contrib; q0 += 4) {
                        float4 v[4][4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int qd = base + u * NTHR;
#pragma unroll
                            for (int w = 0; w < 4; ++w) {
                                const int q = q0 + w;
                                v[u][w] = (qd < QUADS && q < n_contrib)
                                              ? __ldcg(reinterpret_cast<const float4 *>(prm.partial + ((size_t)(c_first + q) * 2 + (q == 0 ? 0 : 1)) * slot_elems) + qd)
                                              : make_float4(0.f, 0.f, 0.f, 0.f);
                            }
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u)
#pragma unroll
                            for (int w = 0; w < 4; ++w) { sum[u].x += v[u][w].x; sum[u].y += v[u][w].y; sum[u].z += v[u][w].z; sum[u].w += v[u][w].w; }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int qd = base + u * NTHR;
                        if (qd >= QUADS) continue;
                        const int ml = qd / (TILE / 4), ch = (qd % (TILE / 4)) * 4;
                        const int64_t m = (int64_t)seg.mt * BNT + ml, n = (int64_t)seg.nb * TILE + ch;
                        if (m >= prm.M) continue;
                        const float o[4] = {sum[u].x, sum[u].y, sum[u].z, sum[u].w};
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (n + e < d.N) prm.y[m * d.N + n + e] = float_to_act(o[e], prm.f16);
                    }
                }
                if (dec_tid == 0) prm.counters[seg.tile] = 0;  // leave the workspace ready for the next call
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
}

// ---------------------------------------------------------------- host side
template <int B, int G, int BN, int NACC, bool SK>
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
    const TcPlan plan = gemm_tc_plan(d, M);
    if (plan.bnt != BN * NACC || (plan.p2 > 0) != SK) return cudaErrorInvalidConfiguration;
    TcParams p;
    p.layout = (const uint8_t *)layout; p.y = y; p.status = status; p.d = d; p.M = (int)M;
    p.raw_stage_bytes = (d.tile_bytes + 1023) / 1024 * 1024;
    p.MT = plan.token_tiles; p.t_full = plan.t_full; p.p2 = plan.p2;
    constexpr int RAW_STAGES = tc_raw_stages(B, G, BN, NACC);
    if (p.raw_stage_bytes != tc_raw_stage_bytes(B, G)) return cudaErrorInvalidConfiguration;
    const size_t smem = (size_t)tc_ring_bytes(B, G, BN, NACC) + (size_t)RAW_STAGES * p.raw_stage_bytes + 256;
    static_assert(tc_ring_bytes(B, G, BN, NACC) + tc_raw_stages(B, G, BN, NACC) * tc_raw_stage_bytes(B, G) + 256 <= 227 * 1024, "shared memory");
    auto kern = gemm_tc_kernel<B, G, BN, NACC, SK>;
    static std::atomic<uint64_t> attr_done{0};   // per kernel instantiation: the devices it has been set on
    cudaError_t ea = ensure_func_attr(kern, attr_done, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (ea != cudaSuccess) return ea;
    p.partial = partial; p.counters = counters; p.f16 = act_f16;
    kern<<<dim3((unsigned)plan.ctas), TC_THREADS, smem, st>>>(xmap, p);
    return cudaGetLastError();
}

template <int B, int G, bool SK>
cudaError_t launch_g(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int *status,
                     float *partial, int *counters, bool act_f16, cudaStream_t st) {
    if (M <= 32) return launch_bn<B, G, 32, 1, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    if (M <= 64) return launch_bn<B, G, 64, 1, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    if (M <= 128) return launch_bn<B, G, 128, 1, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    if (M <= 256) return launch_bn<B, G, 256, 1, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    return launch_bn<B, G, 256, 2, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
}

template <int B, bool SK>
cudaError_t launch_b(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int *status,
                     float *partial, int *counters, bool act_f16, cudaStream_t st) {
    switch (d.G) {
        case 32: return launch_g<B, 32, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 64: return launch_g<B, 64, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        default: return launch_g<B, 128, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    }
}

template <bool SK>
cudaError_t launch_tc_variant(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int *status,
                              float *partial, int *counters, bool act_f16, cudaStream_t st) {
    switch (d.B) {
        case 1: return launch_b<1, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 2: return launch_b<2, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 3: return launch_b<3, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 4: return launch_b<4, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 5: return launch_b<5, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 6: return launch_b<6, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        case 7: return launch_b<7, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
        default: return launch_b<8, SK>(layout, d, x, y, M, status, partial, counters, act_f16, st);
    }
}

}  // namespace
}  // namespace cq
