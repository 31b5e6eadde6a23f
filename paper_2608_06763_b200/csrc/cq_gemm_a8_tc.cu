// Large-M Dynamic-A8 GEMM on tcgen05 (Section 5.4): INT8 activation carriers x INT8 weight
// carriers -> int32 group partials in TMEM -> fp32 rescale by s_g (and d_x / 127 at the end).
//
// CTA = 128 output channels x BN tokens, K (or one slice of it, for a tile of the last round) walked in 128-wide
// blocks (one layout tile).
//   warp 0       TMA of the x8 tiles [BN x 128] (swizzled) into a ring of two stages
//   warp 18      bulk copies of the raw layout tiles into their own ring (2-4 deep)
//   warp 1       TMEM allocation, tcgen05.mma kind::i8 (K = 32 per instruction); every group of
//                the block accumulates into its own BN columns of one of two TMEM buffers
//   warps 2..17  work warps, two jobs per K block, interleaved so the tensor core never waits on both:
//                (a) decode block t: a signed carrier table r(k) per (row, group) (Eq. carrier, the
//                    fp32 sequence of cq_common.cuh), then the carriers of the block (byte-permute look-ups
//                    in register tables for B <= 4, one shared-memory look-up per weight otherwise) go
//                    into the K-major swizzled INT8 operand tile in the operand order of cq_decode.cuh;
//                (b) drain block t-1: tcgen05.ld of its int32 partials P_g, acc += s_g * P_g in fp32
//                    registers (Eq. a8-output), which frees that TMEM buffer for block t+1.
//                At the end y = (d_x / 127) * acc, rounded to bf16.
// All mbarrier waits are bounded and report through the workspace status word.
#include "cq_common.cuh"
#include "cq_decode.cuh"
#include "cq_internal.h"
#include "cq_tc_ptx.cuh"

namespace cq {

// Token tile of the Dynamic-A8 GEMM (two accumulator buffers of (128 / G) x tile columns fill at most
// the 512 TMEM columns).
int gemm_a8_token_tile(const Dims &d, int64_t M) {
    const int bmax = 256 / d.gpt;
    const int bn = M <= 64 ? 64 : M <= 128 ? 128 : 256;
    return bn < bmax ? bn : bmax;
}
// How the Dynamic-A8 GEMM is spread over the SMs: whole tiles, one CTA each, round after round; when the last
// round would leave SMs idle, each of its r tiles is cut along K into the same number s of slices (one CTA each;
// the last CTA of a tile to arrive adds the partial tiles in K order).  In units of one 128-wide K block of main
// loop: a whole tile costs KT + 3, a slice KT / s + 3 + up to 4 for the partial tile's trip through L2 and its share
// of the addition; r s slices take ceil(r s / SMs) rounds.  Slices are used when that saves more than 3 % of the
// whole launch.
A8Plan gemm_a8_plan(const Dims &d, int64_t M) {
    A8Plan p;
    p.bn = gemm_a8_token_tile(d, M);
    p.token_tiles = (int)((M + p.bn - 1) / p.bn);
    const int64_t T = (int64_t)d.NB * p.token_tiles, sms = sm_count();
    const int64_t r = T % sms;
    p.t_full = T; p.slices = 1;
    if (r != 0) {
        const double wide = (double)p.bn / 256.0;
        const double whole = (double)(d.KT + 3), all = (double)(T / sms + 1) * whole;
        double best = whole;
        for (int64_t s = 2; s <= 8 && s * 4 <= d.KT; ++s) {
            const double c = (double)((r * s + sms - 1) / sms) * ((double)d.KT / (double)s + 3.0 + 4.0 * wide);
            if (c < best) { best = c; p.slices = (int)s; }
        }
        if ((whole - best) / all > 0.03) p.t_full = T - r; else p.slices = 1;
    }
    p.ctas = (int)(p.t_full + (T - p.t_full) * p.slices);
    return p;
}

namespace {

using namespace tc;

constexpr int A8_WORK_WARPS = 16;
constexpr int A8_THREADS = 32 * (3 + A8_WORK_WARPS);   // producer of activations, MMA issuer, work warps, producer of raw tiles
constexpr int A8_STAGES = 2;     // operand stages (one 128-wide k block each)
// Raw layout tiles in flight per CTA: as many as the shared memory left by the rest holds, two to four.
constexpr int a8_raw_stage_bytes(int B, int G) { return (2048 * B + 1024 * (TILE / G) + 1023) / 1024 * 1024; }
constexpr int a8_fixed_smem(int B, int G, int BN) {
    return 2 * (128 * 128 + BN * 128) + 8 * 2 * 16 * carrier_table_stride(B) + 8 * 128 * (TILE / G) * 4 + 512 + 256;
}
constexpr int a8_raw_stages(int B, int G, int BN) {
    const int n = (226 * 1024 - a8_fixed_smem(B, G, BN)) / a8_raw_stage_bytes(B, G);
    return n > 4 ? 4 : n < 2 ? 2 : n;
}
constexpr int A8_SRING = 8;      // ring of per-block scale snapshots for the drain warps
constexpr int A8_A_STAGE_BYTES = 128 * 128;

struct A8Params {
    const uint8_t *layout;
    const float *dx;
    uint16_t *y;
    int *status;
    Dims d;
    int M;
    int raw_stage_bytes;
    float *partial;       // sliced tiles: fp32 partial tiles [shared tile][slice][BN][128] (before the d_x / 127 factor)
    int *counters;        // sliced tiles: arrival counters, one per output tile
    int t_full;           // CTAs 0 .. t_full - 1 compute one whole tile each (tile = mt * NB + nb)
    int slices;           // every later tile is cut along K into this many slices, one CTA each
    bool f16;             // y is written as binary16 instead of bfloat16
};

__device__ __forceinline__ void named_barrier_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <int B, int G, int BN>
__global__ void __launch_bounds__(A8_THREADS, 1)
gemm_a8_kernel(const __grid_constant__ CUtensorMap xmap, A8Params prm) {
    constexpr int GPT = TILE / G;                 // groups per 128-wide block
    constexpr int MPG = 4 / GPT;                  // K = 32 MMAs per group
    constexpr int NCODE = carrier_table_stride(B);   // bytes per table row (2^B entries indexed by the stored code u, padded)
    constexpr int Mx = B == 1 ? 1 : (1 << (B - 1)) - 1;
    constexpr int B_STAGE_BYTES = BN * 128;
    constexpr uint32_t ACC_COLS = GPT * BN;       // columns of one accumulator buffer
    constexpr uint32_t TMEM_COLS = 2 * ACC_COLS;  // 512
    constexpr int QCOLS = BN / 4;                 // columns per work thread in the drain
    constexpr int A8_RAW_STAGES = a8_raw_stages(B, G, BN);
    static_assert(TMEM_COLS <= 512 && (TMEM_COLS & (TMEM_COLS - 1)) == 0, "TMEM columns");
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *sA = smem;
    uint8_t *sB = sA + A8_STAGES * A8_A_STAGE_BYTES;
    uint8_t *sRaw = sB + A8_STAGES * B_STAGE_BYTES;
    int8_t *sTab = reinterpret_cast<int8_t *>(sRaw + A8_RAW_STAGES * prm.raw_stage_bytes);   // [8 row blocks][2][16 rows][NCODE]
    float *sScale = reinterpret_cast<float *>(sTab + 8 * 2 * 16 * NCODE);                      // [SRING][128][GPT]
    float *sT = sScale + A8_SRING * 128 * GPT;                                                 // t_i = i / M, i = 0..127
    uint64_t *bars = reinterpret_cast<uint64_t *>(sT + 128);
    uint64_t *a_full = bars, *b_full = a_full + A8_STAGES, *st_empty = b_full + A8_STAGES;
    uint64_t *raw_full = st_empty + A8_STAGES, *raw_empty = raw_full + A8_RAW_STAGES;
    uint64_t *acc_full = raw_empty + A8_RAW_STAGES, *acc_empty = acc_full + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);

    const Dims &d = prm.d;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // This CTA's tile and, for a tile of the last round, its slice z of nz: the layout tiles [kt0, kt0 + KT)
    int kt0, KT, p_nb, p_mt;
    {
        const int bid = (int)blockIdx.x;
        const int nz = bid < prm.t_full ? 1 : prm.slices;
        const int tile_id = bid < prm.t_full ? bid : prm.t_full + (bid - prm.t_full) / prm.slices;
        const int z = bid < prm.t_full ? 0 : (bid - prm.t_full) % prm.slices;
        p_mt = tile_id / d.NB; p_nb = tile_id - p_mt * d.NB;
        kt0 = (int)(((int64_t)d.KT * z) / nz);
        KT = (int)(((int64_t)d.KT * (z + 1)) / nz) - kt0;
        if (threadIdx.x == 0) {   // what only the epilogue needs is parked in shared memory (set up below, before the barrier)
            uint32_t *park = reinterpret_cast<uint32_t *>(acc_empty + 2);
            park[4] = (uint32_t)nz; park[5] = (uint32_t)z; park[6] = (uint32_t)tile_id; park[7] = (uint32_t)p_nb; park[8] = (uint32_t)p_mt;
        }
    }
    const int nb = p_nb, mt = p_mt;   // the producer's coordinates

    if ((smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicCAS(prm.status, 0, 9);
        return;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < A8_STAGES; ++s) { mbar_init(&a_full[s], A8_WORK_WARPS); mbar_init(&b_full[s], 1); mbar_init(&st_empty[s], 1); }
        for (int s = 0; s < A8_RAW_STAGES; ++s) { mbar_init(&raw_full[s], 1); mbar_init(&raw_empty[s], A8_WORK_WARPS); }
        for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], A8_WORK_WARPS); }
        fence_barrier_init();
        tmem_slot[2] = 0;   // the work warps' "a wait gave up" flag
        tmem_slot[3] = prm.f16 ? 1u : 0u;   // the output dtype, parked in shared memory: a register held across the main loop is one too many
        // tmem_slot[4 .. 8]: slice count, slice, tile, row block and token tile of this CTA (written above)
    }
    if (threadIdx.x < 128) sT[threadIdx.x] = __fdiv_rn((float)threadIdx.x, (float)Mx);  // the pinned t = i / M
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ===== producer of the activation tiles: only the wait for the stage stands between the MMAs that free it
        // and the TMA that refills it (with two stages that latency is on the critical path)
        if (lane == 0) {
            bool ok = true;
            for (int t = 0; t < KT && ok; ++t) {
                const int s = t % A8_STAGES;
                if (t >= A8_STAGES) ok = mbar_wait(&st_empty[s], ((t / A8_STAGES) - 1) & 1, prm.status, 12);
                if (!ok) break;
                mbar_arrive_expect_tx(&b_full[s], B_STAGE_BYTES);
                tma_load_2d(sB + s * B_STAGE_BYTES, &xmap, &b_full[s], (kt0 + t) * 128, mt * BN);
            }
        }
    } else if (warp == 2 + A8_WORK_WARPS) {
        // ===== producer of the raw layout tiles (its own warp: a wait for the work warps never delays an activation tile)
        if (lane == 0) {
            const uint8_t *tiles = prm.layout + ((size_t)nb * d.KT + kt0) * (size_t)d.tile_bytes;
            bool ok = true;
            for (int t = 0; t < KT && ok; ++t) {
                const int rs = t % A8_RAW_STAGES;
                if (t >= A8_RAW_STAGES) ok = mbar_wait(&raw_empty[rs], ((t / A8_RAW_STAGES) - 1) & 1, prm.status, 11);
                if (!ok) break;
                mbar_arrive_expect_tx(&raw_full[rs], (uint32_t)d.tile_bytes);
                bulk_load(sRaw + rs * prm.raw_stage_bytes, tiles + (size_t)t * d.tile_bytes, (uint32_t)d.tile_bytes, &raw_full[rs]);
            }
        }
    } else if (warp == 1) {
        // ===== MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_i8(BN);
            bool ok = true;
            for (int t = 0; t < KT && ok; ++t) {
                const int s = t % A8_STAGES, ab = t & 1;
                ok = mbar_wait(&a_full[s], (t / A8_STAGES) & 1, prm.status, 13) &&
                     mbar_wait(&b_full[s], (t / A8_STAGES) & 1, prm.status, 14);
                if (ok && t >= 2) ok = mbar_wait(&acc_empty[ab], ((t >> 1) - 1) & 1, prm.status, 15);
                if (!ok) break;
                tc_fence_after();
                const uint64_t adesc = smem_desc_sw128(smem_u32(sA + s * A8_A_STAGE_BYTES));
                const uint64_t bdesc = smem_desc_sw128(smem_u32(sB + s * B_STAGE_BYTES));
#pragma unroll
                for (int mi = 0; mi < 4; ++mi)   // four K = 32 steps, 32 bytes apart; a new group restarts the sum
                    umma_i8(tmem_base + ab * ACC_COLS + (mi / MPG) * BN, adesc + 2 * mi, bdesc + 2 * mi, idesc, (mi % MPG) != 0);
                umma_commit(&st_empty[s]);
                umma_commit(&acc_full[ab]);
            }
        }
    } else {
        // ===== work warps.  Decode: warp dw owns row block dw / 2 and the 64-wide half dw % 2 of every
        // block.  Drain: TMEM lane quarter warp % 4, column quarter dw / 4.
        const int dw = warp - 2, g = lane >> 2, tq = lane & 3;
        const int rb = dw >> 1, jh = dw & 1;
        const int q4 = warp & 3, cq4 = dw >> 2;
        const int drow = q4 * 32 + lane;
        int8_t *tab = sTab + (rb * 2 + (G == 128 ? 0 : jh)) * 16 * NCODE;   // G = 128: the two halves share one table
        float acc[QCOLS];
#pragma unroll
        for (int i = 0; i < QCOLS; ++i) acc[i] = 0.0f;
        // A wait that gives up (bounded, see mbar_wait) must not make this warp leave the loop: with G = 128
        // its partner of the row block would then wait for it at the 64-thread barrier for ever.  The warp
        // keeps walking the blocks instead, without waiting any more, so every barrier still sees both
        // warps; what it computes from then on is discarded (the status word is set, nothing is stored).
        volatile int *gave_up = reinterpret_cast<volatile int *>(tmem_slot + 2);   // CTA-wide flag, cleared at start
        for (int t = 0; t <= KT; ++t) {
            if (t < KT) {
                // ---------------- (a) decode block t
                const int rs = t % A8_RAW_STAGES, s = t % A8_STAGES;
                if (!*gave_up && !mbar_wait(&raw_full[rs], (t / A8_RAW_STAGES) & 1, prm.status, 16)) *gave_up = 1;
                if (t >= A8_STAGES && !*gave_up && !mbar_wait(&st_empty[s], ((t / A8_STAGES) - 1) & 1, prm.status, 17)) *gave_up = 1;
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
                uint8_t *a_stage = sA + s * A8_A_STAGE_BYTES;
                uint8_t *row_lo = a_stage + (rb * 2 + 0) * 1024 + g * 128;
                uint8_t *row_hi = a_stage + (rb * 2 + 1) * 1024 + g * 128;
                float *sc = sScale + (size_t)(t % A8_SRING) * 128 * GPT;
                constexpr int GH = GPT >= 2 ? GPT / 2 : 1;   // groups this warp's 64-wide half touches
                constexpr int CPGH = 4 / GH;                 // 16-wide chunks of the half per such group
                auto do_half = [&](auto jhc) {
                    constexpr int JH = decltype(jhc)::value;
                    static_for<GH>([&](auto gc) {
                        constexpr int gi = (GPT >= 2) ? JH * GH + decltype(gc)::value : 0;
                        const uint2 p_lo = *(const uint2 *)(prow + gi * 8), p_hi = *(const uint2 *)(prow + (8 * GPT + gi) * 8);
                        if (tq == 0 && (G != 128 || JH == 0)) {
                            sc[(rb * 16 + g) * GPT + gi] = __uint_as_float(p_lo.x & 0x7FFFFFFFu);
                            sc[(rb * 16 + g + 8) * GPT + gi] = __uint_as_float(p_hi.x & 0x7FFFFFFFu);
                        }
                        if constexpr (B >= 3) {
                            // signed carrier table: index = stored code u; u = 0 (reserved) -> 0,
                            // u = 2^(B-1) + k -> sign(k) r(|k|).  With G = 128 the two warps of a row block
                            // build eight rows each and meet at a 64-thread barrier.
                            constexpr int bias = 1 << (B - 1);
                            if constexpr (G == 128) named_barrier_sync(1 + rb, 64); else __syncwarp();
                            auto build_row = [&](int row, uint32_t abbits) {
                                const __half2 ab = as_h2(abbits);
                                const float a = __low2float(ab), b = __high2float(ab);
                                const float c = __fsub_rn(__fsub_rn(1.0f, a), b);
                                int8_t *tr = tab + row * NCODE;
                                if (tq == 0) tr[0] = 0;
                                for (int i = tq; i <= Mx; i += 4) {
                                    const float tt = sT[i];
                                    const float q = __fmul_rn(tt, fmaf(tt, fmaf(tt, c, b), a));
                                    int r = __float2int_rn(__fmul_rn(127.0f, q));
                                    r = min(max(r, 0), 127);
                                    tr[bias + i] = (int8_t)r;
                                    tr[bias - i] = (int8_t)(-r);
                                }
                            };
                            if constexpr (G == 128) {
                                if (JH == 0) build_row(g, p_lo.y); else build_row(g + 8, p_hi.y);
                                named_barrier_sync(1 + rb, 64);
                            } else {
                                build_row(g, p_lo.y);
                                build_row(g + 8, p_hi.y);
                                __syncwarp();
                            }
                        }
                        // carriers of the group's 32-wide k blocks, straight into the MMA operand order
                        // (a8_row_regs): lane tq holds bytes 8 tq .. 8 tq + 7 of block m for rows g and g + 8
                        const int8_t *t_lo = tab + g * NCODE, *t_hi = tab + (g + 8) * NCODE;
                        uint4 tab_lo = make_uint4(0, 0, 0, 0), tab_hi = make_uint4(0, 0, 0, 0);
                        if constexpr (B == 4) {
                            tab_lo = *reinterpret_cast<const uint4 *>(t_lo);
                            tab_hi = *reinterpret_cast<const uint4 *>(t_hi);
                        } else if constexpr (B == 3) {
                            const uint2 v0 = *reinterpret_cast<const uint2 *>(t_lo), v1 = *reinterpret_cast<const uint2 *>(t_hi);
                            tab_lo.x = v0.x; tab_lo.y = v0.y; tab_hi.x = v1.x; tab_hi.y = v1.y;
                        }
                        static_for<CPGH / 2>([&](auto mc) {
                            constexpr int MI = 2 * JH + decltype(gc)::value * (CPGH / 2) + decltype(mc)::value;
                            uint2 lo, hi;
                            a8_row_regs<B, 0, MI>(w, tab_lo, t_lo, lo.x, lo.y);
                            a8_row_regs<B, 1, MI>(w, tab_hi, t_hi, hi.x, hi.y);
                            // bytes 32 MI + 8 tq of the row: 16-byte chunk 2 MI + tq / 2, swizzled by the row
                            const int off = (((2 * MI + (tq >> 1)) ^ g) * 16) + (tq & 1) * 8;
                            *(uint2 *)(row_lo + off) = lo;
                            *(uint2 *)(row_hi + off) = hi;
                        });
                    });
                };
                if (jh == 0) do_half(std::integral_constant<int, 0>{}); else do_half(std::integral_constant<int, 1>{});
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&a_full[s]); mbar_arrive(&raw_empty[rs]); }
            }
            if (t >= 1) {
                // ---------------- (b) drain block t - 1
                const int td = t - 1, ab = td & 1;
                if (!*gave_up && !mbar_wait(&acc_full[ab], (td >> 1) & 1, prm.status, 18)) *gave_up = 1;
                tc_fence_after();
                const float *scd = sScale + (size_t)(td % A8_SRING) * 128 * GPT + drow * GPT;
#pragma unroll
                for (int gi = 0; gi < GPT; ++gi) {
                    const float sg = scd[gi];
#pragma unroll
                    for (int c0 = 0; c0 < QCOLS; c0 += 16) {
                        uint32_t r[16];
                        tmem_ld16(tmem_base + ((uint32_t)(q4 * 32) << 16) + ab * ACC_COLS + gi * BN + cq4 * QCOLS + c0, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 16; ++i) acc[c0 + i] = fmaf(sg, (float)(int)r[i], acc[c0 + i]);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[ab]);
            }
        }
        if (!*gave_up) {
            const int e_nb = (int)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 7);
            const int e_mt = (int)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 8);
            const int64_t n = (int64_t)e_nb * TILE + drow;
            const int e_nz = (int)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 4);
            if (n < d.N || e_nz > 1) {   // partial sums of padding channels are written too (zeros), never read back as y
                // the output dtype is decided once, outside the loop over the 64 accumulators (a select inside it
                // costs the registers this kernel does not have)
                // partial tile of this slice: [token of the tile][128 channels]
                const int e_z = (int)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 5);
                const int e_tile = (int)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 6);
                float *pslot = prm.partial + ((size_t)(e_tile - prm.t_full) * prm.slices + e_z) * (size_t)(BN * TILE) + drow;
                auto store_all = [&](auto f16c, auto stagedc) {
                    constexpr bool F16 = decltype(f16c)::value, STAGED = decltype(stagedc)::value;
#pragma unroll
                    for (int i = 0; i < QCOLS; ++i) {
                        const int64_t m = (int64_t)e_mt * BN + cq4 * QCOLS + i;
                        if (m < prm.M) {
                            if (e_nz == 1) {
                                const float v = acc[i] * (prm.dx[m] * (1.0f / 127.0f));
                                if constexpr (STAGED) reinterpret_cast<uint16_t *>(sB)[(cq4 * QCOLS + i) * TILE + drow] = float_to_act(v, F16);
                                else prm.y[m * d.N + n] = float_to_act(v, F16);
                            } else {
                                pslot[(size_t)(cq4 * QCOLS + i) * TILE] = acc[i];
                            }
                        }
                    }
                };
                // A whole tile whose rows of y start on 16-byte boundaries goes through shared memory (the activation
                // ring is idle: every MMA has completed) and is copied out in 16-byte pieces after the CTA's barrier.
                const bool f16o = *reinterpret_cast<volatile uint32_t *>(tmem_slot + 3) != 0;
                if (e_nz == 1 && (d.N & 7) == 0) { if (f16o) store_all(std::true_type{}, std::true_type{}); else store_all(std::false_type{}, std::true_type{}); }
                else { if (f16o) store_all(std::true_type{}, std::false_type{}); else store_all(std::false_type{}, std::false_type{}); }
            }
        }
    }
    if (*reinterpret_cast<volatile int *>(prm.status) != 0) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
    if (*reinterpret_cast<volatile uint32_t *>(tmem_slot + 4) == 1 && (d.N & 7) == 0 && !*reinterpret_cast<volatile uint32_t *>(tmem_slot + 2)) {
        // the staged tile [token][128 channels]: eight channels of one token per thread and step
        const int64_t m0 = (int64_t)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 8) * BN;
        const int64_t n0 = (int64_t)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 7) * TILE;
        const uint16_t *stage = reinterpret_cast<const uint16_t *>(sB);
        for (int c = threadIdx.x; c < BN * (TILE / 8); c += A8_THREADS) {
            const int tok = c / (TILE / 8), part = c % (TILE / 8);
            if (m0 + tok < prm.M && n0 + part * 8 < d.N)
                *reinterpret_cast<uint4 *>(prm.y + (m0 + tok) * d.N + n0 + part * 8) = *reinterpret_cast<const uint4 *>(stage + tok * TILE + part * 8);
        }
    }
    if (*reinterpret_cast<volatile uint32_t *>(tmem_slot + 4) > 1) {
        // The last CTA of this output tile to arrive adds the slices in K order and applies d_x / 127.  The barrier
        // above ordered the CTA's partial stores before thread 0's release.  (Tile, slice count and position are read
        // back from shared memory: held in registers they would stay live across the main loop.)
        const int nz = (int)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 4), tile_id = (int)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 6);
        const int nb = (int)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 7), mt = (int)*reinterpret_cast<volatile uint32_t *>(tmem_slot + 8);
        volatile int *s_last_p = reinterpret_cast<volatile int *>(tmem_slot + 1);   // scratch word after the TMEM slot
        int *ctr = prm.counters + tile_id;
        if (threadIdx.x == 0) {
            int old;
            asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(ctr) : "memory");
            *s_last_p = (old == nz - 1);
        }
        __syncthreads();
        if (*s_last_p) {
            const bool out_f16 = *reinterpret_cast<volatile uint32_t *>(tmem_slot + 3) != 0;
            constexpr int QUADS = BN * TILE / 4;   // four consecutive channels of one token per 128-bit load
            const float4 *src = reinterpret_cast<const float4 *>(prm.partial + (size_t)(tile_id - prm.t_full) * prm.slices * (size_t)(BN * TILE));
            for (int qd = threadIdx.x; qd < QUADS; qd += A8_THREADS) {
                const int64_t m = (int64_t)mt * BN + qd / (TILE / 4), n = (int64_t)nb * TILE + (qd % (TILE / 4)) * 4;
                if (m >= prm.M) continue;
                float4 v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    v[q] = q < nz ? __ldcg(src + (size_t)q * QUADS + qd) : make_float4(0.f, 0.f, 0.f, 0.f);
                float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int q = 0; q < 8; ++q) { sum.x += v[q].x; sum.y += v[q].y; sum.z += v[q].z; sum.w += v[q].w; }  // slice order
                const float f = prm.dx[m] * (1.0f / 127.0f);
                const float o[4] = {sum.x * f, sum.y * f, sum.z * f, sum.w * f};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (n + e < d.N) prm.y[m * d.N + n + e] = float_to_act(o[e], out_f16);
            }
            if (threadIdx.x == 0) *ctr = 0;  // leave the workspace ready for the next call
        }
    }
}

template <int B, int G, int BN>
cudaError_t launch_a8(const void *layout, const Dims &d, const int8_t *x8, int64_t pitch, const float *dx, uint16_t *y,
                      int64_t M, int *status, float *partial, int *counters, bool act_f16, cudaStream_t st) {
    constexpr int GPT = TILE / G;
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return cudaErrorNotSupported;
    CUtensorMap xmap;
    const cuuint64_t dims[2] = {(cuuint64_t)pitch, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)pitch};
    const cuuint32_t box[2] = {128, (cuuint32_t)BN};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&xmap, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t *>(x8), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    A8Params p;
    p.layout = (const uint8_t *)layout; p.dx = dx; p.y = y; p.status = status; p.d = d; p.M = (int)M;
    p.partial = partial; p.counters = counters; p.f16 = act_f16;
    p.raw_stage_bytes = (d.tile_bytes + 1023) / 1024 * 1024;
    static_assert(A8_STAGES == 2 && A8_A_STAGE_BYTES == 128 * 128 && A8_SRING == 8, "a8_fixed_smem spells these out");
    if (p.raw_stage_bytes != a8_raw_stage_bytes(B, G)) return cudaErrorInvalidConfiguration;
    const size_t smem = (size_t)a8_fixed_smem(B, G, BN) + (size_t)a8_raw_stages(B, G, BN) * p.raw_stage_bytes;
    auto kern = gemm_a8_kernel<B, G, BN>;
    static std::atomic<uint64_t> attr_done{0};   // per kernel instantiation: the devices it has been set on
    cudaError_t ea = ensure_func_attr(kern, attr_done, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (ea != cudaSuccess) return ea;
    const A8Plan plan = gemm_a8_plan(d, M);
    if (plan.bn != BN) return cudaErrorInvalidConfiguration;
    p.t_full = (int)plan.t_full; p.slices = plan.slices;
    kern<<<dim3((unsigned)plan.ctas), A8_THREADS, smem, st>>>(xmap, p);
    return cudaGetLastError();
}

// token tile: two accumulator buffers of GPT x BN columns must fit the 512 TMEM columns
template <int B, int G>
cudaError_t launch_a8_bn(const void *layout, const Dims &d, const int8_t *x8, int64_t pitch, const float *dx, uint16_t *y,
                         int64_t M, int *status, float *partial, int *counters, bool act_f16, cudaStream_t st) {
    constexpr int BMAX = 256 / (TILE / G);
    const int bn = gemm_a8_token_tile(d, M);
    if constexpr (BMAX >= 256) if (bn == 256) return launch_a8<B, G, 256>(layout, d, x8, pitch, dx, y, M, status, partial, counters, act_f16, st);
    if constexpr (BMAX >= 128) if (bn == 128) return launch_a8<B, G, 128>(layout, d, x8, pitch, dx, y, M, status, partial, counters, act_f16, st);
    return launch_a8<B, G, 64>(layout, d, x8, pitch, dx, y, M, status, partial, counters, act_f16, st);
}

template <int B>
cudaError_t launch_a8_b(const void *layout, const Dims &d, const int8_t *x8, int64_t pitch, const float *dx, uint16_t *y,
                        int64_t M, int *status, float *partial, int *counters, bool act_f16, cudaStream_t st) {
    switch (d.G) {
        case 32: return launch_a8_bn<B, 32>(layout, d, x8, pitch, dx, y, M, status, partial, counters, act_f16, st);
        case 64: return launch_a8_bn<B, 64>(layout, d, x8, pitch, dx, y, M, status, partial, counters, act_f16, st);
        default: return launch_a8_bn<B, 128>(layout, d, x8, pitch, dx, y, M, status, partial, counters, act_f16, st);
    }
}

}  // namespace

// Quantise the activations (one block per row), then run the tcgen05 INT8 GEMM on the carriers.
cudaError_t launch_gemm_a8_tc(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, bool act_f16,
                              uint8_t *ws, const Workspace &plan, cudaStream_t st, bool prequantized) {
    int8_t *xq = reinterpret_cast<int8_t *>(ws + plan.x8_off);
    float *dxs = reinterpret_cast<float *>(ws + plan.dx_off);
    int *status = reinterpret_cast<int *>(ws + plan.status_off);
    float *partial = reinterpret_cast<float *>(ws + plan.partial_off);
    int *counters = reinterpret_cast<int *>(ws + plan.counters_off);
    const int64_t pitch = (int64_t)d.KT * TILE;
    if (!prequantized) {
        cudaError_t e = launch_quantize_a8(x, M, d.K, xq, pitch, dxs, true, act_f16, st);
        if (e != cudaSuccess) return e;
    }
    switch (d.B) {
        case 1: return launch_a8_b<1>(layout, d, xq, pitch, dxs, y, M, status, partial, counters, act_f16, st);
        case 2: return launch_a8_b<2>(layout, d, xq, pitch, dxs, y, M, status, partial, counters, act_f16, st);
        case 3: return launch_a8_b<3>(layout, d, xq, pitch, dxs, y, M, status, partial, counters, act_f16, st);
        case 4: return launch_a8_b<4>(layout, d, xq, pitch, dxs, y, M, status, partial, counters, act_f16, st);
        case 5: return launch_a8_b<5>(layout, d, xq, pitch, dxs, y, M, status, partial, counters, act_f16, st);
        case 6: return launch_a8_b<6>(layout, d, xq, pitch, dxs, y, M, status, partial, counters, act_f16, st);
        case 7: return launch_a8_b<7>(layout, d, xq, pitch, dxs, y, M, status, partial, counters, act_f16, st);
        default: return launch_a8_b<8>(layout, d, xq, pitch, dxs, y, M, status, partial, counters, act_f16, st);
    }
}

}  // namespace cq
