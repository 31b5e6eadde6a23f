// Large-M packed GEMM on the 5th-generation tensor cores (Section 5.3 dense path, re-done for
// sm_100a): weights stay packed in HBM and are decoded into bf16 shared-memory operand tiles
// right before tcgen05.mma consumes them; accumulators live in TMEM.
//
// Roles inside a CTA (output tiles of 128 channels x BN or 2 BN tokens):
//   warp 0      TMA-loads activation tiles x[BN x 64] (128-byte swizzle) into a ring of stages; nothing but the wait
//               for a stage stands between the MMAs that free it and the copy that refills it
//   warp 18     bulk-copies raw layout tiles (codes + co-located group parameters) into their own ring (2-4 deep)
//   warp 1      allocates TMEM, issues tcgen05.mma (one elected lane), commits to mbarriers
//   warps 2..17 decode: raw tile -> s_g * q(|k|/M) * sign (Eq. cubic; q by the half2 Horner form of
//               Eq. gpu-horner on the power-of-two-normalised code, scale in fp32), rounded to bf16 and stored in
//               the K-major 128-byte-swizzled layout the MMA reads; then the epilogue
//               (tcgen05.ld -> bf16 -> y)
// Weights sit on the MMA's M side (TMEM lane = output channel), tokens on its N side, so any
// token count maps to a legal instruction shape and each epilogue thread owns one output channel.
//
// Every wait on an mbarrier is bounded: a wait that runs out sets a status word in global memory and a
// flag in shared memory, after which no role of the CTA waits any more; the CTA still walks its loops to
// the end, releases TMEM and exits.
//
// This file holds the plan (which CTA computes what) and the instantiations that compute one whole tile
// per CTA; cq_gemm_tc_sk.cu holds those that also share tiles between CTAs (stream-K); the kernel itself is
// in cq_gemm_tc_impl.cuh.
#include "cq_gemm_tc_impl.cuh"

namespace cq {

int gemm_tc_available() { return 1; }

// Token tile of the model-dtype GEMM for M rows.
int gemm_tc_token_tile(int64_t M) { return M <= 32 ? 32 : M <= 64 ? 64 : M <= 128 ? 128 : M <= 256 ? 256 : 512; }
// How the model-dtype GEMM is spread over the SMs.  Whole tiles, one CTA each, fill the SMs round after
// round.  When the last round would leave SMs idle, its r tiles are cut along K as well (stream-K) -- if that
// pays.  In units of one layout tile of main loop: a whole tile costs KT + 4 (pipeline fill, epilogue).
//   (b) every tile cut into the same number s of runs, so that a run lies inside its tile: a run costs its
//       length + 4 .. 10 (the fill, the partial tile's trip through L2 and, for one CTA per tile, the addition
//       of the partial tiles; the more the wider the token tile), and r s runs take ceil(r s / SMs) rounds;
//   (a) one run per SM, cut anywhere: the best balance, but most runs cross from one tile into the next (two
//       fills, two partial tiles: length + 10 .. 22; recalibrated against forced plans at M = 64 .. 4096).
// The kernel that can share tiles runs about 5 % slower on every tile of the launch than the one that cannot
// (measured at M = 4096, N = 57344, K = 8192, and at M = 1024, N = 6144, K = 4096; merely compiling the partial-tile
// code into the kernel costs that much), so it is a separate instantiation and sharing has to save more.
TcPlan gemm_tc_plan(const Dims &d, int64_t M) {
    TcPlan p;
    p.bnt = gemm_tc_token_tile(M);
    p.token_tiles = (int)((M + p.bnt - 1) / p.bnt);
    const int64_t T = (int64_t)d.NB * p.token_tiles, sms = sm_count();
    const int64_t r = T % sms;                      // tiles of the last, partial round
    p.t_full = T; p.p2 = 0; p.crossing = 0;
    if (r != 0) {
        const int64_t V2 = r * d.KT;
        const double wide = (double)p.bnt / 512.0;   // the partial tiles grow with the token tile
        const double whole = (double)(d.KT + 4), all = (double)(T / sms + 1) * whole;
        double best = 1e30;
        int64_t best_p2 = 0;
        int best_crossing = 0;
        for (int64_t s = 2; s <= 16 && s * 4 <= d.KT; ++s) {
            const double c = (double)((r * s + sms - 1) / sms) * ((double)d.KT / (double)s + 4.0 + 6.0 * wide);
            if (c < best) { best = c; best_p2 = r * s; best_crossing = 0; }
        }
        int64_t pa = sms;
        if (pa > V2 / 4) pa = V2 / 4;               // at least four layout tiles per run
        if (pa > r) {
            const double c = (double)V2 / (double)pa + 10.0 + 12.0 * wide;
            if (c < best) { best = c; best_p2 = pa; best_crossing = 1; }
        }
        if (best_p2 > 0 && (whole - best) / all > 0.06) { p.p2 = (int)best_p2; p.crossing = best_crossing; p.t_full = T - r; }
    }
    p.ctas = (int)(p.t_full + p.p2);
    p.stream_k = p.p2 > 0;
    return p;
}

// stream-K instantiations: cq_gemm_tc_sk.cu
cudaError_t launch_gemm_tc_streamk(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int *status,
                                   float *partial, int *counters, bool act_f16, cudaStream_t st);

cudaError_t launch_gemm_tc(const void *layout, const Dims &d, const uint16_t *x, uint16_t *y, int64_t M, int mode,
                           bool act_f16, uint8_t *ws, const Workspace &plan, cudaStream_t st) {
    if (mode != 0) return cudaErrorNotSupported;
    int *status = reinterpret_cast<int *>(ws + plan.status_off);
    float *partial = reinterpret_cast<float *>(ws + plan.partial_off);
    int *counters = reinterpret_cast<int *>(ws + plan.counters_off);
    if (gemm_tc_plan(d, M).p2 > 0) return launch_gemm_tc_streamk(layout, d, x, y, M, status, partial, counters, act_f16, st);
    return launch_tc_variant<false>(layout, d, x, y, M, status, partial, counters, act_f16, st);
}

}  // namespace cq
