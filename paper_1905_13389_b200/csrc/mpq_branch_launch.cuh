// Launch policy of the branch-fused kernel: which tile width, and whether the CTA is split into
// k-groups, for a given problem on the device at hand.
#pragma once
#include "mpq_branch_kernel.cuh"

namespace mpq {

// Streamed-side tile width (16*TS items): the widest tile has the least shared-memory traffic per
// population count, but a grid of few large tiles leaves SMs idle in its last wave.  Pick the
// width with the smallest estimated makespan: waves of (resident CTAs x SM count) tiles, each
// costing its width times the CTAs that share an SM times a measured per-width inefficiency.
// A GEMM with a long k whose tiles would occupy at most one CTA per multiprocessor (a fully-connected
// layer at small batch) takes the narrowest such tile and splits the CTA into k-groups instead:
// two or three times the warps per SM on the same tiles.
template <int HB, int SB, int MODE>
static int launch_auto(const BranchParams& p, cudaStream_t st) {
    using T = BranchTile<HB, SB>;
    const int64_t held_tiles = ceil_div(p.held_rows, 16 * T::TH);
    const int sms = sm_count();
    if (sms <= 0) return MPQ_ERR_CUDA;
    if (MODE == kModeGemm && ceil_div(p.rw / 4, T::KQ) >= 12) {
        // three k-groups where the thread tile fits 80 registers, else two
        constexpr int KS = HB * SB <= 16 ? 3 : 2;
        if (ceil_div(p.streamed_rows, 32) * held_tiles <= sms) return launch_branch<HB, SB, 2, kModeGemm, KS>(p, st);
        if (ceil_div(p.streamed_rows, 64) * held_tiles <= sms) return launch_branch<HB, SB, 4, kModeGemm, KS>(p, st);
    }
    // (with 7 or 8 streamed planes the 128-wide tile's loop body outgrows the instruction cache)
    const double penalty[3] = {SB >= 7 ? 1.10 : 1.00, T::resident(4) == 3 ? 0.98 : 1.05, 1.20};      // TS = 8, 4, 2
    int best = 0;
    double best_cost = 0.0;
    for (int c = 0; c < (MODE == kModeConv ? 2 : 3); ++c) {      // the 32-wide tile never won for a convolution
        const int ts = 8 >> c;
        const int per_sm = T::resident(ts);
        const int64_t slots = (int64_t)per_sm * sms;
        const int64_t tiles = ceil_div(p.streamed_rows, 16 * ts) * held_tiles;
        // a grid that fits the resident slots takes one tile time; a longer one its share of waves
        // plus half a wave of tail; a tile's time grows with its width and with the CTAs sharing the SM
        const double waves = tiles <= slots ? 1.0 : (double)tiles / (double)slots + 0.5;
        const double cost = waves * ts * per_sm * penalty[c];
        if (c == 0 || cost < best_cost) { best = c; best_cost = cost; }
    }
    if (best == 0) return launch_branch<HB, SB, 8, MODE>(p, st);
    if (best == 1) return launch_branch<HB, SB, 4, MODE>(p, st);
    return launch_branch<HB, SB, 2, kModeGemm>(p, st);
}

}  // namespace mpq
