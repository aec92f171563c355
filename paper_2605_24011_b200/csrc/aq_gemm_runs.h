// Host-only: how the prefill GEMM's work is cut into one contiguous run per CTA.  Plain C++ (no CUDA), so that the
// partition can be tested with the host compiler alone.
#pragma once
#include <cstdint>

namespace aq {

constexpr int GM_MAX_GRID = 192;   // CTAs of one launch (one per SM)
// What ending one piece of a tile costs a CTA (accumulator drain, epilogue, refilling the pipeline), in units of one
// slab-accumulator of MMA work (measured: about 8 us against 0.88 us); the runs are cut so that work + pieces balance.
constexpr int GM_SEG_COST = 9;

// Cuts [0, total) into `grid` contiguous runs with even bounds (bounds[0] = 0 .. bounds[grid] = total).  The work is a
// sequence of tiles: n_two tiles of c2 units first, then tiles of c1 units.  A run costs its units plus GM_SEG_COST per
// tile it touches; the smallest budget under which a greedy walk places everything is found by bisection.
inline void cut_runs(long long total, long long n_two, long long c2, long long c1, int grid, int* bounds) {
    auto tile_end = [&](long long pos) {
        const long long reg2 = n_two * c2;
        return pos < reg2 ? (pos / c2 + 1) * c2 : reg2 + ((pos - reg2) / c1 + 1) * c1;
    };
    auto walk = [&](long long budget, int* out) {
        long long pos = 0;
        for (int c = 0; c < grid; ++c) {
            if (out) out[c] = (int)pos;
            long long left = budget;
            while (pos < total) {
                const long long te = tile_end(pos), need = GM_SEG_COST + (te - pos);
                if (need <= left) { pos = te; left -= need; continue; }
                const long long take = (left - GM_SEG_COST) & ~1LL;
                if (take >= 2) pos += take;
                break;
            }
        }
        if (out) out[grid] = (int)total;
        return pos >= total;
    };
    long long lo = total / grid, hi = total / grid + c2 + 4 * GM_SEG_COST + 2;
    while (!walk(hi, nullptr)) hi *= 2;
    while (lo < hi) {
        const long long mid = (lo + hi) / 2;
        if (walk(mid, nullptr)) hi = mid; else lo = mid + 1;
    }
    walk(hi, bounds);   // (a tail of CTAs may be left without work: their runs are empty)
}

// Cost of the run [lo, hi) under the model above.
inline long long run_cost(long long lo, long long hi, long long n_two, long long c2, long long c1) {
    long long cost = 0;
    const long long reg2 = n_two * c2;
    for (long long pos = lo; pos < hi;) {
        const long long te = pos < reg2 ? (pos / c2 + 1) * c2 : reg2 + ((pos - reg2) / c1 + 1) * c1;
        const long long end = te < hi ? te : hi;
        cost += GM_SEG_COST + (end - pos);
        pos = end;
    }
    return cost;
}

}  // namespace aq
