// Single-pass, order-preserving stream compaction with decoupled look-back.
//
// A tile is kCompactThreads x kCompactRows float4.  Tiles are handed out
// through an atomic ticket, so every tile a CTA may have to wait for is
// already resident or finished.  A CTA publishes its tile's survivor count
// (flag "aggregate") in a 64-bit status word, walks back over its
// predecessors' words until it meets an inclusive prefix, and then publishes
// its own inclusive prefix.  Every wait is bounded: when the poll limit runs
// out the CTA records GK_DEV_TIMEOUT, assumes a zero prefix and carries on, so
// the kernel always terminates.
#pragma once

#include "gk_common.cuh"

namespace gk {

// Exclusive offsets, in (row, thread) order, of per-thread per-row counts.
// c[j] in 0..4 is the number of survivors this thread holds in row j.
// Returns the tile total; off[j] is the number of survivors that precede this
// thread's row-j elements inside the tile.
struct TileScanSmem {
    unsigned int wtot[kCompactRows / 4][kCompactThreads / 32];
    unsigned int off[kCompactRows][kCompactThreads / 32];
    unsigned int total;
};

__device__ __forceinline__ unsigned int tile_scan(const unsigned int (&c)[kCompactRows],
                                                  unsigned int (&off)[kCompactRows],
                                                  TileScanSmem& sm) {
    constexpr int NW = kCompactThreads / 32;
    static_assert(NW == 8 && kCompactRows % 4 == 0, "scan layout assumes 8 warps, rows in fours");
    constexpr int G = kCompactRows / 4;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    unsigned int incl[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        unsigned int p = c[4 * g] | (c[4 * g + 1] << 8) | (c[4 * g + 2] << 16) | (c[4 * g + 3] << 24);
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            unsigned int t = __shfl_up_sync(0xffffffffu, p, o);
            if (lane >= o) p += t;  // byte lanes hold at most 32 * 4 = 128: no carry
        }
        incl[g] = p;
        if (lane == 31) sm.wtot[g][w] = p;
    }
    __syncthreads();
    if (w == 0) {
        unsigned int run = 0;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int j = lane >> 3, ww = lane & 7;  // lane enumerates (row in group, warp)
            const unsigned int v = (sm.wtot[g][ww] >> (8 * j)) & 0xffu;
            unsigned int s = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                unsigned int t = __shfl_up_sync(0xffffffffu, s, o);
                if (lane >= o) s += t;
            }
            sm.off[4 * g + j][ww] = run + s - v;
            run += __shfl_sync(0xffffffffu, s, 31);
        }
        if (lane == 0) sm.total = run;
    }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
        for (int j = 0; j < 4; ++j)
            off[4 * g + j] = sm.off[4 * g + j][w] + ((incl[g] >> (8 * j)) & 0xffu) - c[4 * g + j];
    return sm.total;
}

// Look-back by one full warp.  `aggregate` is this tile's payload (< 2^62; the
// exact Top_k path packs two 31-bit counts, whose sums never carry into each
// other because d < 2^31).  Returns the sum of the payloads of all earlier
// tiles and publishes this tile's inclusive prefix.
__device__ __forceinline__ unsigned long long lookback_warp(unsigned long long* status, int tile,
                                                            unsigned long long aggregate,
                                                            int* dev_status) {
    const int lane = threadIdx.x & 31;
    if (tile == 0) {
        if (lane == 0) st_status(&status[0], (kFlagPrefix << kFlagShift) | aggregate);
        return 0ull;
    }
    if (lane == 0) st_status(&status[tile], (kFlagAggregate << kFlagShift) | aggregate);
    unsigned long long excl = 0ull;
    int pos = tile - 1;
    bool gave_up = false;
    while (true) {
        const int mine = pos - lane;
        // before tile 0 sits a virtual inclusive prefix of zero
        unsigned long long wd = (mine >= 0) ? ld_status(&status[mine]) : (kFlagPrefix << kFlagShift);
        int polls = 0;
        while (__any_sync(0xffffffffu, (wd >> kFlagShift) == 0ull)) {
            if (++polls > kLookbackPollLimit) { gave_up = true; break; }
            __nanosleep(20);
            if ((wd >> kFlagShift) == 0ull) wd = ld_status(&status[mine]);
        }
        if (gave_up) break;
        const unsigned int pm = __ballot_sync(0xffffffffu, (wd >> kFlagShift) == kFlagPrefix);
        const int stop = pm ? (__ffs(pm) - 1) : 31;  // nearest predecessor holding a prefix
        unsigned long long v = (lane <= stop) ? (wd & kPayloadMask) : 0ull;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        excl += v;
        if (pm) break;
        pos -= 32;
    }
    if (gave_up) {
        if (lane == 0) atomicOr(dev_status, GK_DEV_TIMEOUT);
        excl = 0ull;
    }
    if (lane == 0) st_status(&status[tile], (kFlagPrefix << kFlagShift) | (excl + aggregate));
    return excl;
}

}  // namespace gk
