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

// Look-back by the whole CTA: every thread inspects one predecessor, so one round trip to
// memory covers kCompactThreads tiles (with a few hundred tiles in flight at once, a
// warp-wide window would need many round trips to reach a tile that already knows its
// prefix).  `aggregate` is this tile's payload (< 2^62; the exact Top_k path packs two
// 31-bit counts, whose sums never carry into each other because d < 2^31).  Called by all
// threads; returns to all of them the sum of the payloads of all earlier tiles, and
// publishes this tile's inclusive prefix.
// Test hooks of this translation unit: the poll limit of the look-back, and a tile that keeps
// its status word to itself (-1: none), which makes its successors' bounded waits run out.
static __device__ int g_lookback_poll_limit = kLookbackPollLimit;
static __device__ int g_lookback_mute_tile = -1;
static int set_compact_knob(int key, int value) {
    if (key == kKnobLookbackPolls) return (int)cudaMemcpyToSymbol(g_lookback_poll_limit, &value, sizeof(int));
    if (key == kKnobMuteTile) return (int)cudaMemcpyToSymbol(g_lookback_mute_tile, &value, sizeof(int));
    return 0;
}
static const int g_compact_knob_registered = register_knob_setter(&set_compact_knob);

struct LookbackSmem {
    unsigned long long sum_all[kCompactThreads / 32];
    unsigned long long sum_upto[kCompactThreads / 32];
    int first[kCompactThreads / 32];  // lane of the nearest prefix holder in the warp, 32 if none
    int gave_up;
    unsigned long long result;
};

__device__ __forceinline__ unsigned long long lookback_block(unsigned long long* status, int tile,
                                                             unsigned long long aggregate, int* dev_status,
                                                             LookbackSmem& sm) {
    constexpr int NW = kCompactThreads / 32;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const bool mute = (tile == g_lookback_mute_tile);
    const int poll_limit = g_lookback_poll_limit;
    if (tile == 0) {
        if (tid == 0 && !mute) st_status(&status[0], (kFlagPrefix << kFlagShift) | aggregate);
        return 0ull;
    }
    if (tid == 0) {
        if (!mute) st_status(&status[tile], (kFlagAggregate << kFlagShift) | aggregate);
        sm.gave_up = 0;
    }
    __syncthreads();
    unsigned long long excl = 0ull;
    int pos = tile - 1;
    while (true) {
        const int mine = pos - tid;
        // before tile 0 sits a virtual inclusive prefix of zero
        unsigned long long wd = (mine >= 0) ? ld_status(&status[mine]) : (kFlagPrefix << kFlagShift);
        int polls = 0;
        while ((wd >> kFlagShift) == 0ull) {  // bounded wait for this predecessor's word
            if (++polls > poll_limit) { sm.gave_up = 1; break; }
            __nanosleep(20);
            wd = ld_status(&status[mine]);
        }
        const unsigned int pm = __ballot_sync(0xffffffffu, (wd >> kFlagShift) == kFlagPrefix);
        const int fl = pm ? (__ffs(pm) - 1) : 32;
        unsigned long long all = wd & kPayloadMask;
        unsigned long long upto = (lane <= fl) ? all : 0ull;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            all += __shfl_xor_sync(0xffffffffu, all, o);
            upto += __shfl_xor_sync(0xffffffffu, upto, o);
        }
        if (lane == 0) { sm.sum_all[w] = all; sm.sum_upto[w] = upto; sm.first[w] = fl; }
        __syncthreads();
        // warps are in order of distance: the first warp that holds a prefix ends the walk
        unsigned long long total = 0ull;
        bool found = false;
#pragma unroll
        for (int q = 0; q < NW; ++q) {
            if (!found) {
                if (sm.first[q] < 32) { total += sm.sum_upto[q]; found = true; }
                else total += sm.sum_all[q];
            }
        }
        const bool stop = found || sm.gave_up;
        excl += total;
        __syncthreads();  // the arrays are rewritten by the next window
        if (stop) break;
        pos -= kCompactThreads;
    }
    if (sm.gave_up) {
        if (tid == 0) atomicOr(dev_status, GK_DEV_TIMEOUT);
        excl = 0ull;
    }
    if (tid == 0 && !mute) st_status(&status[tile], (kFlagPrefix << kFlagShift) | (excl + aggregate));
    return excl;
}

// Host side: launch a compaction kernel whose last parameter is the `persistent` flag.
// Where the device supports it the kernel is launched cooperatively with as many CTAs as are
// resident at once (persistent = 1: static tile assignment, no ticket); otherwise one CTA per
// tile with ticketed tiles.  The arguments must have exactly the kernel's parameter types.
template <class Kernel, class... Args>
inline cudaError_t launch_compaction(Kernel kernel, int n_tiles, int sm_count, cudaStream_t st, Args... a) {
    int dev = 0, coop = 0, occ = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    int persistent = 0;
    int grid = n_tiles;
    if (coop && cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kCompactThreads, 0) == cudaSuccess &&
        occ > 0) {
        persistent = 1;
        grid = occ * sm_count < n_tiles ? occ * sm_count : n_tiles;
    } else {
        cudaGetLastError();
    }
    void* args[] = {(void*)&a..., (void*)&persistent};
    if (persistent)
        return cudaLaunchCooperativeKernel((const void*)kernel, dim3((unsigned)grid), dim3(kCompactThreads), args, 0, st);
    return cudaLaunchKernel((const void*)kernel, dim3((unsigned)grid), dim3(kCompactThreads), args, 0, st);
}

}  // namespace gk
