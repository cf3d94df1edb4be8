// Pieces shared by the persistent cooperative selection kernels (exact Top_k and
// DGC_k): shared-memory layout, magnitude keys, warp scans, the merged radix
// histogram and the choice of a digit from it.  Internal.
#pragma once

#include "gk_common.cuh"
#include "gk_coop.cuh"

namespace gk {

constexpr int kTkTableMaxRows = 448;                                   // rows per CTA the maximum table covers
constexpr int kTkTableBytes = kTkTableMaxRows * kFusedWarps * 2;       // 28 KB: one uint16 per (row, warp)
constexpr int kTkSmemRows = 11;                                        // 16 KB rows of dynamic shared memory
constexpr int kTkSmemBytes = kTkSmemRows * kRowBytes + kTkTableBytes;  // g ring (ACCUM), u slots, table
// rows in flight in pass 1, plus one: with ACCUM every row is two copies (g and eps), else one,
// and about 100 KB in flight per SM are what it takes to keep HBM busy
template <bool ACCUM> struct TkStages { static constexpr int value = ACCUM ? 4 : 8; };
constexpr int kTkGroupRows = 8;                                        // rows a warp gathers per batch
constexpr int kTkBins = 2048;
// The write-out keeps the places of a CTA's selected entries in shared memory, two words each:
// in rows the first pass no longer needs (the g ring) or, when u is given, in two rows set aside.
constexpr int kTkStageRows = 2;
constexpr unsigned short kTkPending = 0xffffu;                         // table entry: segment still to be counted

struct __align__(128) TopkShared {
    unsigned int hist[kTkBins];      // this CTA's histogram of the current digit
    unsigned int wsum[kFusedWarps];
    unsigned long long wsum2[kFusedWarps];
    // keys above T (low word) and equal to T (high word): per round of G consecutive rows, and
    // in the vector before each row of this CTA
    unsigned long long roundtot[kTkTableMaxRows];
    unsigned long long rowpre[kTkTableMaxRows];
    unsigned short qrow[kFusedWarps][kTkGroupRows];
    unsigned long long need;         // entries still to take among the keys that match the digits so far
    unsigned int digit;
    unsigned int n_staged;           // selected entries whose places were put aside for the write-out
    int ok;
};
static_assert((sizeof(TopkShared) + 1023) / 1024 * 1024 + kTkSmemBytes <= 232448,
              "over the 227 KB of shared memory per CTA (the dynamic part starts on a 1 KB boundary)");

__device__ __forceinline__ unsigned int tk_key(float x) { return __float_as_uint(x) & 0x7fffffffu; }

__device__ __forceinline__ unsigned int warp_incl_scan(unsigned int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}
__device__ __forceinline__ unsigned long long warp_incl_scan64(unsigned long long v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Called by every CTA after a grid barrier.  ghist: the level's NB merged bins.  Finds the
// largest digit D with  #(keys in bins > D) < need <= #(keys in bins >= D),  leaves D in
// sh.digit and need - #(keys in bins > D) in sh.need.
__device__ __forceinline__ void pick_digit(const unsigned int* __restrict__ ghist, int NB, TopkShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const unsigned long long need = sh.need;
    // thread 0 owns the two highest bins, thread 1 the next two, ...
    const int hi = NB - 1 - 2 * tid, lo = hi - 1;
    const unsigned int g_hi = hi >= 0 ? __ldcg(ghist + hi) : 0u;
    const unsigned int g_lo = lo >= 0 ? __ldcg(ghist + lo) : 0u;
    const unsigned int mine = g_hi + g_lo;
    const unsigned int s = warp_incl_scan(mine, lane);
    if (lane == 31) sh.wsum[w] = s;
    __syncthreads();
    const unsigned int x = sh.wsum[lane];
    const unsigned int y = warp_incl_scan(x, lane);
    const unsigned int wpre = __shfl_sync(0xffffffffu, y - x, w);
    const unsigned long long above = (unsigned long long)wpre + s - mine;  // keys in the bins above `hi`
    __syncthreads();  // every thread has read sh.need and sh.wsum
    if (above < need && need <= above + mine) {  // true in exactly one thread
        if (need <= above + g_hi) { sh.digit = (unsigned int)hi; sh.need = need - above; }
        else { sh.digit = (unsigned int)lo; sh.need = need - above - g_hi; }
    }
    __syncthreads();
}

// Adds this CTA's histogram to the merged one and clears it.
__device__ __forceinline__ void merge_hist(unsigned int* __restrict__ ghist, int NB, TopkShared& sh) {
    for (int b = threadIdx.x; b < NB; b += kFusedThreads) {
        const unsigned int c = sh.hist[b];
        if (c) { atomicAdd(ghist + b, c); sh.hist[b] = 0u; }
    }
}

}  // namespace gk
