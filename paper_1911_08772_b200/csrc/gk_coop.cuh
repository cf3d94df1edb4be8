// Pieces shared by the persistent cooperative kernels (one CTA of 1024 threads
// per SM, rows of 1024 float4): asynchronous copies, the L2-retaining store,
// and the bounded grid barrier.  Internal.
#pragma once

#include "gk_common.cuh"

namespace gk {

constexpr int kFusedThreads = 1024;
constexpr int kFusedWarps = kFusedThreads / 32;
constexpr int kRowF4 = kFusedThreads;    // float4 per row
constexpr int kRowBytes = kRowF4 * 16;   // 16 KB
constexpr int kBarrierPollLimit = 1 << 24;

#ifdef __CUDACC__

// Poll limit of grid_barrier in this translation unit (a test may lower it).
static __device__ int g_barrier_poll_limit = kBarrierPollLimit;
static int set_coop_knob(int key, int value) {
    if (key != kKnobBarrierPolls) return 0;
    return (int)cudaMemcpyToSymbol(g_barrier_poll_limit, &value, sizeof(int));
}
static const int g_coop_knob_registered = register_knob_setter(&set_coop_knob);

// 16-byte asynchronous copy global -> shared, bypassing L1.
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    const unsigned int s = (unsigned int)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// 32-byte store that asks L2 to keep the line longer than ordinary traffic (the eviction
// priority is only available on 256-bit accesses).  p must be 32-byte aligned.
__device__ __forceinline__ void st_keep32(float4* p, const float4 a, const float4 b) {
    asm volatile("st.global.L2::evict_last.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(a.x), "f"(a.y),
                 "f"(a.z), "f"(a.w), "f"(b.x), "f"(b.y), "f"(b.z), "f"(b.w)
                 : "memory");
}

// Arrive at a barrier counter and wait until all G CTAs have arrived.
// Returns false when the bounded wait ran out.
__device__ __forceinline__ bool grid_barrier(unsigned int* counter, unsigned int G, int* ok_flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        int polls = 0;
        const int limit = g_barrier_poll_limit;
        bool ok = true;
        while (true) {
            unsigned int v;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
            if (v >= G) break;
            if (++polls > limit) { ok = false; break; }
            __nanosleep(40);
        }
        *ok_flag = ok ? 1 : 0;
    }
    __syncthreads();
    return *ok_flag != 0;
}

// The per-(row, warp) table of the persistent kernels: one uint16 per cell of 128 elements.
constexpr int kGroupRows = 8;                // rows a warp gathers per batch
constexpr unsigned int kFlagBit = 0x8000u;   // fused sparsifier: the cell has not been counted yet
constexpr unsigned int kMaxMask = 0x7fffu;   // fused sparsifier: the cell's maximum (top 16 bits, rounded up)

// Up to kGroupRows of this warp's cells (local rows) that meet a condition, from row `cursor`
// on: their rows go to qrow[0 ..), the cursor moves past the last one taken.  Called by all
// lanes of a warp; returns the number of rows gathered.
enum GatherWhat { kGatherFlagged, kGatherPending, kGatherNonZero };
constexpr unsigned short kPending = 0xffffu;   // the cell is marked, its count is still to come
template <GatherWhat WHAT>
__device__ __forceinline__ int gather_cells(const unsigned short* table, const int nrows, int& cursor,
                                            unsigned short* qrow, const unsigned int above = 0u) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int n = 0;
    while (n < kGroupRows && cursor < nrows) {
        const int r = cursor + lane;
        unsigned int e = 0u;
        if (r < nrows) e = table[r * kFusedWarps + w];
        // (flagged cells only count when their maximum reaches the lowest threshold of interest)
        const bool hit = WHAT == kGatherFlagged ? (e & kFlagBit) != 0u && (e & kMaxMask) > above
                         : WHAT == kGatherPending ? e == kPending : e != 0u;
        unsigned int b = __ballot_sync(0xffffffffu, hit);
        while (b && n < kGroupRows) {
            const int bit = __ffs(b) - 1;
            if (lane == 0) qrow[n] = (unsigned short)(cursor + bit);
            ++n;
            b &= b - 1u;
        }
        if (b) { cursor += __ffs(b) - 1; break; }
        cursor += 32;
    }
    __syncwarp();
    return n;
}

#endif  // __CUDACC__

}  // namespace gk
