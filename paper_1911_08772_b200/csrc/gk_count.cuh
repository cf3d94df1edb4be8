// Exact multi-threshold counting: #{|u| > candidate} for the ten candidates of
// Algorithm 1 (arXiv 1911.08772), shared by the fused kernel and the segmented count stage.
#pragma once

#include "gk_common.cuh"

namespace gk {

// 1.0f when a > c, else 0.0f: one compare instruction with a float result.
__device__ __forceinline__ float gt_as_float(float a, float c) {
    float r;
    asm("set.gt.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(c));
    return r;
}

// Candidates LO..HI-1 (in ascending order of value) against the four magnitudes of one
// float4.  The counters are floats: exact up to 2^24 per thread, far above a thread's share.
template <int LO, int HI, int N>
__device__ __forceinline__ void count_tier(const float a0, const float a1, const float a2, const float a3,
                                           const float (&cs)[N], float (&acc)[N]) {
#pragma unroll
    for (int j = LO; j < HI; ++j)
        acc[j] += (gt_as_float(a0, cs[j]) + gt_as_float(a1, cs[j])) + (gt_as_float(a2, cs[j]) + gt_as_float(a3, cs[j]));
}

// rm: the cell's largest magnitude (top 16 bits, rounded up).  A candidate whose top 16
// bits (rounded down) are not below rm cannot be exceeded by any element of the cell, nor
// can any larger candidate: candidates 0..1, 2..4, 5..6 and 7..9 (in ascending order) are
// evaluated only as far as the cell's maximum reaches.
struct Tiers { unsigned int t0, t2, t5, t7; };
__device__ __forceinline__ void count_float4(const float4 v, const unsigned int rm, const float (&cs)[kNumCand],
                                             const Tiers& tier, float (&acc)[kNumCand]) {
    if (rm <= tier.t0) return;  // warp-uniform, as are the tests below
    const float a0 = fabsf(v.x), a1 = fabsf(v.y), a2 = fabsf(v.z), a3 = fabsf(v.w);
    count_tier<0, 2>(a0, a1, a2, a3, cs, acc);
    if (rm > tier.t2) {
        count_tier<2, 5>(a0, a1, a2, a3, cs, acc);
        if (rm > tier.t5) {
            count_tier<5, 7>(a0, a1, a2, a3, cs, acc);
            if (rm > tier.t7) count_tier<7, kNumCand>(a0, a1, a2, a3, cs, acc);
        }
    }
}

__device__ __forceinline__ unsigned int max_mag_bits(const float4 u) {
    return __float_as_uint(fmaxf(fmaxf(fabsf(u.x), fabsf(u.y)), fmaxf(fabsf(u.z), fabsf(u.w))));
}


// Tier limits for candidates cs[] in ascending order: the top 16 bits of each tier's lowest
// candidate, rounded down.  A negative candidate is exceeded by every magnitude; since the
// candidates ascend it is enough to test the lowest one (callers then pass rm = 0x10000).
__device__ __forceinline__ Tiers make_tiers(const float (&cs)[kNumCand]) {
    Tiers t;
    t.t0 = __float_as_uint(fmaxf(cs[0], 0.f)) >> 16;
    t.t2 = __float_as_uint(fmaxf(cs[2], 0.f)) >> 16;
    t.t5 = __float_as_uint(fmaxf(cs[5], 0.f)) >> 16;
    t.t7 = __float_as_uint(fmaxf(cs[7], 0.f)) >> 16;
    return t;
}

}  // namespace gk
