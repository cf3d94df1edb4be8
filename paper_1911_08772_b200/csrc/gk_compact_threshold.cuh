// Ordered compaction of the survivors |u_i| > threshold into (index, value)
// pairs, with the selected slots of u cleared (Eq. 2: eps = u - Comp(u)).
// Used by the whole-vector and by the segmented sparsifier.
#pragma once

#include "gk_common.cuh"
#include "gk_compact.cuh"

namespace gk {

// Segment that holds element i: the s in [0, S) with off[s] <= i < off[s + 1].
// Called by all 32 lanes of a warp with the same arguments: a 32-ary search, so that a table
// of a few hundred segments costs two rounds of global loads instead of eight.
__device__ __forceinline__ int find_segment(const int64_t* __restrict__ off, int S, int64_t i) {
    const int lane = threadIdx.x & 31;
    int lo = 0, hi = S - 1;  // the answer is the first s in [lo, hi] with off[s + 1] > i
    while (lo < hi) {
        const int n = hi - lo + 1;
        const int step = (n + 31) / 32;
        // lane l asks about the last segment of its group: s_l = lo + (l + 1) * step - 1
        int sl = lo + (lane + 1) * step - 1;
        if (sl > hi) sl = hi;
        const bool above = off[sl + 1] > i;
        const unsigned int m = __ballot_sync(0xffffffffu, above);
        if (m == 0u) { lo = hi; break; }  // malformed table: settle on the last segment
        const int g = __ffs(m) - 1;       // first group whose last segment ends above i
        int nhi = lo + (g + 1) * step - 1;
        if (nhi > hi) nhi = hi;
        lo = lo + g * step;
        hi = nhi;
        if (step == 1) { lo = hi; break; }
    }
    return lo;
}

// ---------------------------------------------------------------------------
// Kernel C.  Survivors |u_i| > thr_sel -> ordered pairs; eps slot cleared (CLEAR; the
// operator form leaves the vector as it is).
// ---------------------------------------------------------------------------
template <bool SEG, bool CLEAR = true>
__global__ void __launch_bounds__(kCompactThreads)
k_compact_threshold(float* __restrict__ u, int64_t d, Ctrl* __restrict__ ctrl,
                    unsigned long long* __restrict__ tile_status, int n_tiles,
                    int32_t* __restrict__ idx_out, float* __restrict__ val_out,
                    int64_t* __restrict__ nnz_out, int64_t cap,
                    const int64_t* __restrict__ seg_off, int S, const float* __restrict__ seg_thr,
                    int persistent) {
    __shared__ TileScanSmem scan;
    __shared__ int s_tile;
    __shared__ LookbackSmem lb;
    __shared__ unsigned int s_tailcnt;
    const int tid = threadIdx.x;
    // persistent: launched cooperatively with all CTAs resident, CTA b takes tiles b, b + grid, ...
    // (every earlier tile belongs to a resident CTA, so the look-back always makes progress);
    // otherwise one tile per CTA, handed out by an atomic ticket in the order the CTAs start.
    for (int pass = 0;; ++pass) {
    if (persistent) {
        if ((int64_t)blockIdx.x + (int64_t)pass * gridDim.x >= n_tiles) break;
        if (tid == 0) { s_tile = (int)(blockIdx.x + pass * gridDim.x); s_tailcnt = 0u; }
    } else {
        if (pass > 0) break;
        if (tid == 0) {
            s_tile = (int)atomicAdd(&ctrl->tile_ticket, 1u);
            s_tailcnt = 0u;
        }
    }
    __syncthreads();
    const int tile = s_tile;
    const int64_t n4 = d >> 2;
    const int64_t base4 = (int64_t)tile * (kCompactThreads * kCompactRows);
    const float4* u4 = reinterpret_cast<const float4*>(u);
    // Threshold lookup.  Unsegmented: one threshold.  Segmented: the tile's first and last
    // segment; when they coincide the tile is uniform, otherwise each element searches
    // the boundaries between them.
    int s_lo = 0, s_hi = 0;
    float thr_u;
    if (SEG) {
        const int64_t t_lo = base4 << 2;
        int64_t t_hi = t_lo + kCompactTileElems;
        if (t_hi > d) t_hi = d;
        s_lo = find_segment(seg_off, S, t_lo);
        s_hi = find_segment(seg_off, S, t_hi - 1);
        thr_u = seg_thr[s_lo];
    } else {
        thr_u = ctrl->thr_sel;
    }
    auto thr_of = [&](int64_t e) -> float {
        if (!SEG || s_lo == s_hi) return thr_u;
        int lo = s_lo, hi = s_hi;  // first s in [s_lo, s_hi] with seg_off[s + 1] > e
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (seg_off[mid + 1] > e) hi = mid; else lo = mid + 1;
        }
        return seg_thr[lo];
    };

    float4 v[kCompactRows];
#pragma unroll
    for (int j = 0; j < kCompactRows; ++j) {
        const int64_t i4 = base4 + j * kCompactThreads + tid;
        v[j] = (i4 < n4) ? __ldcs(u4 + i4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    unsigned int mask = 0u, c[kCompactRows], off[kCompactRows];
#pragma unroll
    for (int j = 0; j < kCompactRows; ++j) {
        const int64_t i4 = base4 + j * kCompactThreads + tid;
        unsigned int m = 0u;
        if (i4 < n4) {
            if (!SEG || s_lo == s_hi) {
                m = (unsigned)(fabsf(v[j].x) > thr_u) | ((unsigned)(fabsf(v[j].y) > thr_u) << 1) |
                    ((unsigned)(fabsf(v[j].z) > thr_u) << 2) | ((unsigned)(fabsf(v[j].w) > thr_u) << 3);
            } else {
                const int64_t e0 = i4 << 2;
                m = (unsigned)(fabsf(v[j].x) > thr_of(e0)) | ((unsigned)(fabsf(v[j].y) > thr_of(e0 + 1)) << 1) |
                    ((unsigned)(fabsf(v[j].z) > thr_of(e0 + 2)) << 2) |
                    ((unsigned)(fabsf(v[j].w) > thr_of(e0 + 3)) << 3);
            }
        }
        c[j] = __popc(m);
        mask |= m << (4 * j);
    }
    // the ragged tail (d mod 4 elements) belongs to the last thread of the last tile
    const bool owns_tail = (tile == n_tiles - 1) && (tid == kCompactThreads - 1) && (d & 3);
    float tailv[3] = {0.f, 0.f, 0.f};
    unsigned int tail_mask = 0u;
    if (owns_tail) {
        for (int t = 0; t < (int)(d & 3); ++t) {
            tailv[t] = u[(n4 << 2) + t];
            tail_mask |= (unsigned)(fabsf(tailv[t]) > thr_of((n4 << 2) + t)) << t;
        }
    }
    if (owns_tail) s_tailcnt = __popc(tail_mask);
    const unsigned int total = tile_scan(c, off, scan);  // synchronises the CTA
    const unsigned int tile_total = total + s_tailcnt;

    const unsigned long long prefix =
        lookback_block(tile_status, tile, (unsigned long long)tile_total, &ctrl->stats.status, lb);

    if (mask) {
#pragma unroll
        for (int j = 0; j < kCompactRows; ++j) {
            unsigned int m = (mask >> (4 * j)) & 0xfu;
            if (m) {
                const int64_t e0 = (base4 + j * kCompactThreads + tid) << 2;
                unsigned long long pos = prefix + off[j];
                const float vv[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    if (m & (1u << t)) {
                        if ((int64_t)pos < cap) {
                            idx_out[pos] = (int32_t)(e0 + t);
                            val_out[pos] = vv[t];
                            if (CLEAR) u[e0 + t] = 0.0f;
                        }
                        ++pos;
                    }
                }
            }
        }
    }
    if (owns_tail && tail_mask) {
        unsigned long long pos = prefix + total;
        for (int t = 0; t < (int)(d & 3); ++t) {
            if (tail_mask & (1u << t)) {
                if ((int64_t)pos < cap) {
                    idx_out[pos] = (int32_t)((n4 << 2) + t);
                    val_out[pos] = tailv[t];
                    if (CLEAR) u[(n4 << 2) + t] = 0.0f;
                }
                ++pos;
            }
        }
    }
    if (tile == n_tiles - 1 && tid == 0) {
        const long long all = (long long)(prefix + tile_total);
        const long long written = all < cap ? all : cap;
        *nnz_out = written;
        ctrl->stats.emitted = written;
        if (all > cap) atomicOr(&ctrl->stats.status, GK_DEV_TRUNCATED);
        ctrl->tile_ticket = 0u;
    }
    __syncthreads();  // shared arrays are reused by the next tile
    }
}


}  // namespace gk
