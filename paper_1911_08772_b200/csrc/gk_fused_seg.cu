// gk_sparsify_segmented as ONE persistent cooperative kernel: Algorithm 1 of
// arXiv 1911.08772 run independently on every contiguous segment of the vector
// (layer-wise selection), for tables of up to kSegFusedMax segments.
//
// One CTA per SM owns a contiguous run of rows of 1024 float4 (with its own
// thresholds every segment looks alike to the count phase, so contiguous runs
// stay balanced, and a run meets only a few segments).  The runs are cut to
// equal cost, a segment boundary counting as two rows, so that a stretch of
// many short layers does not leave one CTA behind.  The phases are those of the
// whole-vector kernel:
//
//   phase A  u = g + eps over eps through the ring of asynchronous copies; the
//            per-thread fp64 sums belong to the segment the run is in and are
//            reduced over the CTA whenever the run leaves a segment, into slot
//            (CTA + segment) -- unique, because both only grow along the vector;
//            a row that holds a segment boundary attributes its elements one by
//            one.
//   barrier  every CTA adds, per segment, the slots of the CTAs the segment
//            spans in ascending order, and forms that segment's ten candidates.
//   phase B  candidate counts per segment (integer atomics).
//   barrier  every CTA replays the rounds for every segment: all thresholds are
//            known everywhere.
//   phase C  survivors per (row, warp) with the threshold of each element's
//            segment; the runs' totals exchanged through a third barrier give
//            every run its output offset; pairs written, slots cleared.
//
// Larger tables, vectors of more than kTableMaxRows rows per SM and devices
// without cooperative launch take the three-kernel form in gk_segmented.cu.
#include <math.h>

#include <mutex>

#include "gk_alg1.cuh"
#include "gk_common.cuh"
#include "gk_coop.cuh"
#include "gk_count.cuh"
#include "gk_segmented.cuh"

namespace gk {

constexpr int kSegFusedMax = 256;                      // segments the single-kernel form takes
constexpr int kSfTableMaxRows = 448;                   // most rows a CTA may own
constexpr int kSfTableRowBytes = kFusedWarps * 2;
constexpr int kSfStages = 4;                           // phase A: rows of g and eps in flight, plus one
constexpr int kSfRing = 8;                             // ring slots; phase B has kSfRing - 1 rows in flight
constexpr int kSfGroupRows = 8;
constexpr unsigned short kSfPending = 0xffffu;
// phase C keeps the places of a run's survivors (row, warp, lane, element, rank within the
// 128-element segment: one word each) in the ring's shared memory between counting and write-out
constexpr int kSfStageCap = kSfRing * kFusedThreads * 4;
constexpr int kSfLocal = 8;                           // segments of a run whose partial results wait in shared memory

struct __align__(128) SegFusedShared {
    double2 red[kFusedWarps];
    long long off[kSegFusedMax + 1];                   // segment offsets
    double piv[kSegFusedMax];                          // pivot of each segment's sums: g[off[s]]
    float cs[kSegFusedMax][kNumCand];                  // candidates in ascending order
    unsigned char ord[kSegFusedMax][kNumCand];         // their candidate indices
    float thr[kSegFusedMax];                           // threshold of the mask returned
    unsigned char counted[kSegFusedMax];               // 0: nothing to count (all or nothing selected)
    double2 wpart[kSfLocal][kFusedWarps];              // phase A: per-warp sums of the run's first segments
    unsigned int cnt2[kSfLocal][kNumCand];             // phase B: counts of the run's first segments
    unsigned int wsum[kFusedWarps];
    unsigned int rowpre[kSfTableMaxRows];              // survivors in the vector before each row of this CTA
    unsigned short qrow[kFusedWarps][kSfGroupRows];
    int runrow[kFusedGridCap + 1];                     // first row of every CTA's run; [G] = rows of the vector
    unsigned long long total;                          // survivors in the runs before this one
    unsigned int n_staged;                             // survivors whose places were put aside in phase C
    int ok;
};
constexpr int kSfSmemBudget = (232448 - (int)((sizeof(SegFusedShared) + 1023) / 1024 * 1024));

// First segment s >= from with off[s + 1] > e (the segment that holds element e, skipping
// empty ones); S when there is none.  Sequential: runs meet few segments.
__device__ __forceinline__ int seg_advance(const long long* off, int S, int from, int64_t e) {
    int s = from;
    while (s < S && off[s + 1] <= e) ++s;
    return s;
}
// The same by bisection, for a cold start.
__device__ __forceinline__ int seg_find(const long long* off, int S, int64_t e) {
    int lo = 0, hi = S;  // first s in [0, S] with s == S or off[s + 1] > e
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (off[mid + 1] > e) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// n_rows: rows of 1024 float4 in the vector (at least as many as CTAs); max_rows: the most rows a
// run may have (table entries); u_slots: row slots of shared memory that hold u after phase A
// (the last u_slots rows of the run).
// Shared memory: [ring of kSfRing rows][u_slots rows][table of table_rows x 32 uint16].
__global__ void __launch_bounds__(kFusedThreads, 1)
k_gk_fused_seg(const float* __restrict__ g, float* __restrict__ eps, int64_t d, const int64_t* __restrict__ off_g,
               const int64_t* __restrict__ seg_k, int S, int n_rows, int max_rows, int u_slots, Ctrl* __restrict__ ctrl,
               SegScratch v, unsigned int* __restrict__ bars, unsigned int* __restrict__ cta_tot,
               int32_t* __restrict__ idx_out, float* __restrict__ val_out, int64_t* __restrict__ seg_nnz_out,
               int64_t* __restrict__ nnz_out, int64_t cap, unsigned long long* __restrict__ trace) {
    extern __shared__ __align__(1024) float4 smem4[];
    __shared__ SegFusedShared sh;
    float4* gring = smem4;
    float4* uslot = smem4 + (size_t)kSfRing * kRowF4;
    unsigned short* table = reinterpret_cast<unsigned short*>(smem4 + (size_t)(kSfRing + u_slots) * kRowF4);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int c = blockIdx.x, G = gridDim.x;
    const int64_t n4 = d >> 2;

    const bool owns_tail = (c == G - 1) && (w == kFusedWarps - 1) && (lane < (int)(d & 3));
    const int64_t tail_i = (n4 << 2) + lane;
    const float4* g4 = reinterpret_cast<const float4*>(g);
    float4* e4 = reinterpret_cast<float4*>(eps);
    float tail_u = 0.f;
    const bool wide_ok = ((reinterpret_cast<uintptr_t>(eps) & 31u) == 0);

    if (c == 0 && tid == 0) {
        ctrl->stats.status = GK_DEV_OK;
        ctrl->phase_t[0] = global_timer_ns();
    }
    // optional per-CTA trace: start, table read, end of phase A, after barrier 1, thresholds
    // formed, end of phase B, after barrier 2, end
    auto stamp = [&](int slot) {
        if (trace != nullptr && tid == 0) trace[(size_t)c * 8 + slot] = global_timer_ns();
    };
    stamp(0);

    // ------------------------------------------------------------ the table
    // Offsets and pivots go to shared memory; every CTA checks the table for itself.
    int bad = 0;
    long long kq = 1;
    if (tid <= S) sh.off[tid] = off_g[tid];  // S <= kSegFusedMax < the number of threads
    if (tid < S) kq = seg_k[tid];
    __syncthreads();
    if (tid == 0 && (sh.off[0] != 0 || sh.off[S] != d)) bad = 1;
    if (tid < S) {
        const long long a = sh.off[tid], b = sh.off[tid + 1];
        if (a < 0 || b > d || b < a || kq < 1) bad = 1;
    }
    bad = __syncthreads_or(bad);
    if (tid < S) {
        const long long a = sh.off[tid];
        sh.piv[tid] = (!bad && a < d) ? (double)g[a] : 0.0;
    }
    // candidate counts start at zero
    if (c == 0) for (int j = tid; j < S * kNumCand; j += kFusedThreads) v.counts[j] = 0ull;
    __syncthreads();
    const int S_use = bad ? 0 : S;  // a malformed table: u is still formed, nothing is selected

    // ------------------------------------------------------------ the runs
    // Every CTA owns a contiguous run of rows.  A segment boundary costs a run about as much as
    // two rows (its sums and counts are closed warp by warp, the next segment's scalars
    // fetched), and layer tables have stretches of many short segments: runs of equal length
    // left the CTA with the most boundaries 5 us behind in phase A and 14 us in phase B, with
    // everyone else waiting at the barriers.  So the runs are cut to equal COST,
    // cost(row) = row + 2 (boundaries before the row): thread t finds the first row of run t by
    // bisection; every CTA computes the same cuts.
    {
        // With j boundaries before it a row costs row + 2 j, and that holds for the rows from
        // range_lo(j) to the row that holds boundary j + 1: one bisection over the boundaries finds
        // the range of a target cost, the row follows by division.
        const int nbnd = S_use > 0 ? S_use - 1 : 0;                  // boundaries off[1 .. S_use - 1]
        auto range_lo = [&](const int j) -> long long { return j == 0 ? 0 : sh.off[j] / (4 * kRowF4) + 1; };
        if (tid <= G) {
            int cut = tid == G ? n_rows : 0;
            if (tid > 0 && tid < G) {
                const long long target = (long long)tid * (1ll * n_rows + 2ll * nbnd) / G;
                int lo = 0, hi = nbnd;   // last j with 2 range_lo(j) + 3 j <= target
                while (lo < hi) {
                    const int mid = (lo + hi + 1) >> 1;
                    if (range_lo(mid) + 2ll * mid <= target) lo = mid; else hi = mid - 1;
                }
                long long row = target - 2ll * lo;
                if (row < range_lo(lo)) row = range_lo(lo);
                if (lo < nbnd && row > sh.off[lo + 1] / (4 * kRowF4)) row = sh.off[lo + 1] / (4 * kRowF4) + 1;
                cut = row < n_rows ? (int)row : n_rows;
            }
            sh.runrow[tid] = cut;
        }
        __syncthreads();
        // every run needs a row at least (a single row can hold dozens of boundaries) and none may
        // have more than the table has entries for.  The cuts usually are like that as they stand;
        // otherwise one thread moves them apart, and failing that the runs get equal lengths.
        int good = 1;
        if (tid < G) {
            const int len = sh.runrow[tid + 1] - sh.runrow[tid];
            good = (len >= 1 && len <= max_rows) ? 1 : 0;
        }
        good = __syncthreads_and(good);
        if (!good && tid == 0) {
            for (int t = 1; t < G; ++t) if (sh.runrow[t] <= sh.runrow[t - 1]) sh.runrow[t] = sh.runrow[t - 1] + 1;
            for (int t = G - 1; t >= 1; --t) if (sh.runrow[t] >= sh.runrow[t + 1]) sh.runrow[t] = sh.runrow[t + 1] - 1;
            bool fits = true;
            for (int t = 0; t < G; ++t) {
                const int len = sh.runrow[t + 1] - sh.runrow[t];
                fits = fits && len >= 1 && len <= max_rows;
            }
            if (!fits) for (int t = 0; t <= G; ++t) sh.runrow[t] = (int)((long long)t * n_rows / G);
        }
        __syncthreads();
    }
    // this CTA's run of float4 and of elements
    int64_t lo4 = (int64_t)sh.runrow[c] * kRowF4, hi4 = (int64_t)sh.runrow[c + 1] * kRowF4;
    if (lo4 > n4) lo4 = n4;
    if (hi4 > n4) hi4 = n4;
    const int nrows = (int)((hi4 - lo4 + kRowF4 - 1) / kRowF4);
    const int first_kept = nrows > u_slots ? nrows - u_slots : 0;  // rows from here on stay on chip
    const int64_t run_lo = lo4 << 2;
    const int64_t run_hi = (c == G - 1) ? d : (hi4 << 2);           // the last CTA also owns the d mod 4 tail
    stamp(1);

    // rows are fetched kSfStages - 1 ahead by asynchronous copies: g into a ring, eps into the slot
    // that will hold u
    auto fetch = [&](int r) {
        const int64_t i = lo4 + (int64_t)r * kRowF4 + tid;
        if (r < nrows && i < hi4) {
            cp_async16(gring + (size_t)(r % kSfStages) * kRowF4 + tid, g4 + i);
            cp_async16(uslot + (size_t)(r % u_slots) * kRowF4 + tid, e4 + i);
        }
        cp_async_commit();
    };
#pragma unroll
    for (int r = 0; r < kSfStages - 1; ++r) fetch(r);


    // ------------------------------------------------------------------ phase A
    {
        double s0 = 0.0, q0 = 0.0, s1 = 0.0, q1 = 0.0;
        bool dirty = false;                          // this thread has added something for segment s
        int s = seg_find(sh.off, S_use, run_lo);     // the segment the run is in (S_use: none)
        long long send = s < S_use ? sh.off[s + 1] : (long long)d + 1;
        double pv = s < S_use ? sh.piv[s] : 0.0;
        const int s_first = s;
        // Closes segment s for this thread's warp, then moves on to the segment of `e`.  The sums
        // of the run's first kSfLocal segments wait per warp in shared memory and are added up
        // after the last row, so that the warps need not meet at every boundary (all warps see
        // the same boundaries, each in its own time); later segments are reduced on the spot.
        auto leave_segment = [&](int64_t e) {
            const int li = s - s_first;
            if (li < kSfLocal) {
                // a short segment lies in a few warps only: the others have nothing to add up
                double a = 0.0, b = 0.0;
                if (__any_sync(0xffffffffu, dirty)) { a = warp_sum(s0 + s1); b = warp_sum(q0 + q1); }
                if (lane == 0) sh.wpart[li][w] = make_double2(a, b);
            } else {
                const double2 part = block_sum2<kFusedThreads>(s0 + s1, q0 + q1, sh.red);
                if (tid == 0) v.partials[c + s] = part;
            }
            s0 = q0 = s1 = q1 = 0.0;
            dirty = false;
            s = seg_advance(sh.off, S_use, s + 1, e);
            send = s < S_use ? sh.off[s + 1] : (long long)d + 1;
            pv = s < S_use ? sh.piv[s] : 0.0;
        };
        // one row: u formed, stored, its maxima recorded; the caller does the statistics
        auto row_u = [&](int r, float4& u0, bool& one) {
            fetch(r + kSfStages - 1);
            cp_async_wait<kSfStages - 1>();
            const int64_t i = lo4 + (int64_t)r * kRowF4 + tid;
            one = i < hi4;
            u0 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (one) {
                float4* us = uslot + (size_t)(r % u_slots) * kRowF4 + tid;
                const float4 a0 = gring[(size_t)(r % kSfStages) * kRowF4 + tid], b0 = *us;
                u0 = make_float4(a0.x + b0.x, a0.y + b0.y, a0.z + b0.z, a0.w + b0.w);
                *us = u0;
            }
            float4 nb;
            nb.x = __shfl_down_sync(0xffffffffu, u0.x, 1); nb.y = __shfl_down_sync(0xffffffffu, u0.y, 1);
            nb.z = __shfl_down_sync(0xffffffffu, u0.z, 1); nb.w = __shfl_down_sync(0xffffffffu, u0.w, 1);
            const bool pair = wide_ok && (i + 1 < hi4);
            if ((lane & 1) == 0) {
                if (pair) st_keep32(e4 + i, u0, nb);
                else if (one) e4[i] = u0;
            } else if (one && !wide_ok) {
                e4[i] = u0;
            }
            const unsigned int m0 = __reduce_max_sync(0xffffffffu, one ? max_mag_bits(u0) : 0u);
            if (lane == 0) table[r * kFusedWarps + w] = (unsigned short)((m0 + 0xffffu) >> 16);
        };
        const int64_t rows_hi = hi4 << 2;  // end of the run's rows
        int r = 0;
        while (r < nrows) {
            // rows [r, pure_end) lie wholly inside segment s (or beyond the table)
            int pure_end = nrows;
            if (send < rows_hi) {
                const int64_t m = (send - run_lo) / (4 * kRowF4);
                pure_end = m < nrows ? (int)m : nrows;
            }
            const bool in_seg = s < S_use;
            for (; r < pure_end; ++r) {
                float4 u0;
                bool one;
                row_u(r, u0, one);
                if (one && in_seg) {
                    const double x0 = (double)u0.x - pv, x1 = (double)u0.y - pv, x2 = (double)u0.z - pv,
                                 x3 = (double)u0.w - pv;
                    s0 += x0; q0 = fma(x0, x0, q0); s1 += x1; q1 = fma(x1, x1, q1);
                    s0 += x2; q0 = fma(x2, x2, q0); s1 += x3; q1 = fma(x3, x3, q1);
                    dirty = true;
                }
            }
            if (r >= nrows) break;
            const int64_t re0 = run_lo + (int64_t)r * (4 * kRowF4);
            if (send <= re0) {  // the segment ended exactly where this row begins
                leave_segment(re0);
                continue;
            }
            // a boundary inside row r: element by element, segment by segment
            {
                float4 u0;
                bool one;
                row_u(r, u0, one);
                int64_t re1 = re0 + 4 * kRowF4;
                if (re1 > rows_hi) re1 = rows_hi;
                const int64_t e0 = (lo4 + (int64_t)r * kRowF4 + tid) << 2;
                const float uu[4] = {u0.x, u0.y, u0.z, u0.w};
                const int64_t we0 = re0 + 128 * w;  // this warp's 128 elements of the row
                int64_t cur = re0;
                while (cur < re1 && s < S_use) {
                    const int64_t seg_hi = send < re1 ? send : re1;
                    if (one && we0 < seg_hi && we0 + 128 > cur) {
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            const int64_t e = e0 + t;
                            if (e >= cur && e < seg_hi) {
                                const double x = (double)uu[t] - pv;
                                s0 += x; q0 = fma(x, x, q0);
                                dirty = true;
                            }
                        }
                    }
                    cur = seg_hi;
                    if (send <= re1) leave_segment(cur); else break;
                }
                ++r;
            }
        }
        // a segment that ends exactly where the run's rows end
        if (s < S_use && send == rows_hi) leave_segment(rows_hi);
        cp_async_wait<0>();
        if (c == G - 1 && (d & 3)) {
            // the d mod 4 trailing elements, held by the last lanes of the last warp
            if (owns_tail) {
                tail_u = g[tail_i] + eps[tail_i];
                eps[tail_i] = tail_u;
            }
            int64_t cur = n4 << 2;
            while (cur < d && s < S_use) {
                const int64_t seg_hi = send < d ? send : d;
                if (owns_tail && tail_i >= cur && tail_i < seg_hi) {
                    const double x = (double)tail_u - pv;
                    s0 += x; q0 = fma(x, x, q0);
                    dirty = true;
                }
                cur = seg_hi;
                if (send <= d) leave_segment(cur); else break;
            }
        }
        // the segment the run ends in has not been closed yet
        if (s < S_use && sh.off[s] < run_hi) leave_segment(run_hi);
        __syncthreads();
        // the waiting sums: thread t adds the 32 warps of the run's t-th segment in warp order, as
        // block_sum2 would, into slot (c + segment); segments the run does not touch have no slot
        if (tid < kSfLocal && s_first + tid < S_use) {
            const int q = s_first + tid;
            if (sh.off[q + 1] > sh.off[q] && sh.off[q] < run_hi && sh.off[q + 1] > run_lo) {
                double a = 0.0, b = 0.0;
#pragma unroll
                for (int i = 0; i < kFusedWarps; ++i) { a += sh.wpart[tid][i].x; b += sh.wpart[tid][i].y; }
                v.partials[c + q] = make_double2(a, b);
            }
        }
        // The normal quantiles depend only on (k_s, d_s).  Whoever has finished its rows takes
        // segments from a shared ticket until none is left: the CTAs that are early at the barrier
        // anyway do most of them.
        if (tid == 0 && !bad) {
            while (true) {
                const unsigned int q = atomicAdd(&bars[4], 1u);
                if (q >= (unsigned)S) break;
                const long long n = sh.off[q + 1] - sh.off[q];
                long long kk = seg_k[q];
                if (kk > n) kk = n;
                double zq = -INFINITY;
                if (n > 0 && kk >= 1 && kk < n) {
                    const double pq = 1.0 - (double)kk / (double)n;  // Algorithm 1: p = 1 - k/d
                    zq = normal_quantile_upper(1.0 - pq);
                }
                v.zs[q] = zq;
            }
        }
        stamp(2);
        if (!grid_barrier(&bars[0], (unsigned)G, &sh.ok)) {
            if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
            goto leave;
        }
        stamp(3);
    }

    // --------------------------------------------------- thresholds of every segment
    // Thread q takes segment q: adds the slots of the CTAs the segment spans in ascending order
    // (the same order in every CTA), forms the candidates, and leaves them sorted in shared
    // memory.  CTA 0 also writes the records that the host can read back.
    for (int q = tid; q < S; q += kFusedThreads) {
        const long long a = sh.off[q], b = sh.off[q + 1], n = b - a;
        gk_stats rec;
        double c64[kNumCand];
        float c32[kNumCand];
        unsigned long long dummy[kNumCand];
        float tsel;
#pragma unroll
        for (int i = 0; i < kNumCand; ++i) { c32[i] = INFINITY; c64[i] = INFINITY; }
        const Alg1State st{&rec, c64, c32, dummy, &tsel};
        bool counted = false;
        if (bad || n <= 0) {
            rec.mu = rec.sigma = rec.z = rec.thres0 = rec.thr_final = 0.0;
            for (int i = 0; i < kMaxRounds; ++i) rec.counts[i] = 0;
            rec.rounds = 0; rec.status = bad ? GK_DEV_BAD_SEGMENTS : GK_DEV_OK; rec.nnz = 0; rec.emitted = 0;
            tsel = INFINITY;  // nothing passes
            for (int i = 0; i < kNumCand; ++i) { c32[i] = INFINITY; c64[i] = INFINITY; }
        } else {
            // the CTAs whose runs hold the segment's first and last element
            auto cta_of = [&](const long long e) -> int {
                const long long row = (e >> 2) / kRowF4;
                int lo = 0, hi = G - 1;   // last t in [0, G - 1] with runrow[t] <= row
                while (lo < hi) {
                    const int mid = (lo + hi + 1) >> 1;
                    if (sh.runrow[mid] <= row) lo = mid; else hi = mid - 1;
                }
                return lo;
            };
            const int c0 = cta_of(a), c1 = cta_of(b - 1);
            double s1 = 0.0, s2 = 0.0;
            for (int cc = c0; cc <= c1; cc += 8) {
                double2 p[8];
#pragma unroll
                for (int t = 0; t < 8; ++t)
                    p[t] = (cc + t <= c1) ? __ldcg(&v.partials[cc + t + q]) : make_double2(0.0, 0.0);
#pragma unroll
                for (int t = 0; t < 8; ++t) { s1 += p[t].x; s2 += p[t].y; }
            }
            long long kk = seg_k[q];
            if (kk > n) kk = n;
            alg1_thresholds(st, s1, s2, sh.piv[q], n, kk, __ldcg(&v.zs[q]));
            counted = !(rec.rounds == 0 && rec.thr_final == -INFINITY);  // not "everything selected"
        }
        sh.counted[q] = counted ? 1 : 0;
        sh.thr[q] = tsel;
        // the ten thresholds in ascending order (all equal when nothing is counted)
        const bool neg = counted && rec.thres0 < 0.0;
#pragma unroll
        for (int j = 0; j < kNumCand; ++j) {
            const int oj = cand_ascending(j, neg);
            sh.cs[q][j] = c32[oj];
            sh.ord[q][j] = (unsigned char)oj;
        }
        if (c == 0) {
            v.stats[q] = rec;
            v.thr_sel[q] = tsel;
            for (int j = 0; j < kNumCand; ++j) {
                v.cand64[(size_t)q * kNumCand + j] = c64[j];
                v.cand32[(size_t)q * kNumCand + j] = c32[j];
            }
        }
    }
    for (int j = tid; j < kSfLocal * kNumCand; j += kFusedThreads) (&sh.cnt2[0][0])[j] = 0u;
    if (c == 0 && tid == 0) ctrl->phase_t[1] = global_timer_ns();
    __syncthreads();
    stamp(4);

    // ------------------------------------------------------------------ phase B
    {
        float cs[kNumCand], acc[kNumCand];
        Tiers tier;
        bool any_neg = false, counted = false, dirty = false;
        int s = seg_find(sh.off, S_use, run_lo);
        long long send = s < S_use ? sh.off[s + 1] : (long long)d + 1;
        auto enter_segment = [&]() {
            counted = s < S_use && sh.counted[s] != 0;
#pragma unroll
            for (int j = 0; j < kNumCand; ++j) { cs[j] = counted ? sh.cs[s][j] : INFINITY; acc[j] = 0.f; }
            tier = make_tiers(cs);
            any_neg = cs[0] < 0.f;
        };
        const int s_first = s;
        // Closes segment s for this thread's warp (integer counts: any order).  The counts of the
        // run's first kSfLocal segments are collected in shared memory and go out after the last
        // row; later segments go to the global counters directly.  No warp waits for another.
        auto leave_segment = [&](int64_t e) {
            // a short segment lies in a few warps only: the others have counted nothing
            if (counted && __any_sync(0xffffffffu, dirty)) {
                const int li = s - s_first;
#pragma unroll
                for (int j = 0; j < kNumCand; ++j) {
                    const unsigned int ws = __reduce_add_sync(0xffffffffu, (unsigned int)acc[j]);
                    if (lane == 0 && ws) {
                        const int oj = sh.ord[s][j];
                        if (li < kSfLocal) atomicAdd(&sh.cnt2[li][oj], ws);
                        else atomicAdd(&v.counts[(size_t)s * kNumCand + oj], (unsigned long long)ws);
                    }
                }
            }
            dirty = false;
            s = seg_advance(sh.off, S_use, s + 1, e);
            send = s < S_use ? sh.off[s + 1] : (long long)d + 1;
            enter_segment();
        };
        enter_segment();
        const float4* src = e4 + lo4 + tid;
        const unsigned short* trow = table + w;
        auto fetch_u = [&](int r) {
            if (r < first_kept) cp_async16(gring + ((r & (kSfRing - 1)) << 10) + tid, src + ((size_t)r << 10));
            cp_async_commit();
        };
#pragma unroll
        for (int r = 0; r < kSfRing - 1; ++r) fetch_u(r);
        static_assert(kRowF4 == 1024 && (kSfRing & (kSfRing - 1)) == 0, "ring indexing assumes 1024-float4 rows");
        // this thread's float4 of row r: through the ring when the row is not on chip (those are
        // all full rows), else from its slot
        auto row_x = [&](int r, float4& x, bool& one) {
            one = lo4 + (int64_t)r * kRowF4 + tid < hi4;
            x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < first_kept) {
                fetch_u(r + kSfRing - 1);
                cp_async_wait<kSfRing - 1>();
                x = gring[((r & (kSfRing - 1)) << 10) + tid];
            } else {
                if (r == first_kept) cp_async_wait<0>();
                if (one) x = uslot[(size_t)(r % u_slots) * kRowF4 + tid];
            }
        };
        const int64_t rows_hi = hi4 << 2;
        int r = 0;
        while (r < nrows) {
            int pure_end = nrows;
            if (send < rows_hi) {
                const int64_t m = (send - run_lo) / (4 * kRowF4);
                pure_end = m < nrows ? (int)m : nrows;
            }
            if (counted) {
#pragma unroll 2
                for (; r < pure_end; ++r) {
                    float4 x;
                    bool one;
                    row_x(r, x, one);
                    if (one) count_float4(x, any_neg ? 0x10000u : (unsigned int)trow[r * kFusedWarps], cs, tier, acc);
                }
                dirty = true;  // (rows were counted, or the loop did not run and it does not matter)
            } else {
                // nothing to count here, but the ring keeps turning
                for (; r < pure_end; ++r) {
                    float4 x;
                    bool one;
                    row_x(r, x, one);
                }
            }
            if (r >= nrows) break;
            const int64_t re0 = run_lo + (int64_t)r * (4 * kRowF4);
            if (send <= re0) {
                leave_segment(re0);
                continue;
            }
            {
                float4 x;
                bool one;
                row_x(r, x, one);
                int64_t re1 = re0 + 4 * kRowF4;
                if (re1 > rows_hi) re1 = rows_hi;
                const int64_t e0 = (lo4 + (int64_t)r * kRowF4 + tid) << 2;
                const float xx[4] = {fabsf(x.x), fabsf(x.y), fabsf(x.z), fabsf(x.w)};
                const int64_t we0 = re0 + 128 * w;  // this warp's 128 elements of the row
                int64_t cur = re0;
                while (cur < re1 && s < S_use) {
                    const int64_t seg_hi = send < re1 ? send : re1;
                    if (one && counted && we0 < seg_hi && we0 + 128 > cur) {
                        dirty = true;
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            const int64_t e = e0 + t;
                            if (e >= cur && e < seg_hi) {
#pragma unroll
                                for (int j = 0; j < kNumCand; ++j) acc[j] += gt_as_float(xx[t], cs[j]);
                            }
                        }
                    }
                    cur = seg_hi;
                    if (send <= re1) leave_segment(cur); else break;
                }
                ++r;
            }
        }
        if (s < S_use && send == rows_hi) leave_segment(rows_hi);
        cp_async_wait<0>();
        if (c == G - 1 && (d & 3)) {
            int64_t cur = n4 << 2;
            const float a = fabsf(tail_u);
            while (cur < d && s < S_use) {
                const int64_t seg_hi = send < d ? send : d;
                if (owns_tail && counted && tail_i >= cur && tail_i < seg_hi) {
#pragma unroll
                    for (int j = 0; j < kNumCand; ++j) acc[j] += gt_as_float(a, cs[j]);
                    dirty = true;
                }
                cur = seg_hi;
                if (send <= d) leave_segment(cur); else break;
            }
        }
        if (s < S_use && sh.off[s] < run_hi) leave_segment(run_hi);
        __syncthreads();
        for (int j = tid; j < kSfLocal * kNumCand; j += kFusedThreads) {
            const unsigned int x = sh.cnt2[j / kNumCand][j % kNumCand];
            const int q = s_first + j / kNumCand;
            if (x && q < S_use) atomicAdd(&v.counts[(size_t)q * kNumCand + j % kNumCand], (unsigned long long)x);
        }
        if (c == 0 && tid == 0) ctrl->phase_t[2] = global_timer_ns();
        stamp(5);
        if (!grid_barrier(&bars[1], (unsigned)G, &sh.ok)) {
            if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
            goto leave;
        }
        if (c == 0 && tid == 0) ctrl->phase_t[3] = global_timer_ns();
        stamp(6);
    }

    // ------------------------------------------------------------------ resolve
    // Thread q replays the rounds of segment q on its final counts: its threshold is then known
    // in this CTA.  CTA 0 also completes the records and adds up the survivors.
    {
        unsigned long long my_nnz = 0ull;
        for (int q = tid; q < S; q += kFusedThreads) {
            const long long n = sh.off[q + 1] - sh.off[q];
            long long kk = bad ? 1 : seg_k[q];
            if (kk > n) kk = n;
            unsigned long long nz = 0ull;
            if (!bad && n > 0) {
                if (sh.counted[q]) {
                    // the ten counts come in together; the rounds are then replayed on the copy
                    unsigned long long cnt[kNumCand];
#pragma unroll
                    for (int j = 0; j < kNumCand; ++j) cnt[j] = __ldcg(&v.counts[(size_t)q * kNumCand + j]);
                    const Alg1Path p = alg1_replay(cnt, kk);
                    float t = INFINITY;
                    for (int j = 0; j < kNumCand; ++j) if (sh.ord[q][j] == p.chosen) t = sh.cs[q][j];
                    sh.thr[q] = t;
                    nz = (unsigned long long)alg1_last_est(p);
                } else {
                    nz = (unsigned long long)n;  // everything selected
                }
            }
            if (c == 0 && seg_nnz_out) seg_nnz_out[q] = (int64_t)nz;
            my_nnz += nz;
        }
        if (c == 0) {
            // total over the segments (integers: any order)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) my_nnz += __shfl_xor_sync(0xffffffffu, my_nnz, o);
            if (tid == 0) sh.total = 0ull;
            __syncthreads();
            if (lane == 0 && my_nnz) atomicAdd(&sh.total, my_nnz);
            __syncthreads();
            if (tid == 0) {
                const long long all = (long long)sh.total;
                const long long written = all < cap ? all : cap;
                gk_stats* o = &ctrl->stats;
                o->nnz = all; o->emitted = written;
                int flags = bad ? GK_DEV_BAD_SEGMENTS : 0;
                if (all > cap) flags |= GK_DEV_TRUNCATED;
                if (flags) atomicOr(&o->status, flags);
                *nnz_out = written;
                ctrl->phase_t[4] = global_timer_ns();
            }
        }
        __syncthreads();
    }

    // ------------------------------------------------------------------ phase C
    if (tid == 0) sh.n_staged = 0u;
    __syncthreads();
    {
        // threshold of element e, given a segment sx at or before its own (empty segments skipped)
        auto thr_at = [&](int& sx, int64_t e) -> float {
            while (sx < S_use && sh.off[sx + 1] <= e) ++sx;
            return sx < S_use ? sh.thr[sx] : INFINITY;
        };
        // survivors of the float4 at element index e0, starting the segment walk at sx
        auto mask_of = [&](const float4 x, int64_t e0, int sx) -> unsigned int {
            while (sx < S_use && sh.off[sx + 1] <= e0) ++sx;
            if (sx < S_use && sh.off[sx + 1] >= e0 + 4) {  // the four elements share a segment
                const float t = sh.thr[sx];
                return (unsigned)(fabsf(x.x) > t) | ((unsigned)(fabsf(x.y) > t) << 1) |
                       ((unsigned)(fabsf(x.z) > t) << 2) | ((unsigned)(fabsf(x.w) > t) << 3);
            }
            unsigned int m = 0u;
            m |= (unsigned)(fabsf(x.x) > thr_at(sx, e0));
            m |= (unsigned)(fabsf(x.y) > thr_at(sx, e0 + 1)) << 1;
            m |= (unsigned)(fabsf(x.z) > thr_at(sx, e0 + 2)) << 2;
            m |= (unsigned)(fabsf(x.w) > thr_at(sx, e0 + 3)) << 3;
            return m;
        };
        auto gather = [&](int& cursor, const bool want_pending) -> int {
            return want_pending ? gather_cells<kGatherPending>(table, nrows, cursor, sh.qrow[w])
                                : gather_cells<kGatherNonZero>(table, nrows, cursor, sh.qrow[w]);
        };
        auto load_row = [&](int r, int64_t i) -> float4 {
            return (r >= first_kept) ? uslot[(size_t)(r % u_slots) * kRowF4 + tid] : __ldcg(e4 + i);
        };
        // step 0: which (row, warp) segments of 128 elements can hold a survivor: all of one
        // layer-segment, the recorded maximum decides; with a boundary inside, always read
        const int s_run = seg_find(sh.off, S_use, run_lo);  // the segment the run starts in
        int su0 = s_run;                                     // this lane's walk through the segments
        for (int r = lane; r < nrows; r += 32) {
            const int64_t ue0 = ((lo4 + (int64_t)r * kRowF4) << 2) + 128 * w;
            int64_t ue1 = ue0 + 128;
            if (ue1 > (hi4 << 2)) ue1 = hi4 << 2;
            bool ql = false;
            if (ue0 < ue1) {
                const int su = su0 = seg_advance(sh.off, S_use, su0, ue0);
                if (su < S_use) {
                    if (sh.off[su + 1] >= ue1) {
                        const float t = sh.thr[su];
                        ql = t < 0.f || (unsigned int)table[r * kFusedWarps + w] > (__float_as_uint(fmaxf(t, 0.f)) >> 16);
                    } else {
                        ql = true;
                    }
                }
            }
            table[r * kFusedWarps + w] = ql ? kSfPending : (unsigned short)0;
        }
        __syncwarp();
        // step 1: survivors of every qualifying segment into the table (rows come in ascending
        // order, so the warp's position among the segments only moves forward)
        int su1 = s_run;
        unsigned int* st_tag = reinterpret_cast<unsigned int*>(gring);
        for (int cursor = 0; cursor < nrows;) {
            const int n = gather(cursor, true);
            float4 x[kSfGroupRows];
#pragma unroll
            for (int q = 0; q < kSfGroupRows; ++q) {
                x[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (q < n) {
                    const int r = sh.qrow[w][q];
                    const int64_t i = lo4 + (int64_t)r * kRowF4 + tid;
                    if (i < hi4) x[q] = load_row(r, i);
                }
            }
#pragma unroll
            for (int q = 0; q < kSfGroupRows; ++q) {
                if (q < n) {
                    const int r = sh.qrow[w][q];
                    const int64_t i = lo4 + (int64_t)r * kRowF4 + tid;
                    // every lane starts its walk at the segment of the warp's first element
                    const int su = su1 = seg_advance(sh.off, S_use, su1, ((lo4 + (int64_t)r * kRowF4) << 2) + 128 * w);
                    const unsigned int m = i < hi4 ? mask_of(x[q], i << 2, su) : 0u;
                    const unsigned int cnt = __reduce_add_sync(0xffffffffu, __popc(m));
                    if (lane == 0) table[r * kFusedWarps + w] = (unsigned short)cnt;
                    if (cnt != 0u) {
                        // the survivors' places are put aside for the write-out (as long as they fit)
                        unsigned int base = 0u;
                        if (lane == 0) base = atomicAdd(&sh.n_staged, cnt);
                        base = __shfl_sync(0xffffffffu, base, 0);
                        unsigned int rank = 0u;
                        if (cnt > 1u) {
                            const unsigned int b0 = __ballot_sync(0xffffffffu, m & 1u), b1 = __ballot_sync(0xffffffffu, m & 2u),
                                               b2 = __ballot_sync(0xffffffffu, m & 4u), b3 = __ballot_sync(0xffffffffu, m & 8u);
                            const unsigned int below = (1u << lane) - 1u;
                            rank = __popc(b0 & below) + __popc(b1 & below) + __popc(b2 & below) + __popc(b3 & below);
                        }
                        if (m && base + cnt <= (unsigned)kSfStageCap) {
                            const unsigned int place = ((unsigned int)r << 19) | ((unsigned int)w << 14) | ((unsigned int)lane << 9);
#pragma unroll
                            for (int t = 0; t < 4; ++t) {
                                if (m & (1u << t)) {
                                    st_tag[base + rank] = place | ((unsigned int)t << 7) | rank;
                                    ++rank;
                                }
                            }
                        }
                    }
                }
            }
            __syncwarp();
        }
        __syncthreads();
        // all places kept: the write-out is one thread per survivor; else one warp per segment
        const bool staged = sh.n_staged <= (unsigned)kSfStageCap;
        // step 2: survivors per row (thread t takes row t), a scan over this run's rows, and the
        // run's total to this CTA's word in global memory
        unsigned int mine_row = 0u;
        if (tid < nrows) {
            uint4* tv = reinterpret_cast<uint4*>(table + (size_t)tid * kFusedWarps);
#pragma unroll
            for (int q = 0; q < kSfTableRowBytes / 16; ++q) {
                const uint4 y = tv[q];
                if (staged) {
                    // the entries become the survivors of the row in the warps before each one
                    // (at most 3968), which is what the write-out needs
                    unsigned int ws[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const unsigned int lo = ws[j] & 0xffffu, hi = ws[j] >> 16;
                        ws[j] = mine_row | ((mine_row + lo) << 16);
                        mine_row += lo + hi;
                    }
                    tv[q] = make_uint4(ws[0], ws[1], ws[2], ws[3]);
                } else {
                    mine_row += (y.x & 0xffffu) + (y.x >> 16) + (y.y & 0xffffu) + (y.y >> 16) +
                                (y.z & 0xffffu) + (y.z >> 16) + (y.w & 0xffffu) + (y.w >> 16);
                }
            }
        }
        unsigned int run_total;
        {
            unsigned int sc = mine_row;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int t = __shfl_up_sync(0xffffffffu, sc, o);
                if (lane >= o) sc += t;
            }
            if (lane == 31) sh.wsum[w] = sc;
            __syncthreads();
            const unsigned int y0 = sh.wsum[lane];
            unsigned int y = y0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int t = __shfl_up_sync(0xffffffffu, y, o);
                if (lane >= o) y += t;
            }
            const unsigned int wpre = __shfl_sync(0xffffffffu, y - y0, w);
            run_total = __shfl_sync(0xffffffffu, y, 31);
            if (tid < nrows) sh.rowpre[tid] = wpre + sc - mine_row;
            if (tid == 0) { cta_tot[c] = run_total; sh.total = 0ull; }
        }
        if (!grid_barrier(&bars[3], (unsigned)G, &sh.ok)) {
            if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
            goto leave;
        }
        // survivors in the runs before this one (integers: any order): thread t reads CTA t's word
        {
            unsigned long long before = 0ull;
            for (int t = tid; t < c; t += kFusedThreads) before += __ldcg(cta_tot + t);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
            if (lane == 0 && before) atomicAdd(&sh.total, before);
            __syncthreads();
            const unsigned long long base = sh.total;
            if (staged) {
                // step 3: one thread per survivor put aside: its place gives its index, where its
                // value is, and its position in the output
                const unsigned int n_st = sh.n_staged;
                for (unsigned int j = tid; j < n_st; j += kFusedThreads) {
                    const unsigned int tag = st_tag[j];
                    const unsigned int r = tag >> 19, cell = (tag >> 14) & 31u, ln = (tag >> 9) & 31u, t = (tag >> 7) & 3u,
                                       rank = tag & 127u;
                    const long long p = (long long)base + sh.rowpre[r] + table[r * kFusedWarps + cell] + rank;
                    if (p < cap) {
                        const unsigned int in_row = ((cell << 5) | ln) << 2 | t;   // element within the row
                        const int64_t at = run_lo + ((int64_t)r << 12) + in_row;
                        const float xv = ((int)r >= first_kept)
                                             ? reinterpret_cast<const float*>(uslot + (size_t)(r % u_slots) * kRowF4)[in_row]
                                             : __ldcg(eps + at);
                        idx_out[p] = (int32_t)at;
                        val_out[p] = xv;
                        eps[at] = 0.0f;
                    }
                }
            }
            // step 3 without the places: every warp writes the survivors of its segments that have any
            int su3 = s_run;
            for (int cursor = staged ? nrows : 0; cursor < nrows;) {
                const int n = gather(cursor, false);
                float4 x[kSfGroupRows];
#pragma unroll
                for (int q = 0; q < kSfGroupRows; ++q) {
                    x[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (q < n) {
                        const int r = sh.qrow[w][q];
                        const int64_t i = lo4 + (int64_t)r * kRowF4 + tid;
                        if (i < hi4) x[q] = load_row(r, i);
                    }
                }
#pragma unroll
                for (int q = 0; q < kSfGroupRows; ++q) {
                    if (q >= n) continue;
                    const int r = sh.qrow[w][q];
                    const int64_t i = lo4 + (int64_t)r * kRowF4 + tid;
                    const int su = su3 = seg_advance(sh.off, S_use, su3, ((lo4 + (int64_t)r * kRowF4) << 2) + 128 * w);
                    const unsigned int m = i < hi4 ? mask_of(x[q], i << 2, su) : 0u;
                    const unsigned int earlier =
                        __reduce_add_sync(0xffffffffu, lane < w ? (unsigned int)table[r * kFusedWarps + lane] : 0u);
                    const unsigned int c_m = __popc(m);
                    unsigned int s2 = c_m;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned int t = __shfl_up_sync(0xffffffffu, s2, o);
                        if (lane >= o) s2 += t;
                    }
                    if (m) {
                        long long p = (long long)base + sh.rowpre[r] + earlier + (s2 - c_m);
                        const int64_t e0 = i << 2;
                        const float vv[4] = {x[q].x, x[q].y, x[q].z, x[q].w};
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            if (m & (1u << t)) {
                                if (p < cap) {
                                    idx_out[p] = (int32_t)(e0 + t);
                                    val_out[p] = vv[t];
                                    eps[e0 + t] = 0.0f;
                                }
                                ++p;
                            }
                        }
                    }
                }
                __syncwarp();
            }
            // the ragged tail comes last in index order
            if ((c == G - 1) && (w == kFusedWarps - 1) && (d & 3)) {
                int sx = seg_find(sh.off, S_use, n4 << 2);
                const bool hit = owns_tail && (fabsf(tail_u) > thr_at(sx, tail_i));
                const unsigned int bal = __ballot_sync(0xffffffffu, hit);
                if (hit) {
                    const long long p = (long long)base + run_total + __popc(bal & ((1u << lane) - 1u));
                    if (p < cap) {
                        idx_out[p] = (int32_t)tail_i;
                        val_out[p] = tail_u;
                        eps[tail_i] = 0.0f;
                    }
                }
            }
        }
    }
    // CTA 0 completes the records that the host can read back, off everybody's way
    if (c == 0 && !bad) {
        for (int q = tid; q < S; q += kFusedThreads) {
            const long long n = sh.off[q + 1] - sh.off[q];
            if (n <= 0 || !sh.counted[q]) continue;
            long long kk = seg_k[q];
            if (kk > n) kk = n;
            unsigned long long cnt[kNumCand];
#pragma unroll
            for (int j = 0; j < kNumCand; ++j) cnt[j] = __ldcg(&v.counts[(size_t)q * kNumCand + j]);
            gk_stats rec = v.stats[q];
            const Alg1Path p = alg1_replay(cnt, kk);
#pragma unroll
            for (int r = 0; r < kMaxRounds; ++r) rec.counts[r] = p.est[r];   // rounds not run: 0
            rec.rounds = p.rounds;
            rec.thr_final = v.cand64[(size_t)q * kNumCand + p.chosen];
            rec.nnz = alg1_last_est(p);
            v.stats[q] = rec;
            v.thr_sel[q] = sh.thr[q];
        }
    }
    if (c == 0 && tid == 0) ctrl->phase_t[5] = global_timer_ns();
    stamp(7);

leave:
    // the CTA that leaves last clears the barrier counters for the next call
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(&bars[2], 1u);
        if (t == (unsigned)G - 1) {
            ctrl->phase_t[6] = global_timer_ns();
            bars[0] = 0u; bars[1] = 0u; bars[3] = 0u; bars[4] = 0u;
            // (no fence: the end of the kernel orders these stores before the next launch on this
            // stream, the only reader)
            bars[2] = 0u;
        }
    }
}

// Host side -----------------------------------------------------------------
struct SegFusedPlan {
    bool ready = false, usable = false;
    int grid = 0;
};
static SegFusedPlan g_sf_plan[64];

static SegFusedPlan* seg_fused_plan(int dev, int sm_count) {
    if (dev < 0 || dev >= 64) return nullptr;
    // built once per device, under a lock: a second thread's first call waits for the finished plan
    static std::mutex plan_mu;
    std::lock_guard<std::mutex> plan_lock(plan_mu);
    SegFusedPlan& p = g_sf_plan[dev];
    if (p.ready) return &p;
    p.ready = true;
    int coop = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return &p;
    if (cudaFuncSetAttribute(k_gk_fused_seg, cudaFuncAttributeMaxDynamicSharedMemorySize, kSfSmemBudget) !=
        cudaSuccess) {
        cudaGetLastError();
        return &p;
    }
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_gk_fused_seg, kFusedThreads, kSfSmemBudget) !=
            cudaSuccess || occ < 1) {
        cudaGetLastError();
        return &p;
    }
    p.grid = sm_count < kFusedGridCap ? sm_count : kFusedGridCap;
    p.usable = true;
    return &p;
}

// Returns GK_OK when the fused kernel was enqueued, 1 when it cannot serve this call (the
// caller then takes the three-kernel form), or an error.
int enqueue_gk_fused_seg(Workspace* ws, const float* g, float* eps, int64_t d, const int64_t* seg_offsets,
                         const int64_t* seg_k, int32_t S, int32_t* idx_out, float* val_out, int64_t* seg_nnz_out,
                         int64_t* nnz_out, cudaStream_t st) {
    if (S > kSegFusedMax) return 1;
    int dev = 0;
    GK_CUDA_TRY(cudaGetDevice(&dev));
    SegFusedPlan* p = seg_fused_plan(dev, ws->sm_count);
    if (!p || !p->usable) return 1;
    const int64_t n4 = d >> 2;
    const int64_t n_rows = (n4 + kRowF4 - 1) / kRowF4;
    int64_t G = n_rows < p->grid ? n_rows : p->grid;
    if (G < 1) G = 1;
    // the longest run the kernel's cut can produce: a run's cost is (n_rows + 2 (S - 1)) / G, a row costs 1
    int64_t max_rows = (n_rows + 2 * (int64_t)(S - 1) + G - 1) / G + 2;
    if (max_rows > kSfTableMaxRows) return 1;
    int rpc = (int)max_rows;
    const int64_t left = (int64_t)kSfSmemBudget - (int64_t)kSfRing * kRowBytes - (int64_t)rpc * kSfTableRowBytes;
    int u_slots = (int)(left / kRowBytes);
    if (u_slots > rpc) u_slots = rpc;
    // a slot is written again kSfStages - 1 rows later: with fewer slots than rows in flight the
    // copy for a later row would land on the row being read
    if (u_slots < kSfStages && u_slots < rpc) return 1;
    const size_t smem = (size_t)(kSfRing + u_slots) * kRowBytes + (size_t)rpc * kSfTableRowBytes;
    int n_rows_arg = (int)n_rows;
    int S_arg = (int)S;
    Ctrl* ctrl = ws->ctrl;
    SegScratch v = segmented_views(ws);
    unsigned int* bars = ws->bars + 10;  // counters 10..14: three barriers, the exit, the quantile ticket
    unsigned int* cta_tot = ws->cta_counts;  // one word per CTA: the survivors of its run
    int64_t cap = output_capacity(d);
    unsigned long long* trace = ws->cta_trace;
    void* args[] = {(void*)&g, (void*)&eps, (void*)&d, (void*)&seg_offsets, (void*)&seg_k, (void*)&S_arg,
                    (void*)&n_rows_arg, (void*)&rpc, (void*)&u_slots, (void*)&ctrl, (void*)&v, (void*)&bars, (void*)&cta_tot,
                    (void*)&idx_out, (void*)&val_out, (void*)&seg_nnz_out, (void*)&nnz_out, (void*)&cap,
                    (void*)&trace};
    static_assert(sizeof(args) / sizeof(args[0]) == 19, "k_gk_fused_seg takes 19 arguments");
    stage_mark(ws, st, 0);
    GK_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)k_gk_fused_seg, dim3((unsigned)G), dim3(kFusedThreads), args,
                                            smem, st));
    note_launch();
    stage_mark(ws, st, 1);
    ws->last_grid = (int)G;
    ws->last_fused = true;  // the per-CTA trace is this kernel's
    ws->phase_spans = 6;
    return GK_OK;
}

}  // namespace gk
