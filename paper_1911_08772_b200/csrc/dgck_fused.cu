// DGC_k, the hierarchical sampling selector that arXiv 1911.08772 compares
// Gaussian_k with (Section 3.3; a 1 % sample in Section 4.3), as ONE persistent
// cooperative kernel.  The paper describes it in one sentence: a small random
// sample gives the threshold, and top-k selection runs twice on subsets of the
// vector.  As built here:
//
//   sample   the caller passes the m sampled positions.  Every CTA takes a
//            share of them, reads |u| there (u = g + eps in the sparsifier
//            form) and the k_m-th largest sampled magnitude tau,
//            k_m = ceil(k m / d), is found by a radix select on the 31
//            magnitude bits (11 + 10 + 10) over histograms merged in global
//            memory: the first top-k, on the sample.
//   stream   the vector streams through once (sparsifier form: u = g + eps goes
//            back over eps, Eq. 2); per (row, warp) segment of 128 elements the
//            number of magnitudes >= tau goes to a table in shared memory, the
//            CTAs' totals to global memory; after a barrier every CTA knows
//            n = #{ |u_i| >= tau }.
//   select   n <= k: every candidate is returned.  n > k: the second top-k, on
//            the candidates: a radix select for the k-th largest among the keys
//            >= tau, reading only segments that hold a candidate (shared memory
//            or L2); ties go to the lower index.
//   compact  per-row counts are exchanged through one more barrier, which gives
//            every row its output offset; pairs come out in ascending index.
//
// Rows of 1024 float4 are dealt to one CTA per SM in turn, as in the other
// persistent kernels.  All waits are bounded (grid_barrier).
#include <mutex>

#include "gk_common.cuh"
#include "gk_coop.cuh"
#include "gk_radix.cuh"

namespace gk {

constexpr int kDgCacheKeys = kTkSmemRows * kRowF4 * 4;  // sampled keys a CTA keeps in shared memory

template <bool ACCUM> struct DgStages { static constexpr int value = ACCUM ? 4 : 8; };

// ACCUM: src = g, eps in/out (u stored over eps, selected slots cleared).  Otherwise src = u,
// read-only, eps unused.  sample_idx: m positions in [0, d).  km: rank taken in the sample.
// ghist: 2048 + 1024 + 1024 merged bins, zero on entry and on exit.  cta_cnt: one word per CTA.
// rowcnt: two words per row of the vector.  bars: [0] barrier counter (the i-th barrier waits for
// i * G arrivals), [1] exit counter; zero on entry and on exit.
// Shared memory: [g ring of kStages rows (ACCUM only)][u_slots rows][table]; before the stream
// phase the rows hold this CTA's sampled keys.
template <bool ACCUM>
__global__ void __launch_bounds__(kFusedThreads, 1)
k_dgck_fused(const float* __restrict__ src, float* __restrict__ eps, int64_t d, int64_t k,
             const int32_t* __restrict__ sample_idx, int64_t m, int64_t km, int n_rows, int u_slots,
             Ctrl* __restrict__ ctrl, unsigned int* __restrict__ ghist, unsigned int* __restrict__ cta_cnt,
             uint2* __restrict__ rowcnt, unsigned int* __restrict__ bars, int32_t* __restrict__ idx_out,
             float* __restrict__ val_out, int64_t* __restrict__ nnz_out) {
    extern __shared__ __align__(1024) float4 smem4[];
    __shared__ TopkShared sh;
    __shared__ unsigned int cta_total;
    __shared__ unsigned long long n_all;
    float4* gring = smem4;
    constexpr int kStages = DgStages<ACCUM>::value;
    float4* uslot = smem4 + (ACCUM ? (size_t)kStages * kRowF4 : 0);
    unsigned short* table = reinterpret_cast<unsigned short*>(smem4 + (size_t)kTkSmemRows * kRowF4);
    unsigned int* skeys = reinterpret_cast<unsigned int*>(smem4);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int c = blockIdx.x, G = gridDim.x;
    const int64_t n4 = d >> 2;
    unsigned int* ghist1 = ghist;
    unsigned int* ghist2 = ghist + 2048;
    unsigned int* ghist3 = ghist + 3072;

    const int nrows = c < n_rows ? (n_rows - c + G - 1) / G : 0;
    const int64_t stride4 = (int64_t)G * kRowF4;
    const int64_t first4 = (int64_t)c * kRowF4 + tid;
    const int first_kept = nrows > u_slots ? nrows - u_slots : 0;  // rows from here on stay on chip
    const bool owns_tail = (c == G - 1) && (w == kFusedWarps - 1) && (lane < (int)(d & 3));
    const int64_t tail_i = (n4 << 2) + lane;
    const float4* s4 = reinterpret_cast<const float4*>(src);
    float4* e4 = reinterpret_cast<float4*>(eps);
    const float4* uglob = ACCUM ? reinterpret_cast<const float4*>(eps) : s4;  // where u is after the stream phase
    float tail_u = 0.f;
    const bool wide_ok = ACCUM && ((reinterpret_cast<uintptr_t>(eps) & 31u) == 0);
    int bar_no = 0;
    // the i-th barrier of the call: all CTAs arrive at the same sequence of barriers
    auto barrier = [&]() -> bool {
        ++bar_no;
        if (grid_barrier(&bars[0], (unsigned)G * (unsigned)bar_no, &sh.ok)) return true;
        if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
        return false;
    };

    if (c == 0 && tid == 0) {
        ctrl->stats.status = GK_DEV_OK;
        ctrl->phase_t[0] = global_timer_ns();
    }
    for (int b = tid; b < kTkBins; b += kFusedThreads) sh.hist[b] = 0u;
    if (tid == 0) { sh.need = (unsigned long long)km; sh.digit = 0u; sh.n_staged = 0u; cta_total = 0u; }
    __syncthreads();

    // ------------------------------------------------------------------ sample: tau
    unsigned int tau;
    {
        const int64_t s_lo = m * c / G, s_hi = m * (c + 1) / G;  // this CTA's share of the sample
        bool bad = false;
        auto sample_key = [&](int64_t j) -> unsigned int {
            int64_t i = sample_idx[j];
            if (i < 0 || i >= d) { bad = true; i = i < 0 ? 0 : d - 1; }
            const float x = ACCUM ? src[i] + eps[i] : src[i];
            return tk_key(x);
        };
        for (int64_t j = s_lo + tid; j < s_hi; j += kFusedThreads) {
            const unsigned int key = sample_key(j);
            if (j - s_lo < kDgCacheKeys) skeys[j - s_lo] = key;
            atomicAdd(&sh.hist[key >> 20], 1u);
        }
        __syncthreads();
        merge_hist(ghist1, 2048, sh);
        if (!barrier()) goto leave;
        if (bad) atomicOr(&ctrl->stats.status, GK_DEV_BAD_SAMPLE);  // after CTA 0 has cleared the word
        pick_digit(ghist1, 2048, sh);
        const unsigned int b1 = sh.digit;
        for (int64_t j = s_lo + tid; j < s_hi; j += kFusedThreads) {
            const unsigned int key = (j - s_lo < kDgCacheKeys) ? skeys[j - s_lo] : sample_key(j);
            if ((key >> 20) == b1) atomicAdd(&sh.hist[(key >> 10) & 1023u], 1u);
        }
        __syncthreads();
        merge_hist(ghist2, 1024, sh);
        if (!barrier()) goto leave;
        // every CTA has read the first level's merged bins before it arrived here
        if (c == 0) for (int b = tid; b < 2048; b += kFusedThreads) ghist1[b] = 0u;
        pick_digit(ghist2, 1024, sh);
        const unsigned int p21 = (b1 << 10) | sh.digit;
        for (int64_t j = s_lo + tid; j < s_hi; j += kFusedThreads) {
            const unsigned int key = (j - s_lo < kDgCacheKeys) ? skeys[j - s_lo] : sample_key(j);
            if ((key >> 10) == p21) atomicAdd(&sh.hist[key & 1023u], 1u);
        }
        __syncthreads();
        merge_hist(ghist3, 1024, sh);
        if (!barrier()) goto leave;
        if (c == 0) for (int b = tid; b < 1024; b += kFusedThreads) ghist2[b] = 0u;
        pick_digit(ghist3, 1024, sh);
        tau = (p21 << 10) | sh.digit;
        if (c == 0 && tid == 0) ctrl->phase_t[1] = global_timer_ns();
    }

    // ------------------------------------------------------------------ stream: candidates per segment
    {
        int64_t fi = first4;  // the row the next fetch brings in
        auto fetch = [&](int r) {
            if (r < nrows && fi < n4) {
                if (ACCUM) {
                    cp_async16(gring + (size_t)(r % kStages) * kRowF4 + tid, s4 + fi);
                    cp_async16(uslot + (size_t)(r % u_slots) * kRowF4 + tid, e4 + fi);
                } else {
                    cp_async16(uslot + (size_t)(r % u_slots) * kRowF4 + tid, s4 + fi);
                }
            }
            cp_async_commit();
            fi += stride4;
        };
#pragma unroll
        for (int r = 0; r < kStages - 1; ++r) fetch(r);
        int64_t i = first4;
        unsigned int warp_total = 0u;
        for (int r = 0; r < nrows; ++r, i += stride4) {
            fetch(r + kStages - 1);
            cp_async_wait<kStages - 1>();
            const bool one = i < n4;
            float4 u0 = make_float4(0.f, 0.f, 0.f, 0.f);
            unsigned int c4 = 0u;
            if (one) {
                float4* us = uslot + (size_t)(r % u_slots) * kRowF4 + tid;
                u0 = *us;
                if (ACCUM) {
                    const float4 a0 = gring[(size_t)(r % kStages) * kRowF4 + tid];
                    u0 = make_float4(a0.x + u0.x, a0.y + u0.y, a0.z + u0.z, a0.w + u0.w);
                    *us = u0;
                }
                c4 = (unsigned)(tk_key(u0.x) >= tau) + (unsigned)(tk_key(u0.y) >= tau) +
                     (unsigned)(tk_key(u0.z) >= tau) + (unsigned)(tk_key(u0.w) >= tau);
            }
            if (ACCUM) {
                // u goes out in 32-byte stores by the even lanes (own float4 and the right
                // neighbour's), marked to stay in L2: the later passes read parts of u again
                float4 nb;
                nb.x = __shfl_down_sync(0xffffffffu, u0.x, 1); nb.y = __shfl_down_sync(0xffffffffu, u0.y, 1);
                nb.z = __shfl_down_sync(0xffffffffu, u0.z, 1); nb.w = __shfl_down_sync(0xffffffffu, u0.w, 1);
                const bool pair = wide_ok && (i + 1 < n4);
                if ((lane & 1) == 0) {
                    if (pair) st_keep32(e4 + i, u0, nb);
                    else if (one) e4[i] = u0;
                } else if (one && !wide_ok) {
                    e4[i] = u0;
                }
            }
            const unsigned int wc = __reduce_add_sync(0xffffffffu, c4);
            if (lane == 0) table[r * kFusedWarps + w] = (unsigned short)wc;
            warp_total += wc;
        }
        cp_async_wait<0>();
        if (owns_tail) {
            tail_u = ACCUM ? src[tail_i] + eps[tail_i] : src[tail_i];
            if (ACCUM) eps[tail_i] = tail_u;
            if (tk_key(tail_u) >= tau) atomicAdd(&cta_total, 1u);
        }
        if (lane == 0 && warp_total) atomicAdd(&cta_total, warp_total);
        __syncthreads();
        if (tid == 0) cta_cnt[c] = cta_total;
        if (c == 0 && tid == 0) ctrl->phase_t[2] = global_timer_ns();
        if (!barrier()) goto leave;
        if (c == 0) for (int b = tid; b < 1024; b += kFusedThreads) ghist3[b] = 0u;
        // n: candidates in the whole vector (integer sum, the same in every CTA)
        unsigned long long s = 0ull;
        for (int t = tid; t < G; t += kFusedThreads) s += __ldcg(cta_cnt + t);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) sh.wsum2[w] = s;
        __syncthreads();
        if (tid == 0) {
            unsigned long long t = 0ull;
            for (int q = 0; q < kFusedWarps; ++q) t += sh.wsum2[q];
            n_all = t;
            sh.need = (unsigned long long)k;
        }
        __syncthreads();
    }

    {
        const unsigned long long n = n_all;
        const bool second = n > (unsigned long long)k;   // the same decision in every CTA
        const long long out_n = (long long)(second ? (unsigned long long)k : n);
        if (c == 0 && tid == 0) {
            *nnz_out = out_n;
            ctrl->dgc[0] = tau; ctrl->dgc[1] = n; ctrl->dgc[2] = (unsigned long long)km;
            ctrl->dgc[3] = (unsigned long long)out_n;
            ctrl->phase_t[3] = global_timer_ns();
        }
        // segments that hold a candidate are the only ones read again
        for (int r = lane; r < nrows; r += 32)
            if (table[r * kFusedWarps + w] != 0) table[r * kFusedWarps + w] = kTkPending;
        __syncthreads();

        auto gather = [&](int& cursor, const bool want_pending) -> int {
            return want_pending ? gather_cells<kGatherPending>(table, nrows, cursor, sh.qrow[w])
                                : gather_cells<kGatherNonZero>(table, nrows, cursor, sh.qrow[w]);
        };
        auto load_row = [&](int r) -> float4 {
            const int64_t i = first4 + (int64_t)r * stride4;
            if (i >= n4) return make_float4(0.f, 0.f, 0.f, 0.f);
            return (r >= first_kept) ? uslot[(size_t)(r % u_slots) * kRowF4 + tid] : __ldcg(uglob + i);
        };
#define DG_FOR_EACH_MARKED(want_pending, ...)                                       \
    for (int cursor_ = 0; cursor_ < nrows;) {                                         \
        const int n_ = gather(cursor_, want_pending);                                 \
        float4 v_[kTkGroupRows];                                                      \
        _Pragma("unroll") for (int q_ = 0; q_ < kTkGroupRows; ++q_) {                 \
            v_[q_] = make_float4(0.f, 0.f, 0.f, 0.f);                                 \
            if (q_ < n_) v_[q_] = load_row(sh.qrow[w][q_]);                           \
        }                                                                             \
        _Pragma("unroll") for (int q_ = 0; q_ < kTkGroupRows; ++q_) {                 \
            if (q_ < n_) {                                                            \
                const int r = sh.qrow[w][q_];                                         \
                const float4 v = v_[q_];                                              \
                const bool in = first4 + (int64_t)r * stride4 < n4;                   \
                __VA_ARGS__                                                           \
            }                                                                         \
        }                                                                             \
        __syncwarp();                                                                 \
    }

        unsigned int T = tau;                     // key of the last entry taken
        unsigned long long need_eq = 1ull << 62;  // entries equal to T to take: all of them when n <= k
        const unsigned int tail_key = tk_key(tail_u);
        const bool tail_cand = owns_tail && tail_key >= tau;
        if (second) {
            // ---------------------------------------------------------- second top-k, on the candidates
            DG_FOR_EACH_MARKED(true, {
                if (in) {
                    const unsigned int key[4] = {tk_key(v.x), tk_key(v.y), tk_key(v.z), tk_key(v.w)};
#pragma unroll
                    for (int t = 0; t < 4; ++t)
                        if (key[t] >= tau) atomicAdd(&sh.hist[key[t] >> 20], 1u);
                }
            })
            if (tail_cand) atomicAdd(&sh.hist[tail_key >> 20], 1u);
            __syncthreads();
            merge_hist(ghist1, 2048, sh);
            if (!barrier()) goto leave;
            pick_digit(ghist1, 2048, sh);
            const unsigned int b1 = sh.digit;
            DG_FOR_EACH_MARKED(true, {
                if (in) {
                    const unsigned int key[4] = {tk_key(v.x), tk_key(v.y), tk_key(v.z), tk_key(v.w)};
#pragma unroll
                    for (int t = 0; t < 4; ++t)
                        if (key[t] >= tau && (key[t] >> 20) == b1) atomicAdd(&sh.hist[(key[t] >> 10) & 1023u], 1u);
                }
            })
            if (tail_cand && (tail_key >> 20) == b1) atomicAdd(&sh.hist[(tail_key >> 10) & 1023u], 1u);
            __syncthreads();
            merge_hist(ghist2, 1024, sh);
            if (!barrier()) goto leave;
            if (c == 0) for (int b = tid; b < 2048; b += kFusedThreads) ghist1[b] = 0u;
            pick_digit(ghist2, 1024, sh);
            const unsigned int p21 = (b1 << 10) | sh.digit;
            DG_FOR_EACH_MARKED(true, {
                if (in) {
                    const unsigned int key[4] = {tk_key(v.x), tk_key(v.y), tk_key(v.z), tk_key(v.w)};
#pragma unroll
                    for (int t = 0; t < 4; ++t)
                        if (key[t] >= tau && (key[t] >> 10) == p21) atomicAdd(&sh.hist[key[t] & 1023u], 1u);
                }
            })
            if (tail_cand && (tail_key >> 10) == p21) atomicAdd(&sh.hist[tail_key & 1023u], 1u);
            __syncthreads();
            merge_hist(ghist3, 1024, sh);
            if (!barrier()) goto leave;
            if (c == 0) for (int b = tid; b < 1024; b += kFusedThreads) ghist2[b] = 0u;
            pick_digit(ghist3, 1024, sh);
            T = (p21 << 10) | sh.digit;
            need_eq = sh.need;
        }
        if (c == 0 && tid == 0) {
            ctrl->key_threshold = T;
            ctrl->need_eq = need_eq;
            ctrl->phase_t[4] = global_timer_ns();
        }

        // ---------------------------------------------------------- compaction
        // step 1: keys above / equal to T per marked segment; the table entry becomes
        // (above) | (equal << 8), at most 128 each
        // The places of the entries counted here -- row, warp, lane, element, above or equal, and
        // their ranks among the segment's keys above and equal to T -- are put aside in shared
        // memory, two words each, as long as they fit: the write-out is then one thread per
        // entry instead of one warp per segment.
        unsigned int* st_ent = ACCUM ? reinterpret_cast<unsigned int*>(gring)
                                     : reinterpret_cast<unsigned int*>(smem4 + (size_t)(kTkSmemRows - kTkStageRows) * kRowF4);
        constexpr unsigned int kStageCap = (ACCUM ? kStages : kTkStageRows) * kRowBytes / 8;
        const unsigned int lanes_below = (1u << lane) - 1u;
        DG_FOR_EACH_MARKED(true, {
            unsigned int gm = 0u, em = 0u;
            if (in) {
                const unsigned int key[4] = {tk_key(v.x), tk_key(v.y), tk_key(v.z), tk_key(v.w)};
#pragma unroll
                for (int t = 0; t < 4; ++t) { gm |= (unsigned)(key[t] > T) << t; em |= (unsigned)(key[t] == T) << t; }
            }
            const unsigned int ge = __reduce_add_sync(0xffffffffu, __popc(gm) | (__popc(em) << 8));
            if (lane == 0) table[r * kFusedWarps + w] = (unsigned short)ge;
            if (ge != 0u) {
                const unsigned int total = (ge & 0xffu) + (ge >> 8);
                unsigned int base = 0u;
                if (lane == 0) base = atomicAdd(&sh.n_staged, total);
                base = __shfl_sync(0xffffffffu, base, 0);
                unsigned int rank_g = 0u, rank_e = 0u;
                if (total > 1u) {
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        rank_g += __popc(__ballot_sync(0xffffffffu, gm & (1u << t)) & lanes_below);
                        rank_e += __popc(__ballot_sync(0xffffffffu, em & (1u << t)) & lanes_below);
                    }
                }
                if ((gm | em) && base + total <= kStageCap) {
                    const unsigned int place = ((unsigned int)r << 19) | ((unsigned int)w << 14) | ((unsigned int)lane << 9);
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const bool isg = gm & (1u << t), ise = em & (1u << t);
                        if (isg || ise) {
                            const unsigned int slot = base + rank_g + rank_e;
                            st_ent[2 * slot] = place | ((unsigned int)t << 7) | (isg ? 1u : 0u);
                            st_ent[2 * slot + 1] = rank_g | (rank_e << 8);
                            rank_g += isg; rank_e += ise;
                        }
                    }
                }
            }
        })
        __syncthreads();
        const bool staged = sh.n_staged <= kStageCap;
        // step 2: per row (thread t takes local row t) the two counts go to the row's words
        bool any_mine = false;
        if (tid < nrows) {
            const uint4* tv = reinterpret_cast<const uint4*>(table + (size_t)tid * kFusedWarps);
            unsigned int lo8 = 0u, hi8 = 0u;
#pragma unroll
            for (int q = 0; q < kFusedWarps * 2 / 16; ++q) {
                const uint4 x = tv[q];
                const unsigned int ws[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    lo8 += (ws[j] & 0xffu) + ((ws[j] >> 16) & 0xffu);
                    hi8 += ((ws[j] >> 8) & 0xffu) + (ws[j] >> 24);
                }
            }
            rowcnt[c + tid * G] = make_uint2(lo8, hi8);
            any_mine = (lo8 | hi8) != 0u;
        }
        any_mine = __syncthreads_or(any_mine) != 0;
        if (!barrier()) goto leave;
        if (second && c == 0) for (int b = tid; b < 1024; b += kFusedThreads) ghist3[b] = 0u;
        if (c == 0 && tid == 0) ctrl->phase_t[5] = global_timer_ns();
        const bool tail_cta = (c == G - 1) && (d & 3);
        unsigned long long all_rows = 0ull;  // keys above / equal to T in all rows (tail CTA only)
        if (any_mine || tail_cta) {
            // entries before local row r of this CTA = those of the rounds before r (round r is the
            // G consecutive rows r * G ... r * G + G - 1) + those of the CTAs before this one in
            // round r; a count pair travels as one 64-bit word (above low, equal high)
            for (int r = w; r < nrows; r += kFusedWarps) {
                unsigned long long tot = 0ull, pre = 0ull;
                const int R0 = r * G;
                for (int t = lane; t < G; t += 32) {
                    uint2 x = make_uint2(0u, 0u);
                    if (R0 + t < n_rows) x = __ldcg(rowcnt + R0 + t);
                    const unsigned long long v = (unsigned long long)x.x | ((unsigned long long)x.y << 32);
                    tot += v;
                    pre += (t < c) ? v : 0ull;
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    tot += __shfl_xor_sync(0xffffffffu, tot, o);
                    pre += __shfl_xor_sync(0xffffffffu, pre, o);
                }
                if (lane == 0) { sh.roundtot[r] = tot; sh.rowpre[r] = pre; }
            }
            __syncthreads();
            {
                const unsigned long long mine_round = tid < nrows ? sh.roundtot[tid] : 0ull;
                const unsigned long long s = warp_incl_scan64(mine_round, lane);
                if (lane == 31) sh.wsum2[w] = s;
                __syncthreads();
                const unsigned long long x = sh.wsum2[lane];
                const unsigned long long y = warp_incl_scan64(x, lane);
                const unsigned long long wpre = __shfl_sync(0xffffffffu, y - x, w);
                if (tid < nrows) sh.rowpre[tid] += wpre + s - mine_round;
                all_rows = __shfl_sync(0xffffffffu, y, 31);
                __syncthreads();
            }
        }
        if (any_mine && staged) {
            // step 3: one thread per entry put aside: keys above T always, keys equal to T while
            // fewer than need_eq of them came before
            const unsigned int n_st = sh.n_staged;
            for (unsigned int j = tid; j < n_st; j += kFusedThreads) {
                const unsigned int tag = st_ent[2 * j], rk = st_ent[2 * j + 1];
                const unsigned int r = tag >> 19, cell = (tag >> 14) & 31u, ln = (tag >> 9) & 31u, t = (tag >> 7) & 3u;
                const bool isg = tag & 1u;
                unsigned int bg = 0u, be = 0u;   // keys above / equal to T in the warps before this one
                for (unsigned int ww = 0; ww < cell; ++ww) {
                    const unsigned int x = table[r * kFusedWarps + ww];
                    bg += x & 0xffu; be += x >> 8;
                }
                const unsigned long long rp = sh.rowpre[r];
                const unsigned long long ng = (rp & 0xffffffffull) + bg + (rk & 0xffu);
                const unsigned long long ne = (rp >> 32) + be + (rk >> 8);
                if (isg || ne < need_eq) {
                    const unsigned long long pos = ng + (ne < need_eq ? ne : need_eq);
                    if ((long long)pos < out_n) {
                        const unsigned int in_row = ((cell << 5) | ln) << 2 | t;   // element within the row
                        const int64_t at = (((int64_t)c + (int64_t)r * G) << 12) + in_row;
                        const float x = ((int)r >= first_kept)
                                            ? reinterpret_cast<const float*>(uslot + (size_t)(r % u_slots) * kRowF4)[in_row]
                                            : __ldcg(reinterpret_cast<const float*>(uglob) + at);
                        idx_out[pos] = (int32_t)at;
                        val_out[pos] = x;
                        if (ACCUM) eps[at] = 0.0f;
                    }
                }
            }
        } else if (any_mine) {
            // step 3 without the places: every warp writes the selected entries of its segments
            // that have any
            DG_FOR_EACH_MARKED(false, {
                unsigned int gm = 0u, em = 0u;
                if (in) {
                    const unsigned int key[4] = {tk_key(v.x), tk_key(v.y), tk_key(v.z), tk_key(v.w)};
#pragma unroll
                    for (int t = 0; t < 4; ++t) { gm |= (unsigned)(key[t] > T) << t; em |= (unsigned)(key[t] == T) << t; }
                }
                const unsigned int e_before = lane < w ? (unsigned int)table[r * kFusedWarps + lane] : 0u;
                const unsigned int wb = __reduce_add_sync(0xffffffffu, (e_before & 0xffu) | ((e_before >> 8) << 16));
                const unsigned int mine_ge = __popc(gm) | (__popc(em) << 16);
                const unsigned int sc = warp_incl_scan(mine_ge, lane) - mine_ge;
                if (gm | em) {
                    const unsigned long long rp = sh.rowpre[r];
                    unsigned long long ng = (rp & 0xffffffffull) + (wb & 0xffffu) + (sc & 0xffffu);
                    unsigned long long ne = (rp >> 32) + (wb >> 16) + (sc >> 16);
                    const int64_t e0 = (first4 + (int64_t)r * stride4) << 2;
                    const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const bool isg = gm & (1u << t), ise = em & (1u << t);
                        if (isg || (ise && ne < need_eq)) {
                            const unsigned long long pos = ng + (ne < need_eq ? ne : need_eq);
                            if ((long long)pos < out_n) {
                                idx_out[pos] = (int32_t)(e0 + t);
                                val_out[pos] = vv[t];
                                if (ACCUM) eps[e0 + t] = 0.0f;
                            }
                        }
                        ng += isg; ne += ise;
                    }
                }
            })
        }
        // the ragged tail comes last in index order
        if (tail_cta && w == kFusedWarps - 1) {
            unsigned long long extra = 0ull;  // rounds this CTA has no row in are missing from its scan
            const int rounds = (n_rows + G - 1) / G;
            if (rounds > nrows) {
                for (int t = lane; t < G; t += 32) {
                    const int R = (rounds - 1) * G + t;
                    if (R < n_rows) {
                        const uint2 x = __ldcg(rowcnt + R);
                        extra += (unsigned long long)x.x | ((unsigned long long)x.y << 32);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) extra += __shfl_xor_sync(0xffffffffu, extra, o);
            }
            const unsigned long long tot = all_rows + extra;
            const bool isg = owns_tail && tail_key > T, ise = owns_tail && tail_key == T;
            const unsigned int bg = __ballot_sync(0xffffffffu, isg), be = __ballot_sync(0xffffffffu, ise);
            const unsigned int below = (1u << lane) - 1u;
            const unsigned long long ng = (tot & 0xffffffffull) + __popc(bg & below);
            const unsigned long long ne = (tot >> 32) + __popc(be & below);
            if (isg || (ise && ne < need_eq)) {
                const unsigned long long pos = ng + (ne < need_eq ? ne : need_eq);
                if ((long long)pos < out_n) {
                    idx_out[pos] = (int32_t)tail_i;
                    val_out[pos] = tail_u;
                    if (ACCUM) eps[tail_i] = 0.0f;
                }
            }
        }
#undef DG_FOR_EACH_MARKED
    }
    if (c == 0 && tid == 0) ctrl->phase_t[6] = global_timer_ns();

leave:
    // the CTA that leaves last clears the counters for the next call
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(&bars[1], 1u);
        if (t == (unsigned)G - 1) {
            ctrl->phase_t[7] = global_timer_ns();
            bars[0] = 0u;
            // (no fence: the end of the kernel orders these stores before the next launch on this
            // stream, the only reader)
            bars[1] = 0u;
        }
    }
}

// Host side -----------------------------------------------------------------
struct DgPlan {
    bool ready = false, usable = false;
    int grid = 0;
};
static DgPlan g_dg_plan[64];

template <bool ACCUM>
static bool dgck_kernel_ready() {
    if (cudaFuncSetAttribute(k_dgck_fused<ACCUM>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTkSmemBytes) !=
        cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_dgck_fused<ACCUM>, kFusedThreads, kTkSmemBytes) !=
            cudaSuccess || occ < 1) {
        cudaGetLastError();
        return false;
    }
    return true;
}

static DgPlan* dgck_plan(int dev, int sm_count) {
    if (dev < 0 || dev >= 64) return nullptr;
    // built once per device, under a lock: a second thread's first call waits for the finished plan
    static std::mutex plan_mu;
    std::lock_guard<std::mutex> plan_lock(plan_mu);
    DgPlan& p = g_dg_plan[dev];
    if (p.ready) return &p;
    p.ready = true;
    int coop = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return &p;
    if (!dgck_kernel_ready<false>() || !dgck_kernel_ready<true>()) return &p;
    p.grid = sm_count < kFusedGridCap ? sm_count : kFusedGridCap;
    p.usable = true;
    return &p;
}

// With eps != nullptr: src = g, u = g + eps is formed, stored over eps and cleared where
// selected; else src = u, read-only.
static int enqueue_dgck(const float* src, float* eps, int64_t d, int64_t k, const int32_t* sample_idx, int64_t m,
                        int32_t* idx_out, float* val_out, int64_t* nnz_out, cudaStream_t st) {
    Workspace* ws = nullptr;
    const int wrc = acquire_workspace(d, 1, st, &ws);
    if (wrc != GK_OK) return wrc;
    int dev = 0;
    GK_CUDA_TRY(cudaGetDevice(&dev));
    DgPlan* p = dgck_plan(dev, ws->sm_count);
    if (!p || !p->usable) return GK_ERR_LIMIT;  // no cooperative launch on this device
    const int64_t n4 = d >> 2;
    const int64_t rows = (n4 + kRowF4 - 1) / kRowF4;
    int64_t G = rows < p->grid ? rows : p->grid;
    if (G < 1) G = 1;
    int64_t most = (rows + G - 1) / G;  // rows of CTA 0
    if (most < 1) most = 1;
    if (most > kTkTableMaxRows) return GK_ERR_LIMIT;
    int n_rows = (int)rows;
    const bool accum = eps != nullptr;
    // with u given there is no g ring to reuse: two rows are set aside for the places of the selected entries
    int u_slots = accum ? kTkSmemRows - DgStages<true>::value : kTkSmemRows - kTkStageRows;
    static_assert(kTkSmemRows - DgStages<true>::value >= DgStages<true>::value && kTkSmemRows - kTkStageRows >= DgStages<false>::value,
                  "not enough row slots for the rows in flight");
    if (u_slots > most) u_slots = (int)most;
    int64_t km = (k * m + d - 1) / d;  // the density k/d applied to the sample size
    Ctrl* ctrl = ws->ctrl;
    unsigned int* ghist = ws->hist;
    unsigned int* cta_cnt = ws->cta_counts;
    uint2* rowcnt = reinterpret_cast<uint2*>(ws->rowcnt);
    unsigned int* bars = ws->bars + 14;  // the other persistent kernels own the counters before these two
    void* args[] = {(void*)&src, (void*)&eps, (void*)&d, (void*)&k, (void*)&sample_idx, (void*)&m, (void*)&km,
                    (void*)&n_rows, (void*)&u_slots, (void*)&ctrl, (void*)&ghist, (void*)&cta_cnt, (void*)&rowcnt,
                    (void*)&bars, (void*)&idx_out, (void*)&val_out, (void*)&nnz_out};
    static_assert(sizeof(args) / sizeof(args[0]) == 17, "k_dgck_fused takes 17 arguments");
    stage_mark(ws, st, 0);
    const void* fn = accum ? (const void*)k_dgck_fused<true> : (const void*)k_dgck_fused<false>;
    GK_CUDA_TRY(cudaLaunchCooperativeKernel(fn, dim3((unsigned)G), dim3(kFusedThreads), args, (size_t)kTkSmemBytes, st));
    note_launch();
    stage_mark(ws, st, 1);
    ws->last_grid = (int)G;
    ws->last_fused = false;
    ws->phase_spans = 7;
    return GK_OK;
}

}  // namespace gk

using namespace gk;

extern "C" int dgck_select(const float* u, int64_t d, int64_t k, const int32_t* sample_idx, int64_t m,
                           int32_t* idx_out, float* val_out, int64_t* nnz_out, gk_stream_t stream) {
    if (!u || !sample_idx || !idx_out || !val_out || !nnz_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll || m < 1 || m > 2147483647ll) return GK_ERR_SIZE;
    if (k < 1 || k > d) return GK_ERR_K;
    if ((uintptr_t)u & 15u) return GK_ERR_ALIGN;
    return enqueue_dgck(u, nullptr, d, k, sample_idx, m, idx_out, val_out, nnz_out, (cudaStream_t)stream);
}

extern "C" int dgck_sparsify(const float* g, float* eps, int64_t d, int64_t k, const int32_t* sample_idx,
                             int64_t m, int32_t* idx_out, float* val_out, int64_t* nnz_out, gk_stream_t stream) {
    if (!g || !eps || !sample_idx || !idx_out || !val_out || !nnz_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll || m < 1 || m > 2147483647ll) return GK_ERR_SIZE;
    if (k < 1 || k > d) return GK_ERR_K;
    if (((uintptr_t)g & 15u) || ((uintptr_t)eps & 15u)) return GK_ERR_ALIGN;
    const uintptr_t a = (uintptr_t)g, b = (uintptr_t)eps, n = (uintptr_t)d * 4u;
    if (a < b + n && b < a + n) return GK_ERR_ALIAS;
    return enqueue_dgck(g, eps, d, k, sample_idx, m, idx_out, val_out, nnz_out, (cudaStream_t)stream);
}
