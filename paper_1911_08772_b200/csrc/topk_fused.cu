// Exact Top_k (Section 1 of arXiv 1911.08772) as ONE persistent cooperative
// kernel: most-significant-digit radix select on the 31 magnitude bits of the
// fp32 pattern, followed by the ordered compaction, with what fits of u kept
// on chip between the passes.
//
// The vector is cut into rows of 1024 float4, dealt to one CTA per SM in turn (CTA c owns
// rows c, c + G, ...), so that every CTA gets the same mix of quiet and loud stretches.
//
//   pass 1   the run streams in through asynchronous copies (with ACCUM, g and
//            eps: u = g + eps goes back over eps, Eq. 2); every key's top 11
//            bits are counted in a shared-memory histogram; per (row, warp)
//            segment of 128 elements the largest magnitude goes to a table.
//   barrier  histograms are merged in global memory; every CTA finds the digit
//            that holds the k-th largest key.
//   pass 2/3 the next 10 + 10 bits, among the keys that match the digits found
//            so far.  Only segments whose recorded maximum reaches the first
//            digit are read again (a few percent of them when k << d), from
//            shared memory or L2.
//   barrier  after the third digit the threshold key T and the number of keys
//            equal to T still to take are known.
//   compact  every CTA counts the keys above / equal to T per row (the same few
//            segments again), the rows' counts are exchanged through a fourth
//            barrier, which gives every row its output offset -- no look-back;
//            keys above T are all taken, keys equal to T in order of increasing
//            index until k pairs are out.
//
// All waits are bounded (grid_barrier); a CTA whose wait runs out records
// GK_DEV_TIMEOUT and leaves.  Vectors whose runs exceed the table (more than
// kTkTableMaxRows rows per CTA) and devices without cooperative launch take
// the multi-kernel path in topk_exact.cu.
#include <mutex>

#include "gk_common.cuh"
#include "gk_coop.cuh"
#include "gk_count.cuh"
#include "gk_radix.cuh"

namespace gk {

// ACCUM: src = g, eps in/out (u stored over eps, selected slots cleared).  Otherwise src = u,
// read-only, eps unused.  n_rows: rows of 1024 float4 in the vector; CTA c owns rows c, c + G,
// c + 2G, ... so that stretches of large values are spread over all CTAs.  ghist: 2048 + 1024 +
// 1024 merged bins, zero on entry and on exit.  rowcnt: two words per row of the vector.
// bars: four barrier counters and an exit counter, zero on entry and on exit.
// Shared memory: [g ring of kStages rows (ACCUM only)][u_slots rows][table].
template <bool ACCUM>
__global__ void __launch_bounds__(kFusedThreads, 1)
k_topk_fused(const float* __restrict__ src, float* __restrict__ eps, int64_t d, int64_t k, int n_rows, int u_slots,
             Ctrl* __restrict__ ctrl, unsigned int* __restrict__ ghist, uint2* __restrict__ rowcnt,
             unsigned int* __restrict__ bars, int32_t* __restrict__ idx_out, float* __restrict__ val_out,
             int64_t* __restrict__ nnz_out) {
    // 1 KB alignment keeps every warp's 512 bytes of a row within four 128-byte lines of shared
    // memory, whatever the size of the static part
    extern __shared__ __align__(1024) float4 smem4[];
    __shared__ TopkShared sh;
    float4* gring = smem4;
    constexpr int kStages = TkStages<ACCUM>::value;
    float4* uslot = smem4 + (ACCUM ? (size_t)kStages * kRowF4 : 0);
    unsigned short* table = reinterpret_cast<unsigned short*>(smem4 + (size_t)kTkSmemRows * kRowF4);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int c = blockIdx.x, G = gridDim.x;
    const int64_t n4 = d >> 2;
    unsigned int* ghist1 = ghist;
    unsigned int* ghist2 = ghist + 2048;
    unsigned int* ghist3 = ghist + 3072;

    // this CTA's rows: local row r is row c + r * G of the vector (at most kTkTableMaxRows of
    // them); only the last row of the vector can be short
    const int nrows = c < n_rows ? (n_rows - c + G - 1) / G : 0;
    const int64_t stride4 = (int64_t)G * kRowF4;
    const int64_t first4 = (int64_t)c * kRowF4 + tid;
    const int first_kept = nrows > u_slots ? nrows - u_slots : 0;  // rows from here on stay on chip
    const bool owns_tail = (c == G - 1) && (w == kFusedWarps - 1) && (lane < (int)(d & 3));
    const int64_t tail_i = (n4 << 2) + lane;
    const float4* s4 = reinterpret_cast<const float4*>(src);
    float4* e4 = reinterpret_cast<float4*>(eps);
    const float4* uglob = ACCUM ? reinterpret_cast<const float4*>(eps) : s4;  // where u is after pass 1
    float tail_u = 0.f;
    const bool wide_ok = ACCUM && ((reinterpret_cast<uintptr_t>(eps) & 31u) == 0);

    if (c == 0 && tid == 0) {
        ctrl->stats.status = GK_DEV_OK;
        ctrl->phase_t[0] = global_timer_ns();
        if (nnz_out != nullptr) *nnz_out = k;
    }
    for (int b = tid; b < kTkBins; b += kFusedThreads) sh.hist[b] = 0u;
    if (tid == 0) { sh.need = (unsigned long long)k; sh.digit = 0u; sh.n_staged = 0u; }
    __syncthreads();

    // up to kTkGroupRows rows of this warp whose table entry is pending (want_pending) or
    // non-zero, from `cursor` on; they are left in sh.qrow[w]
    auto gather = [&](int& cursor, const bool want_pending) -> int {
        return want_pending ? gather_cells<kGatherPending>(table, nrows, cursor, sh.qrow[w])
                            : gather_cells<kGatherNonZero>(table, nrows, cursor, sh.qrow[w]);
    };
    // this thread's float4 of local row r (zeros beyond the end of the vector)
    auto load_row = [&](int r) -> float4 {
        const int64_t i = first4 + (int64_t)r * stride4;
        if (i >= n4) return make_float4(0.f, 0.f, 0.f, 0.f);
        return (r >= first_kept) ? uslot[(size_t)(r % u_slots) * kRowF4 + tid] : __ldcg(uglob + i);
    };
    // body(r, v, in_range) for every marked segment of this warp, rows gathered eight at a time
    // so that their loads overlap
#define TK_FOR_EACH_MARKED(want_pending, ...)                                       \
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

    // ------------------------------------------------------------------ pass 1
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
        for (int r = 0; r < nrows; ++r, i += stride4) {
            fetch(r + kStages - 1);
            cp_async_wait<kStages - 1>();
            const bool one = i < n4;
            float4 u0 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (one) {
                float4* us = uslot + (size_t)(r % u_slots) * kRowF4 + tid;
                u0 = *us;
                if (ACCUM) {
                    const float4 a0 = gring[(size_t)(r % kStages) * kRowF4 + tid];
                    u0 = make_float4(a0.x + u0.x, a0.y + u0.y, a0.z + u0.z, a0.w + u0.w);
                    *us = u0;
                }
                atomicAdd(&sh.hist[tk_key(u0.x) >> 20], 1u);
                atomicAdd(&sh.hist[tk_key(u0.y) >> 20], 1u);
                atomicAdd(&sh.hist[tk_key(u0.z) >> 20], 1u);
                atomicAdd(&sh.hist[tk_key(u0.w) >> 20], 1u);
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
            // largest magnitude of each (row, warp) segment, top 16 bits rounded up
            const unsigned int m0 = __reduce_max_sync(0xffffffffu, one ? max_mag_bits(u0) : 0u);
            if (lane == 0) table[r * kFusedWarps + w] = (unsigned short)((m0 + 0xffffu) >> 16);
        }
        cp_async_wait<0>();
        if (owns_tail) {
            tail_u = ACCUM ? src[tail_i] + eps[tail_i] : src[tail_i];
            if (ACCUM) eps[tail_i] = tail_u;
            atomicAdd(&sh.hist[tk_key(tail_u) >> 20], 1u);
        }
        __syncthreads();
        merge_hist(ghist1, 2048, sh);
        if (c == 0 && tid == 0) ctrl->phase_t[1] = global_timer_ns();
        if (!grid_barrier(&bars[0], (unsigned)G, &sh.ok)) {
            if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
            goto leave;
        }
        pick_digit(ghist1, 2048, sh);
    }

    {
        const unsigned int b1 = sh.digit;
        // a segment can hold a key with first digit >= b1 only if its recorded maximum
        // (top 16 bits, rounded up) reaches b1's lower bound; the others are never read again
        const unsigned int low16 = b1 << 4;
        for (int r = lane; r < nrows; r += 32) {
            const bool ql = table[r * kFusedWarps + w] >= low16;
            table[r * kFusedWarps + w] = ql ? kTkPending : (unsigned short)0;
        }
        if (c == 0 && tid == 0) ctrl->phase_t[2] = global_timer_ns();
        __syncthreads();

        // -------------------------------------------------------------- pass 2
        TK_FOR_EACH_MARKED(true, {
            if (in) {
                const unsigned int key[4] = {tk_key(v.x), tk_key(v.y), tk_key(v.z), tk_key(v.w)};
#pragma unroll
                for (int t = 0; t < 4; ++t)
                    if ((key[t] >> 20) == b1) atomicAdd(&sh.hist[(key[t] >> 10) & 1023u], 1u);
            }
        })
        if (owns_tail && (tk_key(tail_u) >> 20) == b1) atomicAdd(&sh.hist[(tk_key(tail_u) >> 10) & 1023u], 1u);
        __syncthreads();
        merge_hist(ghist2, 1024, sh);
        if (!grid_barrier(&bars[1], (unsigned)G, &sh.ok)) {
            if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
            goto leave;
        }
        // every CTA has read the first level's merged bins before it arrived here
        if (c == 0) for (int b = tid; b < 2048; b += kFusedThreads) ghist1[b] = 0u;
        pick_digit(ghist2, 1024, sh);
        const unsigned int p21 = (b1 << 10) | sh.digit;
        if (c == 0 && tid == 0) ctrl->phase_t[3] = global_timer_ns();

        // -------------------------------------------------------------- pass 3
        TK_FOR_EACH_MARKED(true, {
            if (in) {
                const unsigned int key[4] = {tk_key(v.x), tk_key(v.y), tk_key(v.z), tk_key(v.w)};
#pragma unroll
                for (int t = 0; t < 4; ++t)
                    if ((key[t] >> 10) == p21) atomicAdd(&sh.hist[key[t] & 1023u], 1u);
            }
        })
        if (owns_tail && (tk_key(tail_u) >> 10) == p21) atomicAdd(&sh.hist[tk_key(tail_u) & 1023u], 1u);
        __syncthreads();
        merge_hist(ghist3, 1024, sh);
        if (!grid_barrier(&bars[2], (unsigned)G, &sh.ok)) {
            if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
            goto leave;
        }
        if (c == 0) for (int b = tid; b < 1024; b += kFusedThreads) ghist2[b] = 0u;
        pick_digit(ghist3, 1024, sh);
        const unsigned int T = (p21 << 10) | sh.digit;
        const unsigned long long need_eq = sh.need;  // >= 1: entries equal to T to take, lowest indices first
        if (c == 0 && tid == 0) {
            ctrl->key_threshold = T;
            ctrl->need_eq = need_eq;
            ctrl->phase_t[4] = global_timer_ns();
        }

        // ---------------------------------------------------------- compaction
        // step 1: every warp counts the keys above / equal to T of its marked segments; the
        // table entry becomes (above) | (equal << 8), at most 128 each
        // The places of the entries counted here -- row, warp, lane, element, above or equal, and
        // their ranks among the segment's keys above and equal to T -- are put aside in shared
        // memory, two words each, as long as they fit: the write-out is then one thread per
        // entry instead of one warp per segment.
        unsigned int* st_ent = ACCUM ? reinterpret_cast<unsigned int*>(gring)
                                     : reinterpret_cast<unsigned int*>(smem4 + (size_t)(kTkSmemRows - kTkStageRows) * kRowF4);
        constexpr unsigned int kStageCap = (ACCUM ? kStages : kTkStageRows) * kRowBytes / 8;
        const unsigned int lanes_below = (1u << lane) - 1u;
        TK_FOR_EACH_MARKED(true, {
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
        // step 2: per row (thread t takes local row t) the two counts go to the row's words in
        // global memory; every row of the vector gets them from the CTA that owns it
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
        if (!grid_barrier(&bars[3], (unsigned)G, &sh.ok)) {
            if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
            goto leave;
        }
        if (c == 0) for (int b = tid; b < 1024; b += kFusedThreads) ghist3[b] = 0u;
        if (c == 0 && tid == 0) ctrl->phase_t[5] = global_timer_ns();
        const bool tail_cta = (c == G - 1) && (d & 3);
        unsigned long long all_rows = 0ull;  // keys above / equal to T in all rows (tail CTA only)
        if (any_mine || tail_cta) {
            // Keys above / equal to T before local row r of this CTA = those of the rounds before r
            // (round r is the G consecutive rows r * G ... r * G + G - 1) + those of the CTAs
            // before this one in round r.  Warp j takes rounds j, j + 32, ...; a count pair
            // travels as one 64-bit word (above in the low half, equal in the high half).
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
            // exclusive scan of the round totals (thread t takes round t; at most kTkTableMaxRows).
            // CTA 0 owns a row of every round, so its number of rows is the number of rounds; the
            // tail CTA may own one row fewer and then adds the last round separately.
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
                    if ((long long)pos < k) {
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
            TK_FOR_EACH_MARKED(false, {
                unsigned int gm = 0u, em = 0u;
                if (in) {
                    const unsigned int key[4] = {tk_key(v.x), tk_key(v.y), tk_key(v.z), tk_key(v.w)};
#pragma unroll
                    for (int t = 0; t < 4; ++t) { gm |= (unsigned)(key[t] > T) << t; em |= (unsigned)(key[t] == T) << t; }
                }
                // counts of this row in the warps before this one, then in the lanes before this one
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
                            if ((long long)pos < k) {
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
            // rounds this CTA has no row in (the last one, possibly) are missing from its scan
            unsigned long long extra = 0ull;
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
            const unsigned int key = tk_key(tail_u);
            const bool isg = owns_tail && key > T, ise = owns_tail && key == T;
            const unsigned int bg = __ballot_sync(0xffffffffu, isg), be = __ballot_sync(0xffffffffu, ise);
            const unsigned int below = (1u << lane) - 1u;
            const unsigned long long ng = (tot & 0xffffffffull) + __popc(bg & below);
            const unsigned long long ne = (tot >> 32) + __popc(be & below);
            if (isg || (ise && ne < need_eq)) {
                const unsigned long long pos = ng + (ne < need_eq ? ne : need_eq);
                if ((long long)pos < k) {
                    idx_out[pos] = (int32_t)tail_i;
                    val_out[pos] = tail_u;
                    if (ACCUM) eps[tail_i] = 0.0f;
                }
            }
        }
    }
#undef TK_FOR_EACH_MARKED
    if (c == 0 && tid == 0) ctrl->phase_t[6] = global_timer_ns();

leave:
    // the CTA that leaves last clears the barrier counters for the next call
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(&bars[4], 1u);
        if (t == (unsigned)G - 1) {
            ctrl->phase_t[7] = global_timer_ns();
            bars[0] = 0u; bars[1] = 0u; bars[2] = 0u; bars[3] = 0u;
            // (no fence: the end of the kernel orders these stores before the next launch on this
            // stream, the only reader)
            bars[4] = 0u;
        }
    }
}

// Host side -----------------------------------------------------------------
struct TopkPlan {
    bool ready = false, usable = false;
    int grid = 0;
};
static TopkPlan g_tk_plan[64];

template <bool ACCUM>
static bool topk_kernel_ready(int sm_count) {
    if (cudaFuncSetAttribute(k_topk_fused<ACCUM>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTkSmemBytes) !=
        cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_topk_fused<ACCUM>, kFusedThreads, kTkSmemBytes) !=
            cudaSuccess || occ < 1) {
        cudaGetLastError();
        return false;
    }
    (void)sm_count;
    return true;
}

static TopkPlan* topk_plan(int dev, int sm_count) {
    if (dev < 0 || dev >= 64) return nullptr;
    // built once per device, under a lock: a second thread's first call waits for the finished plan
    static std::mutex plan_mu;
    std::lock_guard<std::mutex> plan_lock(plan_mu);
    TopkPlan& p = g_tk_plan[dev];
    if (p.ready) return &p;
    p.ready = true;
    int coop = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return &p;
    if (!topk_kernel_ready<false>(sm_count) || !topk_kernel_ready<true>(sm_count)) return &p;
    p.grid = sm_count < kFusedGridCap ? sm_count : kFusedGridCap;
    p.usable = true;
    return &p;
}

// Returns GK_OK when the fused kernel was enqueued, 1 when it cannot serve this call (the
// caller then takes the multi-kernel path), or an error.  With eps != nullptr: src = g and
// u = g + eps is formed, stored over eps and cleared where selected; else src = u, read-only.
int enqueue_topk_fused(Workspace* ws, const float* src, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                       float* val_out, int64_t* nnz_out, cudaStream_t st) {
    int dev = 0;
    GK_CUDA_TRY(cudaGetDevice(&dev));
    TopkPlan* p = topk_plan(dev, ws->sm_count);
    if (!p || !p->usable) return 1;
    // With more than one selected entry per 128-element segment on average nearly every
    // segment is read again in every later pass, through gathers; on large vectors the
    // streaming passes of the multi-kernel form are then faster (measured: from about 2^25).
    if (k * 128 > d && d > (int64_t(1) << 25)) return 1;
    const int64_t n4 = d >> 2;
    const int64_t rows = (n4 + kRowF4 - 1) / kRowF4;
    int64_t G = rows < p->grid ? rows : p->grid;
    if (G < 1) G = 1;
    int64_t most = (rows + G - 1) / G;  // rows of CTA 0
    if (most < 1) most = 1;
    if (most > kTkTableMaxRows) return 1;
    int n_rows = (int)rows;
    const bool accum = eps != nullptr;
    // a slot is reused kStages - 1 rows later at the earliest: u_slots >= kStages in both forms
    // with u given there is no g ring to reuse: two rows are set aside for the places of the selected entries
    int u_slots = accum ? kTkSmemRows - TkStages<true>::value : kTkSmemRows - kTkStageRows;
    static_assert(kTkSmemRows - TkStages<true>::value >= TkStages<true>::value && kTkSmemRows - kTkStageRows >= TkStages<false>::value,
                  "not enough row slots for the rows in flight");
    if (u_slots > most) u_slots = (int)most;
    Ctrl* ctrl = ws->ctrl;
    unsigned int* ghist = ws->hist;
    uint2* rowcnt = reinterpret_cast<uint2*>(ws->rowcnt);
    unsigned int* bars = ws->bars + 4;  // the sparsifier's fused kernel owns the first four counters
    void* args[] = {(void*)&src, (void*)&eps, (void*)&d, (void*)&k, (void*)&n_rows, (void*)&u_slots, (void*)&ctrl,
                    (void*)&ghist, (void*)&rowcnt, (void*)&bars, (void*)&idx_out, (void*)&val_out,
                    (void*)&nnz_out};
    static_assert(sizeof(args) / sizeof(args[0]) == 13, "k_topk_fused takes 13 arguments");
    stage_mark(ws, st, 0);
    const void* fn = accum ? (const void*)k_topk_fused<true> : (const void*)k_topk_fused<false>;
    GK_CUDA_TRY(cudaLaunchCooperativeKernel(fn, dim3((unsigned)G), dim3(kFusedThreads), args, (size_t)kTkSmemBytes, st));
    note_launch();
    stage_mark(ws, st, 1);
    ws->last_grid = (int)G;
    ws->last_fused = false;
    ws->phase_spans = 7;
    return GK_OK;
}

}  // namespace gk
