// gk_sparsify_segmented: Algorithm 1 of arXiv 1911.08772 run independently on
// every contiguous segment of the vector (layer-wise selection), with one
// batched launch per stage for all segments.
//
// Every CTA of the two reduction kernels owns a contiguous run of float4 and
// walks the spans in which that run meets the segments.  Per-span partial sums
// go to slot (cta + segment): along the vector both indices only grow, so the
// slot is unique, and the slots of one segment are consecutive CTAs, which the
// finalising CTA adds in ascending order -- the statistics do not depend on
// scheduling.  Candidate counts are integer atomics.  The compaction pass is
// the whole-vector one with a per-element threshold lookup.
#include <math.h>

#include "gk_alg1.cuh"
#include "gk_common.cuh"
#include "gk_compact.cuh"
#include "gk_compact_threshold.cuh"
#include "gk_count.cuh"
#include "gk_segmented.cuh"

namespace gk {

constexpr int kSegThreads = 512;
constexpr int kSegWindow = 128;  // segments whose scalars a CTA keeps in shared memory at a time

struct Span {
    int64_t lo, hi;      // elements [lo, hi)
    int64_t a_lo, a_hi;  // the float4-aligned interior [a_lo, a_hi)
};

__device__ __forceinline__ Span make_span(int64_t lo, int64_t hi) {
    Span s;
    s.lo = lo; s.hi = hi;
    int64_t a = (lo + 3) & ~(int64_t)3;
    if (a > hi) a = hi;
    int64_t b = hi & ~(int64_t)3;
    if (b < a) b = a;
    s.a_lo = a; s.a_hi = b;
    return s;
}

// Elements [lo, hi) owned by CTA c: float4 groups [c * r4, (c + 1) * r4), the
// last CTA also takes the d mod 4 trailing elements.
__device__ __forceinline__ void cta_range(int c, int G, int64_t r4, int64_t d, int64_t* lo, int64_t* hi) {
    const int64_t n4 = d >> 2;
    int64_t a = (int64_t)c * r4, b = a + r4;
    if (a > n4) a = n4;
    if (b > n4) b = n4;
    *lo = a << 2;
    *hi = (c == G - 1) ? d : (b << 2);
}
__device__ __forceinline__ int owner_cta(int64_t i, int G, int64_t r4) {
    const int64_t c = (i >> 2) / r4;
    return (int)(c < G - 1 ? c : G - 1);
}

__device__ __forceinline__ Alg1State seg_state(const SegScratch& v, int s) {
    return Alg1State{&v.stats[s], v.cand64 + (size_t)s * kNumCand, v.cand32 + (size_t)s * kNumCand,
                     v.counts + (size_t)s * kNumCand, &v.thr_sel[s]};
}

// ---------------------------------------------------------------------------
// Stage 1: u = g + eps over eps; per-span sums; last CTA: per-segment thresholds.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kSegThreads)
k_seg_accumulate_stats(const float* __restrict__ g, float* __restrict__ eps, int64_t d, int64_t r4,
                       const int64_t* __restrict__ off, const int64_t* __restrict__ seg_k, int S,
                       Ctrl* __restrict__ ctrl, SegScratch v, unsigned long long* __restrict__ tile_status,
                       int n_tiles) {
    __shared__ double2 red[kSegThreads / 32];
    __shared__ bool is_last;
    const int tid = threadIdx.x, c = blockIdx.x, G = gridDim.x;
    for (int64_t t = (int64_t)c * kSegThreads + tid; t < n_tiles; t += (int64_t)G * kSegThreads)
        tile_status[t] = 0ull;

    // the normal quantiles depend only on (k_s, d_s): thread t of CTA c takes segment c + t * G
    // now, while the other threads stream, so that the finalising CTA only has to read them
    {
        const int64_t q = (int64_t)c + (int64_t)tid * G;
        if (q < S) {
            const int64_t n = off[q + 1] - off[q];
            int64_t kk = seg_k[q];
            if (kk > n) kk = n;
            double zq = -INFINITY;
            if (n > 0 && kk >= 1 && kk < n) {
                const double p = 1.0 - (double)kk / (double)n;  // Algorithm 1: p = 1 - k/d
                zq = normal_quantile_upper(1.0 - p);
            }
            v.zs[q] = zq;
        }
    }
    int64_t lo, hi;
    cta_range(c, G, r4, d, &lo, &hi);
    const float4* g4 = reinterpret_cast<const float4*>(g);
    float4* e4 = reinterpret_cast<float4*>(eps);
    int s = (lo < hi) ? find_segment(off, S, lo) : S;
    int64_t cur = lo;
    // offsets and pivots of the next kSegWindow segments are fetched together into shared
    // memory, so that a run crossing many short segments does not pay a chain of global
    // round trips for each of them
    __shared__ int64_t w_off[kSegWindow + 1];
    __shared__ double w_piv[kSegWindow];
    int w0 = -kSegWindow;  // first segment of the window (none loaded yet)
    while (cur < hi && s < S) {
        if (s >= w0 + kSegWindow) {
            __syncthreads();
            w0 = s;
            if (tid <= kSegWindow) w_off[tid] = off[(w0 + tid) <= S ? (w0 + tid) : S];
            if (tid < kSegWindow) {
                int64_t pi = off[(w0 + tid) < S ? (w0 + tid) : S - 1];
                if (pi < 0 || pi >= d) pi = lo;
                w_piv[tid] = (double)g[pi];  // the segment's pivot
            }
            __syncthreads();
        }
        const int64_t seg_end = w_off[s - w0 + 1];
        const int64_t sp_hi = seg_end < hi ? seg_end : hi;
        if (sp_hi > cur) {
            const Span sp = make_span(cur, sp_hi);
            const double pv = w_piv[s - w0];
            double sum = 0.0, sq = 0.0;
            // unaligned head and tail of the span: one element per thread
            const int nh = (int)(sp.a_lo - sp.lo), nt = (int)(sp.hi - sp.a_hi);
            if (tid < nh || (tid >= 32 && tid < 32 + nt)) {
                const int64_t i = tid < nh ? sp.lo + tid : sp.a_hi + (tid - 32);
                const float u = g[i] + eps[i];
                eps[i] = u;
                const double x = (double)u - pv;
                sum += x; sq = fma(x, x, sq);
            }
            double sum1 = 0.0, sq1 = 0.0;
            const int64_t i4_hi = sp.a_hi >> 2;
            for (int64_t i4 = (sp.a_lo >> 2) + tid; i4 < i4_hi; i4 += 2 * kSegThreads) {
                const int64_t j4 = i4 + kSegThreads;
                const bool two = j4 < i4_hi;
                const float4 a0 = ld_stream(g4 + i4), b0 = ld_stream(e4 + i4);
                float4 a1, b1;
                if (two) { a1 = ld_stream(g4 + j4); b1 = ld_stream(e4 + j4); }
                float4 u0 = make_float4(a0.x + b0.x, a0.y + b0.y, a0.z + b0.z, a0.w + b0.w);
                e4[i4] = u0;
                double x0 = (double)u0.x - pv, x1 = (double)u0.y - pv, x2 = (double)u0.z - pv, x3 = (double)u0.w - pv;
                sum += x0; sq = fma(x0, x0, sq); sum1 += x1; sq1 = fma(x1, x1, sq1);
                sum += x2; sq = fma(x2, x2, sq); sum1 += x3; sq1 = fma(x3, x3, sq1);
                if (two) {
                    float4 u1 = make_float4(a1.x + b1.x, a1.y + b1.y, a1.z + b1.z, a1.w + b1.w);
                    e4[j4] = u1;
                    x0 = (double)u1.x - pv; x1 = (double)u1.y - pv; x2 = (double)u1.z - pv; x3 = (double)u1.w - pv;
                    sum += x0; sq = fma(x0, x0, sq); sum1 += x1; sq1 = fma(x1, x1, sq1);
                    sum += x2; sq = fma(x2, x2, sq); sum1 += x3; sq1 = fma(x3, x3, sq1);
                }
            }
            const double2 part = block_sum2<kSegThreads>(sum + sum1, sq + sq1, red);
            if (tid == 0) v.partials[c + s] = part;
            cur = sp_hi;
        }
        if (cur >= seg_end) ++s;
    }
    // elements past the last segment boundary (malformed table only) still receive u
    if (cur < hi) {
        for (int64_t i = cur + tid; i < hi; i += kSegThreads) eps[i] = g[i] + eps[i];
    }

    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(&ctrl->ticket_a, 1u);
        is_last = (t == (unsigned)G - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();

    // per-segment finalisation, one thread per segment
    int bad = 0;
    if (tid == 0 && (off[0] != 0 || off[S] != d)) bad = 1;
    for (int q = tid; q < S; q += kSegThreads) {
        const int64_t a = off[q], b = off[q + 1];
        if (a < 0 || b > d || b < a || seg_k[q] < 1) bad = 1;
    }
    bad = __syncthreads_or(bad);
    for (int q = tid; q < S; q += kSegThreads) {
        const Alg1State st = seg_state(v, q);
        const int64_t a = off[q], b = off[q + 1], n = b - a;
        if (bad || n <= 0) {
            gk_stats z0;
            z0.mu = z0.sigma = z0.z = z0.thres0 = z0.thr_final = 0.0;
            for (int i = 0; i < kMaxRounds; ++i) z0.counts[i] = 0;
            z0.rounds = 0; z0.status = bad ? GK_DEV_BAD_SEGMENTS : GK_DEV_OK; z0.nnz = 0; z0.emitted = 0;
            *st.stats = z0;
            *st.thr_sel = INFINITY;  // nothing passes
            for (int i = 0; i < kNumCand; ++i) { st.cand32[i] = INFINITY; st.cand64[i] = INFINITY; st.counts[i] = 0ull; }
            continue;
        }
        const int c0 = owner_cta(a, G, r4), c1 = owner_cta(b - 1, G, r4);
        // the slots of one segment are added in ascending CTA order; loads go out sixteen at a
        // time so that their latencies overlap
        double s1 = 0.0, s2 = 0.0;
        for (int cc = c0; cc <= c1; cc += 16) {
            double2 p[16];
#pragma unroll
            for (int t = 0; t < 16; ++t)
                p[t] = (cc + t <= c1) ? __ldcg(&v.partials[cc + t + q]) : make_double2(0.0, 0.0);
#pragma unroll
            for (int t = 0; t < 16; ++t) { s1 += p[t].x; s2 += p[t].y; }
        }
        int64_t kk = seg_k[q];
        if (kk > n) kk = n;
        const double zq = __ldcg(&v.zs[q]);
        alg1_thresholds(st, s1, s2, (double)g[a], n, kk, zq);
    }
    if (tid == 0) {
        ctrl->stats.status = bad ? GK_DEV_BAD_SEGMENTS : GK_DEV_OK;
        ctrl->stats.emitted = 0;
        ctrl->ticket_a = 0u;
    }
}

// ---------------------------------------------------------------------------
// Stage 2: candidate counts per segment; last CTA: replay of the rounds.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kSegThreads)
k_seg_count_candidates(const float* __restrict__ u, int64_t d, int64_t r4, const int64_t* __restrict__ off,
                       const int64_t* __restrict__ seg_k, int S, Ctrl* __restrict__ ctrl, SegScratch v,
                       int64_t* __restrict__ seg_nnz_out) {
    __shared__ unsigned int s_cnt[kNumCand];
    __shared__ int s_ord[kNumCand];
    __shared__ bool is_last;
    const int tid = threadIdx.x, c = blockIdx.x, G = gridDim.x;
    int64_t lo, hi;
    cta_range(c, G, r4, d, &lo, &hi);
    const float4* u4 = reinterpret_cast<const float4*>(u);
    const bool table_ok = (ctrl->stats.status & GK_DEV_BAD_SEGMENTS) == 0;
    int s = (lo < hi && table_ok) ? find_segment(off, S, lo) : S;
    int64_t cur = lo;
    // per window of kSegWindow segments: end offsets, candidates in ascending order with their
    // indices, and whether the segment needs counting at all; thread t prepares segment w0 + t
    __shared__ int64_t w_end[kSegWindow];
    __shared__ float w_cs[kSegWindow][kNumCand];
    __shared__ unsigned char w_ord[kSegWindow][kNumCand];
    __shared__ bool w_counted[kSegWindow];
    int w0 = -kSegWindow;
    while (cur < hi && s < S) {
        if (s >= w0 + kSegWindow) {
            __syncthreads();
            w0 = s;
            if (tid < kSegWindow && w0 + tid < S) {
                const int q = w0 + tid;
                w_end[tid] = off[q + 1];
                // segments that select everything need no counts
                w_counted[tid] = v.stats[q].thr_final != -INFINITY;
                float cd[kNumCand];
                int od[kNumCand];
#pragma unroll
                for (int j = 0; j < kNumCand; ++j) cd[j] = v.cand32[(size_t)q * kNumCand + j];
                for (int j = 0; j < kNumCand; ++j) {  // insertion sort of the ten thresholds
                    int pos = j;
                    while (pos > 0 && cd[od[pos - 1]] > cd[j]) { od[pos] = od[pos - 1]; --pos; }
                    od[pos] = j;
                }
                for (int j = 0; j < kNumCand; ++j) { w_cs[tid][j] = cd[od[j]]; w_ord[tid][j] = (unsigned char)od[j]; }
            }
            __syncthreads();
        }
        const int ws = s - w0;
        const int64_t seg_end = w_end[ws];
        const int64_t sp_hi = seg_end < hi ? seg_end : hi;
        const bool counted = w_counted[ws];
        if (sp_hi > cur && counted) {
            const Span sp = make_span(cur, sp_hi);
            if (tid < kNumCand) { s_cnt[tid] = 0u; s_ord[tid] = w_ord[ws][tid]; }
            __syncthreads();
            float cs[kNumCand], acc[kNumCand];
#pragma unroll
            for (int j = 0; j < kNumCand; ++j) { cs[j] = w_cs[ws][j]; acc[j] = 0.f; }
            const Tiers tier = make_tiers(cs);
            const bool any_neg = cs[0] < 0.f;
            const int nh = (int)(sp.a_lo - sp.lo), nt = (int)(sp.hi - sp.a_hi);
            if (tid < nh || (tid >= 32 && tid < 32 + nt)) {
                const float a = fabsf(u[tid < nh ? sp.lo + tid : sp.a_hi + (tid - 32)]);
#pragma unroll
                for (int j = 0; j < kNumCand; ++j) acc[j] += gt_as_float(a, cs[j]);
            }
            // the warp's largest magnitude in each row of 32 float4 decides how many tiers to evaluate
            const int64_t i4_hi = sp.a_hi >> 2;
            const int64_t i4_lo = sp.a_lo >> 2;
            const int64_t n_it = (i4_hi - i4_lo + kSegThreads - 1) / kSegThreads;  // same for the whole warp
            for (int64_t it = 0; it < n_it; it += 4) {
                float4 x[4];
                bool in[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int64_t i4 = i4_lo + (it + q) * kSegThreads + tid;
                    in[q] = i4 < i4_hi;
                    x[q] = in[q] ? __ldg(u4 + i4) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    unsigned int rm = (__reduce_max_sync(0xffffffffu, max_mag_bits(x[q])) + 0xffffu) >> 16;
                    if (any_neg) rm = 0x10000u;
                    if (in[q]) count_float4(x[q], rm, cs, tier, acc);
                }
            }
            __syncthreads();
#pragma unroll
            for (int j = 0; j < kNumCand; ++j) {
                const unsigned int w = __reduce_add_sync(0xffffffffu, (unsigned int)acc[j]);
                if ((tid & 31) == 0 && w) atomicAdd(&s_cnt[s_ord[j]], w);
            }
            __syncthreads();
            if (tid < kNumCand && s_cnt[tid]) {
                atomicAdd(&v.counts[(size_t)s * kNumCand + tid], (unsigned long long)s_cnt[tid]);
                __threadfence();
            }
            __syncthreads();
        }
        if (sp_hi > cur) cur = sp_hi;
        if (cur >= seg_end) ++s;
    }
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(&ctrl->ticket_b, 1u);
        is_last = (t == (unsigned)G - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int q = tid; q < S; q += kSegThreads) {
        const int64_t n = off[q + 1] - off[q];
        if (table_ok && n > 0) {
            int64_t kk = seg_k[q];
            if (kk > n) kk = n;
            alg1_resolve(seg_state(v, q), kk);
        }
        if (seg_nnz_out) seg_nnz_out[q] = v.stats[q].nnz;
    }
    if (tid == 0) ctrl->ticket_b = 0u;
}

}  // namespace gk

using namespace gk;

extern "C" int gk_sparsify_segmented(const float* g, float* eps, int64_t d, const int64_t* seg_offsets,
                                     const int64_t* seg_k, int32_t S, int32_t* idx_out, float* val_out,
                                     int64_t* seg_nnz_out, int64_t* nnz_out, gk_stream_t stream) {
    if (!g || !eps || !seg_offsets || !seg_k || !idx_out || !val_out || !nnz_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll || S < 1 || S > kMaxSegments) return GK_ERR_SIZE;
    if (((uintptr_t)g & 15u) || ((uintptr_t)eps & 15u)) return GK_ERR_ALIGN;
    const uintptr_t a = (uintptr_t)g, b = (uintptr_t)eps, n = (uintptr_t)d * 4u;
    if (a < b + n && b < a + n) return GK_ERR_ALIAS;
    cudaStream_t st = (cudaStream_t)stream;
    Workspace* ws = nullptr;
    const int wrc = acquire_workspace(d, S, st, &ws);
    if (wrc != GK_OK) return wrc;
    if (selected_path() == 0) {
        const int frc = enqueue_gk_fused_seg(ws, g, eps, d, seg_offsets, seg_k, S, idx_out, val_out, seg_nnz_out,
                                             nnz_out, st);
        if (frc != 1) return frc;  // 1: the single-kernel form cannot serve this call
    }
    const SegScratch v = segmented_views(ws);
    const int n_tiles = (int)num_compact_tiles(d);
    // contiguous float4 runs of r4 per CTA, no CTA empty
    const int64_t n4 = d >> 2;
    int64_t gmax = (int64_t)ws->sm_count * 2;  // two CTAs of 512 threads are resident per SM: one wave
    if (gmax > kMaxPartials) gmax = kMaxPartials;
    const int64_t min_run = 2 * kSegThreads;  // at least one full iteration per CTA
    int64_t r4 = (n4 + gmax - 1) / gmax;
    if (r4 < min_run) r4 = min_run;
    int64_t G = (n4 + r4 - 1) / r4;
    if (G < 1) G = 1;
    stage_mark(ws, st, 0);
    k_seg_accumulate_stats<<<(int)G, kSegThreads, 0, st>>>(g, eps, d, r4, seg_offsets, seg_k, S, ws->ctrl, v,
                                                           ws->tile_status, n_tiles);
    stage_mark(ws, st, 1);
    k_seg_count_candidates<<<(int)G, kSegThreads, 0, st>>>(eps, d, r4, seg_offsets, seg_k, S, ws->ctrl, v,
                                                           seg_nnz_out);
    stage_mark(ws, st, 2);
    GK_CUDA_TRY(launch_compaction(k_compact_threshold<true>, n_tiles, ws->sm_count, st, eps, d, ws->ctrl,
                                  ws->tile_status, n_tiles, idx_out, val_out, nnz_out, output_capacity(d),
                                  seg_offsets, (int)S, (const float*)v.thr_sel));
    stage_mark(ws, st, 3);
    ws->last_fused = false;
    ws->phase_spans = 0;
    note_launch(3);
    GK_CUDA_TRY(cudaGetLastError());
    return GK_OK;
}
