// The step that follows the sparsifier in Eq. 2 of arXiv 1911.08772: the model
// update from the P workers' messages,
//     x <- x + alpha * sum_p Comp_k(u^p)         (alpha = -eta / P in the paper).
//
// Every message is the ascending (index, value) list its sparsifier wrote.  The
// lists may sit in one gathered buffer (after an all-gather) or each in its
// owner's memory (peer pointers over NVLink): the kernel only follows the P
// base pointers it is given, with plain loads.
//
// One block per 256 consecutive entries of one list p.  The lists are ascending, so the
// block's entries can only meet a short window of every other list q: the two ends of that
// window are found by 16-way searches (sixteen lanes probe sixteen positions of list q at
// once, a search ends in about five rounds), the windows are copied to shared memory, and
// every thread then looks its own index up there.  The entry of the lowest rank that holds
// index i owns the position: it adds the terms in rank order (fp32, one addition per term),
// multiplies by alpha and adds to x[i].  No atomics, no scratch vector, no zero-filled
// dense sum: only positions that occur in some message are touched, and the result does
// not depend on timing.
#include "gk_common.cuh"

namespace gk {

constexpr int kApplyMaxRanks = 64;
constexpr int kApplyChunk = 8;      // lists searched in lockstep
constexpr int kApplyThreads = 256;

struct ApplyLists {
    const int32_t* idx[kApplyMaxRanks];
    const float* val[kApplyMaxRanks];
};

// First position in [0, n) of the ascending list `a` whose entry is >= target, found by the
// 16 lanes of a half-warp together: every round probes 16 positions that cut the interval
// into 17 parts.  All 32 lanes of the warp must call this (the two halves may search
// different lists).  Safe on unsorted input: the result stays in [0, n].
__device__ __forceinline__ int search16(const int32_t* a, int n, long long target, int lane16, int half) {
    int lo = 0, hi = n;
    while (__any_sync(0xffffffffu, lo < hi)) {
        const long long w = hi - lo;
        const int m = lo + (int)((w * (lane16 + 1)) / 17);     // in [lo, hi) when lo < hi
        const bool below = (lo < hi) && ((long long)a[m] < target);
        const unsigned int bal = (__ballot_sync(0xffffffffu, below) >> (16 * half)) & 0xffffu;
        if (lo < hi) {
            const int c = __popc(bal);                           // probes 0 .. c-1 lie below the target
            const int m_prev = lo + (int)((w * c) / 17);         // probe c - 1
            const int m_next = lo + (int)((w * (c + 1)) / 17);   // probe c
            if (c > 0) lo = m_prev + 1;
            if (c < 16) hi = m_next;
        }
    }
    return lo;
}

constexpr int kApplyWindow = 1024;   // entries of a list's window kept in shared memory

// grid: blocks_per_list blocks for each of the P lists.
__global__ void __launch_bounds__(kApplyThreads)
k_apply_sparse(float* __restrict__ x, int64_t d, const ApplyLists L, const int64_t* __restrict__ nnz, int P,
               int64_t cap, int blocks_per_list, float alpha, int* __restrict__ status) {
    __shared__ int32_t win[kApplyChunk][kApplyWindow];
    __shared__ int win_lo[kApplyChunk], win_hi[kApplyChunk];
    const int tid = threadIdx.x;
    const int p = blockIdx.x / blocks_per_list;
    const int64_t j0 = (int64_t)(blockIdx.x % blocks_per_list) * kApplyThreads;
    long long n_own = nnz[p];
    if (n_own > cap) n_own = cap;
    if (j0 >= n_own) return;                                    // the whole block: nothing here
    const int n_here = (int)(n_own - j0 < kApplyThreads ? n_own - j0 : kApplyThreads);
    const int32_t* own = L.idx[p] + j0;
    const bool live = tid < n_here;
    const int32_t i = live ? own[tid] : 0;
    const bool valid = live && i >= 0 && (int64_t)i < d;
    if (live && !valid) atomicOr(status, GK_DEV_BAD_INDEX);
    const long long first = own[0], last = own[n_here - 1];
    float s = live ? L.val[p][j0 + tid] : 0.f;
    bool owned_below = false;
    const int group = tid >> 4, lane16 = tid & 15, half = (tid >> 4) & 1;
    for (int q0 = 0; q0 < P; q0 += kApplyChunk) {
        // the window of every list of the chunk that can meet this block's entries:
        // half-warp 2t finds its start in list q0 + t, half-warp 2t + 1 its end
        {
            const int q = q0 + (group >> 1);
            int n = 0;
            const int32_t* a = own;
            if (q < P && q != p) {
                long long nq = nnz[q];
                if (nq < 0) nq = 0;
                if (nq > cap) nq = cap;
                n = (int)nq;
                a = L.idx[q];
            }
            const int r = search16(a, n, (group & 1) ? last + 1 : first, lane16, half);
            if (lane16 == 0) { if (group & 1) win_hi[group >> 1] = r; else win_lo[group >> 1] = r; }
        }
        __syncthreads();
#pragma unroll 1
        for (int t = 0; t < kApplyChunk; ++t) {
            const int a0 = win_lo[t], w = win_hi[t] - a0;
            if (w > 0 && w <= kApplyWindow) {
                const int32_t* a = L.idx[q0 + t];
                for (int y = tid; y < w; y += kApplyThreads) win[t][y] = a[a0 + y];
            }
        }
        __syncthreads();
        // every entry looks its index up in the windows, lists in rank order
        int pos[kApplyChunk];
#pragma unroll
        for (int t = 0; t < kApplyChunk; ++t) {
            pos[t] = -1;
            const int a0 = win_lo[t], w = win_hi[t] - a0;
            if (valid && !owned_below && w > 0) {
                int lo = 0, hi = w;
                if (w <= kApplyWindow) {
                    while (lo < hi) {
                        const int mid = lo + ((hi - lo) >> 1);
                        if (win[t][mid] < i) lo = mid + 1; else hi = mid;
                    }
                    if (lo < w && win[t][lo] == i) pos[t] = a0 + lo;
                } else {   // a window too long for shared memory: the same search in the list itself
                    const int32_t* a = L.idx[q0 + t] + a0;
                    while (lo < hi) {
                        const int mid = lo + ((hi - lo) >> 1);
                        if (a[mid] < i) lo = mid + 1; else hi = mid;
                    }
                    if (lo < w && a[lo] == i) pos[t] = a0 + lo;
                }
            }
        }
        float v[kApplyChunk];
#pragma unroll
        for (int t = 0; t < kApplyChunk; ++t) {
            v[t] = 0.f;
            if (pos[t] >= 0) {
                if (q0 + t < p) owned_below = true;   // a lower rank holds i and owns the position
                else v[t] = L.val[q0 + t][pos[t]];
            }
        }
#pragma unroll
        for (int t = 0; t < kApplyChunk; ++t)
            if (pos[t] >= 0 && q0 + t > p) s = __fadd_rn(s, v[t]);   // the higher ranks' terms, in rank order
        __syncthreads();   // the windows are overwritten by the next chunk
    }
    if (valid && !owned_below) x[i] = __fadd_rn(x[i], __fmul_rn(alpha, s));
}

static int enqueue_apply(float* x, int64_t d, const ApplyLists& L, const int64_t* nnz, int32_t P, int64_t cap,
                         float alpha, cudaStream_t st) {
    Workspace* ws = nullptr;
    const int wrc = acquire_workspace(1, 1, st, &ws);
    if (wrc != GK_OK) return wrc;
    GK_CUDA_TRY(cudaMemsetAsync(&ws->ctrl->stats.status, 0, sizeof(int), st));
    const int64_t bpl = (cap + kApplyThreads - 1) / kApplyThreads;   // blocks per list
    const int64_t grid = bpl * P;
    if (grid > 2147483647ll) return GK_ERR_LIMIT;
    stage_mark(ws, st, 0);
    k_apply_sparse<<<(unsigned)grid, kApplyThreads, 0, st>>>(x, d, L, nnz, P, cap, (int)bpl, alpha,
                                                            &ws->ctrl->stats.status);
    GK_CUDA_TRY(cudaGetLastError());
    note_launch();
    stage_mark(ws, st, 1);
    ws->phase_spans = 0;
    return GK_OK;
}

}  // namespace gk

using namespace gk;

extern "C" int gk_apply_sparse(float* x, int64_t d, const int32_t* const* idx_lists, const float* const* val_lists,
                               const int64_t* nnz, int32_t P, int64_t cap, float alpha, gk_stream_t stream) {
    if (!x || !idx_lists || !val_lists || !nnz) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll || P < 1 || P > kApplyMaxRanks || cap < 1 || cap > 2147483647ll) return GK_ERR_SIZE;
    ApplyLists L;
    for (int p = 0; p < kApplyMaxRanks; ++p) {
        L.idx[p] = p < P ? idx_lists[p] : nullptr;
        L.val[p] = p < P ? val_lists[p] : nullptr;
        if (p < P && (!L.idx[p] || !L.val[p])) return GK_ERR_NULL;
    }
    return enqueue_apply(x, d, L, nnz, P, cap, alpha, (cudaStream_t)stream);
}

extern "C" int gk_apply_gathered(float* x, int64_t d, const int32_t* idx, const float* val, const int64_t* nnz,
                                 int32_t P, int64_t cap, float alpha, gk_stream_t stream) {
    if (!x || !idx || !val || !nnz) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll || P < 1 || P > kApplyMaxRanks || cap < 1 || cap > 2147483647ll) return GK_ERR_SIZE;
    ApplyLists L;
    for (int p = 0; p < kApplyMaxRanks; ++p) {
        L.idx[p] = p < P ? idx + (int64_t)p * cap : nullptr;
        L.val[p] = p < P ? val + (int64_t)p * cap : nullptr;
    }
    return enqueue_apply(x, d, L, nnz, P, cap, alpha, (cudaStream_t)stream);
}
