// gk_sparsify: error-compensated Gaussian_k sparsification of one vector
// (Eq. 2 and Algorithm 1 of arXiv 1911.08772) in three streaming kernels.
//
//   accumulate_stats   u = g + eps, stored over eps; block partials of
//                      sum(u - c) and sum((u - c)^2) in fp64; the CTA that
//                      retires last reduces the partials in a fixed order and
//                      forms mu, sigma, thres0 and the ten candidate thresholds.
//   count_candidates   one read of u: #{|u| > cand} for all ten candidates;
//                      the last CTA replays Algorithm 1's decisions on the
//                      counts and fixes the threshold of the returned mask.
//   compact            one read of u: ordered (index, value) pairs of the
//                      survivors by decoupled look-back; their eps slots are
//                      cleared, which makes eps = u - Comp(u).
#include <math.h>

#include "gk_alg1.cuh"
#include "gk_common.cuh"
#include "gk_compact.cuh"
#include "gk_compact_threshold.cuh"

namespace gk {

constexpr int kAccThreads = 512;
constexpr int kAccUnroll = 2;   // float4 pairs in flight per thread
constexpr int kCntThreads = 512;
constexpr int kCntUnroll = 4;

__device__ __forceinline__ Alg1State state_of(Ctrl* ctrl) {
    return Alg1State{&ctrl->stats, ctrl->cand64, ctrl->cand32, ctrl->counts, &ctrl->thr_sel};
}

// ---------------------------------------------------------------------------
// Kernel A.  Grid-stride over float4; every CTA writes one partial.  ACC: u = g + eps is
// formed and stored over eps; !ACC: g is the vector u itself and nothing is stored.
// ---------------------------------------------------------------------------
template <bool ACC>
__global__ void __launch_bounds__(kAccThreads)
k_accumulate_stats(const float* __restrict__ g, float* __restrict__ eps, int64_t d, int64_t k, double z,
                   Ctrl* __restrict__ ctrl, double2* __restrict__ partials,
                   unsigned long long* __restrict__ tile_status, int n_tiles) {
    __shared__ double2 red[kAccThreads / 32];
    __shared__ bool is_last;
    const int tid = threadIdx.x;
    const int64_t gtid = (int64_t)blockIdx.x * kAccThreads + tid;
    const int64_t gstride = (int64_t)gridDim.x * kAccThreads;

    // clear the look-back words the compaction kernel will use
    for (int64_t t = gtid; t < n_tiles; t += gstride) tile_status[t] = 0ull;

    const double c = (double)g[0];  // pivot: keeps the one-pass variance well conditioned
    const int64_t n4 = d >> 2;
    const float4* g4 = reinterpret_cast<const float4*>(g);
    float4* e4 = reinterpret_cast<float4*>(eps);
    double s0 = 0.0, q0 = 0.0, s1 = 0.0, q1 = 0.0;

    for (int64_t i = gtid; i < n4; i += gstride * kAccUnroll) {
        float4 a[kAccUnroll], b[kAccUnroll];
#pragma unroll
        for (int j = 0; j < kAccUnroll; ++j) {
            const int64_t ii = i + j * gstride;
            if (ii < n4) {
                a[j] = ld_stream(g4 + ii);
                b[j] = ACC ? ld_stream(e4 + ii) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int j = 0; j < kAccUnroll; ++j) {
            const int64_t ii = i + j * gstride;
            if (ii < n4) {
                float4 u = a[j];
                if (ACC) {
                    u.x = a[j].x + b[j].x; u.y = a[j].y + b[j].y;
                    u.z = a[j].z + b[j].z; u.w = a[j].w + b[j].w;
                    e4[ii] = u;
                }
                const double x0 = (double)u.x - c, x1 = (double)u.y - c;
                const double x2 = (double)u.z - c, x3 = (double)u.w - c;
                s0 += x0; q0 = fma(x0, x0, q0);
                s1 += x1; q1 = fma(x1, x1, q1);
                s0 += x2; q0 = fma(x2, x2, q0);
                s1 += x3; q1 = fma(x3, x3, q1);
            }
        }
    }
    // ragged tail (d not a multiple of 4)
    if (blockIdx.x == 0 && tid < (int)(d & 3)) {
        const int64_t i = (n4 << 2) + tid;
        const float u = ACC ? g[i] + eps[i] : g[i];
        if (ACC) eps[i] = u;
        const double x = (double)u - c;
        s0 += x; q0 = fma(x, x, q0);
    }

    const double2 part = block_sum2<kAccThreads>(s0 + s1, q0 + q1, red);
    if (tid == 0) {
        partials[blockIdx.x] = part;
        __threadfence();
        const unsigned int t = atomicAdd(&ctrl->ticket_a, 1u);
        is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // fixed-order reduction of the partials: thread t takes t, t + T, ...; then the block tree
    double s = 0.0, q = 0.0;
    for (int i = tid; i < (int)gridDim.x; i += kAccThreads) {
        const double2 p = __ldcg(&partials[i]);
        s += p.x; q += p.y;
    }
    const double2 tot = block_sum2<kAccThreads>(s, q, red);
    if (tid == 0) {
        alg1_thresholds(state_of(ctrl), tot.x, tot.y, c, d, k, z);
        ctrl->ticket_a = 0u;
    }
}

// ---------------------------------------------------------------------------
// Kernel B.  Per-thread counters for the ten candidates, reduced with
// redux.sync / shared atomics / one global atomic per candidate per CTA.
// Integer sums: the result does not depend on the order.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kCntThreads)
k_count_candidates(const float* __restrict__ u, int64_t d, int64_t k, Ctrl* __restrict__ ctrl) {
    __shared__ unsigned int s_cnt[kNumCand];
    __shared__ bool is_last;
    const int tid = threadIdx.x;
    if (tid < kNumCand) s_cnt[tid] = 0u;
    float cand[kNumCand];
#pragma unroll
    for (int j = 0; j < kNumCand; ++j) cand[j] = ctrl->cand32[j];
    unsigned int cnt[kNumCand];
#pragma unroll
    for (int j = 0; j < kNumCand; ++j) cnt[j] = 0u;

    const int64_t n4 = d >> 2;
    const float4* u4 = reinterpret_cast<const float4*>(u);
    const int64_t gtid = (int64_t)blockIdx.x * kCntThreads + tid;
    const int64_t gstride = (int64_t)gridDim.x * kCntThreads;
    for (int64_t i = gtid; i < n4; i += gstride * kCntUnroll) {
        float4 v[kCntUnroll];
#pragma unroll
        for (int j = 0; j < kCntUnroll; ++j) {
            const int64_t ii = i + j * gstride;
            v[j] = (ii < n4) ? __ldg(u4 + ii) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < kCntUnroll; ++j) {
            const int64_t ii = i + j * gstride;
            if (ii < n4) {
                const float a0 = fabsf(v[j].x), a1 = fabsf(v[j].y), a2 = fabsf(v[j].z), a3 = fabsf(v[j].w);
#pragma unroll
                for (int c = 0; c < kNumCand; ++c)
                    cnt[c] += (unsigned)(a0 > cand[c]) + (unsigned)(a1 > cand[c]) +
                              (unsigned)(a2 > cand[c]) + (unsigned)(a3 > cand[c]);
            }
        }
    }
    if (blockIdx.x == 0 && tid < (int)(d & 3)) {
        const float a = fabsf(u[(n4 << 2) + tid]);
#pragma unroll
        for (int c = 0; c < kNumCand; ++c) cnt[c] += (unsigned)(a > cand[c]);
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < kNumCand; ++c) {
        const unsigned int w = __reduce_add_sync(0xffffffffu, cnt[c]);
        if ((tid & 31) == 0 && w) atomicAdd(&s_cnt[c], w);
    }
    __syncthreads();
    if (tid < kNumCand && s_cnt[tid]) {
        atomicAdd(&ctrl->counts[tid], (unsigned long long)s_cnt[tid]);
        __threadfence();
    }
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(&ctrl->ticket_b, 1u);
        is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    if (tid == 0) {
        __threadfence();
        alg1_resolve(state_of(ctrl), k);
        ctrl->ticket_b = 0u;
    }
}

static int check_vectors(const float* g, float* eps, int64_t d, int64_t k, const void* idx_out,
                         const void* val_out, const void* nnz_out) {
    if (!g || !eps || !idx_out || !val_out || !nnz_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll) return GK_ERR_SIZE;
    if (k < 1 || k > d) return GK_ERR_K;
    if (((uintptr_t)g & 15u) || ((uintptr_t)eps & 15u)) return GK_ERR_ALIGN;
    const uintptr_t a = (uintptr_t)g, b = (uintptr_t)eps, n = (uintptr_t)d * 4u;
    if (a < b + n && b < a + n) return GK_ERR_ALIAS;
    return GK_OK;
}

static int reduction_grid(const Workspace* ws, int64_t d, int threads, int unroll, int ctas_per_sm) {
    const int64_t n4 = d >> 2;
    int64_t want = (n4 + (int64_t)threads * unroll - 1) / ((int64_t)threads * unroll);
    if (want < 1) want = 1;
    int64_t cap = (int64_t)ws->sm_count * ctas_per_sm;
    if (cap > kMaxPartials) cap = kMaxPartials;
    return (int)(want < cap ? want : cap);
}

// Enqueue the three-kernel (look-back) path on an already validated call.  eps == nullptr:
// the operator form (src = u, read only).
int enqueue_gk_three_kernel(Workspace* ws, const float* src, float* eps, int64_t d, int64_t k,
                        int32_t* idx_out, float* val_out, int64_t* nnz_out, cudaStream_t st) {
    const int n_tiles = (int)num_compact_tiles(d);
    double z = -INFINITY;
    if (k < d) {
        const double p = 1.0 - (double)k / (double)d;  // Algorithm 1: p = 1 - k/d
        z = normal_quantile_upper(1.0 - p);
    }
    const int grid_a = reduction_grid(ws, d, kAccThreads, kAccUnroll, 4);
    stage_mark(ws, st, 0);
    if (eps != nullptr)
        k_accumulate_stats<true><<<grid_a, kAccThreads, 0, st>>>(src, eps, d, k, z, ws->ctrl, ws->partials,
                                                                 ws->tile_status, n_tiles);
    else
        k_accumulate_stats<false><<<grid_a, kAccThreads, 0, st>>>(src, nullptr, d, k, z, ws->ctrl, ws->partials,
                                                                  ws->tile_status, n_tiles);
    note_launch();
    stage_mark(ws, st, 1);
    float* uvec = eps != nullptr ? eps : const_cast<float*>(src);   // the operator form never writes it
    if (k < d) {
        const int grid_b = reduction_grid(ws, d, kCntThreads, kCntUnroll, 4);
        k_count_candidates<<<grid_b, kCntThreads, 0, st>>>(uvec, d, k, ws->ctrl);
        note_launch();
    }
    stage_mark(ws, st, 2);
    if (eps != nullptr)
        GK_CUDA_TRY(launch_compaction(k_compact_threshold<false, true>, n_tiles, ws->sm_count, st, uvec, d, ws->ctrl,
                                      ws->tile_status, n_tiles, idx_out, val_out, nnz_out, output_capacity(d),
                                      (const int64_t*)nullptr, 0, (const float*)nullptr));
    else
        GK_CUDA_TRY(launch_compaction(k_compact_threshold<false, false>, n_tiles, ws->sm_count, st, uvec, d, ws->ctrl,
                                      ws->tile_status, n_tiles, idx_out, val_out, nnz_out, output_capacity(d),
                                      (const int64_t*)nullptr, 0, (const float*)nullptr));
    note_launch();
    stage_mark(ws, st, 3);
    ws->last_fused = false;
    ws->phase_spans = 0;
    GK_CUDA_TRY(cudaGetLastError());
    return GK_OK;
}

// Enqueue one step by the selected path: the cluster kernel for small vectors, else the fused
// cooperative kernel, unless they cannot be used on this device (or for this call), else the
// three-kernel path.
// eps == nullptr: the operator form on src = u.
int enqueue_gk_sparsify(Workspace* ws, const float* src, float* eps, int64_t d, int64_t k,
                        int32_t* idx_out, float* val_out, int64_t* nnz_out, cudaStream_t st) {
    if (selected_path() == 0) {
        const int rc = enqueue_gk_small(ws, src, eps, d, k, idx_out, val_out, nnz_out, st);
        if (rc != 1) return rc;
    }
    if (selected_path() != 1) {
        const int rc = enqueue_gk_fused(ws, src, eps, d, k, idx_out, val_out, nnz_out, st);
        if (rc != 1) return rc;
    }
    return enqueue_gk_three_kernel(ws, src, eps, d, k, idx_out, val_out, nnz_out, st);
}

}  // namespace gk

extern "C" int gk_sparsify(const float* g, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                           float* val_out, int64_t* nnz_out, gk_stream_t stream) {
    const int rc = gk::check_vectors(g, eps, d, k, idx_out, val_out, nnz_out);
    if (rc != GK_OK) return rc;
    gk::Workspace* ws = nullptr;
    const int wrc = gk::acquire_workspace(d, 1, (cudaStream_t)stream, &ws);
    if (wrc != GK_OK) return wrc;
    return gk::enqueue_gk_sparsify(ws, g, eps, d, k, idx_out, val_out, nnz_out, (cudaStream_t)stream);
}

extern "C" int gk_select(const float* u, int64_t d, int64_t k, int32_t* idx_out, float* val_out,
                         int64_t* nnz_out, gk_stream_t stream) {
    if (!u || !idx_out || !val_out || !nnz_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll) return GK_ERR_SIZE;
    if (k < 1 || k > d) return GK_ERR_K;
    if ((uintptr_t)u & 15u) return GK_ERR_ALIGN;
    gk::Workspace* ws = nullptr;
    const int wrc = gk::acquire_workspace(d, 1, (cudaStream_t)stream, &ws);
    if (wrc != GK_OK) return wrc;
    return gk::enqueue_gk_sparsify(ws, u, nullptr, d, k, idx_out, val_out, nnz_out, (cudaStream_t)stream);
}
