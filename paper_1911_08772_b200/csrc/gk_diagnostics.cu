// gk_error_ratio: the compression error ratio the paper analyses (Eq. 5 and
// Section 3.2): ||u - Comp(u)||^2 / ||u||^2, to be held against the classical
// bound 1 - k/d (Eq. 4) and the bound (1 - k/d)^2 that the paper derives for
// bell-shaped u (Theorem 1).
//
// After a sparsification step eps holds u - Comp(u) (selected slots are zero)
// and val the selected entries, so ||u||^2 = ||eps||^2 + ||val||^2: one pass
// over eps (4 d bytes) and the short list, whatever compressor produced them.
//
// Deterministic: a fixed grid, every CTA sums its strided share in fp64 in a
// fixed order, the CTA that retires last adds the per-CTA partials in a fixed
// order.
#include "gk_common.cuh"

namespace gk {

constexpr int kDiagThreads = 512;

__global__ void __launch_bounds__(kDiagThreads)
k_error_ratio(const float* __restrict__ eps, int64_t d, const float* __restrict__ val,
              const int64_t* __restrict__ nnz, Ctrl* __restrict__ ctrl, double2* __restrict__ partials) {
    __shared__ double2 red[kDiagThreads / 32];
    __shared__ bool is_last;
    const int tid = threadIdx.x, c = blockIdx.x, G = gridDim.x;
    const int64_t gtid = (int64_t)c * kDiagThreads + tid, gstride = (int64_t)G * kDiagThreads;
    const int64_t n4 = d >> 2;
    const float4* e4 = reinterpret_cast<const float4*>(eps);
    double e0 = 0.0, e1 = 0.0;
    for (int64_t i = gtid; i < n4; i += 4 * gstride) {
        float4 a[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t ii = i + j * gstride;
            a[j] = ii < n4 ? ld_stream(e4 + ii) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            e0 = fma((double)a[j].x, (double)a[j].x, e0); e1 = fma((double)a[j].y, (double)a[j].y, e1);
            e0 = fma((double)a[j].z, (double)a[j].z, e0); e1 = fma((double)a[j].w, (double)a[j].w, e1);
        }
    }
    if (gtid < (d & 3)) {
        const double x = (double)eps[(n4 << 2) + gtid];
        e0 = fma(x, x, e0);
    }
    int64_t m = *nnz;
    if (m < 0) m = 0;
    double v0 = 0.0;
    for (int64_t i = gtid; i < m; i += gstride) {
        const double x = (double)val[i];
        v0 = fma(x, x, v0);
    }
    const double2 part = block_sum2<kDiagThreads>(e0 + e1, v0, red);
    if (tid == 0) {
        partials[c] = part;
        __threadfence();
        const unsigned int t = atomicAdd(&ctrl->ticket_a, 1u);
        is_last = (t == (unsigned)G - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // thread t adds partials t, t + 512, ... in that order; then the fixed-order block sum
    double e = 0.0, v = 0.0;
    for (int i = tid; i < G; i += kDiagThreads) {
        const double2 p = __ldcg(&partials[i]);
        e += p.x; v += p.y;
    }
    const double2 tot = block_sum2<kDiagThreads>(e, v, red);
    if (tid == 0) {
        ctrl->diag[0] = (tot.x + tot.y) > 0.0 ? tot.x / (tot.x + tot.y) : 0.0;
        ctrl->diag[1] = tot.x;
        ctrl->diag[2] = tot.x + tot.y;
        ctrl->ticket_a = 0u;
    }
}

// ---------------------------------------------------------------------------
// gk_histogram: the histogram of u the paper's gradient-distribution figures
// show (Section 3.1, Fig. 2; the running sum over d is the cumulative curve of
// the appendix).  nbins equal bins from lo, one count below, one above:
//     t = (u_i - lo) * inv_w in fp32 (one subtraction, one multiplication),
//     bin = floor(t);  t < 0: below;  t >= nbins or NaN: above.
// One pass over u (4 d bytes): a shared-memory histogram per CTA, merged with
// 64-bit global atomics (integers: the order does not matter).
// ---------------------------------------------------------------------------
constexpr int kHistThreads = 512;
constexpr int kHistMaxBins = 8192;

__device__ __forceinline__ int hist_slot(float x, float lo, float inv_w, int nbins) {
    const float t = __fmul_rn(__fsub_rn(x, lo), inv_w);
    if (t < 0.0f) return 0;
    if (!(t < (float)nbins)) return nbins + 1;
    return 1 + __float2int_rd(t);
}

__global__ void __launch_bounds__(kHistThreads)
k_histogram(const float* __restrict__ u, int64_t d, float lo, float inv_w, int nbins,
            unsigned long long* __restrict__ counts) {
    extern __shared__ unsigned int hist_sm[];   // nbins + 2
    const int tid = threadIdx.x;
    for (int b = tid; b < nbins + 2; b += kHistThreads) hist_sm[b] = 0u;
    __syncthreads();
    const int64_t gtid = (int64_t)blockIdx.x * kHistThreads + tid, gstride = (int64_t)gridDim.x * kHistThreads;
    const int64_t n4 = d >> 2;
    const float4* u4 = reinterpret_cast<const float4*>(u);
    for (int64_t i = gtid; i < n4; i += 4 * gstride) {
        float4 a[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t ii = i + j * gstride;
            if (ii < n4) a[j] = ld_stream(u4 + ii);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (i + j * gstride < n4) {
                atomicAdd(&hist_sm[hist_slot(a[j].x, lo, inv_w, nbins)], 1u);
                atomicAdd(&hist_sm[hist_slot(a[j].y, lo, inv_w, nbins)], 1u);
                atomicAdd(&hist_sm[hist_slot(a[j].z, lo, inv_w, nbins)], 1u);
                atomicAdd(&hist_sm[hist_slot(a[j].w, lo, inv_w, nbins)], 1u);
            }
        }
    }
    if (gtid < (d & 3)) atomicAdd(&hist_sm[hist_slot(u[(n4 << 2) + gtid], lo, inv_w, nbins)], 1u);
    __syncthreads();
    for (int b = tid; b < nbins + 2; b += kHistThreads) {
        const unsigned int c = hist_sm[b];
        if (c) atomicAdd(&counts[b], (unsigned long long)c);
    }
}

}  // namespace gk

using namespace gk;

extern "C" int gk_histogram(const float* u, int64_t d, float lo, float inv_w, int32_t nbins, int64_t* counts_out,
                            gk_stream_t stream) {
    if (!u || !counts_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll || nbins < 1 || nbins > kHistMaxBins) return GK_ERR_SIZE;
    if (!(inv_w > 0.0f)) return GK_ERR_SIZE;
    if ((uintptr_t)u & 15u) return GK_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    Workspace* ws = nullptr;
    const int wrc = acquire_workspace(1, 1, st, &ws);
    if (wrc != GK_OK) return wrc;
    GK_CUDA_TRY(cudaMemsetAsync(counts_out, 0, sizeof(int64_t) * (size_t)(nbins + 2), st));
    const int64_t n4 = d >> 2;
    int64_t grid = (n4 + 4 * kHistThreads - 1) / (4 * kHistThreads);
    if (grid < 1) grid = 1;
    // a few CTAs per SM: each per-element cost is one shared-memory atomic, the merge is per CTA
    if (grid > (int64_t)ws->sm_count * 4) grid = (int64_t)ws->sm_count * 4;
    stage_mark(ws, st, 0);
    k_histogram<<<(int)grid, kHistThreads, sizeof(unsigned int) * (size_t)(nbins + 2), st>>>(
        u, d, lo, inv_w, nbins, reinterpret_cast<unsigned long long*>(counts_out));
    GK_CUDA_TRY(cudaGetLastError());
    note_launch();
    stage_mark(ws, st, 1);
    ws->last_fused = false;
    ws->phase_spans = 0;
    return GK_OK;
}

extern "C" int gk_error_ratio(const float* eps, int64_t d, const float* val, const int64_t* nnz,
                              gk_stream_t stream, double* host_out) {
    if (!eps || !val || !nnz || !host_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll) return GK_ERR_SIZE;
    if ((uintptr_t)eps & 15u) return GK_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    Workspace* ws = nullptr;
    const int wrc = acquire_workspace(d, 1, st, &ws);
    if (wrc != GK_OK) return wrc;
    const int64_t n4 = d >> 2;
    int64_t grid = (n4 + 4 * kDiagThreads - 1) / (4 * kDiagThreads);
    if (grid < 1) grid = 1;
    if (grid > (int64_t)ws->sm_count * 4) grid = (int64_t)ws->sm_count * 4;
    if (grid > kMaxPartials) grid = kMaxPartials;
    stage_mark(ws, st, 0);
    k_error_ratio<<<(int)grid, kDiagThreads, 0, st>>>(eps, d, val, nnz, ws->ctrl, ws->partials);
    GK_CUDA_TRY(cudaGetLastError());
    note_launch();
    stage_mark(ws, st, 1);
    ws->last_fused = false;
    ws->phase_spans = 0;
    GK_CUDA_TRY(cudaStreamSynchronize(st));
    GK_CUDA_TRY(cudaMemcpy(host_out, ws->ctrl->diag, 3 * sizeof(double), cudaMemcpyDeviceToHost));
    return GK_OK;
}
