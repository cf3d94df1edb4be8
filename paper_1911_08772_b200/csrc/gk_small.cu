// gk_sparsify / gk_select for SMALL vectors (Eq. 2 and Algorithm 1 of arXiv 1911.08772) as one
// thread-block cluster.
//
// A vector of a megabyte or two is over before a grid of 148 CTAs has finished its three grid
// barriers (a counter in global memory costs two round trips to L2 per barrier, 1.5-2 us): the
// persistent kernel of gk_fused.cu spends 24 us on 270,000 elements.  Here sixteen CTAs of one
// cluster hold the whole of u in their shared memory (up to nine rows of 1024 float4 each), talk
// through distributed shared memory, and synchronise with the hardware's cluster barrier:
//
//   phase A  CTA c owns rows c R .. c R + R - 1 (contiguous, so that output offsets are a sum over
//            lower ranks); g and eps arrive through a ring of asynchronous copies, u = g + eps goes
//            back over eps and stays in shared memory; fp64 partial sums per CTA; per (row, warp)
//            cell the largest magnitude.
//   cluster barrier; every CTA reads the sixteen partials in rank order and forms mu, sigma,
//            thres0 and the ten candidates for itself.
//   phase B  counts of |u| > candidate for all ten candidates, from shared memory.
//   cluster barrier; every CTA adds the sixteen CTAs' counts and replays the rounds.
//   phase C  survivors per cell, an exclusive scan over the CTA's cells, the CTA totals exchanged
//            through a third cluster barrier; pairs written in index order, slots cleared.
//
// The arithmetic is that of the persistent kernel (same helpers), so the results are identical.
// No global scratch is used but the statistics record.  A cluster barrier is a hardware barrier
// among CTAs that the hardware schedules together: its waits end.
#include <math.h>

#include <mutex>

#include "gk_alg1.cuh"
#include "gk_common.cuh"
#include "gk_coop.cuh"
#include "gk_count.cuh"

namespace gk {

constexpr int kSmallCluster = 16;                   // CTAs of the cluster
constexpr int kSmallMaxRows = 9;                    // rows of 1024 float4 a CTA holds
constexpr int kSmallStages = 4;                     // rows of g in flight, plus one
constexpr int64_t kSmallMaxElems = (int64_t)kSmallCluster * kSmallMaxRows * kRowF4 * 4;   // 589,824
constexpr int kSmallCells = kSmallMaxRows * kFusedWarps;

struct __align__(128) SmallShared {
    double2 red[kFusedWarps];
    double2 part;                        // this CTA's sums, read by the others
    double2 tot;                         // the cluster's sums
    unsigned int before;                 // survivors in the CTAs before this one
    unsigned int cta_counts[kNumCand];   // this CTA's counts, read by the others
    unsigned int total;                  // this CTA's survivors, read by the others
    unsigned long long col[kNumCand];
    double cand64[kNumCand];
    float cand32[kNumCand];
    int order[kNumCand];
    float thr_sel;
    int chosen;
    gk_stats stats;
    unsigned int wsum[kFusedWarps];
    unsigned short maxtab[kSmallCells];  // largest magnitude of each cell (top 16 bits, rounded up)
    unsigned int cellcnt[kSmallCells];   // survivors of each cell, then survivors before it in the CTA
};
constexpr int kSmallSmemBytes = (kSmallMaxRows + kSmallStages) * kRowBytes;
static_assert((sizeof(SmallShared) + 1023) / 1024 * 1024 + kSmallSmemBytes <= 232448, "over the shared memory of one CTA");

// Distributed shared memory and the cluster barrier, in PTX.
__device__ __forceinline__ unsigned int cluster_rank() {
    unsigned int r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address, in the cluster's shared window, of the variable at `p` in CTA `rank` of the cluster.
__device__ __forceinline__ unsigned int remote_shared(const void* p, unsigned int rank) {
    const unsigned int local = (unsigned int)__cvta_generic_to_shared(p);
    unsigned int remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    return remote;
}
__device__ __forceinline__ unsigned int ld_remote_u32(const void* p, unsigned int rank) {
    unsigned int v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(remote_shared(p, rank)) : "memory");
    return v;
}
__device__ __forceinline__ double ld_remote_f64(const void* p, unsigned int rank) {
    double v;
    asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(v) : "r"(remote_shared(p, rank)) : "memory");
    return v;
}

__device__ __forceinline__ unsigned int small_mask_above(const float4 v, const float thr) {
    return (unsigned)(fabsf(v.x) > thr) | ((unsigned)(fabsf(v.y) > thr) << 1) |
           ((unsigned)(fabsf(v.z) > thr) << 2) | ((unsigned)(fabsf(v.w) > thr) << 3);
}

// ACC: the sparsifier (src = g, eps in / out); !ACC: the operator on src = u (eps unused).
// rows_per_cta = R: CTA c of the cluster owns rows c R .. c R + R - 1 of the n_rows rows.
template <bool ACC>
__global__ void __launch_bounds__(kFusedThreads, 1)
k_gk_small(const float* __restrict__ src, float* __restrict__ eps, int64_t d, int64_t k, double z, int n_rows,
           int rows_per_cta, Ctrl* __restrict__ ctrl, int32_t* __restrict__ idx_out, float* __restrict__ val_out,
           int64_t* __restrict__ nnz_out, int64_t cap) {
    extern __shared__ __align__(1024) float4 smem4[];
    __shared__ SmallShared sh;
    float4* gring = smem4;                                        // kSmallStages rows of g
    float4* urow = smem4 + (size_t)kSmallStages * kRowF4;         // rows_per_cta rows of u
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const unsigned int c = cluster_rank();
    const int64_t n4 = d >> 2;
    const int row0 = (int)c * rows_per_cta;
    int nrows = n_rows - row0;
    nrows = nrows < 0 ? 0 : (nrows > rows_per_cta ? rows_per_cta : nrows);
    const int64_t first4 = (int64_t)row0 * kRowF4 + tid;          // this thread's float4 in local row 0
    const bool owns_tail = (c == kSmallCluster - 1) && (w == kFusedWarps - 1) && (lane < (int)(d & 3));
    const int64_t tail_i = (n4 << 2) + lane;
    const float4* g4 = reinterpret_cast<const float4*>(src);
    float4* e4 = reinterpret_cast<float4*>(eps);
    float tail_u = 0.f;
    const double pv = (double)src[0];

    // ------------------------------------------------------------------ phase A
    {
        double s0 = 0.0, q0 = 0.0, s1 = 0.0, q1 = 0.0;
        auto fetch = [&](int r) {
            const int64_t i = first4 + (int64_t)r * kRowF4;
            if (r < nrows && i < n4) {
                if (ACC) {
                    cp_async16(gring + (size_t)(r % kSmallStages) * kRowF4 + tid, g4 + i);
                    cp_async16(urow + (size_t)r * kRowF4 + tid, e4 + i);
                } else {
                    cp_async16(urow + (size_t)r * kRowF4 + tid, g4 + i);
                }
            }
            cp_async_commit();
        };
#pragma unroll
        for (int r = 0; r < kSmallStages - 1; ++r) fetch(r);
        for (int r = 0; r < nrows; ++r) {
            fetch(r + kSmallStages - 1);
            cp_async_wait<kSmallStages - 1>();
            const int64_t i = first4 + (int64_t)r * kRowF4;
            const bool one = i < n4;
            float4 u0 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (one) {
                float4* us = urow + (size_t)r * kRowF4 + tid;
                if (ACC) {
                    const float4 a0 = gring[(size_t)(r % kSmallStages) * kRowF4 + tid], b0 = *us;
                    u0 = make_float4(a0.x + b0.x, a0.y + b0.y, a0.z + b0.z, a0.w + b0.w);
                    *us = u0;
                    e4[i] = u0;
                } else {
                    u0 = *us;
                }
                const double x0 = (double)u0.x - pv, x1 = (double)u0.y - pv, x2 = (double)u0.z - pv,
                             x3 = (double)u0.w - pv;
                s0 += x0; q0 = fma(x0, x0, q0); s1 += x1; q1 = fma(x1, x1, q1);
                s0 += x2; q0 = fma(x2, x2, q0); s1 += x3; q1 = fma(x3, x3, q1);
            } else {
                urow[(size_t)r * kRowF4 + tid] = u0;   // beyond the end of the vector: zeros, so that later phases need no test
            }
            const unsigned int m0 = __reduce_max_sync(0xffffffffu, max_mag_bits(u0));
            if (lane == 0) sh.maxtab[r * kFusedWarps + w] = (unsigned short)((m0 + 0xffffu) >> 16);
        }
        cp_async_wait<0>();
        if (owns_tail) {
            tail_u = ACC ? src[tail_i] + eps[tail_i] : src[tail_i];
            if (ACC) eps[tail_i] = tail_u;
            const double x = (double)tail_u - pv;
            s0 += x; q0 = fma(x, x, q0);
        }
        const double2 part = block_sum2<kFusedThreads>(s0 + s1, q0 + q1, sh.red);
        if (tid == 0) sh.part = part;
        cluster_sync();
        if (w == 0) {
            // lane r fetches CTA r's sums (the loads of all ranks are in flight together); they are
            // then added in rank order, the same in every CTA: identical statistics everywhere
            double ps = 0.0, pq = 0.0;
            if (lane < kSmallCluster) {
                ps = ld_remote_f64(&sh.part.x, (unsigned int)lane);
                pq = ld_remote_f64(&sh.part.y, (unsigned int)lane);
            }
            double s = 0.0, q = 0.0;
#pragma unroll
            for (int r = 0; r < kSmallCluster; ++r) {
                s += __shfl_sync(0xffffffffu, ps, r);
                q += __shfl_sync(0xffffffffu, pq, r);
            }
            if (lane == 0) sh.tot = make_double2(s, q);
        }
        __syncthreads();
        if (tid == 0) {
            const double s = sh.tot.x, q = sh.tot.y;
            const Alg1State st{&sh.stats, sh.cand64, sh.cand32, sh.col, &sh.thr_sel};
            alg1_thresholds(st, s, q, pv, d, k, z);
            const bool neg = sh.stats.thres0 < 0.0;
#pragma unroll
            for (int j = 0; j < kNumCand; ++j) sh.order[j] = cand_ascending(j, neg);
        }
        if (tid < kNumCand) sh.cta_counts[tid] = 0u;
        __syncthreads();
    }

    // ------------------------------------------------------------------ phase B
    {
        float cs[kNumCand], acc[kNumCand];
#pragma unroll
        for (int j = 0; j < kNumCand; ++j) { cs[j] = sh.cand32[sh.order[j]]; acc[j] = 0.f; }
        const Tiers tier = make_tiers(cs);
        const bool any_neg = cs[0] < 0.f;
        for (int r = 0; r < nrows; ++r) {
            const unsigned int rm = any_neg ? 0x10000u : (unsigned int)sh.maxtab[r * kFusedWarps + w];
            // (zeros beyond the end of the vector exceed no candidate unless one is negative)
            if (first4 + (int64_t)r * kRowF4 < n4) count_float4(urow[(size_t)r * kRowF4 + tid], rm, cs, tier, acc);
        }
        if (owns_tail) {
            const float a = fabsf(tail_u);
#pragma unroll
            for (int j = 0; j < kNumCand; ++j) acc[j] += gt_as_float(a, cs[j]);
        }
#pragma unroll
        for (int j = 0; j < kNumCand; ++j) {
            const unsigned int ws = __reduce_add_sync(0xffffffffu, (unsigned int)acc[j]);
            if (lane == 0 && ws) atomicAdd(&sh.cta_counts[sh.order[j]], ws);
        }
        cluster_sync();
        // thread (j, r) fetches CTA r's count of candidate j; sixteen lanes add up one candidate
        if (tid < kNumCand * kSmallCluster) {
            unsigned long long v = ld_remote_u32(&sh.cta_counts[tid / kSmallCluster], (unsigned int)(tid % kSmallCluster));
#pragma unroll
            for (int o = kSmallCluster / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (tid % kSmallCluster == 0) sh.col[tid / kSmallCluster] = v;
        }
        __syncthreads();
        if (tid == 0) {
            const Alg1State st{&sh.stats, sh.cand64, sh.cand32, sh.col, &sh.thr_sel};
            sh.chosen = alg1_resolve(st, k);
        }
        __syncthreads();
    }

    // ------------------------------------------------------------------ phase C
    {
        const float thr = sh.thr_sel;
        const bool all_pass = thr < 0.0f;
        const unsigned int thr16 = __float_as_uint(fmaxf(thr, 0.0f)) >> 16;
        // survivors of each of this warp's cells
        for (int r = 0; r < nrows; ++r) {
            unsigned int cnt = 0u;
            if (all_pass || sh.maxtab[r * kFusedWarps + w] > thr16) {
                const bool in = first4 + (int64_t)r * kRowF4 < n4;
                cnt = __reduce_add_sync(0xffffffffu, in ? __popc(small_mask_above(urow[(size_t)r * kRowF4 + tid], thr)) : 0u);
            }
            if (lane == 0) sh.cellcnt[r * kFusedWarps + w] = cnt;
        }
        __syncthreads();
        // exclusive scan over the CTA's cells in index order (thread t takes cell t)
        {
            const int ncells = nrows * kFusedWarps;
            const unsigned int mine = tid < ncells ? sh.cellcnt[tid] : 0u;
            unsigned int s = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int t = __shfl_up_sync(0xffffffffu, s, o);
                if (lane >= o) s += t;
            }
            if (lane == 31) sh.wsum[w] = s;
            __syncthreads();
            const unsigned int x = sh.wsum[lane];
            unsigned int y = x;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int t = __shfl_up_sync(0xffffffffu, y, o);
                if (lane >= o) y += t;
            }
            const unsigned int wpre = __shfl_sync(0xffffffffu, y - x, w);
            const unsigned int tot = __shfl_sync(0xffffffffu, y, 31);
            if (tid < ncells) sh.cellcnt[tid] = wpre + s - mine;
            if (tid == 0) sh.total = tot;
        }
        cluster_sync();
        // survivors in the CTAs before this one (the ragged tail comes last of all)
        if (w == 0) {
            const unsigned int t = lane < kSmallCluster ? ld_remote_u32(&sh.total, (unsigned int)lane) : 0u;
            const unsigned int b = __reduce_add_sync(0xffffffffu, (unsigned int)lane < c ? t : 0u);
            if (lane == 0) sh.before = b;
        }
        __syncthreads();
        const unsigned long long before = sh.before;
        for (int r = 0; r < nrows; ++r) {
            if (!(all_pass || sh.maxtab[r * kFusedWarps + w] > thr16)) continue;
            const int64_t i = first4 + (int64_t)r * kRowF4;
            const float4 x = urow[(size_t)r * kRowF4 + tid];
            const unsigned int m = i < n4 ? small_mask_above(x, thr) : 0u;
            if (__ballot_sync(0xffffffffu, m != 0u) == 0u) continue;
            // rank of this thread's first survivor within the cell: the survivors of the lanes below
            unsigned int sc = __popc(m);
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int t = __shfl_up_sync(0xffffffffu, sc, o);
                if (lane >= o) sc += t;
            }
            if (m) {
                long long p = (long long)before + sh.cellcnt[r * kFusedWarps + w] + (sc - __popc(m));
                const int64_t e0 = i << 2;
                const float vv[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    if (m & (1u << t)) {
                        if (p < cap) {
                            idx_out[p] = (int32_t)(e0 + t);
                            val_out[p] = vv[t];
                            if (ACC) eps[e0 + t] = 0.0f;
                        }
                        ++p;
                    }
                }
            }
        }
        if ((c == kSmallCluster - 1) && (w == kFusedWarps - 1) && (d & 3)) {
            const bool hit = owns_tail && (fabsf(tail_u) > thr);
            const unsigned int bal = __ballot_sync(0xffffffffu, hit);
            if (hit) {
                const long long p = (long long)sh.stats.nnz - __popc(bal) + __popc(bal & ((1u << lane) - 1u));
                if (p < cap) {
                    idx_out[p] = (int32_t)tail_i;
                    val_out[p] = tail_u;
                    if (ACC) eps[tail_i] = 0.0f;
                }
            }
        }
        if (c == 0 && tid == 0) {
            const long long all = sh.stats.nnz;
            const long long written = all < cap ? all : cap;
            gk_stats o = sh.stats;
            o.emitted = written;
            o.status = sh.stats.status | (all > cap ? GK_DEV_TRUNCATED : 0);
            ctrl->stats = o;
            *nnz_out = written;
        }
    }
    // no CTA may leave while another can still read its shared memory
    cluster_sync();
}

// Host side -----------------------------------------------------------------
struct SmallPlan {
    bool ready = false, usable = false;
};
static SmallPlan g_small_plan[64];

template <bool ACC>
static bool small_kernel_ready() {
    if (cudaFuncSetAttribute(k_gk_small<ACC>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmallSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(k_gk_small<ACC>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    // can the device hold one cluster of this shape at all?
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kSmallCluster);
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = kSmallSmemBytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = kSmallCluster;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, k_gk_small<ACC>, &cfg) != cudaSuccess || clusters < 1) {
        cudaGetLastError();
        return false;
    }
    return true;
}

static SmallPlan* small_plan(int dev) {
    if (dev < 0 || dev >= 64) return nullptr;
    static std::mutex plan_mu;
    std::lock_guard<std::mutex> plan_lock(plan_mu);
    SmallPlan& p = g_small_plan[dev];
    if (p.ready) return &p;
    p.ready = true;
    int cc_major = 0;
    if (cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || cc_major < 9) return &p;
    p.usable = small_kernel_ready<true>() && small_kernel_ready<false>();
    return &p;
}

// Returns GK_OK when the cluster kernel was enqueued, 1 when it cannot serve this call (the
// caller then takes the persistent kernel), or an error.  eps == nullptr: the operator form.
int enqueue_gk_small(Workspace* ws, const float* src, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                     float* val_out, int64_t* nnz_out, cudaStream_t st) {
    if (d > kSmallMaxElems || k >= d) return 1;
    int dev = 0;
    GK_CUDA_TRY(cudaGetDevice(&dev));
    SmallPlan* p = small_plan(dev);
    if (!p || !p->usable) return 1;
    const int64_t n4 = d >> 2;
    int n_rows = (int)((n4 + kRowF4 - 1) / kRowF4);
    int rows_per_cta = (n_rows + kSmallCluster - 1) / kSmallCluster;
    if (rows_per_cta < 1) rows_per_cta = 1;
    if (rows_per_cta > kSmallMaxRows) return 1;
    const double pq = 1.0 - (double)k / (double)d;  // Algorithm 1: p = 1 - k/d
    const double z = normal_quantile_upper(1.0 - pq);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kSmallCluster);
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = (size_t)(rows_per_cta + kSmallStages) * kRowBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = kSmallCluster;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    Ctrl* ctrl = ws->ctrl;
    const int64_t cap = output_capacity(d);
    stage_mark(ws, st, 0);
    if (eps != nullptr)
        GK_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_gk_small<true>, src, eps, d, k, z, n_rows, rows_per_cta, ctrl, idx_out,
                                       val_out, nnz_out, cap));
    else
        GK_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_gk_small<false>, src, (float*)nullptr, d, k, z, n_rows, rows_per_cta,
                                       ctrl, idx_out, val_out, nnz_out, cap));
    note_launch();
    stage_mark(ws, st, 1);
    ws->last_fused = false;
    ws->phase_spans = 0;
    return GK_OK;
}

}  // namespace gk
