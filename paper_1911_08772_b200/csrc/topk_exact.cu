// topk_exact: the Top_k operator of Section 1 of arXiv 1911.08772 -- the k
// entries of largest magnitude with their indices -- by most-significant-digit
// radix select on the 31 magnitude bits of the fp32 pattern (for finite
// floats the order of |x| is the order of those bits as integers).
//
//   three histogram passes (11 + 10 + 10 bits) in shared memory, each followed,
//   in the CTA that retires last, by the choice of the digit that holds the
//   k-th largest key; after the third pass the full threshold key T and the
//   number of entries equal to T that still fit are known;
//   one ordered compaction pass: keys above T are all taken, keys equal to T in
//   order of increasing index until k pairs are out.
#include "gk_common.cuh"
#include "gk_compact.cuh"

namespace gk {

constexpr int kHistThreads = 512;
constexpr int kHistUnroll = 4;
constexpr int kHistBins = 2048;

__device__ __forceinline__ unsigned int mag_key(float x) { return __float_as_uint(x) & 0x7fffffffu; }

// PASS 0: digit = key[30:20]; PASS 1: key[19:10] among keys whose top 11 bits
// equal the prefix; PASS 2: key[9:0] among keys whose top 21 bits equal it.
template <int PASS>
__global__ void __launch_bounds__(kHistThreads)
k_radix_histogram(const float* __restrict__ u, int64_t d, int64_t k, Ctrl* __restrict__ ctrl,
                  unsigned int* __restrict__ ghist, unsigned long long* __restrict__ tile_status,
                  int n_tiles) {
    constexpr int SHIFT = PASS == 0 ? 20 : PASS == 1 ? 10 : 0;
    constexpr int BITS = PASS == 0 ? 11 : 10;
    constexpr int NB = 1 << BITS;
    constexpr int PSHIFT = SHIFT + BITS;  // bits above the digit form the prefix
    __shared__ unsigned int sh[kHistBins];
    __shared__ unsigned int s_part[kHistThreads];
    __shared__ bool is_last;
    const int tid = threadIdx.x;
    for (int b = tid; b < NB; b += kHistThreads) sh[b] = 0u;
    const int64_t gtid = (int64_t)blockIdx.x * kHistThreads + tid;
    const int64_t gstride = (int64_t)gridDim.x * kHistThreads;
    if (PASS == 0) {
        for (int64_t t = gtid; t < n_tiles; t += gstride) tile_status[t] = 0ull;
    }
    const unsigned int prefix = PASS == 0 ? 0u : ctrl->key_prefix;
    __syncthreads();

    const int64_t n4 = d >> 2;
    const float4* u4 = reinterpret_cast<const float4*>(u);
    for (int64_t i = gtid; i < n4; i += gstride * kHistUnroll) {
        float4 v[kHistUnroll];
#pragma unroll
        for (int j = 0; j < kHistUnroll; ++j) {
            const int64_t ii = i + j * gstride;
            v[j] = (ii < n4) ? __ldg(u4 + ii) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < kHistUnroll; ++j) {
            const int64_t ii = i + j * gstride;
            if (ii < n4) {
                const unsigned int key[4] = {mag_key(v[j].x), mag_key(v[j].y), mag_key(v[j].z), mag_key(v[j].w)};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    if (PASS == 0 || (key[t] >> PSHIFT) == prefix)
                        atomicAdd(&sh[(key[t] >> SHIFT) & (NB - 1)], 1u);
                }
            }
        }
    }
    if (blockIdx.x == 0 && tid < (int)(d & 3)) {
        const unsigned int key = mag_key(u[(n4 << 2) + tid]);
        if (PASS == 0 || (key >> PSHIFT) == prefix) atomicAdd(&sh[(key >> SHIFT) & (NB - 1)], 1u);
    }
    __syncthreads();
    for (int b = tid; b < NB; b += kHistThreads) {
        const unsigned int c = sh[b];
        if (c) atomicAdd(&ghist[b], c);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned int t = atomicAdd(&ctrl->ticket_h, 1u);
        is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();

    // Choose the digit: the largest D with  sum_{b > D} hist[b] < need <= sum_{b >= D} hist[b].
    const unsigned long long need = PASS == 0 ? (unsigned long long)k : ctrl->need;
    constexpr int PER = kHistBins / kHistThreads;  // bins per thread (4)
    unsigned int loc[PER];
    unsigned int mine = 0u;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        const int b = tid * PER + j;
        loc[j] = (b < NB) ? __ldcg(&ghist[b]) : 0u;
        if (b < NB) ghist[b] = 0u;  // leave the histogram clear for the next pass / call
        mine += loc[j];
    }
    // suffix sums over threads (counts fit 32 bits: d < 2^31)
    s_part[tid] = mine;
    __syncthreads();
    for (int o = 1; o < kHistThreads; o <<= 1) {
        const unsigned int add = (tid + o < kHistThreads) ? s_part[tid + o] : 0u;
        __syncthreads();
        s_part[tid] += add;
        __syncthreads();
    }
    const unsigned long long above_mine = (tid + 1 < kHistThreads) ? s_part[tid + 1] : 0u;
    if (above_mine < need && need <= above_mine + mine) {
        unsigned long long above = above_mine;
        for (int j = PER - 1; j >= 0; --j) {
            if (need <= above + loc[j]) {
                const unsigned int digit = (unsigned int)(tid * PER + j);
                const unsigned int np = (prefix << BITS) | digit;
                ctrl->key_prefix = np;
                ctrl->need = need - above;
                if (PASS == 2) {
                    ctrl->key_threshold = np;
                    ctrl->need_eq = need - above;
                }
                break;
            }
            above += loc[j];
        }
    }
    if (tid == 0) ctrl->ticket_h = 0u;
}

// Ordered compaction for the exact path.  gt: key > T, eq: key == T.  An entry
// goes out at position (#gt before it) + min(#eq before it, need_eq); eq
// entries only while #eq before it < need_eq.
template <bool CLEAR>
__global__ void __launch_bounds__(kCompactThreads)
k_compact_topk(float* __restrict__ u, int64_t d, Ctrl* __restrict__ ctrl,
               unsigned long long* __restrict__ tile_status, int n_tiles,
               int32_t* __restrict__ idx_out, float* __restrict__ val_out, int persistent) {
    __shared__ TileScanSmem scan;
    __shared__ int s_tile;
    __shared__ LookbackSmem lb;
    __shared__ unsigned int s_tail_gt, s_tail_eq;
    const int tid = threadIdx.x;
    const unsigned int T = ctrl->key_threshold;
    const unsigned long long need_eq = ctrl->need_eq;
    // persistent: cooperative launch, CTA b takes tiles b, b + grid, ...; else one ticketed tile
    for (int pass = 0;; ++pass) {
    if (persistent) {
        if ((int64_t)blockIdx.x + (int64_t)pass * gridDim.x >= n_tiles) break;
        if (tid == 0) { s_tile = (int)(blockIdx.x + pass * gridDim.x); s_tail_gt = 0u; s_tail_eq = 0u; }
    } else {
        if (pass > 0) break;
        if (tid == 0) {
            s_tile = (int)atomicAdd(&ctrl->tile_ticket, 1u);
            s_tail_gt = 0u;
            s_tail_eq = 0u;
        }
    }
    __syncthreads();
    const int tile = s_tile;
    const int64_t n4 = d >> 2;
    const int64_t base4 = (int64_t)tile * (kCompactThreads * kCompactRows);
    const float4* u4 = reinterpret_cast<const float4*>(u);

    float4 v[kCompactRows];
#pragma unroll
    for (int j = 0; j < kCompactRows; ++j) {
        const int64_t i4 = base4 + j * kCompactThreads + tid;
        v[j] = (i4 < n4) ? __ldcs(u4 + i4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    unsigned int mgt = 0u, meq = 0u, cg[kCompactRows], ce[kCompactRows], og[kCompactRows], oe[kCompactRows];
#pragma unroll
    for (int j = 0; j < kCompactRows; ++j) {
        const int64_t i4 = base4 + j * kCompactThreads + tid;
        unsigned int g = 0u, e = 0u;
        if (i4 < n4) {
            const unsigned int key[4] = {mag_key(v[j].x), mag_key(v[j].y), mag_key(v[j].z), mag_key(v[j].w)};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                g |= (unsigned)(key[t] > T) << t;
                e |= (unsigned)(key[t] == T) << t;
            }
        }
        cg[j] = __popc(g); ce[j] = __popc(e);
        mgt |= g << (4 * j); meq |= e << (4 * j);
    }
    const bool owns_tail = (tile == n_tiles - 1) && (tid == kCompactThreads - 1) && (d & 3);
    float tailv[3] = {0.f, 0.f, 0.f};
    unsigned int tail_gt = 0u, tail_eq = 0u;
    if (owns_tail) {
        for (int t = 0; t < (int)(d & 3); ++t) {
            tailv[t] = u[(n4 << 2) + t];
            const unsigned int key = mag_key(tailv[t]);
            tail_gt |= (unsigned)(key > T) << t;
            tail_eq |= (unsigned)(key == T) << t;
        }
        s_tail_gt = __popc(tail_gt);
        s_tail_eq = __popc(tail_eq);
    }
    const unsigned int tot_gt = tile_scan(cg, og, scan);
    const unsigned int tot_eq = tile_scan(ce, oe, scan);
    const unsigned long long agg =
        (unsigned long long)(tot_gt + s_tail_gt) | ((unsigned long long)(tot_eq + s_tail_eq) << 31);
    const unsigned long long excl = lookback_block(tile_status, tile, agg, &ctrl->stats.status, lb);
    const unsigned long long pre_gt = excl & 0x7fffffffull;
    const unsigned long long pre_eq = excl >> 31;

    if (mgt | meq) {
#pragma unroll
        for (int j = 0; j < kCompactRows; ++j) {
            const unsigned int g = (mgt >> (4 * j)) & 0xfu, e = (meq >> (4 * j)) & 0xfu;
            if (g | e) {
                const int64_t e0 = (base4 + j * kCompactThreads + tid) << 2;
                unsigned long long ng = pre_gt + og[j], ne = pre_eq + oe[j];
                const float vv[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const bool isg = g & (1u << t), ise = e & (1u << t);
                    if (isg || (ise && ne < need_eq)) {
                        const unsigned long long pos = ng + (ne < need_eq ? ne : need_eq);
                        idx_out[pos] = (int32_t)(e0 + t);
                        val_out[pos] = vv[t];
                        if (CLEAR) u[e0 + t] = 0.0f;
                    }
                    ng += isg; ne += ise;
                }
            }
        }
    }
    if (owns_tail && (tail_gt | tail_eq)) {
        unsigned long long ng = pre_gt + tot_gt, ne = pre_eq + tot_eq;
        for (int t = 0; t < (int)(d & 3); ++t) {
            const bool isg = tail_gt & (1u << t), ise = tail_eq & (1u << t);
            if (isg || (ise && ne < need_eq)) {
                const unsigned long long pos = ng + (ne < need_eq ? ne : need_eq);
                idx_out[pos] = (int32_t)((n4 << 2) + t);
                val_out[pos] = tailv[t];
                if (CLEAR) u[(n4 << 2) + t] = 0.0f;
            }
            ng += isg; ne += ise;
        }
    }
    if (tile == n_tiles - 1 && tid == 0) ctrl->tile_ticket = 0u;
    __syncthreads();  // shared arrays are reused by the next tile
    }
}

// u = g + eps stored over eps (Eq. 2), no statistics.
__global__ void __launch_bounds__(512)
k_accumulate_only(const float* __restrict__ g, float* __restrict__ eps, int64_t d, Ctrl* ctrl,
                  int64_t* nnz_out, int64_t k) {
    const int64_t gtid = (int64_t)blockIdx.x * 512 + threadIdx.x;
    const int64_t gstride = (int64_t)gridDim.x * 512;
    const int64_t n4 = d >> 2;
    const float4* g4 = reinterpret_cast<const float4*>(g);
    float4* e4 = reinterpret_cast<float4*>(eps);
    for (int64_t i = gtid; i < n4; i += gstride) {
        const float4 a = ld_stream(g4 + i), b = ld_stream(e4 + i);
        e4[i] = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
    }
    if (gtid < (d & 3)) {
        const int64_t i = (n4 << 2) + gtid;
        eps[i] = g[i] + eps[i];
    }
    if (gtid == 0) { ctrl->stats.status = GK_DEV_OK; *nnz_out = k; }
}

static int hist_grid(const Workspace* ws, int64_t d) {
    const int64_t n4 = d >> 2;
    int64_t want = (n4 + (int64_t)kHistThreads * kHistUnroll - 1) / ((int64_t)kHistThreads * kHistUnroll);
    if (want < 1) want = 1;
    const int64_t cap = (int64_t)ws->sm_count * 4;
    return (int)(want < cap ? want : cap);
}

template <bool CLEAR>
static int enqueue_topk(Workspace* ws, float* u, int64_t d, int64_t k, int32_t* idx_out, float* val_out,
                        cudaStream_t st, int ev0) {
    const int n_tiles = (int)num_compact_tiles(d);
    const int grid = hist_grid(ws, d);
    stage_mark(ws, st, ev0);
    k_radix_histogram<0><<<grid, kHistThreads, 0, st>>>(u, d, k, ws->ctrl, ws->hist, ws->tile_status, n_tiles);
    stage_mark(ws, st, ev0 + 1);
    k_radix_histogram<1><<<grid, kHistThreads, 0, st>>>(u, d, k, ws->ctrl, ws->hist, ws->tile_status, n_tiles);
    stage_mark(ws, st, ev0 + 2);
    k_radix_histogram<2><<<grid, kHistThreads, 0, st>>>(u, d, k, ws->ctrl, ws->hist, ws->tile_status, n_tiles);
    stage_mark(ws, st, ev0 + 3);
    GK_CUDA_TRY(launch_compaction(k_compact_topk<CLEAR>, n_tiles, ws->sm_count, st, u, d, ws->ctrl, ws->tile_status,
                                  n_tiles, idx_out, val_out));
    stage_mark(ws, st, ev0 + 4);
    note_launch(4);
    GK_CUDA_TRY(cudaGetLastError());
    return GK_OK;
}

}  // namespace gk

using namespace gk;

extern "C" int topk_exact(const float* u, int64_t d, int64_t k, int32_t* idx_out, float* val_out,
                          gk_stream_t stream) {
    if (!u || !idx_out || !val_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll) return GK_ERR_SIZE;
    if (k < 1 || k > d) return GK_ERR_K;
    if ((uintptr_t)u & 15u) return GK_ERR_ALIGN;
    Workspace* ws = nullptr;
    const int wrc = acquire_workspace(d, 1, (cudaStream_t)stream, &ws);
    if (wrc != GK_OK) return wrc;
    if (selected_path() == 0) {
        const int frc = enqueue_topk_fused(ws, u, nullptr, d, k, idx_out, val_out, nullptr, (cudaStream_t)stream);
        if (frc != 1) return frc;  // 1: the single-kernel form cannot serve this call
    }
    ws->phase_spans = 0;
    return enqueue_topk<false>(ws, const_cast<float*>(u), d, k, idx_out, val_out, (cudaStream_t)stream, 0);
}

extern "C" int topk_sparsify(const float* g, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                             float* val_out, int64_t* nnz_out, gk_stream_t stream) {
    if (!g || !eps || !idx_out || !val_out || !nnz_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll) return GK_ERR_SIZE;
    if (k < 1 || k > d) return GK_ERR_K;
    if (((uintptr_t)g & 15u) || ((uintptr_t)eps & 15u)) return GK_ERR_ALIGN;
    const uintptr_t a = (uintptr_t)g, b = (uintptr_t)eps, n = (uintptr_t)d * 4u;
    if (a < b + n && b < a + n) return GK_ERR_ALIAS;
    cudaStream_t st = (cudaStream_t)stream;
    Workspace* ws = nullptr;
    const int wrc = acquire_workspace(d, 1, st, &ws);
    if (wrc != GK_OK) return wrc;
    if (selected_path() == 0) {
        const int frc = enqueue_topk_fused(ws, g, eps, d, k, idx_out, val_out, nnz_out, st);
        if (frc != 1) return frc;
    }
    ws->phase_spans = 0;
    const int64_t n4 = d >> 2;
    int64_t grid = (n4 + 511) / 512;
    if (grid < 1) grid = 1;
    if (grid > (int64_t)ws->sm_count * 8) grid = (int64_t)ws->sm_count * 8;
    stage_mark(ws, st, 0);
    k_accumulate_only<<<(int)grid, 512, 0, st>>>(g, eps, d, ws->ctrl, nnz_out, k);
    note_launch();
    return enqueue_topk<true>(ws, eps, d, k, idx_out, val_out, st, 1);
}
