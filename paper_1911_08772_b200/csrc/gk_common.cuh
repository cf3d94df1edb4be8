// Shared declarations of the CUDA library: workspace layout, small device
// helpers, launch bookkeeping.  Internal; the public interface is include/gk.h.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "gk.h"

namespace gk {

// ---------------------------------------------------------------------------
// Algorithm 1 visits at most four thresholds, each thres0 * 0.5^a * 1.5^b with
// a + b <= 3.  Halving is exact in binary floating point, so the ten products
// do not depend on the order of the adjustments and can all be counted in one
// pass.  Candidate (a, b) lives at index cand_index(a, b).
// ---------------------------------------------------------------------------
constexpr int kMaxRounds = 4;
constexpr int kNumCand = 10;
__host__ __device__ constexpr int cand_index(int a, int b) {
    // b = 0: 0..3, b = 1: 4..6, b = 2: 7..8, b = 3: 9
    return (b == 0 ? 0 : b == 1 ? 4 : b == 2 ? 7 : 9) + a;
}

// Compaction tile: kCompactThreads threads, kCompactRows float4 per thread.
constexpr int kCompactThreads = 256;
constexpr int kCompactRows = 8;
constexpr int kCompactTileElems = kCompactThreads * kCompactRows * 4;  // 8192

constexpr int kFusedGridCap = 512;  // upper bound on the grid of the fused kernel
constexpr int kMaxPartials = 4096;  // upper bound on the grid of the reduction kernels

// Bounded waits: polls of a predecessor's status word before giving up.
constexpr int kLookbackPollLimit = 1 << 22;

// Test hooks (gk_debug_set): knobs that let a test reach the give-up branches of the bounded
// waits and both sides of run-time decisions.  The device-side ones live in one variable per
// translation unit (no relocatable device code); each unit registers a setter for its copy.
enum Knob {
    kKnobBarrierPolls = 0,    // polls of a grid barrier before a CTA gives up
    kKnobLookbackPolls = 1,   // polls of a predecessor's status word before a tile gives up
    kKnobExtraArrivals = 2,   // host: arrivals the fused kernels' barriers expect beyond the grid size
    kKnobMuteTile = 3,        // compaction tile that does not publish its status word (-1: none)
    kKnobPrediction = 4,      // host: -1 automatic, 0 never, 1 whenever possible (gk_fused.cu)
    kKnobSelectedWay = 5,     // phase B of the persistent kernel: -1 automatic, 0 never the selected way, 1 thres0 alone selected
    kKnobBiasedStd = 6,       // gk_set_params: 1 divides the variance by d instead of d - 1
    kKnobMaxRounds = 7,       // gk_set_params: rounds of Algorithm 1's loop, 1 .. 4
    kKnobCount = 8
};
typedef int (*KnobSetter)(int key, int value);   // returns a cudaError_t as int
int register_knob_setter(KnobSetter fn);
int host_knob(int key);

// Tile status word of the decoupled look-back: flag in bits 63..62, payload below.
constexpr unsigned long long kFlagShift = 62;
constexpr unsigned long long kFlagAggregate = 1ull;
constexpr unsigned long long kFlagPrefix = 2ull;
constexpr unsigned long long kPayloadMask = (1ull << kFlagShift) - 1ull;

// Control block at the start of every workspace.  Zeroed when the workspace is
// created; the tickets are reset by the CTA that retires last, so every call
// finds them at zero.
struct Ctrl {
    unsigned int ticket_a;     // CTAs of the accumulate kernel that have finished
    unsigned int ticket_b;     // CTAs of the count kernel that have finished
    unsigned int tile_ticket;  // next compaction tile to hand out
    unsigned int ticket_h;     // CTAs of a histogram kernel that have finished
    unsigned long long counts[kNumCand];  // #{|u| > cand}, filled by the count kernel
    double cand64[kNumCand];              // candidate thresholds, fp64
    float cand32[kNumCand];               // the same rounded toward -inf to fp32
    float thr_sel;                        // threshold of the mask to return (fp32, rounded down)
    gk_stats stats;
    // exact Top_k state
    unsigned int key_prefix;       // magnitude bits fixed so far
    unsigned int key_threshold;    // final k-th largest magnitude key
    unsigned long long need;       // how many still to take among keys matching the prefix
    unsigned long long need_eq;    // how many entries equal to the threshold key to take
    // fused kernel: %globaltimer of CTA 0 at its start, after the first barrier and the
    // thresholds, after its counting loop, after the second barrier, after the replay of the
    // rounds, at the end of its compaction; and of the CTA that leaves last
    unsigned long long phase_t[8];
    // fused Gaussian_k kernel, how the last call counted: CTAs that formed a prediction, CTAs whose
    // predicted bands held the exact thresholds, whether a second full count was needed, cells
    // left to phase B by CTAs with a prediction, CTAs that counted only the candidates they
    // expected the rounds to reach
    unsigned int path_info[6];
    // gk_error_ratio: ratio, ||u - Comp(u)||^2, ||u||^2
    double diag[4];
    // DGC_k: key of the sampled threshold, candidates at or above it, rank taken in the sample,
    // pairs written
    unsigned long long dgc[4];
};

struct Workspace {
    void* base = nullptr;          // device allocation
    size_t bytes = 0;
    int64_t d_cap = 0;             // sizes the allocation was made for
    int32_t s_cap = 0;
    Ctrl* ctrl = nullptr;
    double2* partials = nullptr;            // kMaxPartials
    double2* part_recs = nullptr;           // persistent Gaussian_k kernel: one 32-byte record of partial sums per CTA, and one more
    unsigned int fused_calls = 0;           // launches of that kernel on this workspace (the records carry the number)
    unsigned long long* tile_status = nullptr;  // one per compaction tile
    unsigned int* hist = nullptr;           // 3 x 2048 radix histograms
    unsigned int* cta_counts = nullptr;     // DGC_k and segmented fused kernels: per-CTA words (kFusedGridCap x kNumCand)
    unsigned int* bars = nullptr;           // 128 words: [2..3], [36..56], [64..103] fused sparsifier, [4..8] fused Top_k, [10..13] fused segmented
    unsigned int* rowcnt = nullptr;         // fused kernels: two words per row of 4096 elements
    unsigned long long* cta_trace = nullptr;  // fused kernel: kFusedGridCap x 8 timestamps (tracing aid)
    int last_grid = 0;                      // CTAs of the last fused launch
    // segmented call
    void* seg_block = nullptr;
    int sm_count = 0;
    // per-stage timing (tracing aid)
    cudaEvent_t ev[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    int n_stages = 0;
    bool last_fused = false;  // the last sparsify call on this workspace ran the fused kernel
    int phase_spans = 0;      // spans between the timestamps the last (single) kernel took itself; 0: none
};

// host side (gk_host.cu)
int acquire_workspace(int64_t d, int32_t S, cudaStream_t stream, Workspace** out);
int cuda_fail(cudaError_t e);   // records the error text, returns GK_ERR_CUDA
void note_launch(int n = 1);
// Stage timing: mark(ws, st, i) records event i (0 = before the first kernel) when tracing is on.
void stage_mark(Workspace* ws, cudaStream_t st, int i);
int64_t output_capacity(int64_t d);
int selected_path();  // 0: cluster kernel for small vectors, else the persistent kernel; 1: three kernels; 2: persistent kernel at every size
int enqueue_gk_small(Workspace* ws, const float* src, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                     float* val_out, int64_t* nnz_out, cudaStream_t st);
// eps == nullptr: the operator on a given vector (src = u, read only)
int enqueue_gk_fused(Workspace* ws, const float* src, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                     float* val_out, int64_t* nnz_out, cudaStream_t st);
int enqueue_topk_fused(Workspace* ws, const float* src, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                       float* val_out, int64_t* nnz_out, cudaStream_t st);
int enqueue_gk_fused_seg(Workspace* ws, const float* g, float* eps, int64_t d, const int64_t* seg_offsets,
                         const int64_t* seg_k, int32_t S, int32_t* idx_out, float* val_out, int64_t* seg_nnz_out,
                         int64_t* nnz_out, cudaStream_t st);
int enqueue_gk_sparsify(Workspace* ws, const float* g, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                        float* val_out, int64_t* nnz_out, cudaStream_t st);

inline int64_t num_compact_tiles(int64_t d) {
    return (d + kCompactTileElems - 1) / kCompactTileElems;
}

#define GK_CUDA_TRY(expr)                                  \
    do {                                                   \
        cudaError_t e__ = (expr);                          \
        if (e__ != cudaSuccess) return ::gk::cuda_fail(e__); \
    } while (0)

// ---------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    return v;
}

// Streaming 128-bit load: the line is not expected to be read again.
__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ unsigned long long ld_status(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_status(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Deterministic block reduction of (s, q) pairs: warp shuffles, then a fixed
// order over the warps.  Result valid in thread 0.
template <int THREADS>
__device__ __forceinline__ double2 block_sum2(double s, double q, double2* smem /* THREADS/32 */) {
    s = warp_sum(s);
    q = warp_sum(q);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) smem[w] = make_double2(s, q);
    __syncthreads();
    double2 r = make_double2(0.0, 0.0);
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < THREADS / 32; ++i) { r.x += smem[i].x; r.y += smem[i].y; }
    }
    __syncthreads();
    return r;
}

#endif  // __CUDACC__

}  // namespace gk
