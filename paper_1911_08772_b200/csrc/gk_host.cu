// Host-side plumbing of the library: per-(device, stream) scratch workspaces,
// the normal quantile, capacity, statistics read-back, error text, and the
// host-buffer convenience call.
#include <math.h>
#include <string.h>

#include <atomic>
#include <map>
#include <mutex>
#include <string>
#include <utility>

#include "gk_alg1.cuh"
#include "gk_common.cuh"
#include "gk_segmented.cuh"

namespace gk {

static std::mutex g_mu;
static std::map<std::pair<int, cudaStream_t>, Workspace> g_ws;
static std::atomic<int64_t> g_launches{0};
static std::atomic<int64_t> g_capacity{0};
static thread_local std::string g_cuda_err;

int cuda_fail(cudaError_t e) {
    g_cuda_err = cudaGetErrorString(e);
    return GK_ERR_CUDA;
}

void note_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static std::atomic<int> g_stage_timing{0};

void stage_mark(Workspace* ws, cudaStream_t st, int i) {
    if (!g_stage_timing.load(std::memory_order_relaxed) || i < 0 || i > 5) return;
    if (!ws->ev[i] && cudaEventCreate(&ws->ev[i]) != cudaSuccess) { cudaGetLastError(); return; }
    cudaEventRecord(ws->ev[i], st);
    ws->n_stages = i;
}

int64_t output_capacity(int64_t d) {
    const int64_t c = g_capacity.load(std::memory_order_relaxed);
    return c > 0 ? c : d;
}

// ---------------------------------------------------------------------------
// Workspace layout
// ---------------------------------------------------------------------------
static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
    size_t ctrl, partials, part_recs, hist, cta_counts, bars, cta_trace, rowcnt, tile_status, seg, total;
};

static Layout layout_for(int64_t d, int32_t S) {
    Layout L;
    size_t at = 0;
    L.ctrl = at;        at = align_up(at + sizeof(Ctrl), 256);
    L.partials = at;    at = align_up(at + sizeof(double2) * kMaxPartials, 256);
    L.part_recs = at;   at = align_up(at + (size_t)32 * (kFusedGridCap + 1), 256);
    L.hist = at;        at = align_up(at + sizeof(unsigned int) * 3 * 2048, 256);
    L.cta_counts = at;  at = align_up(at + sizeof(unsigned int) * kFusedGridCap * kNumCand, 256);
    L.bars = at;        at = align_up(at + sizeof(unsigned int) * 128, 256);
    L.cta_trace = at;   at = align_up(at + sizeof(unsigned long long) * kFusedGridCap * 8, 256);
    L.rowcnt = at;      at = align_up(at + sizeof(unsigned int) * 2 * ((size_t)(d >> 12) + 2), 256);
    L.tile_status = at; at = align_up(at + sizeof(unsigned long long) * (size_t)num_compact_tiles(d), 256);
    L.seg = at;         at = align_up(at + segmented_scratch_bytes(d, S), 256);
    L.total = at;
    return L;
}

int acquire_workspace(int64_t d, int32_t S, cudaStream_t stream, Workspace** out) {
    int dev = 0;
    GK_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(g_mu);
    Workspace& ws = g_ws[std::make_pair(dev, stream)];
    if (ws.base == nullptr || d > ws.d_cap || S > ws.s_cap) {
        const int64_t nd = d > ws.d_cap ? d : ws.d_cap;
        const int32_t ns = S > ws.s_cap ? S : ws.s_cap;
        const Layout L = layout_for(nd, ns);
        if (ws.base) {
            // work already enqueued on this stream may still use the old block
            GK_CUDA_TRY(cudaStreamSynchronize(stream));
            GK_CUDA_TRY(cudaFree(ws.base));
            ws.base = nullptr;
        }
        void* p = nullptr;
        cudaError_t e = cudaMalloc(&p, L.total);
        if (e != cudaSuccess) { cudaGetLastError(); return GK_ERR_NOMEM; }
        // cleared on the caller's stream, so that the clear is ordered before the kernels of this and
        // every later call there (a memset on the default stream would not be ordered with a
        // non-blocking stream)
        e = cudaMemsetAsync(p, 0, L.total, stream);
        if (e != cudaSuccess) { cudaFree(p); return cuda_fail(e); }
        char* b = static_cast<char*>(p);
        ws.base = p;
        ws.bytes = L.total;
        ws.d_cap = nd;
        ws.s_cap = ns;
        ws.ctrl = reinterpret_cast<Ctrl*>(b + L.ctrl);
        ws.partials = reinterpret_cast<double2*>(b + L.partials);
        ws.part_recs = reinterpret_cast<double2*>(b + L.part_recs);
        ws.hist = reinterpret_cast<unsigned int*>(b + L.hist);
        ws.cta_counts = reinterpret_cast<unsigned int*>(b + L.cta_counts);
        ws.bars = reinterpret_cast<unsigned int*>(b + L.bars);
        ws.cta_trace = reinterpret_cast<unsigned long long*>(b + L.cta_trace);
        ws.rowcnt = reinterpret_cast<unsigned int*>(b + L.rowcnt);
        ws.tile_status = reinterpret_cast<unsigned long long*>(b + L.tile_status);
        ws.seg_block = b + L.seg;
        GK_CUDA_TRY(cudaDeviceGetAttribute(&ws.sm_count, cudaDevAttrMultiProcessorCount, dev));
    }
    *out = &ws;
    return GK_OK;
}

static Workspace* find_workspace(cudaStream_t stream) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    std::lock_guard<std::mutex> lock(g_mu);
    auto it = g_ws.find(std::make_pair(dev, stream));
    return it == g_ws.end() ? nullptr : &it->second;
}

// staging buffers of gk_sparsify_host, one set per device
struct HostStage {
    float* g = nullptr; float* eps = nullptr; int32_t* idx = nullptr; float* val = nullptr;
    int64_t* nnz = nullptr; int64_t d_cap = 0; int64_t out_cap = 0; cudaStream_t stream = nullptr;
};
static std::map<int, HostStage> g_stage;

static std::atomic<int> g_path{0};
int selected_path() { return g_path.load(std::memory_order_relaxed); }

// Test hooks: setters registered by the translation units that hold device-side knobs, and
// the host-side knobs themselves.
struct KnobRegistry {
    std::mutex mu;
    KnobSetter fn[32];
    int n = 0;
};
static KnobRegistry& knob_registry() {
    static KnobRegistry r;   // constructed on first use: units register during static initialisation
    return r;
}
int register_knob_setter(KnobSetter fn) {
    KnobRegistry& r = knob_registry();
    std::lock_guard<std::mutex> lock(r.mu);
    if (r.n < 32) r.fn[r.n++] = fn;
    return r.n;
}
static std::atomic<int> g_host_knob[kKnobCount] = {};
static std::atomic<bool> g_host_knob_set[kKnobCount] = {};
int host_knob(int key) {
    if (key < 0 || key >= kKnobCount) return 0;
    if (!g_host_knob_set[key].load()) return (key == kKnobPrediction || key == kKnobSelectedWay) ? -1 : 0;
    return g_host_knob[key].load();
}

}  // namespace gk

using namespace gk;

extern "C" int gk_set_capacity(int64_t cap) {
    if (cap < 0) return GK_ERR_CAPACITY;
    g_capacity.store(cap);
    return GK_OK;
}

extern "C" int gk_set_path(int path) {
    if (path < 0 || path > 2) return GK_ERR_SIZE;
    g_path.store(path);
    return GK_OK;
}

static int set_knob_everywhere(int key, int value) {
    g_host_knob[key].store(value);
    g_host_knob_set[key].store(true);
    KnobRegistry& r = knob_registry();
    std::lock_guard<std::mutex> lock(r.mu);
    for (int i = 0; i < r.n; ++i) {
        const int e = r.fn[i](key, value);
        if (e != 0) return cuda_fail((cudaError_t)e);
    }
    return GK_OK;
}

extern "C" int gk_set_params(int unbiased_std, int max_rounds) {
    if (max_rounds < 1 || max_rounds > kMaxRounds) return GK_ERR_SIZE;
    const int rc = set_knob_everywhere(kKnobBiasedStd, unbiased_std ? 0 : 1);
    return rc != GK_OK ? rc : set_knob_everywhere(kKnobMaxRounds, max_rounds);
}

extern "C" int gk_debug_set(int key, int64_t value) {
    if (key < 0 || key >= kKnobBiasedStd || value < -1 || value > 2147483647ll) return GK_ERR_SIZE;
    return set_knob_everywhere(key, (int)value);
}

extern "C" int gk_reserve(int64_t d, int32_t S, gk_stream_t stream) {
    if (d < 1 || d > 2147483647ll || S < 1 || S > kMaxSegments) return GK_ERR_SIZE;
    Workspace* ws = nullptr;
    return acquire_workspace(d, S, (cudaStream_t)stream, &ws);
}

extern "C" int64_t gk_workspace_bytes(int64_t d, int32_t S) {
    if (d < 1 || S < 1) return 0;
    return (int64_t)layout_for(d, S).total;
}

extern "C" int gk_last_stats(gk_stream_t stream, gk_stats* host_out) {
    if (!host_out) return GK_ERR_NULL;
    Workspace* ws = find_workspace((cudaStream_t)stream);
    if (!ws) return GK_ERR_NULL;
    GK_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    GK_CUDA_TRY(cudaMemcpy(host_out, &ws->ctrl->stats, sizeof(gk_stats), cudaMemcpyDeviceToHost));
    return GK_OK;
}

extern "C" int dgck_last_info(gk_stream_t stream, int64_t* host_out) {
    if (!host_out) return GK_ERR_NULL;
    Workspace* ws = find_workspace((cudaStream_t)stream);
    if (!ws) return GK_ERR_NULL;
    GK_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    unsigned long long v[4];
    GK_CUDA_TRY(cudaMemcpy(v, ws->ctrl->dgc, sizeof(v), cudaMemcpyDeviceToHost));
    for (int i = 0; i < 4; ++i) host_out[i] = (int64_t)v[i];
    return GK_OK;
}

extern "C" int gk_last_segment_stats(gk_stream_t stream, int32_t S, gk_stats* host_out) {
    if (!host_out) return GK_ERR_NULL;
    Workspace* ws = find_workspace((cudaStream_t)stream);
    if (!ws || S < 1 || S > ws->s_cap) return GK_ERR_SIZE;
    GK_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    GK_CUDA_TRY(cudaMemcpy(host_out, segmented_stats_ptr(ws), sizeof(gk_stats) * (size_t)S,
                           cudaMemcpyDeviceToHost));
    gk_stats total;
    GK_CUDA_TRY(cudaMemcpy(&total, &ws->ctrl->stats, sizeof(gk_stats), cudaMemcpyDeviceToHost));
    // call-wide flags apply to every record; without truncation every mask went out whole
    for (int32_t s = 0; s < S; ++s) {
        host_out[s].status |= total.status;
        if (!(total.status & (GK_DEV_TRUNCATED | GK_DEV_TIMEOUT))) host_out[s].emitted = host_out[s].nnz;
    }
    return GK_OK;
}

extern "C" int gk_last_path_info(gk_stream_t stream, int64_t* host_out) {
    if (!host_out) return GK_ERR_NULL;
    Workspace* ws = find_workspace((cudaStream_t)stream);
    if (!ws) return GK_ERR_NULL;
    GK_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    unsigned int v[5];
    GK_CUDA_TRY(cudaMemcpy(v, ws->ctrl->path_info, sizeof(v), cudaMemcpyDeviceToHost));
    for (int i = 0; i < 4; ++i) host_out[i] = (int64_t)v[i];
    host_out[4] = ws->last_fused ? ws->last_grid : 0;
    host_out[5] = (int64_t)v[4];
    return GK_OK;
}

extern "C" int gk_stage_timing(int enable) {
    g_stage_timing.store(enable ? 1 : 0);
    return GK_OK;
}

extern "C" int gk_last_stage_ms(gk_stream_t stream, float* ms_out, int* n_stages) {
    if (!ms_out || !n_stages) return GK_ERR_NULL;
    Workspace* ws = find_workspace((cudaStream_t)stream);
    if (!ws) return GK_ERR_NULL;
    GK_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    *n_stages = ws->n_stages;
    for (int i = 0; i < ws->n_stages; ++i)
        GK_CUDA_TRY(cudaEventElapsedTime(&ms_out[i], ws->ev[i], ws->ev[i + 1]));
    if (ws->phase_spans > 0 && ws->n_stages == 1) {
        // one kernel: after its event time, the spans between the kernel's own timestamps
        unsigned long long t[8];
        GK_CUDA_TRY(cudaMemcpy(t, ws->ctrl->phase_t, sizeof(t), cudaMemcpyDeviceToHost));
        for (int i = 0; i < ws->phase_spans; ++i) ms_out[1 + i] = (float)((double)(t[i + 1] - t[i]) * 1e-6);
        *n_stages = 1 + ws->phase_spans;
    }
    return GK_OK;
}

extern "C" int gk_last_cta_trace(gk_stream_t stream, uint64_t* host_out, int* n_ctas) {
    if (!host_out || !n_ctas) return GK_ERR_NULL;
    Workspace* ws = find_workspace((cudaStream_t)stream);
    if (!ws) return GK_ERR_NULL;
    GK_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    *n_ctas = ws->last_fused ? ws->last_grid : 0;
    if (*n_ctas > 0)
        GK_CUDA_TRY(cudaMemcpy(host_out, ws->cta_trace, sizeof(uint64_t) * 8 * (size_t)*n_ctas,
                               cudaMemcpyDeviceToHost));
    return GK_OK;
}

extern "C" int64_t gk_launch_count(void) { return g_launches.load(); }

extern "C" const char* gk_strerror(int code) {
    switch (code) {
        case GK_OK: return "ok";
        case GK_ERR_NULL: return "a required pointer is NULL (or no call was made on this stream)";
        case GK_ERR_SIZE: return "size out of range (need 1 <= d <= 2^31-1, 1 <= S <= 65536)";
        case GK_ERR_K: return "k out of range (need 1 <= k <= d)";
        case GK_ERR_ALIGN: return "vector base pointer is not 16-byte aligned";
        case GK_ERR_ALIAS: return "g overlaps eps";
        case GK_ERR_CUDA: return "CUDA runtime error (see gk_last_cuda_error)";
        case GK_ERR_NOMEM: return "could not allocate the scratch workspace";
        case GK_ERR_CAPACITY: return "capacity must be >= 0";
        case GK_ERR_LIMIT: return "size beyond a built-in limit";
        default: return "unknown gk_status";
    }
}

extern "C" const char* gk_last_cuda_error(void) { return g_cuda_err.c_str(); }

extern "C" int gk_version(void) { return 1000; }

extern "C" int gk_sparsify_host(const float* g, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                                float* val_out, int64_t* nnz_out, gk_stats* stats_out) {
    if (!g || !eps || !idx_out || !val_out || !nnz_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll) return GK_ERR_SIZE;
    if (k < 1 || k > d) return GK_ERR_K;
    int dev = 0;
    GK_CUDA_TRY(cudaGetDevice(&dev));
    const int64_t cap = output_capacity(d);
    // the staging buffers of a device serve one call at a time
    static std::mutex stage_mu;
    std::lock_guard<std::mutex> stage_lock(stage_mu);
    HostStage* hs = &g_stage[dev];
    if (!hs->stream) GK_CUDA_TRY(cudaStreamCreateWithFlags(&hs->stream, cudaStreamNonBlocking));
    if (d > hs->d_cap || cap > hs->out_cap) {
        GK_CUDA_TRY(cudaStreamSynchronize(hs->stream));
        cudaFree(hs->g); cudaFree(hs->eps); cudaFree(hs->idx); cudaFree(hs->val); cudaFree(hs->nnz);
        *hs = HostStage{nullptr, nullptr, nullptr, nullptr, nullptr, 0, 0, hs->stream};
        if (cudaMalloc(&hs->g, sizeof(float) * d) != cudaSuccess ||
            cudaMalloc(&hs->eps, sizeof(float) * d) != cudaSuccess ||
            cudaMalloc(&hs->idx, sizeof(int32_t) * cap) != cudaSuccess ||
            cudaMalloc(&hs->val, sizeof(float) * cap) != cudaSuccess ||
            cudaMalloc(&hs->nnz, sizeof(int64_t)) != cudaSuccess) {
            cudaGetLastError();
            return GK_ERR_NOMEM;
        }
        hs->d_cap = d;
        hs->out_cap = cap;
    }
    cudaStream_t st = hs->stream;
    Workspace* ws = nullptr;
    const int wrc = acquire_workspace(d, 1, st, &ws);
    if (wrc != GK_OK) return wrc;
    GK_CUDA_TRY(cudaMemcpyAsync(hs->g, g, sizeof(float) * d, cudaMemcpyHostToDevice, st));
    GK_CUDA_TRY(cudaMemcpyAsync(hs->eps, eps, sizeof(float) * d, cudaMemcpyHostToDevice, st));
    const int rc = enqueue_gk_sparsify(ws, hs->g, hs->eps, d, k, hs->idx, hs->val, hs->nnz, st);
    if (rc != GK_OK) return rc;
    GK_CUDA_TRY(cudaMemcpyAsync(nnz_out, hs->nnz, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    GK_CUDA_TRY(cudaMemcpyAsync(eps, hs->eps, sizeof(float) * d, cudaMemcpyDeviceToHost, st));
    GK_CUDA_TRY(cudaStreamSynchronize(st));
    const int64_t n = *nnz_out;
    if (n > 0) {
        GK_CUDA_TRY(cudaMemcpyAsync(idx_out, hs->idx, sizeof(int32_t) * n, cudaMemcpyDeviceToHost, st));
        GK_CUDA_TRY(cudaMemcpyAsync(val_out, hs->val, sizeof(float) * n, cudaMemcpyDeviceToHost, st));
    }
    if (stats_out)
        GK_CUDA_TRY(cudaMemcpyAsync(stats_out, &ws->ctrl->stats, sizeof(gk_stats), cudaMemcpyDeviceToHost, st));
    GK_CUDA_TRY(cudaStreamSynchronize(st));
    return GK_OK;
}
