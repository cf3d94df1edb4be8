// Scratch layout of the segmented (layer-wise) sparsifier.  Internal.
#pragma once

#include "gk_common.cuh"

namespace gk {

constexpr int32_t kMaxSegments = 65536;

// Views into Workspace::seg_block for S segments (struct of arrays).
struct SegScratch {
    gk_stats* stats;             // S
    double* cand64;              // S x kNumCand
    unsigned long long* counts;  // S x kNumCand
    float* cand32;               // S x kNumCand
    float* thr_sel;              // S
    double2* partials;           // kMaxPartials + S: slot (cta + segment)
    double* zs;                  // S: normal quantile of each segment's density
};

inline size_t seg_align(size_t x) { return (x + 255) / 256 * 256; }

inline size_t segmented_scratch_bytes(int64_t /*d*/, int32_t S) {
    if (S < 1) S = 1;
    size_t at = 0;
    at = seg_align(at + sizeof(gk_stats) * (size_t)S);
    at = seg_align(at + sizeof(double) * kNumCand * (size_t)S);
    at = seg_align(at + sizeof(unsigned long long) * kNumCand * (size_t)S);
    at = seg_align(at + sizeof(float) * kNumCand * (size_t)S);
    at = seg_align(at + sizeof(float) * (size_t)S);
    at = seg_align(at + sizeof(double2) * ((size_t)kMaxPartials + (size_t)S));
    at = seg_align(at + sizeof(double) * (size_t)S);
    return at;
}

inline SegScratch segmented_views(const Workspace* ws) {
    const size_t S = (size_t)(ws->s_cap < 1 ? 1 : ws->s_cap);
    char* b = static_cast<char*>(ws->seg_block);
    SegScratch v;
    size_t at = 0;
    v.stats = reinterpret_cast<gk_stats*>(b + at);             at = seg_align(at + sizeof(gk_stats) * S);
    v.cand64 = reinterpret_cast<double*>(b + at);              at = seg_align(at + sizeof(double) * kNumCand * S);
    v.counts = reinterpret_cast<unsigned long long*>(b + at);  at = seg_align(at + sizeof(unsigned long long) * kNumCand * S);
    v.cand32 = reinterpret_cast<float*>(b + at);               at = seg_align(at + sizeof(float) * kNumCand * S);
    v.thr_sel = reinterpret_cast<float*>(b + at);              at = seg_align(at + sizeof(float) * S);
    v.partials = reinterpret_cast<double2*>(b + at);           at = seg_align(at + sizeof(double2) * ((size_t)kMaxPartials + S));
    v.zs = reinterpret_cast<double*>(b + at);
    return v;
}

inline gk_stats* segmented_stats_ptr(const Workspace* ws) { return segmented_views(ws).stats; }

}  // namespace gk
