// gk_sparsify (and gk_select, the same selection on a given u) as ONE persistent
// cooperative kernel (Eq. 2 and Algorithm 1 of arXiv 1911.08772).
//
// The vector is cut into rows of 1024 float4 (16 KB; thread t takes float4 t of
// the row), dealt to one CTA per SM in turn (CTA c owns rows c, c + G, ...), so
// that every CTA gets the same mix of the vector's quiet and loud stretches.
// The three phases of the method are separated by grid barriers, and what fits
// of u stays on chip between them:
//
//   phase A  g and eps arrive through a ring of asynchronous copies (cp.async,
//            kStages - 1 rows ahead); u = g + eps is written over eps and into the
//            shared-memory slot its eps came through, so the last rows of the
//            run are still on chip afterwards; fp64 partial sums per CTA; per
//            (row, warp) cell the largest magnitude goes to a small table.
//            On large vectors most of the counting of Algorithm 1 happens here
//            as well, against PREDICTED thresholds (below).
//   barrier  every CTA adds the partials in the same fixed order and forms
//            mu, sigma, thres0 and the ten candidate thresholds for itself.
//   phase B  counts of |u| > candidate, from the on-chip copy where there is
//            one, else from eps (L2 / HBM): for all ten candidates over all
//            cells, or, when the prediction held, for the six upper candidates
//            over the cells that phase A could not settle.
//   barrier  the CTAs' counts meet in ten global sums; every CTA replays the
//            rounds of Algorithm 1: threshold and number of survivors are known.
//   phase C  a cell is read again only if its recorded maximum can exceed the
//            threshold; the survivors of every row are counted and the counts
//            exchanged through a third barrier, which gives every row its output
//            offset -- no look-back, no waiting between CTAs; the survivors are
//            written as (index, value) pairs and their slots cleared.
//
// Counting while the vector streams in.  The thresholds depend on mu and sigma
// of the whole vector, which are known only after phase A.  But they can be
// predicted: every warp first reads one block of 128 elements (the blocks of
// all warps of all CTAs are spread evenly over the vector: a systematic sample
// of about 1/42 of it at the benchmark size), the CTAs publish the sample's
// power sums, and a few rows later every CTA forms a predicted first threshold
// with an error bound delta from the sample's own fourth moment.  From then on
// phase A counts, for each of the six candidates thres0 * {3/4, 1, 9/8, 3/2,
// 9/4, 27/8}, the elements above hi_j = c_j (1 + delta), and notes for every
// cell whether any element lies in a band (lo_j, hi_j].  A cell without such an
// element has the same count for every threshold inside the band, so once the
// exact c_j is known to lie in its band the phase A count of that cell is the
// exact one; cells with a band element ("flagged"), rows that streamed before
// the prediction arrived, and CTAs whose band missed are counted in phase B as
// before.  The four lower candidates (thres0 / 8 ... thres0 / 2) are reached
// only when the first count is below 2k/3; then every CTA that took the short
// way counts again in full and one more barrier follows.  The result is exact
// in every case: prediction only decides where a cell is counted.
//
// HBM traffic: 12 d bytes for phase A (4 d for gk_select), phase B's re-reads
// (L2 mostly), and next to nothing for phase C (survivors are rare, so few
// cells qualify).
//
// The barriers are counters in the workspace.  Every wait is bounded; a CTA
// whose wait runs out records GK_DEV_TIMEOUT and leaves.  The kernel is
// launched cooperatively, so all CTAs are resident and the waits do end.
#include <math.h>

#include <cstddef>
#include <mutex>
#include <type_traits>

#include "gk_alg1.cuh"
#include "gk_common.cuh"
#include "gk_coop.cuh"
#include "gk_count.cuh"

namespace gk {

constexpr int kTableMaxRows = 1024;                    // most rows a CTA may own (entries of its maximum table)
constexpr int kTableRowBytes = kFusedWarps * 2;        // one uint16 per (row, warp)
constexpr int kFusedSmemBudget = 221184;               // dynamic shared memory the kernel may ask for
constexpr int kStages = 4;                             // phase A: rows of g and eps in flight, plus one
constexpr int kRing = 8;                               // ring slots; phase B has kRing - 1 rows in flight
constexpr int kFusedMaxGrid = kFusedGridCap;
constexpr int kTraceSlots = 8;                         // timestamps per CTA in the optional trace
// phase C keeps the places of a CTA's survivors (row, warp, lane, element, rank within the
// segment: one word each) in the ring's shared memory between counting and write-out
constexpr int kStageCap = kRing * kRowF4 * 4;

// Counting during phase A (prediction of the thresholds from a sample).
constexpr int kUpper = 6;               // candidates thres0 * {3/4, 1, 9/8, 3/2, 9/4, 27/8}: sorted places 4..9
// Rows per CTA from which on the prediction is tried without being asked for (39 M elements on 148
// SMs).  Measured on B200: at 110 rows per CTA (2^26 elements) the streaming phase is bound by HBM and
// takes the extra work for free (200 -> 177 us per call); at 42 rows (25.6 M elements, half of eps
// served by L2) it has no issue slots to spare and the two ways take the same time; below, the
// prediction costs more than it saves.
constexpr int kPredMinRows = 64;
constexpr int kPredMaxRows = 511;       // ... and up to which: a thread's counts (4 per row) are kept in 13 bits
constexpr float kPackScale = 8192.f;    // two counts in one float: lo + 8192 * hi, exact below 2^24
constexpr int kSampleElems = kFusedThreads * 4;   // sample elements per CTA: one float4 per thread
constexpr double kPredSigmas = 3.5;     // half width of the bands in standard errors of the predicted threshold
constexpr double kPredSlack = 5e-4;     // added to the relative half width
constexpr double kPredMaxDelta = 0.05;  // wider bands than this are not worth counting against
constexpr unsigned int kSparseWay = 2;  // no prediction: the short way is taken when at most 1 cell in 2 is loud
// candidates that only phase B's full count covers
// The selected way of phase B: at most kSelMax candidates, those that the rounds can reach
// according to an estimate of every candidate's count from this CTA's table of cell maxima.
constexpr int kSelMax = 6;
constexpr float kSelSigmas = 4.0f;     // width of an estimate's band, in standard errors of the loud-cell count
constexpr float kSelSlack = 0.10f;     // added to the band: the maxima are rounded, the cells are not a random sample
constexpr float kSelCluster = 4.0f;    // survivors that sit together in few cells make the estimate too low: upper side only
constexpr int kSelMinRows = 12;        // rows a CTA must own for its cells to stand for the vector's
constexpr float kSelFlat = 0.3f;       // loud cells that stay loud at twice the candidate, as a share: above it, no upper side
constexpr unsigned int kAllCandMask = (1u << kNumCand) - 1u;
// Test hook: -1 decides by itself, 0 never takes the selected way, 1 takes it with thres0 alone
// selected (so that any second round finds a candidate left out and the count is taken again).
static __device__ int g_selected_way = -1;
static int set_fused_knob(int key, int value) {
    if (key == kKnobSelectedWay) return (int)cudaMemcpyToSymbol(g_selected_way, &value, sizeof(int));
    return 0;
}
static const int g_fused_knob_registered = register_knob_setter(&set_fused_knob);

constexpr unsigned int kLowCandMask = (1u << cand_index(1, 0)) | (1u << cand_index(2, 0)) |
                                      (1u << cand_index(3, 0)) | (1u << cand_index(2, 1));
static_assert(cand_by_factor(0) == cand_index(3, 0) && cand_by_factor(1) == cand_index(2, 0) &&
              cand_by_factor(2) == cand_index(2, 1) && cand_by_factor(3) == cand_index(1, 0),
              "the four lowest factors are the candidates of kLowCandMask");

// Words of the barrier block used by this kernel (the exact Top_k kernel has 4..8, the segmented
// one 10..13).  All are zero between calls: the CTA that leaves last clears them.
// (words 0 and 1 are free: the first two barriers are the arrival of the data itself, see the kernel)
constexpr int kBarExit = 2;       // CTAs that have left
constexpr int kBarRows = 3;       // barrier inside phase C
constexpr int kBarTotals = 64;    // 2 x kNumCand 64-bit words (first count, second count), one per candidate:
                                  // CTAs that have added theirs (bits 52..63), CTAs that left the candidate
                                  // out (40..51), the count over the vector (0..39)
constexpr int kTotArriveShift = 52, kTotLeftShift = 40;
constexpr unsigned long long kTotCountMask = (1ull << kTotLeftShift) - 1ull;
constexpr int kBarInfo = 36;      // 5 words: what Ctrl::path_info reports, collected during the call
constexpr int kBarSample = 48;    // 4 doubles: the sample's power sums over all CTAs; then a word: CTAs that are in
constexpr int kBarWords = 128;

struct __align__(128) FusedShared {
    double2 red[kFusedWarps];
    unsigned int cta_counts[kNumCand];
    unsigned long long col[kNumCand];   // counts over the whole vector
    double cand64[kNumCand];
    float cand32[kNumCand];
    int order[kNumCand];                // candidate indices, ascending by threshold
    float plo[kUpper], phi[kUpper];     // predicted bands of the six upper candidates
    float thr_sel;
    int chosen;
    int ok;
    unsigned int samp_n;                // warps whose sums are in
    int pred_ready;                     // 0: no word yet; 1: the predicted bands stand; 2: no prediction
    int fast;                           // phase B of this CTA: 0 in full, 1 a short way over the cells left, 2 the selected way
    long long k_wanted;                 // k, for the functions that are not handed it
    int sel_n;                          // the selected way: how many candidates, which (ascending), as a mask
    int sel_idx[kSelMax];
    unsigned int sel_mask;
    int recount;                        // the rounds need a candidate that some CTA has not counted
    gk_stats stats;
    unsigned int wsum[kFusedWarps];
    // survivors in each round of rows (G consecutive rows); before phase C the first 1 KB holds
    // the warps' sample sums as double2, hence the alignment
    alignas(16) unsigned int roundtot[kTableMaxRows];
    unsigned int rowpre[kTableMaxRows];    // survivors in the vector before each row of this CTA
    unsigned short qrow[kFusedWarps][kGroupRows];  // rows a warp has gathered for one batch
    unsigned int n_staged;                 // survivors put aside in phase C
    unsigned int left_out;                 // candidates (bit = index) that some CTA has not counted
};

static_assert(offsetof(FusedShared, roundtot) % 16 == 0 && sizeof(unsigned int) * kTableMaxRows >= 64 * kFusedWarps,
              "the sample slots (two double2 per warp) borrow roundtot");
// FusedShared sits at the front of the dynamic shared memory, the rows behind it on a 1 KB boundary
constexpr int kFusedStaticBytes = 11264;
static_assert(sizeof(FusedShared) <= kFusedStaticBytes && kFusedStaticBytes % 1024 == 0 &&
                  kFusedStaticBytes + kFusedSmemBudget <= 232448,
              "over the 227 KB of shared memory per CTA");

__device__ __forceinline__ unsigned int mask_above(const float4 v, const float thr) {
    return (unsigned)(fabsf(v.x) > thr) | ((unsigned)(fabsf(v.y) > thr) << 1) |
           ((unsigned)(fabsf(v.z) > thr) << 2) | ((unsigned)(fabsf(v.w) > thr) << 3);
}

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// A CTA's partial sums travel as one 32-byte record, written with one 256-bit store and read with
// one 256-bit load: {call number, 0, s, q, 0, call number}.  The record is its own arrival flag:
// a reader that finds this call's number at both ends has the sums of this call (a 32-byte aligned
// access is one sector to L2; the number at both ends also shows a record torn between its
// 16-byte halves, should a device ever do that).  No fence and no counter: the sums are all that
// the other CTAs need from this one before the second barrier.
__device__ __forceinline__ void store_partial(unsigned int* rec, const unsigned int call_no, const double s, const double q) {
    asm volatile("st.relaxed.gpu.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(rec), "r"(call_no), "r"(0u),
                 "r"((unsigned int)__double2loint(s)), "r"((unsigned int)__double2hiint(s)),
                 "r"((unsigned int)__double2loint(q)), "r"((unsigned int)__double2hiint(q)), "r"(0u), "r"(call_no)
                 : "memory");
}
__device__ __forceinline__ bool load_partial(const unsigned int* rec, const unsigned int call_no, double& s, double& q) {
    unsigned int w0, w1, w2, w3, w4, w5, w6, w7;
    asm volatile("ld.relaxed.gpu.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3), "=r"(w4), "=r"(w5), "=r"(w6), "=r"(w7) : "l"(rec) : "memory");
    s = __hiloint2double((int)w3, (int)w2);
    q = __hiloint2double((int)w5, (int)w4);
    return w0 == call_no && w7 == call_no;
}
constexpr int kPartialWords = 8;   // 32 bytes a record

// The predicted first threshold and its bands, from the sample's power sums about the pivot pv
// (n sample elements).  The half width is kPredSigmas standard errors of mu + sigma z, with the
// standard error of sigma taken from the sample's own fourth moment (heavy tails widen the
// bands by themselves), plus a small slack.  Returns false when no useful prediction exists.
__device__ __noinline__ bool predict_bands(double s1, double s2, double s3, double s4, double n, double pv, double z,
                                     float* plo, float* phi) {
    const double inv_n = 1.0 / n;
    const double m1 = s1 * inv_n, r2 = s2 * inv_n, r3 = s3 * inv_n, r4 = s4 * inv_n;
    const double var_p = r2 - m1 * m1;                    // population variance of the sample
    if (!(var_p > 0.0) || !(n > 2.0)) return false;
    const double c4 = r4 - 4.0 * m1 * r3 + 6.0 * m1 * m1 * r2 - 3.0 * m1 * m1 * m1 * m1;   // central fourth moment
    // from here on single precision is plenty: the half width is a bound, not a result
    const float nf = (float)n, zf = (float)z;
    const float var = (float)var_p * (nf / (nf - 1.0f));
    const float kurt = (float)c4 / ((float)var_p * (float)var_p);
    const float sigma = sqrtf(var);
    const double th = (pv + m1) + (double)sigma * z;
    if (!(th > 0.0) || !(th < 3.0e38)) return false;
    const float se_sigma = 0.5f * sqrtf(fmaxf(kurt - 1.0f, 0.0f) / nf) * sigma;   // standard error of sigma
    const float se_th = sqrtf(var / nf + zf * zf * se_sigma * se_sigma);
    const float delta = (float)kPredSigmas * se_th / (float)th + (float)kPredSlack;
    if (!(delta < (float)kPredMaxDelta)) return false;
    const double f[kUpper] = {0.75, 1.0, 1.125, 1.5, 2.25, 3.375};
    const double dn = 1.0 - (double)delta, up = 1.0 + (double)delta;
#pragma unroll
    for (int j = 0; j < kUpper; ++j) {
        plo[j] = __double2float_rd(th * f[j] * dn);
        phi[j] = __double2float_ru(th * f[j] * up);
    }
    return phi[kUpper - 1] < 3.0e38f;
}

// The sample of one CTA: warp w reads block (c * 32 + w) of G * 32 blocks of 32 float4 spread
// evenly over the vector.  They are read with plain loads before anything else (so that no row
// has been overwritten yet) and parked in two ring slots that phase A does not use once the
// first row has been worked on.
// Nothing here synchronises a CTA or the grid, and nothing waits for memory to settle (a fence
// in a warp that streams rows stalls it for microseconds): every warp leaves the power sums of
// its block's (u - pv) in a slot of shared memory; the warp that comes last adds the 32 slots
// and adds the CTA's sums to four global accumulators, then one to a count, with plain atomics.
// Warp 0 of every CTA reads the accumulators and the count once per row (one sector, issued
// before the row and looked at after it); when the count is complete it forms the bands and
// hands them to its CTA's warps, which change over at their next row.
// The prediction only decides where a cell is counted, never what the count is: sums that are
// incomplete because the count overtook them, or a sample that misleads, give bands that are
// found out when the exact thresholds are known, and the CTA then counts in full.  (For the
// same reason it does no harm that the sums are added in the order of arrival, or that another
// CTA may already have replaced eps by u in a block of the first rows.)
// This thread's float4 of its warp's sample block: block (c * 32 + w) of G * 32 blocks of 32
// float4 spread evenly over the whole vector (leaving a stretch out would bias the prediction
// on vectors whose loud layers are few).
__device__ __forceinline__ int64_t sample_at(const int64_t n4) {
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int64_t nblk = n4 >> 5;
    const int64_t blk = (((int64_t)blockIdx.x * kFusedWarps + w) * nblk) / ((int64_t)gridDim.x * kFusedWarps);
    return (blk << 5) + lane;
}
// Called by whole warps, each once.  Out of line: its temporaries are its own.
template <bool ACC>
__device__ __noinline__ void publish_sample(const float4* gring, double pv, FusedShared* shp, unsigned int* bars) {
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    float4 a = gring[(size_t)kStages * kRowF4 + tid];
    if (ACC) {
        const float4 b = gring[(size_t)(kStages + 1) * kRowF4 + tid];
        a = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
    }
    const double x[4] = {(double)a.x - pv, (double)a.y - pv, (double)a.z - pv, (double)a.w - pv};
    double p1 = 0.0, p2 = 0.0, p3 = 0.0, p4 = 0.0;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const double y = x[t] * x[t];
        p1 += x[t]; p2 += y; p3 = fma(y, x[t], p3); p4 = fma(y, y, p4);
    }
    p1 = warp_sum(p1); p2 = warp_sum(p2); p3 = warp_sum(p3); p4 = warp_sum(p4);
    // the slots borrow an array that only phase C uses
    double2* slots = reinterpret_cast<double2*>(shp->roundtot);
    unsigned int before = 0u;
    if (lane == 0) {
        slots[2 * w] = make_double2(p1, p2);
        slots[2 * w + 1] = make_double2(p3, p4);
        __threadfence_block();
        before = atomicAdd(&shp->samp_n, 1u);
    }
    if (__shfl_sync(0xffffffffu, before, 0) != kFusedWarps - 1) return;
    // all warps are in: the CTA's sums (slot order, then a shuffle tree) join the global ones
    __threadfence_block();
    const volatile double* sv = reinterpret_cast<const volatile double*>(slots);
    p1 = warp_sum(sv[4 * lane]); p2 = warp_sum(sv[4 * lane + 1]);
    p3 = warp_sum(sv[4 * lane + 2]); p4 = warp_sum(sv[4 * lane + 3]);
    if (lane == 0) {
        double* acc = reinterpret_cast<double*>(bars + kBarSample);
        atomicAdd(acc + 0, p1); atomicAdd(acc + 1, p2); atomicAdd(acc + 2, p3); atomicAdd(acc + 3, p4);
        atomicAdd(bars + kBarSample + 8, 1u);
    }
}

// What a thread needs to know about its CTA's share of the vector, derived from the launch
// parameters alone, so that every phase can form it for itself.  Local row r of CTA c is row
// c + r * G of the vector; only the last row of the vector can be short, and it is the last
// local row of the CTA that owns it.
struct Rows {
    int nrows;          // rows of this CTA
    int first_kept;     // rows from here on stay on chip after phase A (the short last row of the
                        // vector, if this CTA owns it, is among them: u_slots >= 1)
    int64_t n4;         // float4 in the vector
    int64_t stride4;    // from a local row to the next
    int64_t first4;     // this thread's float4 in local row 0
    int64_t tail_i;     // this lane's element of the ragged tail (d mod 4 elements)
    bool in_last_row;   // this thread has a float4 in the CTA's last row
    bool owns_tail;     // this thread holds an element of the ragged tail
};
__device__ __forceinline__ Rows rows_of(const int64_t d, const int n_rows, const int u_slots) {
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int c = blockIdx.x, G = gridDim.x;
    Rows q;
    q.n4 = d >> 2;
    q.nrows = c < n_rows ? (n_rows - c + G - 1) / G : 0;
    q.stride4 = (int64_t)G * kRowF4;
    q.first4 = (int64_t)c * kRowF4 + tid;
    const bool has_last = q.nrows > 0 && (c + (q.nrows - 1) * G == n_rows - 1);
    q.in_last_row = !(has_last && (q.n4 & (kRowF4 - 1)) != 0) || tid < (int)(q.n4 & (kRowF4 - 1));
    q.first_kept = q.nrows > u_slots ? q.nrows - u_slots : 0;
    q.owns_tail = (c == G - 1) && (w == kFusedWarps - 1) && (lane < (int)(d & 3));
    q.tail_i = (q.n4 << 2) + lane;
    return q;
}

// Shared memory of the kernel: [FusedShared, kFusedStaticBytes][ring of kRing rows][u_slots rows]
// [table of table_rows x 32 uint16].  The rows start on a 1 KB boundary, which keeps every
// warp's 512 bytes of a row within four 128-byte lines.
struct Smem {
    FusedShared* sh;
    float4* gring;           // kRing x kRowF4 (phase A uses kStages of them for g)
    float4* uslot;           // u_slots x kRowF4
    unsigned short* table;   // one entry per (local row, warp)
};
__device__ __forceinline__ Smem smem_of(const int u_slots) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    Smem m;
    m.sh = reinterpret_cast<FusedShared*>(smem_raw);
    float4* rows = reinterpret_cast<float4*>(smem_raw + kFusedStaticBytes);
    m.gring = rows;
    m.uslot = rows + (size_t)kRing * kRowF4;
    m.table = reinterpret_cast<unsigned short*>(rows + (size_t)(kRing + u_slots) * kRowF4);
    return m;
}
#define GK_FUSED_VIEW(d, n_rows, u_slots)                                               \
    const Rows rows_ = rows_of(d, n_rows, u_slots);                                     \
    const Smem smem_ = smem_of(u_slots);                                                \
    FusedShared& sh = *smem_.sh;                                                        \
    float4* const gring = smem_.gring; float4* const uslot = smem_.uslot;               \
    unsigned short* const table = smem_.table;                                          \
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;                         \
    const int c = blockIdx.x, G = gridDim.x;                                            \
    const int nrows = rows_.nrows, first_kept = rows_.first_kept;                       \
    const int64_t n4 = rows_.n4, stride4 = rows_.stride4, first4 = rows_.first4, tail_i = rows_.tail_i; \
    const bool in_last_row = rows_.in_last_row, owns_tail = rows_.owns_tail;            \
    (void)gring; (void)uslot; (void)table; (void)lane; (void)w; (void)c; (void)G; (void)nrows; (void)first_kept; \
    (void)n4; (void)stride4; (void)first4; (void)tail_i; (void)in_last_row; (void)owns_tail; (void)sh

// With every cell still to be counted after phase A, two ways can beat streaming every row
// against all ten candidates, which is bound by the compare instructions (forty a float4).
//  - Where few of this CTA's cells can reach even thres0 / 2 (loud layers among quiet ones,
//    heavy tails), the short way over those few: the six upper candidates and thres0 / 2; the
//    three lowest candidates then wait for the rounds to ask for them.  sh.fast = 1.
//  - Else the selected way: the rounds of Algorithm 1 visit four of the ten candidates at most,
//    and which ones follows from the counts' rough sizes.  The number of cells whose maximum
//    reaches a candidate gives its count by the Poisson rule (cells without a survivor are
//    exp(-mean) of all), with a band for the noise of this CTA's cells; a candidate is selected
//    when the bands leave a way for the rounds to reach it.  Every row is streamed, but only
//    against the selected candidates.  sh.fast = 2.
// Either way the candidates left out are flagged, and the rounds asking for one of them sends
// the CTAs that took a short way through the count in full.  Out of line.
__device__ __noinline__ void decide_short_way(const int64_t d, const int n_rows, const int u_slots) {
    GK_FUSED_VIEW(d, n_rows, u_slots);
    __syncthreads();   // thread 0 has written the candidates, k and sh.fast
    const long long k = sh.k_wanted;
    const int knob = g_selected_way;
    if (sh.fast != 0 || !(sh.stats.thres0 > 0.0) || nrows == 0) return;   // the same in every thread
    unsigned int* const wsums = sh.rowpre;   // free until phase C: kNumCand / 2 words per warp
    // Every warp looks at 32 of its cells at most, evenly spread over its rows: one pass, and a
    // thousand cells are plenty for the estimate.  (This part and the next are short on work and
    // long on latency: a lone warp issues an instruction every few cycles.)
    const int step = (nrows + 31) >> 5;
    const int looked = (nrows + step - 1) / step;   // rows each warp looks at
    const unsigned int m = lane < looked ? ((unsigned int)table[lane * step * kFusedWarps + w] & kMaxMask) : 0u;
    const float n_cells = (float)(looked * kFusedWarps);
    {
        // the cells that reach thres0 / 2, counted by the barrier itself
        const int loud_half = __syncthreads_count(m > (__float_as_uint(sh.cand32[cand_index(1, 0)]) >> 16));
        if ((float)loud_half * (float)kSparseWay <= n_cells) {
            if (tid == 0) sh.fast = 1;
            return;
        }
    }
    if (!(knob > 0 || (knob < 0 && nrows >= kSelMinRows))) return;
    {
        // loud cells among them, two candidates to a word
        unsigned int loud[kNumCand / 2];
#pragma unroll
        for (int j = 0; j < kNumCand / 2; ++j) {
            const unsigned int l0 = __float_as_uint(sh.cand32[2 * j]) >> 16, l1 = __float_as_uint(sh.cand32[2 * j + 1]) >> 16;
            loud[j] = (m > l0 ? 1u : 0u) + (m > l1 ? 0x10000u : 0u);
        }
#pragma unroll
        for (int j = 0; j < kNumCand / 2; ++j) {
            const unsigned int ws = __reduce_add_sync(0xffffffffu, loud[j]);
            if (lane == j) wsums[w * (kNumCand / 2) + j] = ws;
        }
    }
    __syncthreads();
    if (w != 0) return;
    // warp 0: the CTA's sums; then lane j < 10 judges candidate j and ballots carry the judgements
    float L = 0.f;   // loud cells for this lane's candidate
#pragma unroll
    for (int j = 0; j < kNumCand / 2; ++j) {
        const unsigned int x = __reduce_add_sync(0xffffffffu, wsums[lane * (kNumCand / 2) + j]);
        if ((lane >> 1) == j) L = (float)((x >> ((lane & 1) * 16)) & 0xffffu);
    }
    // Cells that reach a candidate twice as large (the largest there is, for 9/4) in numbers not
    // far below: loud stretches or lone outliers, not the tail of one bell, and the loud cells
    // may hold any number of survivors.  No upper side to the estimate then.
    const int twice = lane == cand_index(0, 0) ? cand_index(0, 2)
                    : lane == cand_index(1, 0) ? cand_index(0, 0)
                    : lane == cand_index(0, 1) ? cand_index(0, 3)
                    : lane == cand_index(2, 0) ? cand_index(1, 0)
                    : lane == cand_index(1, 1) ? cand_index(0, 1)
                    : cand_index(0, 3);
    const float L_twice = __shfl_sync(0xffffffffu, L, twice);
    bool may_down = false, may_up = false;
    if (lane < kNumCand) {
        // the count over the whole vector that this many loud cells among n_cells suggest
        const float Q = n_cells - L, inv_n = __frcp_rn(n_cells);
        float lo = 0.f, hi = 5.f * (float)d * (1.f / 128.f) * inv_n * kSelCluster;   // no loud cell: a handful at most
        if (L > 0.5f) {
            const float pl = L * inv_n;
            const float lam = Q < 0.5f ? __logf(2.f * n_cells) : -__logf(1.f - pl);   // survivors per cell
            const float rel = __fdividef(__fsqrt_rn(pl * inv_n * __frcp_rn(fmaxf(1.f - pl, 0.5f * inv_n))), lam);
            const float m = 1.f + kSelSigmas * rel + kSelSlack;
            const float est = lam * (float)d * (1.f / 128.f);
            lo = __fdividef(est, m);
            hi = (Q < 8.f || L_twice > kSelFlat * L) ? INFINITY : est * m * kSelCluster;
        }
        may_down = 3.f * lo < 2.f * (float)k;
        may_up = 3.f * hi > 4.f * (float)k;
    }
    const unsigned int downs = __ballot_sync(0xffffffffu, may_down), ups = __ballot_sync(0xffffffffu, may_up);
    // The candidates the rounds can reach: round by round, a step down (to the candidate with one
    // more halving) where the count may fall short of 2k/3, a step up where it may pass 4k/3.
    // Lane ci asks whether either of its parents is reached and may step its way.
    const int b_ = lane < 4 ? 0 : lane < 7 ? 1 : lane < 9 ? 2 : 3;
    const int h_ = lane - (b_ == 0 ? 0 : b_ == 1 ? 4 : b_ == 2 ? 7 : 9);
    const int from_above = (lane < kNumCand && h_ > 0) ? cand_index(h_ - 1, b_) : -1;   // reached by a step down
    const int from_below = (lane < kNumCand && b_ > 0) ? cand_index(h_, b_ - 1) : -1;   // reached by a step up
    unsigned int reach = 1u << cand_index(0, 0);
    if (knob != 1) {
#pragma unroll
        for (int lvl = 0; lvl < kMaxRounds - 1; ++lvl) {
            const bool r = (from_above >= 0 && ((reach & downs) >> from_above) & 1u) ||
                           (from_below >= 0 && ((reach & ups) >> from_below) & 1u);
            reach |= __ballot_sync(0xffffffffu, r);
        }
    }
    // in ascending order of the thresholds: lane j looks at the j-th smallest candidate
    int mine_ci = 0;
#pragma unroll
    for (int j = 0; j < kNumCand; ++j) if (lane == j) mine_ci = cand_by_factor(j);
    const bool in = lane < kNumCand && ((reach >> mine_ci) & 1u);
    const unsigned int sorted = __ballot_sync(0xffffffffu, in);
    if (__popc(sorted) <= kSelMax) {
        if (in) sh.sel_idx[__popc(sorted & ((1u << lane) - 1u))] = mine_ci;
        if (lane == 0) { sh.sel_n = __popc(sorted); sh.sel_mask = reach; sh.fast = 2; }
    }
}

// Phase B, the short way: the six upper candidates over the cells that phase A left (flagged),
// added to phase A's own counts (pacc, two candidates to a float).  The cells are few and
// scattered, so every warp gathers its own eight at a time and loads them together, from shared
// memory where the row is on chip, else from L2.  Leaves the CTA's counts in sh.cta_counts.
// Out of line: its registers are its own.
template <int NC>
__device__ __noinline__ void count_short_way(const float* __restrict__ uvec, const int64_t d, const int n_rows,
                                             const int u_slots, const float pacc0, const float pacc1,
                                             const float pacc2, const float tail_u, unsigned int* __restrict__ bars) {
    static_assert(NC == kUpper || NC == kUpper + 1, "the six upper candidates, or those and thres0 / 2");
    GK_FUSED_VIEW(d, n_rows, u_slots);
    const float4* u4 = reinterpret_cast<const float4*>(uvec);
    const float pacc[kUpper / 2] = {pacc0, pacc1, pacc2};
    constexpr int X = NC - kUpper;   // candidates below the six upper ones
    float cs[NC], acc[NC];
#pragma unroll
    for (int j = 0; j < NC; ++j) { cs[j] = sh.cand32[cand_by_factor(kNumCand - NC + j)]; acc[j] = 0.f; }
#pragma unroll
    for (int j = 0; j < kUpper / 2; ++j) {
        const float hi = floorf(pacc[j] * (1.0f / kPackScale));
        acc[X + 2 * j] = pacc[j] - hi * kPackScale;
        acc[X + 2 * j + 1] = hi;
    }
    // tiers: [thres0 / 2], 3/4, {1, 9/8}, {3/2, 9/4, 27/8}: evaluated as far as the cell's maximum reaches
    const unsigned int t0 = __float_as_uint(cs[0]) >> 16, tq = __float_as_uint(cs[X]) >> 16,
                       t1 = __float_as_uint(cs[X + 1]) >> 16, t3 = __float_as_uint(cs[X + 3]) >> 16;
    auto count_upper = [&](const float4 x, const unsigned int rm) {   // rm > t0
        const float a0 = fabsf(x.x), a1 = fabsf(x.y), a2 = fabsf(x.z), a3 = fabsf(x.w);
        if (X == 1) {
            count_tier<0, 1>(a0, a1, a2, a3, cs, acc);
            if (rm <= tq) return;
        }
        count_tier<X, X + 1>(a0, a1, a2, a3, cs, acc);
        if (rm > t1) {
            count_tier<X + 1, X + 3>(a0, a1, a2, a3, cs, acc);
            if (rm > t3) count_tier<X + 3, NC>(a0, a1, a2, a3, cs, acc);
        }
    };
    unsigned int n_left = 0u;   // cells this warp had left
    for (int cursor = 0; cursor < nrows;) {
        const int n = gather_cells<kGatherFlagged>(table, nrows, cursor, sh.qrow[w], t0);
        n_left += (unsigned int)n;
        float4 v[kGroupRows];
#pragma unroll
        for (int q = 0; q < kGroupRows; ++q) {
            v[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (q < n) {
                const int r = sh.qrow[w][q];
                const int64_t i = first4 + (int64_t)r * stride4;
                if (i < n4) v[q] = (r >= first_kept) ? uslot[(size_t)(r % u_slots) * kRowF4 + tid] : __ldcg(u4 + i);
            }
        }
#pragma unroll
        for (int q = 0; q < kGroupRows; ++q) {
            if (q < n) count_upper(v[q], (unsigned int)table[sh.qrow[w][q] * kFusedWarps + w] & kMaxMask);
        }
        __syncwarp();
    }
    if (owns_tail) {
        const float a = fabsf(tail_u);
#pragma unroll
        for (int j = 0; j < NC; ++j) acc[j] += gt_as_float(a, cs[j]);
    }
#pragma unroll
    for (int j = 0; j < NC; ++j) {
        const unsigned int ws = __reduce_add_sync(0xffffffffu, (unsigned int)acc[j]);
        if (lane == 0 && ws) atomicAdd(&sh.cta_counts[cand_by_factor(kNumCand - NC + j)], ws);
    }
    if (lane == 0 && n_left) atomicAdd(&bars[kBarInfo + 3], n_left);
    __syncthreads();
}

// Phase B in full: all ten candidates over all cells of this CTA.  Leaves the CTA's counts in
// sh.cta_counts (cleared first when `again`: a second count after the short way).
__device__ __noinline__ void count_in_full(const float* __restrict__ uvec, const int64_t d, const int n_rows,
                                           const int u_slots, const float tail_u, const bool again) {
    GK_FUSED_VIEW(d, n_rows, u_slots);
    const float4* u4 = reinterpret_cast<const float4*>(uvec);
    // candidates in ascending order of value; cs[j] = value, sh.order[j] = its index
    float cs[kNumCand], acc[kNumCand];
#pragma unroll
    for (int j = 0; j < kNumCand; ++j) { cs[j] = sh.cand32[sh.order[j]]; acc[j] = 0.f; }
    // tier limits: top 16 bits of the tier's lowest candidate, rounded down; a negative
    // candidate is exceeded by everything, and candidates ascend, so testing the lowest suffices
    const Tiers tier = make_tiers(cs);
    const unsigned int always = 0x10000u;  // above every 16-bit maximum
    const bool any_neg = cs[0] < 0.f;
    const unsigned short* trow = table + w;
    auto row_max = [&](int r) -> unsigned int {
        return any_neg ? always : ((unsigned int)trow[r * kFusedWarps] & kMaxMask);
    };
    // rows that are not on chip come back from eps (L2 / HBM) through the ring that carried g
    // in phase A, kRing - 1 rows ahead of the counting; all of them are full rows.  They are
    // taken from the last written to the first: the rows written last are the ones most
    // likely still in L2, and reading them first keeps the misses on the oldest rows from
    // pushing them out before their turn.
    int64_t fo = first4 + (int64_t)(first_kept - 1) * stride4;  // the row the next fetch brings in
    auto fetch_u = [&](int q) {   // q-th row in this order: local row first_kept - 1 - q
        if (q < first_kept) cp_async16(gring + ((q & (kRing - 1)) << 10) + tid, u4 + fo);
        cp_async_commit();
        fo -= stride4;
    };
#pragma unroll
    for (int q = 0; q < kRing - 1; ++q) fetch_u(q);
    static_assert(kRowF4 == 1024 && (kRing & (kRing - 1)) == 0, "ring indexing assumes 1024-float4 rows, 2^n slots");
    // (two rows to an iteration: the counting is bound by its compare instructions, and two
    // independent rows keep the pipes busier than one)
#pragma unroll 2
    for (int q = 0; q < first_kept; ++q) {
        fetch_u(q + kRing - 1);
        cp_async_wait<kRing - 1>();
        count_float4(gring[((q & (kRing - 1)) << 10) + tid], row_max(first_kept - 1 - q), cs, tier, acc);
    }
    cp_async_wait<0>();
#pragma unroll 1
    for (int r = first_kept; r < nrows; ++r) {
        if (r != nrows - 1 || in_last_row)
            count_float4(uslot[(size_t)(r % u_slots) * kRowF4 + tid], row_max(r), cs, tier, acc);
    }
    if (owns_tail) {
        const float a = fabsf(tail_u);
#pragma unroll
        for (int j = 0; j < kNumCand; ++j) acc[j] += gt_as_float(a, cs[j]);
    }
    if (again) {
        __syncthreads();   // the first count's sums have been read by everyone
        if (tid < kNumCand) sh.cta_counts[tid] = 0u;
        __syncthreads();
    }
#pragma unroll
    for (int j = 0; j < kNumCand; ++j) {
        const unsigned int ws = __reduce_add_sync(0xffffffffu, (unsigned int)acc[j]);
        if (lane == 0 && ws) atomicAdd(&sh.cta_counts[sh.order[j]], ws);
    }
    __syncthreads();
}

// Phase B, the selected way: every cell of this CTA against the candidates of sh.sel_idx
// (ascending; empty places hold +inf, which nothing exceeds).  Every candidate is its own tier:
// it is evaluated only where the cell's maximum reaches it.
__device__ __noinline__ void count_selected(const float* __restrict__ uvec, const int64_t d, const int n_rows,
                                            const int u_slots, const float tail_u) {
    GK_FUSED_VIEW(d, n_rows, u_slots);
    const float4* u4 = reinterpret_cast<const float4*>(uvec);
    const int n_sel = sh.sel_n;
    float cs[kSelMax], acc[kSelMax];
    unsigned int lim[kSelMax];
#pragma unroll
    for (int j = 0; j < kSelMax; ++j) {
        cs[j] = j < n_sel ? sh.cand32[sh.sel_idx[j]] : INFINITY;   // all positive: thres0 > 0
        acc[j] = 0.f;
        lim[j] = __float_as_uint(cs[j]) >> 16;
    }
    const unsigned short* trow = table + w;
    auto count4 = [&](const float4 v, const unsigned int rm) {   // rm: the cell's maximum, as in count_float4
        if (rm <= lim[0]) return;
        const float a0 = fabsf(v.x), a1 = fabsf(v.y), a2 = fabsf(v.z), a3 = fabsf(v.w);
        count_tier<0, 1>(a0, a1, a2, a3, cs, acc);
        if (rm <= lim[1]) return;
        count_tier<1, 2>(a0, a1, a2, a3, cs, acc);
        if (rm <= lim[2]) return;
        count_tier<2, 3>(a0, a1, a2, a3, cs, acc);
        if (rm <= lim[3]) return;
        count_tier<3, 4>(a0, a1, a2, a3, cs, acc);
        if (rm <= lim[4]) return;
        count_tier<4, 5>(a0, a1, a2, a3, cs, acc);
        if (rm <= lim[5]) return;
        count_tier<5, 6>(a0, a1, a2, a3, cs, acc);
    };
    static_assert(kSelMax == 6, "one tier per selected candidate");
    // the rows that are not on chip come through the ring, last written first, as in the full count
    int64_t fo = first4 + (int64_t)(first_kept - 1) * stride4;
    auto fetch_u = [&](int q) {
        if (q < first_kept) cp_async16(gring + ((q & (kRing - 1)) << 10) + tid, u4 + fo);
        cp_async_commit();
        fo -= stride4;
    };
#pragma unroll
    for (int q = 0; q < kRing - 1; ++q) fetch_u(q);
#pragma unroll 2
    for (int q = 0; q < first_kept; ++q) {
        fetch_u(q + kRing - 1);
        cp_async_wait<kRing - 1>();
        count4(gring[((q & (kRing - 1)) << 10) + tid], (unsigned int)trow[(first_kept - 1 - q) * kFusedWarps] & kMaxMask);
    }
    cp_async_wait<0>();
#pragma unroll 1
    for (int r = first_kept; r < nrows; ++r) {
        if (r != nrows - 1 || in_last_row)
            count4(uslot[(size_t)(r % u_slots) * kRowF4 + tid], (unsigned int)trow[r * kFusedWarps] & kMaxMask);
    }
    if (owns_tail) {
        const float a = fabsf(tail_u);
#pragma unroll
        for (int j = 0; j < kSelMax; ++j) acc[j] += gt_as_float(a, cs[j]);
    }
#pragma unroll
    for (int j = 0; j < kSelMax; ++j) {
        const unsigned int ws = __reduce_add_sync(0xffffffffu, (unsigned int)acc[j]);
        if (lane == 0 && ws && j < n_sel) atomicAdd(&sh.cta_counts[sh.sel_idx[j]], ws);
    }
    __syncthreads();
}

// Phase C: the survivors |u_i| > threshold of this CTA's rows, counted per cell, the per-row
// totals exchanged through one more grid barrier, then written as ordered pairs (and their
// slots of eps cleared, ACC).  Returns false when the barrier's bounded wait ran out.
template <bool ACC>
__device__ __noinline__ bool compact_survivors(const float* __restrict__ uvec, float* __restrict__ eps, const int64_t d,
                                               const int n_rows, const int u_slots, const unsigned int bar_target,
                                               unsigned int* __restrict__ bars, unsigned int* __restrict__ rowcnt,
                                               int32_t* __restrict__ idx_out, float* __restrict__ val_out,
                                               const int64_t cap, const float tail_u,
                                               unsigned long long* __restrict__ trace) {
    GK_FUSED_VIEW(d, n_rows, u_slots);
    const float4* u4 = reinterpret_cast<const float4*>(uvec);
    auto stamp = [&](int slot) {
        if (trace != nullptr && tid == 0) trace[(size_t)c * kTraceSlots + slot] = global_timer_ns();
    };
    {
        const float thr = sh.thr_sel;
        const unsigned int mine = sh.cta_counts[sh.chosen];  // survivors in this CTA's rows
        // a segment can hold a survivor only if its recorded maximum (rounded up to 16 bits)
        // exceeds the threshold's top 16 bits; a negative threshold admits everything
        const bool all_pass = thr < 0.0f;
        const unsigned int thr16 = __float_as_uint(fmaxf(thr, 0.0f)) >> 16;
        auto load_row = [&](int r, int64_t i) -> float4 {
            return (r >= first_kept) ? uslot[(size_t)(r % u_slots) * kRowF4 + tid] : __ldcg(u4 + i);
        };
        // When this CTA's survivors fit the ring's shared memory (free since phase B), their
        // places -- row, warp, lane, element, rank within the segment: one word -- are put aside
        // while they are counted, and the write-out is one thread per survivor instead of one
        // warp per segment; with many survivors the per-segment work of 32 warps was what the
        // phase cost.
        const bool staged = mine <= (unsigned)kStageCap;
        unsigned int* st_tag = reinterpret_cast<unsigned int*>(gring);
        if (mine != 0u) {
            // step 1: every warp counts the survivors of its qualifying segments; the table
            // entry of a segment is replaced by that count (0 where it cannot qualify).
            int pending = 0;
            for (int r = lane; r < nrows; r += 32) {
                const bool ql = all_pass || ((unsigned int)table[r * kFusedWarps + w] & kMaxMask) > thr16;
                table[r * kFusedWarps + w] = ql ? kPending : (unsigned short)0;
                pending += ql;
            }
            pending = __reduce_add_sync(0xffffffffu, pending);
            const bool many = pending * 4 > nrows;   // then the rows are taken as they come, eight at a time
            __syncwarp();
            const unsigned int lanes_below = (1u << lane) - 1u;
            // one segment of local row r: m has a bit for each survivor in this thread's float4
            auto count_cell = [&](const int r, const unsigned int m) {
                const unsigned int cnt = __reduce_add_sync(0xffffffffu, __popc(m));
                if (lane == 0) table[r * kFusedWarps + w] = (unsigned short)cnt;
                if (staged && cnt != 0u) {
                    unsigned int base = 0u;
                    if (lane == 0) base = atomicAdd(&sh.n_staged, cnt);
                    base = __shfl_sync(0xffffffffu, base, 0);
                    unsigned int rank = 0u;
                    if (cnt > 1u) {
                        // one ballot per element of the float4: the bits below this lane are its rank
                        const unsigned int b0 = __ballot_sync(0xffffffffu, m & 1u), b1 = __ballot_sync(0xffffffffu, m & 2u),
                                           b2 = __ballot_sync(0xffffffffu, m & 4u), b3 = __ballot_sync(0xffffffffu, m & 8u);
                        rank = __popc(b0 & lanes_below) + __popc(b1 & lanes_below) + __popc(b2 & lanes_below) +
                               __popc(b3 & lanes_below);
                    }
                    if (m) {
                        const unsigned int place = ((unsigned int)r << 19) | ((unsigned int)w << 14) | ((unsigned int)lane << 9);
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            if (m & (1u << t)) {
                                st_tag[base + rank] = place | ((unsigned int)t << 7) | rank;
                                ++rank;
                            }
                        }
                    }
                }
            };
            // else the qualifying segments are gathered, eight at a time; either way their loads overlap
            for (int cursor = 0; cursor < nrows;) {
                int n;
                if (many) {
                    n = 0;
                    const int r = cursor + lane;
                    const unsigned int pend = __ballot_sync(0xffffffffu, lane < kGroupRows && r < nrows &&
                                                                             table[r * kFusedWarps + w] == kPending);
                    if (lane < kGroupRows && ((pend >> lane) & 1u)) sh.qrow[w][__popc(pend & ((1u << lane) - 1u))] = (unsigned short)r;
                    n = __popc(pend);
                    cursor += kGroupRows;
                    __syncwarp();
                } else {
                    n = gather_cells<kGatherPending>(table, nrows, cursor, sh.qrow[w]);
                }
                float4 v[kGroupRows];
#pragma unroll
                for (int q = 0; q < kGroupRows; ++q) {
                    v[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (q < n) {
                        const int r = sh.qrow[w][q];
                        const int64_t i = (first4 + (int64_t)r * stride4);
                        if (i < n4) v[q] = load_row(r, i);
                    }
                }
                // the eight masks of this thread in one word, so that the segments can be taken one
                // after the other by one copy of the code
                unsigned int masks = 0u;
#pragma unroll
                for (int q = 0; q < kGroupRows; ++q) {
                    if (q < n && first4 + (int64_t)sh.qrow[w][q] * stride4 < n4) masks |= mask_above(v[q], thr) << (4 * q);
                }
#pragma unroll 1
                for (int q = 0; q < n; ++q) count_cell(sh.qrow[w][q], (masks >> (4 * q)) & 15u);
                __syncwarp();
            }
        }
        __syncthreads();
        // step 2: survivors per row (thread t takes local row t) go to the row's word in global
        // memory; every row of the vector gets its word from the CTA that owns it
        if (tid < nrows) {
            unsigned int mine_row = 0u;
            if (mine != 0u) {
                uint4* tv = reinterpret_cast<uint4*>(table + (size_t)tid * kFusedWarps);
#pragma unroll
                for (int q = 0; q < kTableRowBytes / 16; ++q) {
                    const uint4 x = tv[q];
                    if (staged) {
                        // the entries become the survivors of the row in the warps before each one
                        // (at most 3968: sixteen bits hold it), which is what the write-out needs
                        unsigned int ws[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const unsigned int lo = ws[j] & 0xffffu, hi = ws[j] >> 16;
                            ws[j] = mine_row | ((mine_row + lo) << 16);
                            mine_row += lo + hi;
                        }
                        tv[q] = make_uint4(ws[0], ws[1], ws[2], ws[3]);
                    } else {
                        mine_row += (x.x & 0xffffu) + (x.x >> 16) + (x.y & 0xffffu) + (x.y >> 16) +
                                    (x.z & 0xffffu) + (x.z >> 16) + (x.w & 0xffffu) + (x.w >> 16);
                    }
                }
            }
            rowcnt[c + tid * G] = mine_row;
        }
        stamp(5);
        if (!grid_barrier(&bars[kBarRows], bar_target, &sh.ok)) {
            return false;
        }
        stamp(6);
        if (mine != 0u) {
            // Survivors before local row r of this CTA = those of the rounds before r (round r is
            // the G consecutive rows r * G ... r * G + G - 1) + those of the CTAs before this one
            // in round r.  Warp j takes rounds j, j + 32, ...
            for (int r = w; r < nrows; r += kFusedWarps) {
                unsigned int tot = 0u, pre = 0u;
                const int R0 = r * G;
                for (int t = lane; t < G; t += 32) {
                    const unsigned int v = (R0 + t < n_rows) ? __ldcg(rowcnt + R0 + t) : 0u;
                    tot += v;
                    pre += (t < c) ? v : 0u;
                }
                tot = __reduce_add_sync(0xffffffffu, tot);
                pre = __reduce_add_sync(0xffffffffu, pre);
                if (lane == 0) { sh.roundtot[r] = tot; sh.rowpre[r] = pre; }
            }
            __syncthreads();
            // exclusive scan of the round totals (thread t takes round t; at most kTableMaxRows)
            {
                const unsigned int mine_round = tid < nrows ? sh.roundtot[tid] : 0u;
                unsigned int s = mine_round;
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
                if (tid < nrows) sh.rowpre[tid] += wpre + s - mine_round;
                __syncthreads();
            }
            if (staged) {
                // step 3: one thread per survivor put aside: its place gives its index, where its
                // value is, and its position in the output
                const unsigned int n_st = sh.n_staged;
                for (unsigned int j = tid; j < n_st; j += kFusedThreads) {
                    const unsigned int tag = st_tag[j];
                    const unsigned int r = tag >> 19, cell = (tag >> 14) & 31u, ln = (tag >> 9) & 31u, t = (tag >> 7) & 3u,
                                       rank = tag & 127u;
                    const long long p = (long long)sh.rowpre[r] + table[r * kFusedWarps + cell] + rank;
                    if (p < cap) {
                        const unsigned int in_row = ((cell << 5) | ln) << 2 | t;   // element within the row
                        const int64_t at = (((int64_t)c + (int64_t)r * G) << 12) + in_row;
                        const float x = ((int)r >= first_kept)
                                            ? reinterpret_cast<const float*>(uslot + (size_t)(r % u_slots) * kRowF4)[in_row]
                                            : __ldcg(uvec + at);
                        idx_out[p] = (int32_t)at;
                        val_out[p] = x;
                        if (ACC) eps[at] = 0.0f;
                    }
                }
            } else
            // step 3: every warp writes the survivors of its segments that have any
            for (int cursor = 0; cursor < nrows;) {
                const int n = gather_cells<kGatherNonZero>(table, nrows, cursor, sh.qrow[w]);
                // (the ring holds no places here: the cells that are not on chip land in it, slot q
                // for the q-th, and are then taken one after the other)
#pragma unroll
                for (int q = 0; q < kGroupRows; ++q) {
                    if (q < n) {
                        const int r = sh.qrow[w][q];
                        const int64_t i = (first4 + (int64_t)r * stride4);
                        if (i < n4 && r < first_kept) cp_async16(gring + (q << 10) + tid, u4 + i);
                    }
                }
                cp_async_commit();
                cp_async_wait<0>();
#pragma unroll 1
                for (int q = 0; q < n; ++q) {
                    const int r = sh.qrow[w][q];
                    const int64_t i = (first4 + (int64_t)r * stride4);
                    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (i < n4) x = (r >= first_kept) ? uslot[(size_t)(r % u_slots) * kRowF4 + tid] : gring[(q << 10) + tid];
                    const unsigned int m = i < n4 ? mask_above(x, thr) : 0u;
                    // survivors of this row in the warps before this one
                    const unsigned int before =
                        __reduce_add_sync(0xffffffffu, lane < w ? (unsigned int)table[r * kFusedWarps + lane] : 0u);
                    const unsigned int c_m = __popc(m);
                    unsigned int sc = c_m;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned int t = __shfl_up_sync(0xffffffffu, sc, o);
                        if (lane >= o) sc += t;
                    }
                    if (m) {
                        long long p = (long long)sh.rowpre[r] + before + (sc - c_m);
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
                __syncwarp();
            }
        }
        // the ragged tail comes last in index order
        if ((c == G - 1) && (w == kFusedWarps - 1) && (d & 3)) {
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
    }

    return true;
}

// ACC: the sparsifier (src = g, u = g + eps is formed, stored over eps and cleared where
// selected); !ACC: the operator on a given vector (src = u, read only; eps is not used).
// n_rows: rows of 1024 float4 in the whole vector; CTA c owns rows c, c + G, c + 2G, ...
// (G = gridDim.x), so that stretches of large values are spread over all CTAs.  u_slots: row
// slots of shared memory that receive eps and then hold u (the last u_slots rows of a CTA stay
// on chip); call_no: the number of this launch on its scratch, never 0 (the CTAs' records of partial
// sums carry it; `partials` points to one 32-byte record per CTA and one more).
// PRED: count during phase A against predicted thresholds (the vector must have at least 32
// float4 and no CTA more than kPredMaxRows rows); bar_target: arrivals a grid barrier waits for (the grid size; a test may ask for more
// to see the bounded waits run out).  rowcnt: one word per row.
template <bool ACC, bool PRED>
__global__ void __launch_bounds__(kFusedThreads, 1)
k_gk_fused(const float* __restrict__ src, float* __restrict__ eps, int64_t d, int64_t k, double z,
           int n_rows, int u_slots, unsigned int call_no, unsigned int bar_target, Ctrl* __restrict__ ctrl,
           double2* __restrict__ partials, unsigned int* __restrict__ bars,
           unsigned int* __restrict__ rowcnt, int32_t* __restrict__ idx_out, float* __restrict__ val_out,
           int64_t* __restrict__ nnz_out, int64_t cap, unsigned long long* __restrict__ trace) {
    GK_FUSED_VIEW(d, n_rows, u_slots);
    const float4* g4 = reinterpret_cast<const float4*>(src);
    float4* e4 = reinterpret_cast<float4*>(eps);
    // where u is read again after phase A: eps holds it for the sparsifier, the input itself otherwise
    const float* uvec = ACC ? eps : src;
    float tail_u = 0.f;
    const bool wide_ok = ACC && ((reinterpret_cast<uintptr_t>(eps) & 31u) == 0);  // 32-byte stores possible
    unsigned long long* tot0 = reinterpret_cast<unsigned long long*>(bars + kBarTotals);   // first count
    unsigned long long* tot1 = tot0 + kNumCand;                                            // the second, full one
    if (c == 0 && tid == 0) {
        ctrl->stats.status = GK_DEV_OK;
        ctrl->phase_t[0] = global_timer_ns();
    }
    if (PRED) {
        if (tid == 0) { sh.samp_n = 0u; sh.pred_ready = 0; }
        __syncthreads();
    }
    // optional per-CTA trace: start, before / after each barrier, end
    auto stamp = [&](int slot) {
        if (trace != nullptr && tid == 0) trace[(size_t)c * kTraceSlots + slot] = global_timer_ns();
    };
    stamp(0);

    // phase A's counts of the six upper candidates over the cells it settled
    // (two candidates to a float: counts of candidates 2 j and 2 j + 1 as lo + 8192 * hi)
    float pacc[kUpper / 2];
#pragma unroll
    for (int j = 0; j < kUpper / 2; ++j) pacc[j] = 0.f;

    // ------------------------------------------------------------------ phase A
    {
        const double pv = (double)src[0];
        double s0 = 0.0, q0 = 0.0, s1 = 0.0, q1 = 0.0;
        // rows are fetched kStages - 1 ahead by asynchronous copies: g into a ring, eps into the
        // slot that will hold u.  Every thread copies and later reads only its own 16 bytes.
        // The operator form has one operand, which takes the way of eps.
        int64_t fi = first4;  // the row the next fetch brings in
        // Where the eps of local row r lands.  Normally the slot that will hold u.  A CTA with so
        // many rows that its table leaves fewer slots than rows in flight takes eps through the
        // half of the ring that g does not use, and only its last rows are kept on chip.
        const bool eps_ring = u_slots < kStages;
        auto eps_slot = [&](int r) -> float4* {
            return eps_ring ? gring + (size_t)(kStages + r % kStages) * kRowF4 : uslot + (size_t)(r % u_slots) * kRowF4;
        };
        auto fetch = [&](int r) {
            if (r < nrows && fi < n4) {
                if (ACC) {
                    cp_async16(gring + (size_t)(r % kStages) * kRowF4 + tid, g4 + fi);
                    cp_async16(eps_slot(r) + tid, e4 + fi);
                } else {
                    cp_async16(eps_slot(r) + tid, g4 + fi);
                }
            }
            cp_async_commit();
            fi += stride4;
        };
        int pred_state = PRED ? 1 : 0;   // this warp still waits for the predicted bands
        // the sample's loads go first: they are in flight while the first rows are fetched and are
        // read (and parked in shared memory) only after row 0
        float4 sample_g = make_float4(0.f, 0.f, 0.f, 0.f), sample_e = make_float4(0.f, 0.f, 0.f, 0.f);
        if (PRED) {
            const int64_t at = sample_at(n4);
            sample_g = __ldcg(g4 + at);
            if (ACC) sample_e = __ldcg(e4 + at);
        }
#pragma unroll
        for (int r = 0; r < kStages - 1; ++r) fetch(r);
        // warp 0, lanes 0..4: the global sample sums (lanes 0..3) and the count of CTAs (lane 4) at its last look
        unsigned long long seen = 0ull;
        const unsigned long long* sums = reinterpret_cast<const unsigned long long*>(bars + kBarSample);
        unsigned int ptl0 = 0u, ptl1 = 0u, ptl3 = 0u;   // tier limits of the predicted bands

        // One row: u = g + eps out to eps and into its slot, the fp64 sums, the cell's table entry.
        // COUNTING: the prediction is in place and the six upper candidates are counted on the way.
        auto row_body = [&](const int r, const int64_t i, auto counting) {
            constexpr bool COUNTING = decltype(counting)::value;
            fetch(r + kStages - 1);
            cp_async_wait<kStages - 1>();
            const bool one = i < n4;
            float4 u0 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (one) {
                float4* es = eps_slot(r) + tid;
                if (ACC) {
                    const float4 a0 = gring[(size_t)(r % kStages) * kRowF4 + tid], b0 = *es;
                    u0 = make_float4(a0.x + b0.x, a0.y + b0.y, a0.z + b0.z, a0.w + b0.w);
                    if (!eps_ring) *es = u0;
                } else {
                    u0 = *es;
                }
                if (eps_ring && r >= first_kept) uslot[(size_t)(r % u_slots) * kRowF4 + tid] = u0;
                const double x0 = (double)u0.x - pv, x1 = (double)u0.y - pv, x2 = (double)u0.z - pv,
                             x3 = (double)u0.w - pv;
                s0 += x0; q0 = fma(x0, x0, q0); s1 += x1; q1 = fma(x1, x1, q1);
                s0 += x2; q0 = fma(x2, x2, q0); s1 += x3; q1 = fma(x3, x3, q1);
            }
            // u goes out in 32-byte stores by the even lanes (own float4 and the right neighbour's),
            // marked to stay in L2: the next two phases read most of u again
            if (ACC) {
                float4 nb;
                nb.x = __shfl_down_sync(0xffffffffu, u0.x, 1); nb.y = __shfl_down_sync(0xffffffffu, u0.y, 1);
                nb.z = __shfl_down_sync(0xffffffffu, u0.z, 1); nb.w = __shfl_down_sync(0xffffffffu, u0.w, 1);
                const bool pair = wide_ok && (i + 1 < n4);  // this lane and its right neighbour are in range
                if ((lane & 1) == 0) {
                    if (pair) st_keep32(e4 + i, u0, nb);
                    else if (one) e4[i] = u0;
                } else if (one && !wide_ok) {
                    e4[i] = u0;
                }
            }
            // largest magnitude of each (row, warp) cell, top 16 bits rounded up (15 bits for
            // finite values), and above it the flag "not settled here"
            const unsigned int m0 = __reduce_max_sync(0xffffffffu, one ? max_mag_bits(u0) : 0u);
            unsigned int entry = (m0 + 0xffffu) >> 16;
            if (!COUNTING) {
                entry |= kFlagBit;
            } else if (entry > ptl0) {
                // the cell can reach the lowest band: per candidate the elements above the band's
                // upper edge, and over all candidates those above the lower edges; the two sums
                // differ exactly when an element lies inside a band
                const float a0 = fabsf(u0.x), a1 = fabsf(u0.y), a2 = fabsf(u0.z), a3 = fabsf(u0.w);
                float h[kUpper];
#pragma unroll
                for (int j = 0; j < kUpper; ++j) h[j] = 0.f;
                float below = 0.f;
                auto band = [&](const int j) {
                    const float lo = sh.plo[j], hi = sh.phi[j];
                    h[j] = (gt_as_float(a0, hi) + gt_as_float(a1, hi)) + (gt_as_float(a2, hi) + gt_as_float(a3, hi));
                    below += (gt_as_float(a0, lo) + gt_as_float(a1, lo)) + (gt_as_float(a2, lo) + gt_as_float(a3, lo));
                };
                band(0);
                if (entry > ptl1) {
                    band(1); band(2);
                    if (entry > ptl3) { band(3); band(4); band(5); }
                }
                const float above = ((h[0] + h[1]) + (h[2] + h[3])) + (h[4] + h[5]);
                if (__any_sync(0xffffffffu, below != above)) {
                    entry |= kFlagBit;
                } else {
#pragma unroll
                    for (int j = 0; j < kUpper / 2; ++j) pacc[j] += fmaf(h[2 * j + 1], kPackScale, h[2 * j]);
                }
            }
            if (lane == 0) table[r * kFusedWarps + w] = (unsigned short)entry;
        };

        // The rows stream in three stretches: the first kStages - 1 rows, behind whose copies the
        // sample's were issued; then, the sample having landed, every warp hands its sums in
        // (between the loops: a call inside a streaming loop would cost registers in every
        // iteration) and the rows go on until the predicted bands are there; from then on with
        // the counting.  Each warp changes over by itself, at a row of its own: a cell is
        // flagged or settled by the one warp that handles it.  Warp 0 reads the band block once
        // per row (the load is issued before the row and looked at after it) and gives up after
        // a third of its rows.
        int r = 0;
        int64_t i = first4;
        if (nrows > 0) { row_body(0, i, std::false_type{}); r = 1; i += stride4; }
        if (PRED) {
            gring[(size_t)kStages * kRowF4 + tid] = sample_g;
            if (ACC) gring[(size_t)(kStages + 1) * kRowF4 + tid] = sample_e;
        }
        for (; r < nrows && r < kStages - 1; ++r, i += stride4) row_body(r, i, std::false_type{});
        if (PRED) {
            publish_sample<ACC>(gring, pv, &sh, bars);
            for (; r < nrows; ++r, i += stride4) {
                if (r >= kStages) {
                    const int word = *reinterpret_cast<volatile int*>(&sh.pred_ready);
                    if (word == 1) break;              // on to the counting stretch
                    if (word != 0) pred_state = 0;     // no prediction: nothing to wait for
                }
                const bool looking = pred_state != 0 && w == 0;
                if (looking && lane < 5)
                    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(seen) : "l"(sums + lane));
                row_body(r, i, std::false_type{});
                if (looking) {
                    const unsigned int in = (unsigned int)__shfl_sync(0xffffffffu, seen, 4);
                    const bool late = 3 * r >= nrows;   // too late to be worth having
                    if (in >= (unsigned)G || late) {
                        const double a1 = __longlong_as_double(__shfl_sync(0xffffffffu, seen, 0)),
                                     a2 = __longlong_as_double(__shfl_sync(0xffffffffu, seen, 1)),
                                     a3 = __longlong_as_double(__shfl_sync(0xffffffffu, seen, 2)),
                                     a4 = __longlong_as_double(__shfl_sync(0xffffffffu, seen, 3));
                        if (lane == 0) {
                            const bool ok = in >= (unsigned)G &&
                                            predict_bands(a1, a2, a3, a4, (double)G * kSampleElems, pv, z, sh.plo, sh.phi);
                            __threadfence_block();
                            *reinterpret_cast<volatile int*>(&sh.pred_ready) = ok ? 1 : 2;
                        }
                        pred_state = 0;
                    }
                }
            }
            if (r < nrows) {
                // top 16 bits of each tier's lowest band edge, rounded down (the edges are positive)
                ptl0 = __float_as_uint(sh.plo[0]) >> 16;
                ptl1 = __float_as_uint(sh.plo[1]) >> 16;
                ptl3 = __float_as_uint(sh.plo[3]) >> 16;
                for (; r < nrows; ++r, i += stride4) row_body(r, i, std::true_type{});
            }
            if (w == 0 && lane == 0 && *reinterpret_cast<volatile int*>(&sh.pred_ready) == 0)
                *reinterpret_cast<volatile int*>(&sh.pred_ready) = 2;   // nobody waits for bands any more
        } else {
            for (; r < nrows; ++r, i += stride4) row_body(r, i, std::false_type{});
        }
        cp_async_wait<0>();
        if (owns_tail) {
            tail_u = ACC ? src[tail_i] + eps[tail_i] : src[tail_i];
            if (ACC) eps[tail_i] = tail_u;
            const double x = (double)tail_u - pv;
            s0 += x; q0 = fma(x, x, q0);
        }
        const double2 part = block_sum2<kFusedThreads>(s0 + s1, q0 + q1, sh.red);
        unsigned int* const recs = reinterpret_cast<unsigned int*>(partials);
        if (tid == 0) store_partial(recs + (size_t)c * kPartialWords, call_no, part.x, part.y);
        stamp(1);
        // Grid barrier 1 is the arrival of the sums themselves: thread t waits for the record of
        // CTA t (bounded polls), and every CTA forms the same totals from the same records in the
        // same order.  (A counter would cost a fence that waits for this CTA's stores of u, which
        // nobody else reads, then the counter's round trip, then the records' round trip.)  A
        // test's extra arrivals are records that nobody writes.
        double s = 0.0, q = 0.0;
        bool arrived = true;
        {
            const int limit = g_barrier_poll_limit;
            for (int t = tid; t < (int)bar_target; t += kFusedThreads) {
                double ps = 0.0, pq = 0.0;
                int polls = 0;
                while (!load_partial(recs + (size_t)t * kPartialWords, call_no, ps, pq)) {
                    if (++polls > limit) { arrived = false; break; }
                    __nanosleep(100);
                }
                if (arrived && t < G) { s += ps; q += pq; }
            }
        }
        if (!__syncthreads_and(arrived)) {
            if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
            goto leave;
        }
        stamp(2);
        const double2 tot = block_sum2<kFusedThreads>(s, q, sh.red);
        if (tid == 0) {
            const Alg1State st{&sh.stats, sh.cand64, sh.cand32, sh.col, &sh.thr_sel};
            alg1_thresholds(st, tot.x, tot.y, pv, d, k, z);
            // candidate indices in ascending order of threshold
            const bool neg = sh.stats.thres0 < 0.0;
#pragma unroll
            for (int j = 0; j < kNumCand; ++j) sh.order[j] = cand_ascending(j, neg);
            // phase A's counts stand if every exact candidate lies within its predicted band
            bool fast = PRED && sh.pred_ready == 1 && sh.stats.thres0 > 0.0;
            if (fast) {
#pragma unroll
                for (int j = 0; j < kUpper; ++j) {
                    const float cj = sh.cand32[cand_by_factor(kNumCand - kUpper + j)];
                    fast = fast && sh.plo[j] <= cj && cj <= sh.phi[j];
                }
            }
            sh.fast = fast ? 1 : 0;
            sh.k_wanted = k;
            if (PRED && sh.pred_ready == 1) atomicAdd(&bars[kBarInfo + 0], 1u);
            sh.recount = 0;
        }
        if (tid < kNumCand) sh.cta_counts[tid] = 0u;
        // (vectors large enough for the prediction are left as they are: where it fails, on heavy
        // tails or loud stretches, the estimate behind the selected way fails too)
        if (!PRED) decide_short_way(d, n_rows, u_slots);
        if (c == 0 && tid == 0) ctrl->phase_t[1] = global_timer_ns();
        __syncthreads();
    }

    // ------------------------------------------------------------------ phase B and the rounds
    // First count: the short way where this CTA's prediction held, else in full.  If the rounds
    // then ask for a candidate that some CTA left out, the CTAs that took the short way count
    // again in full and the sums are formed a second time.
    for (int pass = 0; pass < 2; ++pass) {
        const int way = pass == 0 ? sh.fast : 0;
        const bool fast = way != 0;
        if (way == 1) {
            if (PRED) count_short_way<kUpper>(uvec, d, n_rows, u_slots, pacc[0], pacc[1], pacc[2], tail_u, bars);
            else count_short_way<kUpper + 1>(uvec, d, n_rows, u_slots, 0.f, 0.f, 0.f, tail_u, bars);
        }
        else if (way == 2) count_selected(uvec, d, n_rows, u_slots, tail_u);
        else if (pass == 0 || sh.fast != 0) count_in_full(uvec, d, n_rows, u_slots, tail_u, pass == 1);
        // Grid barrier 2 is the arrival of the counts themselves.  This CTA's ten counts join ten
        // 64-bit words, each with a 1 in the word's arrival field and a 1 in its "left out" field
        // where a short way did not count the candidate; lane j of warp 0 then polls word j until
        // every CTA has added to it (bounded), and has count, arrivals and left-out flag in one
        // load: no counter, no fence, no second round trip for the sums.
        if (tid < kNumCand) {
            const unsigned int left = !fast ? 0u : way == 2 ? (kAllCandMask & ~sh.sel_mask)
                                                 : PRED ? kLowCandMask : (kLowCandMask & ~(1u << cand_index(1, 0)));
            atomicAdd((pass == 0 ? tot0 : tot1) + tid,
                      (1ull << kTotArriveShift) | ((unsigned long long)((left >> tid) & 1u) << kTotLeftShift) |
                          (unsigned long long)sh.cta_counts[tid]);
        }
        if (fast && tid == 0) atomicAdd(&bars[kBarInfo + (way == 2 ? 4 : 1)], 1u);
        if (c == 0 && tid == 0) ctrl->phase_t[2] = global_timer_ns();
        stamp(3);
        bool arrived = true;
        if (w == 0) {
            unsigned long long v = 0ull;
            if (lane < kNumCand) {
                const unsigned long long* word = (pass == 0 ? tot0 : tot1) + lane;
                const int limit = g_barrier_poll_limit;
                int polls = 0;
                while (true) {
                    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
                    if ((unsigned int)(v >> kTotArriveShift) >= bar_target) break;
                    if (++polls > limit) { arrived = false; break; }
                    __nanosleep(40);
                }
                sh.col[lane] = v & kTotCountMask;
            }
            // the candidates some CTA left out
            const unsigned int lo = __ballot_sync(0xffffffffu, lane < kNumCand && ((v >> kTotLeftShift) & 0xfffull) != 0ull);
            if (lane == 0) sh.left_out = lo;
        }
        if (!__syncthreads_and(arrived)) {
            if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
            goto leave;
        }
        if (c == 0 && tid == 0) ctrl->phase_t[3] = global_timer_ns();
        stamp(4);

        // -------------------------------------------------------------- the rounds
        if (tid == 0) {
            const Alg1State st{&sh.stats, sh.cand64, sh.cand32, sh.col, &sh.thr_sel};
            unsigned int visited = 0u;
            sh.chosen = alg1_resolve(st, k, &visited);
            sh.n_staged = 0u;
            // a candidate the rounds evaluated but some CTA did not count: count again, in full
            sh.recount = (pass == 0 && (visited & sh.left_out) != 0u) ? 1 : 0;
        }
        __syncthreads();
        if (!sh.recount) break;
        if (c == 0 && tid == 0) bars[kBarInfo + 2] = 1u;
    }
    if (c == 0 && tid == 0) {
        const long long all = sh.stats.nnz;
        const long long written = all < cap ? all : cap;
        // every field but the status word, which was cleared at the start and only ever has
        // flags added to it (a CTA that gave up waiting may have added one already)
        gk_stats* o = &ctrl->stats;
        o->mu = sh.stats.mu; o->sigma = sh.stats.sigma; o->z = sh.stats.z;
        o->thres0 = sh.stats.thres0; o->thr_final = sh.stats.thr_final;
#pragma unroll
        for (int j = 0; j < 4; ++j) o->counts[j] = sh.stats.counts[j];
        o->rounds = sh.stats.rounds; o->nnz = all; o->emitted = written;
        const int flags = sh.stats.status | (all > cap ? GK_DEV_TRUNCATED : 0);
        if (flags) atomicOr(&o->status, flags);
        *nnz_out = written;
        ctrl->phase_t[4] = global_timer_ns();
    }

    // ------------------------------------------------------------------ phase C
    // The survivor count of the whole vector is known to every CTA; with none there is nothing
    // left to do (the same decision in every CTA, so the barrier inside is reached by all or none).
    if (sh.stats.nnz != 0) {
        if (!compact_survivors<ACC>(uvec, eps, d, n_rows, u_slots, bar_target, bars, rowcnt, idx_out, val_out, cap,
                                    tail_u, trace)) {
            if (tid == 0) atomicOr(&ctrl->stats.status, GK_DEV_TIMEOUT);
            goto leave;
        }
    }

    if (c == 0 && tid == 0) ctrl->phase_t[5] = global_timer_ns();
    stamp(7);

leave:
    // the CTA that leaves last clears the barrier counters for the next call
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(&bars[kBarExit], 1u);
        if (t == (unsigned)G - 1) {
            // the words to report are read first, all at once: the kernel ends when this thread
            // does, and a load that waits behind the previous word's stores costs a round trip each
            unsigned int info[5];
#pragma unroll
            for (int j = 0; j < 5; ++j) info[j] = __ldcg(&bars[kBarInfo + j]);
            ctrl->phase_t[6] = global_timer_ns();
            bars[kBarRows] = 0u;
#pragma unroll
            for (int j = 0; j < 2 * kNumCand; ++j) reinterpret_cast<unsigned long long*>(bars + kBarTotals)[j] = 0ull;
#pragma unroll
            for (int j = 0; j < 9; ++j) bars[kBarSample + j] = 0u;
#pragma unroll
            for (int j = 0; j < 5; ++j) { ctrl->path_info[j] = info[j]; bars[kBarInfo + j] = 0u; }
            // (no fence before the last word: the end of the kernel orders all of these stores
            // before the next launch on this stream, the only reader)
            bars[kBarExit] = 0u;
        }
    }
}

// Host side -----------------------------------------------------------------
struct FusedPlan {
    bool ready = false, usable = false;
    int grid = 0;
};
static FusedPlan g_plan[64];

template <bool ACC, bool PRED>
static bool fused_kernel_ready() {
    if (cudaFuncSetAttribute(k_gk_fused<ACC, PRED>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmemBudget + kFusedStaticBytes) !=
        cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_gk_fused<ACC, PRED>, kFusedThreads, kFusedSmemBudget + kFusedStaticBytes) !=
            cudaSuccess || occ < 1) {
        cudaGetLastError();
        return false;
    }
    return true;
}

static FusedPlan* fused_plan(int dev, int sm_count) {
    if (dev < 0 || dev >= 64) return nullptr;
    // built once per device, under a lock: a second thread's first call waits for the finished plan
    static std::mutex plan_mu;
    std::lock_guard<std::mutex> plan_lock(plan_mu);
    FusedPlan& p = g_plan[dev];
    if (p.ready) return &p;
    p.ready = true;
    int coop = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return &p;
    if (!fused_kernel_ready<true, false>() || !fused_kernel_ready<false, false>() ||
        !fused_kernel_ready<true, true>() || !fused_kernel_ready<false, true>()) return &p;
    p.grid = sm_count < kFusedMaxGrid ? sm_count : kFusedMaxGrid;
    p.usable = true;
    return &p;
}

// Launch geometry for a vector of d elements on a grid of at most `grid` CTAs.
struct FusedGeometry {
    bool fits;       // false: a CTA would own more rows than its table holds
    int64_t G;       // CTAs (none without rows, at least one)
    int n_rows;      // rows of 1024 float4 in the vector
    int u_slots;     // row slots of shared memory that end up holding u
    int table_rows;  // the largest number of rows a CTA owns
    size_t smem;     // dynamic shared memory of the launch
};
static FusedGeometry fused_geometry(int64_t d, int grid) {
    FusedGeometry q;
    const int64_t n4 = d >> 2;
    const int64_t n_rows = (n4 + kRowF4 - 1) / kRowF4;
    q.n_rows = (int)n_rows;
    q.G = n_rows < grid ? n_rows : grid;
    if (q.G < 1) q.G = 1;
    int64_t most = (n_rows + q.G - 1) / q.G;  // rows of CTA 0
    if (most < 1) most = 1;
    q.fits = most <= kTableMaxRows;
    q.table_rows = (int)(most < kTableMaxRows ? most : kTableMaxRows);
    // shared memory: the ring and the maximum table claim their share, the rest holds u
    const int64_t left = (int64_t)kFusedSmemBudget - (int64_t)kRing * kRowBytes - (int64_t)q.table_rows * kTableRowBytes;
    q.u_slots = (int)(left / kRowBytes);
    if (q.u_slots > most) q.u_slots = (int)most;
    // (with fewer slots than rows in flight the kernel takes eps through the ring instead; the
    // last row of the vector, which may be short, must stay on chip: one slot at least)
    if (q.u_slots < 1) q.fits = false;
    q.smem = (size_t)kFusedStaticBytes + (size_t)(kRing + q.u_slots) * kRowBytes + (size_t)q.table_rows * kTableRowBytes;
    return q;
}

// Whether the call counts during phase A against predicted thresholds: on vectors large enough
// for the prediction to arrive early in a CTA's run (a test hook can force either answer).
static bool wants_prediction(const FusedGeometry& geo, int64_t d) {
    // one block of 32 float4 at least; a thread's packed counts hold kPredMaxRows rows
    // (and eps arriving in the u slots, which leaves the ring's upper half to the sample)
    const bool possible = (d >> 7) >= 1 && geo.table_rows <= kPredMaxRows && geo.u_slots >= kStages;
    const int knob = host_knob(kKnobPrediction);
    if (knob == 0 || !possible) return false;
    if (knob == 1) return true;
    return (int64_t)geo.n_rows >= (int64_t)kPredMinRows * geo.G;
}

// The one place that builds the kernel's argument list (types checked by the compiler).
// eps == nullptr launches the operator form.
static cudaError_t launch_fused(const FusedGeometry& geo, cudaStream_t st, const float* src, float* eps, int64_t d,
                                int64_t k, double z, Ctrl* ctrl, double2* partials, unsigned int* bars, unsigned int* rowcnt, int32_t* idx_out, float* val_out,
                                int64_t* nnz_out, int64_t cap, unsigned long long* trace, unsigned int call_no) {
    int n_rows = geo.n_rows, u_slots = geo.u_slots;
    // (a test's extra arrivals: one is as good as many, and the first barrier has one spare record)
    unsigned int bar_target = (unsigned int)geo.G + (host_knob(kKnobExtraArrivals) > 0 ? 1u : 0u);
    void* args[] = {(void*)&src, (void*)&eps, (void*)&d, (void*)&k, (void*)&z, (void*)&n_rows, (void*)&u_slots,
                    (void*)&call_no, (void*)&bar_target, (void*)&ctrl, (void*)&partials,
                    (void*)&bars, (void*)&rowcnt, (void*)&idx_out, (void*)&val_out, (void*)&nnz_out, (void*)&cap,
                    (void*)&trace};
    static_assert(sizeof(args) / sizeof(args[0]) == 18, "k_gk_fused takes 18 arguments");
    // the four instances have the same parameter list; naming them keeps the types checked
    typedef void (*Kern)(const float*, float*, int64_t, int64_t, double, int, int, unsigned int, unsigned int, Ctrl*, double2*,
                         unsigned int*, unsigned int*, int32_t*, float*, int64_t*, int64_t, unsigned long long*);
    const bool acc = eps != nullptr, pred = wants_prediction(geo, d);
    const Kern kern = acc ? (pred ? (Kern)k_gk_fused<true, true> : (Kern)k_gk_fused<true, false>)
                          : (pred ? (Kern)k_gk_fused<false, true> : (Kern)k_gk_fused<false, false>);
    return cudaLaunchCooperativeKernel((const void*)kern, dim3((unsigned)geo.G), dim3(kFusedThreads), args,
                                       geo.smem, st);
}

// Returns GK_OK when the fused kernel was enqueued, 1 when it cannot be used on
// this device or for this call (the caller then takes the three-kernel path),
// or an error.
int enqueue_gk_fused(Workspace* ws, const float* src, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                     float* val_out, int64_t* nnz_out, cudaStream_t st) {
    int dev = 0;
    GK_CUDA_TRY(cudaGetDevice(&dev));
    FusedPlan* p = fused_plan(dev, ws->sm_count);
    if (!p || !p->usable || k >= d) return 1;
    const FusedGeometry geo = fused_geometry(d, p->grid);
    if (!geo.fits) return 1;
    const double pq = 1.0 - (double)k / (double)d;  // Algorithm 1: p = 1 - k/d
    const double z = normal_quantile_upper(1.0 - pq);
    ws->last_grid = (int)geo.G;
    stage_mark(ws, st, 0);
    if (++ws->fused_calls == 0u) ws->fused_calls = 1u;   // 0 is what an unwritten record holds
    GK_CUDA_TRY(launch_fused(geo, st, src, eps, d, k, z, ws->ctrl, ws->part_recs, ws->bars, ws->rowcnt, idx_out, val_out, nnz_out, output_capacity(d), ws->cta_trace, ws->fused_calls));
    note_launch();
    stage_mark(ws, st, 1);
    ws->last_fused = true;
    ws->phase_spans = 6;
    return GK_OK;
}

}  // namespace gk

// ---------------------------------------------------------------------------
// gk_sparsify_static: the same kernel for callers that must not allocate.
//
// Some callers cannot let a library call cudaMalloc on their behalf: code that
// runs under a framework's caching allocator with a fixed memory budget, a
// service that forbids device allocations after start-up because cudaMalloc
// synchronises the whole device, or a step that has to behave the same on its
// first and on its millionth call.  For them the scratch of the fused kernel
// (control block, per-CTA partial sums, barrier counters and global counts,
// one word per row of the vector) lives in the fixed array below
// instead of a workspace obtained from cudaMalloc.  The array is part of the
// library image: every GPU that loads the library holds these 544 KB until the
// process exits.
// ---------------------------------------------------------------------------
namespace gk {

constexpr size_t kStaticCtrlBytes = (sizeof(Ctrl) + 255) / 256 * 256;
constexpr size_t kStaticPartialBytes = ((size_t)32 * (kFusedGridCap + 1) + 255) / 256 * 256;   // 16 KB: a 32-byte record per CTA, and one more
constexpr size_t kStaticBarBytes = sizeof(unsigned int) * kBarWords;          // 256 bytes
constexpr size_t kStaticHeadBytes = 32 * 1024;             // everything but the per-row words
constexpr int kStaticRowCap = 1 << 17;                     // rows of 4096 elements: d up to 2^29
constexpr size_t kStaticScratchBytes = kStaticHeadBytes + sizeof(unsigned int) * kStaticRowCap;  // 544 KB
static_assert(kStaticCtrlBytes + kStaticPartialBytes + kStaticBarBytes <= kStaticHeadBytes,
              "static scratch too small");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch per device.  In host code the name of a
// __device__ array is only a handle for the runtime, not an address a kernel
// can use; cudaGetSymbolAddress translates it for the device that is current.
struct StaticScratch {
    bool ready = false;
    unsigned char* base = nullptr;
    int sm_count = 0;
    unsigned int calls = 0;   // launches on this device's array (under g_static_mu)
};
static StaticScratch g_static[64];
static std::mutex g_static_mu;

}  // namespace gk

extern "C" int gk_sparsify_static(const float* g, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                                  float* val_out, int64_t* nnz_out, gk_stream_t stream) {
    using namespace gk;
    if (!g || !eps || !idx_out || !val_out || !nnz_out) return GK_ERR_NULL;
    if (d < 1 || d > 2147483647ll) return GK_ERR_SIZE;
    if (k < 1 || k >= d) return GK_ERR_K;  // k = d (select everything) is served by gk_sparsify only
    if (((uintptr_t)g & 15u) || ((uintptr_t)eps & 15u)) return GK_ERR_ALIGN;
    const uintptr_t ga = (uintptr_t)g, ea = (uintptr_t)eps, nb = (uintptr_t)d * 4u;
    if (ga < ea + nb && ea < ga + nb) return GK_ERR_ALIAS;
    cudaStream_t st = (cudaStream_t)stream;
    int dev = 0;
    GK_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return GK_ERR_LIMIT;
    StaticScratch* ss = &g_static[dev];
    {
        // first call on this device: look the array's device address up once
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!ss->ready) {
            void* p = nullptr;
            GK_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
            GK_CUDA_TRY(cudaDeviceGetAttribute(&ss->sm_count, cudaDevAttrMultiProcessorCount, dev));
            ss->base = static_cast<unsigned char*>(p);
            ss->ready = true;
        }
    }
    FusedPlan* plan = fused_plan(dev, ss->sm_count);
    if (!plan || !plan->usable) return GK_ERR_LIMIT;  // no cooperative launch on this device

    Ctrl* ctrl = reinterpret_cast<Ctrl*>(ss->base);
    double2* partials = reinterpret_cast<double2*>(ss->base + kStaticCtrlBytes);
    unsigned int* bars = reinterpret_cast<unsigned int*>(ss->base + kStaticCtrlBytes + kStaticPartialBytes);

    unsigned int* rowcnt = reinterpret_cast<unsigned int*>(ss->base + kStaticHeadBytes);

    const FusedGeometry geo = fused_geometry(d, plan->grid);
    // more CTAs or rows than the fixed array has slots for, or more rows per CTA than the kernel takes
    if (geo.G > kFusedGridCap || geo.n_rows > kStaticRowCap || !geo.fits) return GK_ERR_LIMIT;
    // The array keeps what the last call left.  The barrier counters and the global counts must
    // start at zero; the kernel resets them when it ends, but a call that was cut short would not have.
    GK_CUDA_TRY(cudaMemsetAsync(bars, 0, kStaticBarBytes, st));
    const double pq = 1.0 - (double)k / (double)d;
    const double z = normal_quantile_upper(1.0 - pq);
    unsigned long long* trace = nullptr;  // no trace array in the fixed scratch
    unsigned int call_no;
    {
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (++ss->calls == 0u) ss->calls = 1u;   // 0 is what an unwritten record holds
        call_no = ss->calls;
    }
    GK_CUDA_TRY(launch_fused(geo, st, g, eps, d, k, z, ctrl, partials, bars, rowcnt, idx_out, val_out, nnz_out,
                             output_capacity(d), trace, call_no));
    note_launch();
    return GK_OK;
}
