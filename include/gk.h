/*
 * gk.h -- C ABI of the B200 error-compensated Gaussian_k gradient sparsifier
 *         and exact Top_k selection (arXiv 1911.08772).
 *
 * Conventions for every call
 *   - Pointers marked DEVICE are caller-owned global memory of the CUDA device
 *     that is current when the call is made; pointers marked HOST are ordinary
 *     host memory.  The library never frees or keeps caller pointers.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  All device work is enqueued on it and the call returns without
 *     synchronising, unless stated otherwise.
 *   - Vectors are fp32, indices int32, so 1 <= d <= 2^31 - 1.  Base pointers of
 *     g, eps and u must be 16-byte aligned.  Inputs must be finite.
 *   - The library owns a small scratch workspace per (device, stream), created
 *     by the first call that needs it (cudaMalloc; use gk_reserve to do that
 *     ahead of time).  Two calls that overlap on the GPU must use different
 *     streams.
 *   - Return value: GK_OK or a negative gk_status for errors detected on the
 *     host before anything is enqueued.  Conditions found on the device
 *     (truncated output, a bounded wait that ran out, a malformed segment
 *     table) are reported in gk_stats.status, never by a trap or a hang.
 */
#ifndef GK_H_
#define GK_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void* gk_stream_t; /* a cudaStream_t */

typedef enum gk_status {
    GK_OK = 0,
    GK_ERR_NULL = -1,      /* a required pointer is NULL */
    GK_ERR_SIZE = -2,      /* d < 1 or d > 2^31 - 1, or S < 1 */
    GK_ERR_K = -3,         /* k < 1 or k > d */
    GK_ERR_ALIGN = -4,     /* g / eps / u not 16-byte aligned */
    GK_ERR_ALIAS = -5,     /* g overlaps eps */
    GK_ERR_CUDA = -6,      /* a CUDA runtime call failed (see gk_last_cuda_error) */
    GK_ERR_NOMEM = -7,     /* workspace allocation failed */
    GK_ERR_CAPACITY = -8,  /* gk_set_capacity: cap < 0 */
    GK_ERR_LIMIT = -9      /* size beyond a fixed built-in limit */
} gk_status;

/* Values of gk_stats.status (bit flags, written by the device). */
#define GK_DEV_OK 0
#define GK_DEV_TRUNCATED 1    /* more survivors than the output capacity */
#define GK_DEV_TIMEOUT 2      /* a bounded look-back wait gave up; outputs invalid */
#define GK_DEV_BAD_SEGMENTS 4 /* seg_offsets not ascending from 0 to d, or seg_k out of range */
#define GK_DEV_BAD_SAMPLE 8   /* dgck_*: a sampled position outside [0, d) (it was clamped) */
#define GK_DEV_BAD_INDEX 16   /* gk_apply_*: a message index outside [0, d) (the entry was skipped) */

/*
 * What one Gaussian_k run decided (Algorithm 1 of the paper).  For the
 * segmented call there is one record per segment.
 */
typedef struct gk_stats {
    double mu;         /* mean of u */
    double sigma;      /* sample standard deviation of u (divisor d - 1) */
    double z;          /* Phi^-1(1 - k/d) */
    double thres0;     /* mu + sigma * z, the first threshold */
    double thr_final;  /* threshold of the mask that was returned */
    int64_t counts[4]; /* #{|u_i| > thres} seen in each executed round */
    int32_t rounds;    /* rounds executed, 0 when k >= d (everything selected) */
    int32_t status;    /* GK_DEV_* flags */
    int64_t nnz;       /* size of the returned mask (before any truncation) */
    int64_t emitted;   /* pairs actually written (= min(nnz, capacity)) */
} gk_stats;

/*
 * gk_sparsify -- one step of error-compensated sparsification, Eq. 2 of the
 * paper with Comp_k = Gaussian_k (Algorithm 1):
 *     u = g + eps;   (idx, val) = Gaussian_k(u);   eps <- u - Comp(u).
 * Gaussian_k takes mean and standard deviation of u, sets the first threshold
 * to the normal quantile at p = 1 - k/d, then for at most four rounds counts
 * #{|u_i| > thres} and halves the threshold when the count is below 2k/3,
 * multiplies it by 1.5 when above 4k/3, and stops otherwise.  The mask of the
 * last round evaluated is returned.
 *
 *   g        DEVICE in   d floats, the stochastic gradient; must not overlap eps
 *   eps      DEVICE i/o  d floats; in: residual eps_t, out: eps_{t+1}
 *                        (+0.0f at selected positions, u_i elsewhere)
 *   d, k     sizes, 1 <= k <= d
 *   idx_out  DEVICE out  capacity ints (see gk_set_capacity; default d):
 *                        positions with |u_i| > threshold, ascending
 *   val_out  DEVICE out  capacity floats: u at those positions
 *   nnz_out  DEVICE out  one int64: number of pairs written
 *   stream   the stream to enqueue on
 *
 * The number of survivors is data dependent and may be below or above k
 * (Appendix A.5 of the paper).  If it exceeds the capacity, only the first
 * `capacity` survivors in index order are written and only their eps slots are
 * cleared, so that Comp(u) + eps_{t+1} == u still holds; status gets
 * GK_DEV_TRUNCATED.
 */
int gk_sparsify(const float* g, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                float* val_out, int64_t* nnz_out, gk_stream_t stream);

/*
 * gk_select -- Gaussian_k as an operator on a given vector (Algorithm 1 of the paper as
 * printed: input u, output the entries with |u_i| > threshold).  The same statistics,
 * first threshold, count-and-adjust rounds and returned mask as gk_sparsify, without the
 * accumulation before and the residual after: this is the form whose running time
 * Section 4.3 / Fig. 4 compares with Top_k and DGC_k (topk_exact and dgck_select here).
 *
 *   u        DEVICE in   d floats, not modified (16-byte aligned)
 *   d, k     sizes, 1 <= k <= d
 *   idx_out  DEVICE out  capacity ints (gk_set_capacity; default d), ascending positions
 *   val_out  DEVICE out  capacity floats: u at those positions
 *   nnz_out  DEVICE out  one int64: number of pairs written
 * Capacity rule, statistics record (gk_last_stats) and the choice of implementation
 * (gk_set_path) as for gk_sparsify.
 */
int gk_select(const float* u, int64_t d, int64_t k, int32_t* idx_out, float* val_out,
              int64_t* nnz_out, gk_stream_t stream);

/*
 * gk_sparsify_segmented -- the same step with Algorithm 1 run independently on
 * every contiguous segment [seg_offsets[s], seg_offsets[s+1]) with its own
 * mean, deviation, k_s and threshold (layer-wise selection).  The paper states
 * Algorithm 1 for the whole vector; applying it per layer is this library's
 * extension.  All S segments are processed by one batched launch per stage.
 *
 *   seg_offsets DEVICE in  S + 1 int64, seg_offsets[0] = 0 <= ... <= seg_offsets[S] = d;
 *                          boundaries need no alignment; empty segments allowed
 *   seg_k       DEVICE in  S int64, 1 <= seg_k[s] (values >= the segment length
 *                          select the whole segment)
 *   S           number of segments, 1 <= S <= 65536
 *   idx_out / val_out      as above; indices are global, segments appear in order,
 *                          so idx_out is ascending overall
 *   seg_nnz_out DEVICE out S int64: size of each segment's mask (may be NULL)
 *   nnz_out     DEVICE out one int64: total pairs written
 * A malformed table sets GK_DEV_BAD_SEGMENTS; nothing is then selected
 * (eps still receives u).
 */
int gk_sparsify_segmented(const float* g, float* eps, int64_t d, const int64_t* seg_offsets,
                          const int64_t* seg_k, int32_t S, int32_t* idx_out, float* val_out,
                          int64_t* seg_nnz_out, int64_t* nnz_out, gk_stream_t stream);

/*
 * topk_exact -- Top_k of Section 1 of the paper: the k entries of largest
 * absolute value with their indices, by radix select on the magnitude bits.
 * Entries of equal magnitude are taken in order of increasing index (+0 and
 * -0 tie).  Exactly k pairs are written, in ascending index order.
 *
 *   u        DEVICE in   d floats, not modified
 *   idx_out  DEVICE out  k ints;   val_out  DEVICE out  k floats
 */
int topk_exact(const float* u, int64_t d, int64_t k, int32_t* idx_out, float* val_out,
               gk_stream_t stream);

/*
 * topk_sparsify -- Eq. 2 of the paper with Comp_k = Top_k: u = g + eps, the exact
 * Top_k of u is written as k pairs, eps <- u - Top_k(u).  Arguments as for
 * gk_sparsify; exactly k pairs are written and *nnz_out = k.
 */
int topk_sparsify(const float* g, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                  float* val_out, int64_t* nnz_out, gk_stream_t stream);

/*
 * dgck_select -- DGC_k, the hierarchical sampling selector the paper compares
 * Gaussian_k with (Section 3.3; Section 4.3 uses a 1 % sample).  The paper says
 * only that a small random sample estimates the threshold and that top-k
 * selection runs twice on subsets of the vector; the steps taken here:
 *   1. tau = the k_m-th largest of { |u[sample_idx[j]]| : j < m },
 *      k_m = ceil(k * m / d)                       (first top-k, on the sample);
 *   2. candidates = { i : |u_i| >= tau }, n of them;
 *   3. n > k: the k largest candidates, ties toward the lower index (second
 *      top-k, on the candidates); otherwise all n candidates.
 * min(n, k) pairs are written in ascending index order.
 *
 *   u          DEVICE in   d floats, not modified (16-byte aligned)
 *   sample_idx DEVICE in   m int32 positions in [0, d), repeats allowed: the random
 *                          draw is the caller's.  A position outside the range is
 *                          clamped and flagged GK_DEV_BAD_SAMPLE.
 *   m          sample size, 1 <= m <= 2^31 - 1
 *   idx_out    DEVICE out  k ints;   val_out  DEVICE out  k floats
 *   nnz_out    DEVICE out  one int64: min(n, k)
 * One cooperative kernel; vectors of more than 448 rows of 4096 elements per SM
 * (271 M elements on 148 SMs) and devices without cooperative launch return
 * GK_ERR_LIMIT.
 */
int dgck_select(const float* u, int64_t d, int64_t k, const int32_t* sample_idx, int64_t m,
                int32_t* idx_out, float* val_out, int64_t* nnz_out, gk_stream_t stream);

/*
 * dgck_sparsify -- Eq. 2 of the paper with Comp_k = DGC_k: u = g + eps (the sample
 * is taken from u), selection as in dgck_select, eps <- u - Comp(u).  g, eps as
 * for gk_sparsify; the other arguments as for dgck_select.
 */
int dgck_sparsify(const float* g, float* eps, int64_t d, int64_t k, const int32_t* sample_idx,
                  int64_t m, int32_t* idx_out, float* val_out, int64_t* nnz_out, gk_stream_t stream);

/* Synchronise `stream` and write what the last dgck_* call on it decided to HOST
 * host_out[0..3]: the fp32 bit pattern of tau, n, k_m, pairs written. */
int dgck_last_info(gk_stream_t stream, int64_t* host_out);

/*
 * gk_apply_sparse -- the model update of Eq. 2 from the P workers' messages:
 *     x <- x + alpha * sum_p Comp_k(u^p)          (alpha = -eta / P in the paper).
 * Message p is the ascending (index, value) list a sparsifier call wrote.  The
 * terms of a position are added in rank order p = 0, 1, ... in fp32 (one
 * addition per term), the sum is multiplied by alpha and added to x; positions
 * that occur in no message are not touched.  The paper does not fix the order
 * of the P terms; rank order makes the result independent of timing.
 *
 *   x          DEVICE i/o  d floats
 *   idx_lists  HOST   in   P pointers to DEVICE int32 lists, each strictly ascending;
 *   val_lists  HOST   in   P pointers to DEVICE float lists.  A list may live in
 *                          another GPU's memory that this device can address (peer
 *                          access): the kernel reads the lists with plain loads.
 *   nnz        DEVICE in   P int64: entries of each list (values above cap count as cap)
 *   P          number of messages, 1 <= P <= 64;  cap: upper bound of every nnz[p]
 * One kernel, no scratch vector, no atomics on x.  An index outside [0, d) is
 * skipped and flagged GK_DEV_BAD_INDEX in the status word gk_last_stats returns.
 *
 * gk_apply_gathered -- the same for messages in one buffer (as an all-gather
 * leaves them): list p starts at idx + p * cap and val + p * cap (DEVICE).
 */
int gk_apply_sparse(float* x, int64_t d, const int32_t* const* idx_lists, const float* const* val_lists,
                    const int64_t* nnz, int32_t P, int64_t cap, float alpha, gk_stream_t stream);
int gk_apply_gathered(float* x, int64_t d, const int32_t* idx, const float* val, const int64_t* nnz,
                      int32_t P, int64_t cap, float alpha, gk_stream_t stream);

/*
 * gk_sparsify_host -- gk_sparsify for HOST buffers (Eq. 2, Algorithm 1): copies g
 * and eps to library-owned device staging buffers, runs the step, copies
 * eps_{t+1}, the pairs and their count back, and synchronises before
 * returning.  All pointers are HOST memory (pinned memory makes the copies
 * faster); idx_out / val_out hold `capacity` entries (default d).
 */
int gk_sparsify_host(const float* g, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                     float* val_out, int64_t* nnz_out, gk_stats* stats_out);

/*
 * gk_error_ratio -- the compression error ratio of Eq. 5 / Section 3.2 of the
 * paper, ||u - Comp(u)||^2 / ||u||^2, for a step that has just run (any of the
 * sparsifiers above): eps then holds u - Comp(u) with the selected slots at
 * zero, so ||u||^2 = ||eps||^2 + ||val||^2.  Hold it against 1 - k/d (Eq. 4)
 * and (1 - k/d)^2 (Theorem 1).
 *
 *   eps      DEVICE in   d floats: the residual the step left (16-byte aligned)
 *   val      DEVICE in   the selected values the step wrote
 *   nnz      DEVICE in   one int64: how many of them
 *   host_out HOST   out  3 doubles: the ratio, ||u - Comp(u)||^2, ||u||^2
 * One pass over eps in fp64, deterministic.  Enqueued on `stream`, which is then
 * synchronised.  A zero vector gives ratio 0.
 */
int gk_error_ratio(const float* eps, int64_t d, const float* val, const int64_t* nnz,
                   gk_stream_t stream, double* host_out);

/*
 * gk_histogram -- the histogram of u shown in the paper's gradient-distribution
 * figures (Section 3.1, Fig. 2; its running sum over d is the cumulative curve
 * of the appendix).  nbins equal bins starting at lo, bin width 1 / inv_w:
 *     t = (u_i - lo) * inv_w in fp32 (one subtraction, one multiplication);
 *     t < 0 counts as "below", t >= nbins (or NaN) as "above", else bin floor(t).
 *
 *   u          DEVICE in   d floats (16-byte aligned), not modified
 *   lo, inv_w  lower edge of the first bin; inv_w = nbins / (hi - lo) > 0, as a float
 *   nbins      1 <= nbins <= 8192
 *   counts_out DEVICE out  nbins + 2 int64: [0] below, [1 .. nbins] the bins,
 *                          [nbins + 1] above (zeroed by the call)
 * One pass over u, enqueued on `stream`; does not synchronise.
 */
int gk_histogram(const float* u, int64_t d, float lo, float inv_w, int32_t nbins, int64_t* counts_out,
                 gk_stream_t stream);

/*
 * gk_sparsify_static -- gk_sparsify for callers that must not allocate device
 * memory (the paper has no counterpart: this is a deployment variant of the
 * same step, not another method).  Think of a step that runs under a framework
 * allocator with a fixed budget, or of a service that bans cudaMalloc once it
 * is serving because that call stalls the whole device.  Same arguments, same
 * results and same capacity rule as gk_sparsify, but the call never reaches
 * cudaMalloc, cudaFree or any routine that allocates: its scratch is a fixed
 * 544 KB array inside the library image, present on every GPU that loads the
 * library for as long as the process lives.
 *
 * Limits: 1 <= k < d <= 2^31 - 1 (d beyond that returns GK_ERR_SIZE; k = d
 * returns GK_ERR_K: selecting everything is left to gk_sparsify); the device
 * must support cooperative launch, the launch must fit the array's 512
 * per-CTA slots, and the vector must not exceed 2^29 elements (the array has one
 * word per row of 4096 elements) nor 1024 rows per SM, else GK_ERR_LIMIT.
 *
 * The first call on a device looks up the array's device address
 * (cudaGetSymbolAddress) and keeps it; make that first call before any stream
 * capture begins.  All calls on a device share the one array, which keeps
 * whatever the previous call left in it; the call clears the words that have
 * to start at zero.  Two calls that overlap on the GPU (different streams)
 * would race on the array: keep them in order.  There is no statistics record
 * to read back for this call.
 */
int gk_sparsify_static(const float* g, float* eps, int64_t d, int64_t k, int32_t* idx_out,
                       float* val_out, int64_t* nnz_out, gk_stream_t stream);

/*
 * gk_set_params -- the two constants of Algorithm 1 that can be read in more than one way.
 *   unbiased_std  non-zero (default): "std" is the sample standard deviation, divisor d - 1
 *                 (the paper's operators are tensor-library calls whose default this is);
 *                 0: the population form, divisor d.
 *   max_rounds    rounds of the loop "for i = 0 -> 3": 4 by default (both bounds included),
 *                 1 .. 4 accepted; the mask of the last round run is returned.
 * Applies to gk_sparsify, gk_select, gk_sparsify_segmented, gk_sparsify_host and
 * gk_sparsify_static from the next call on.  Process-wide; the device-side values are set on
 * the current device.  Returns GK_ERR_SIZE for max_rounds outside 1 .. 4.
 */
int gk_set_params(int unbiased_std, int max_rounds);

/* Output capacity of idx_out / val_out for the sparsify calls, in pairs.
 * 0 (the default) means "d".  Process-wide; returns GK_ERR_CAPACITY if cap < 0. */
int gk_set_capacity(int64_t cap);

/*
 * Which implementation gk_sparsify, gk_select and gk_sparsify_host use.  Process-wide.
 *   0 (default)  vectors of up to 589,824 elements: one thread-block cluster of sixteen CTAs
 *                that holds u in shared memory and synchronises with cluster barriers;
 *                larger ones: one persistent cooperative kernel that keeps what fits of u in
 *                shared memory between the phases of Algorithm 1.  Falls back to path 1 where
 *                neither can be launched and for k = d.
 *   1            three kernels: accumulate + statistics, candidate counts,
 *                compaction by decoupled look-back.
 *   2            the persistent cooperative kernel at every size.
 * All give identical results.  Returns GK_ERR_SIZE for any other value.
 */
int gk_set_path(int path);

/* Create (or grow) the workspace of (current device, stream) for vectors of up
 * to d elements in up to S segments.  Synchronous; call outside timed regions
 * and before stream capture. */
int gk_reserve(int64_t d, int32_t S, gk_stream_t stream);

/* Bytes of scratch workspace a call with these sizes uses. */
int64_t gk_workspace_bytes(int64_t d, int32_t S);

/* Synchronise `stream` and copy the record of the last gk_sparsify (or the S
 * records of the last gk_sparsify_segmented) enqueued on it to HOST memory. */
int gk_last_stats(gk_stream_t stream, gk_stats* host_out);
int gk_last_segment_stats(gk_stream_t stream, int32_t S, gk_stats* host_out);

/*
 * Per-stage device timing (tracing aid, off by default; process-wide switch).
 * While enabled, every call records a CUDA event on its stream before its first
 * kernel and after each kernel.  gk_last_stage_ms synchronises the stream and
 * writes the durations in milliseconds of the stages of the last call enqueued on
 * it to HOST ms_out[0..*n_stages-1] (at most 8).  Single-kernel forms: the kernel,
 * then spans between timestamps the kernel takes itself (CTA 0 and the CTA that
 * leaves last).  gk_sparsify and gk_sparsify_segmented: accumulate incl. first
 * barrier and thresholds, counting loop, second barrier, replay of the rounds,
 * compaction, exit of the last CTA.  topk_exact and topk_sparsify: first pass,
 * barrier and first digit, second pass to second digit, third pass to third digit,
 * counts and fourth barrier, offsets and write-out, exit of the last CTA.
 * Multi-kernel forms, one value per kernel: accumulate, count, compact; for
 * Top_k three histogram passes and compact, with accumulate first in topk_sparsify.
 */
int gk_stage_timing(int enable);
int gk_last_stage_ms(gk_stream_t stream, float* ms_out, int* n_stages);

/*
 * Per-CTA trace of the last single-kernel gk_sparsify or gk_sparsify_segmented
 * call on `stream` (tracing aid).  Synchronises the stream and writes 8 uint64
 * per CTA to HOST host_out (room for 512 x 8), %globaltimer in ns.  gk_sparsify:
 * the CTA's start, before and after the first grid barrier, before and after the
 * second, before and after the third, its end.  gk_sparsify_segmented: start,
 * table read, end of the first phase, after the first barrier, thresholds formed,
 * end of the counting, after the second barrier, end.
 * *n_ctas receives the number of CTAs, 0 if the last call did not run such a kernel.
 */
int gk_last_cta_trace(gk_stream_t stream, uint64_t* host_out, int* n_ctas);

/*
 * gk_debug_set -- test hooks (the paper has no counterpart).  They exist so that tests can
 * reach the give-up branch of every bounded wait without hanging anything, and both sides of
 * the library's run-time decisions.  Process-wide; the device-side values are set on the
 * current device.  Defaults are restored by setting the default value again.
 *   key 0  polls of a grid barrier before a CTA gives up and sets GK_DEV_TIMEOUT (default 2^24)
 *   key 1  polls of a predecessor's status word in the look-back compaction (default 2^22)
 *   key 2  arrivals the barriers of the fused gk_sparsify kernel wait for beyond the grid
 *          size (default 0).  With 1 no barrier can complete: every CTA's wait runs out,
 *          the call ends with GK_DEV_TIMEOUT in gk_stats.status and invalid outputs.
 *   key 3  a tile of the look-back compaction that keeps its status word to itself, so
 *          that its successors' waits run out (default -1: none)
 *   key 4  counting against predicted thresholds in the fused gk_sparsify / gk_select
 *          kernel: -1 automatic (large vectors), 0 never, 1 whenever the vector has 128
 *          elements or more
 *   key 5  the second phase of that kernel counting only the candidates it expects the rounds
 *          to reach: -1 automatic, 0 never, 1 always and with thres0 alone (any further
 *          round then asks for a candidate left out, and the count is taken again in full)
 * Returns GK_ERR_SIZE for an unknown key or a value outside [-1, 2^31 - 1].
 */
int gk_debug_set(int key, int64_t value);

/*
 * How the last single-kernel gk_sparsify / gk_select call on `stream` took its counts
 * (tracing aid).  Synchronises the stream and writes 6 int64 to HOST host_out: CTAs that
 * formed a prediction of the thresholds from the sample; CTAs whose predicted bands held the
 * exact thresholds (their counts come from the first phase plus the cells it left over);
 * 1 if the rounds needed a candidate the short way leaves out, so that a full count followed;
 * (row, warp) cells of 128 elements left to the second phase by CTAs with a prediction; CTAs
 * of the launch (0 if the call did not run that kernel); CTAs that counted, in the second
 * phase, only the candidates they expected the rounds to reach.
 */
int gk_last_path_info(gk_stream_t stream, int64_t* host_out);

/* Number of kernels the library has launched so far in this process. */
int64_t gk_launch_count(void);

/* Text for a gk_status; the CUDA error string of the last GK_ERR_CUDA. */
const char* gk_strerror(int code);
const char* gk_last_cuda_error(void);

/* Library version, major * 1000 + minor. */
int gk_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GK_H_ */
