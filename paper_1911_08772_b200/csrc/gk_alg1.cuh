// Scalar part of Algorithm 1 (arXiv 1911.08772) as device functions: the normal
// quantile, statistics -> candidate thresholds, and the replay of the
// count-and-adjust loop on counts taken for all candidates at once.
#pragma once

#include <math.h>

#include "gk_common.cuh"

namespace gk {

// z with P(Z > z) = q for a standard normal Z, 0 < q < 1: Newton's iteration on
// erfc(z / sqrt 2) / 2 - q (derivative -phi(z)), started from the leading term
// of the tail expansion.
__host__ __device__ inline double normal_quantile_upper(double q) {
    if (!(q > 0.0)) return INFINITY;
    if (!(q < 1.0)) return -INFINITY;
    if (q == 0.5) return 0.0;
    const bool flip = q > 0.5;
    if (flip) q = 1.0 - q;
    double z = sqrt(-2.0 * log(q));
    if (z > 1.0) z -= log(z * 2.5066282746310002) / z;  // q ~ phi(z) / z
    const double inv_sqrt2 = 0.70710678118654752440, inv_sqrt2pi = 0.39894228040143267794;
    // quadratic convergence: a handful of steps reach fp64 precision; the cap keeps the cost
    // bounded when the last bits oscillate
    for (int it = 0; it < 12; ++it) {
        const double f = 0.5 * erfc(z * inv_sqrt2) - q;
        const double phi = inv_sqrt2pi * exp(-0.5 * z * z);
        const double zn = z + f / phi;
        const bool done = fabs(zn - z) <= 1e-15 * fabs(zn);
        z = zn;
        if (done) break;
    }
    return flip ? -z : z;
}

// The candidates thres0 * 0.5^a * 1.5^b listed by ascending factor: 1/8, 1/4, 3/8, 1/2, 3/4, 1,
// 9/8, 3/2, 9/4, 27/8.  For thres0 >= 0 this is the ascending order of the thresholds, for
// thres0 < 0 the descending one (the factors differ by 12 % or more, the roundings of the
// products by 1e-16, and rounding to fp32 is monotone): no sorting is needed.
__host__ __device__ constexpr int cand_by_factor(int j) {
    return j == 0 ? cand_index(3, 0) : j == 1 ? cand_index(2, 0) : j == 2 ? cand_index(2, 1)
         : j == 3 ? cand_index(1, 0) : j == 4 ? cand_index(1, 1) : j == 5 ? cand_index(0, 0)
         : j == 6 ? cand_index(1, 2) : j == 7 ? cand_index(0, 1) : j == 8 ? cand_index(0, 2)
         : cand_index(0, 3);
}
// Index of the j-th smallest candidate threshold.
__host__ __device__ constexpr int cand_ascending(int j, bool thres0_negative) {
    return cand_by_factor(thres0_negative ? kNumCand - 1 - j : j);
}

#ifdef __CUDACC__
// The two constants of Algorithm 1 that the paper leaves open to reading (gk_set_params): the
// divisor of the variance (d - 1 by default, d when `biased`) and the number of rounds (4 by
// default).  One copy per translation unit, set through the registered setter.
static __device__ int g_alg1_biased = 0;
static __device__ int g_alg1_max_rounds = kMaxRounds;
static int set_alg1_knob(int key, int value) {
    if (key == kKnobBiasedStd) return (int)cudaMemcpyToSymbol(g_alg1_biased, &value, sizeof(int));
    if (key == kKnobMaxRounds) return (int)cudaMemcpyToSymbol(g_alg1_max_rounds, &value, sizeof(int));
    return 0;
}
static const int g_alg1_knob_registered = register_knob_setter(&set_alg1_knob);
#endif

// Where one run of Algorithm 1 keeps its scalars.
struct Alg1State {
    gk_stats* stats;
    double* cand64;              // kNumCand
    float* cand32;               // kNumCand
    unsigned long long* counts;  // kNumCand
    float* thr_sel;
};

#ifdef __CUDACC__
// s1 = sum(u - c), s2 = sum((u - c)^2) over the n elements, c the pivot.
// One thread.  k >= n means p = 1 - k/n <= 0: the quantile is -inf and every
// element passes; no statistics are needed.
__device__ inline void alg1_thresholds(const Alg1State& a, double s1, double s2, double c, int64_t n,
                                       int64_t k, double z) {
    gk_stats st;
    st.status = GK_DEV_OK;
    st.emitted = 0;
    for (int i = 0; i < kMaxRounds; ++i) st.counts[i] = 0;
    for (int i = 0; i < kNumCand; ++i) a.counts[i] = 0ull;
    if (k >= n) {
        st.mu = st.sigma = __longlong_as_double(0x7ff8000000000000ll);
        st.z = st.thres0 = st.thr_final = -INFINITY;
        st.rounds = 0;
        st.nnz = n;
        *a.thr_sel = -INFINITY;
        *a.stats = st;
        return;
    }
    const double dn = (double)n;
    const double mean_shift = s1 / dn;
    double var = (s2 - s1 * mean_shift) / (g_alg1_biased ? dn : dn - 1.0);  // sample variance unless asked otherwise
    if (var < 0.0) var = 0.0;
    st.mu = c + mean_shift;
    st.sigma = sqrt(var);
    st.z = z;
    st.thres0 = st.mu + st.sigma * z;
    st.thr_final = st.thres0;
    st.rounds = 0;
    st.nnz = 0;
    *a.stats = st;
    double tb = st.thres0;
    for (int b = 0; b < kMaxRounds; ++b) {
        double t = tb;
        for (int h = 0; h + b < kMaxRounds; ++h) {
            a.cand64[cand_index(h, b)] = t;
            // for fp32 x and fp64 t:  x > t  <=>  x > (t rounded toward -inf to fp32)
            a.cand32[cand_index(h, b)] = __double2float_rd(t);
            t *= 0.5;
        }
        tb *= 1.5;
    }
    *a.thr_sel = __double2float_rd(st.thres0);
}

// Replay of the loop of Algorithm 1 on the ten candidate counts: which candidates the rounds
// visit, what each of them counts, and which one's mask is returned (the last one evaluated).
struct Alg1Path {
    int chosen;                  // candidate index of the returned mask
    int rounds;                  // rounds executed
    unsigned int visited;        // bit ci set: candidate ci was evaluated in some round
    long long est[kMaxRounds];   // the count seen in each round
};
__device__ inline Alg1Path alg1_replay(const unsigned long long* counts, int64_t k) {
    Alg1Path p;
    p.chosen = 0;
    p.rounds = 0;
    p.visited = 0u;
    int h = 0, b = 0;
    bool going = true;
    const int max_rounds = g_alg1_max_rounds;
    // four rounds at most, written out so that nothing is indexed by a run-time value (arrays
    // indexed that way live in local memory, and one thread walks this chain for the whole grid)
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {
        long long est = 0;
        if (going && r < max_rounds) {
            const int ci = cand_index(h, b);
            // the counts may live in global or in shared memory: a generic volatile load serves both
            est = (long long)*reinterpret_cast<const volatile unsigned long long*>(&counts[ci]);
            p.rounds = r + 1;
            p.chosen = ci;
            p.visited |= 1u << ci;
            if (3 * est < 2 * k) ++h;       // thres <- 0.5 * thres
            else if (3 * est > 4 * k) ++b;  // thres <- 1.5 * thres
            else going = false;
        }
        p.est[r] = est;
    }
    return p;
}

// The count of the last round that ran (the size of the returned mask).
__device__ inline long long alg1_last_est(const Alg1Path& p) {
    long long last = p.est[0];
#pragma unroll
    for (int r = 1; r < kMaxRounds; ++r) if (r < p.rounds) last = p.est[r];
    return last;
}

// The same with the record filled in.  One thread.
// Returns the index of the candidate whose mask is returned (-1: everything).  visited_out, when
// given, receives the set of candidates the rounds evaluated (bit = candidate index).
__device__ inline int alg1_resolve(const Alg1State& a, int64_t k, unsigned int* visited_out = nullptr) {
    gk_stats* st = a.stats;
    if (visited_out) *visited_out = 0u;
    if (st->rounds == 0 && st->thr_final == -INFINITY) return -1;  // everything selected
    const Alg1Path p = alg1_replay(a.counts, k);
    if (visited_out) *visited_out = p.visited;
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) st->counts[r] = p.est[r];   // rounds not run keep 0
    st->rounds = p.rounds;
    st->thr_final = a.cand64[p.chosen];  // the mask of the last round evaluated
    st->nnz = alg1_last_est(p);
    *a.thr_sel = a.cand32[p.chosen];
    return p.chosen;
}
#endif

}  // namespace gk
