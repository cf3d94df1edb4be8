// CPU oracle for the error-compensated Gaussian_k sparsifier and exact Top_k.
//
// THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, single-threaded
// restatement of what the paper defines, used only to check the CUDA library
// and to serve as a timed CPU baseline.  It shares no code with the CUDA path
// and nothing in the product may call it.
//
// Every function names the passage of the paper (arXiv 1911.08772) it follows.
// Scalars are fp64; the vectors are fp32 because the paper computes in fp32
// (Section 4.1).  Built with -O2 and without -ffast-math so that signed zeros
// and denormals survive.
//
// Readings taken where the paper is silent (all listed again in the design
// notes of the repository):
//   * "std" is the sample standard deviation (divide by d-1).
//   * ppf(u, p, mu, sigma) is the normal quantile mu + sigma * Phi^-1(p).
//   * the loop "i = 0 -> 3" runs at most four rounds.
//   * 2k/3 and 4k/3 are real numbers: tested as 3*est < 2*k and 3*est > 4*k.
//   * the returned mask is the one last evaluated, i.e. the threshold before
//     the last adjustment.
//   * the comparison |u_i| > thres is taken in fp64 (u_i widened exactly).
//   * k >= d (p <= 0): every element is selected, no statistics.
//   * exact Top_k breaks ties of equal magnitude toward the lower index.
//   * DGC_k (one sentence in the paper): see the comment at oracle_dgck_select.
//
// Pins (tests that do not pass through this file's own formulas): see
// tests/test_oracle_pins.py.  Nothing here is "parity unpinned".
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

extern "C" {

struct oracle_stats {
    double mu;          // mean of u                          (Alg. 1, statistics)
    double sigma;       // sample standard deviation of u     (Alg. 1, statistics)
    double z;           // Phi^-1(1 - k/d)                    (Alg. 1, p and ppf)
    double thres0;      // mu + sigma * z                     (Alg. 1, ppf)
    double thr_final;   // threshold of the last evaluated mask
    int64_t counts[4];  // estimated_k of each executed round (Alg. 1, loop)
    int32_t rounds;     // rounds executed (1..4), 0 when k >= d
    int32_t pad;
    int64_t nnz;        // number of selected elements
};

// ---------------------------------------------------------------------------
// Eq. 2: u = g + eps, one IEEE fp32 addition per element.
// ---------------------------------------------------------------------------
void oracle_accumulate(const float* g, const float* eps, int64_t d, float* u) {
    for (int64_t i = 0; i < d; ++i) {
        u[i] = g[i] + eps[i];
    }
}

// ---------------------------------------------------------------------------
// Alg. 1, "mean and std of vector u": two passes in fp64.
// unbiased != 0 divides the squared deviations by d-1, otherwise by d.
// ---------------------------------------------------------------------------
void oracle_mean_std(const float* u, int64_t d, int unbiased, double* mu, double* sigma) {
    double s = 0.0;
    for (int64_t i = 0; i < d; ++i) s += (double)u[i];
    const double m = s / (double)d;
    double q = 0.0;
    for (int64_t i = 0; i < d; ++i) {
        const double dev = (double)u[i] - m;
        q += dev * dev;
    }
    const double den = unbiased ? (double)(d - 1) : (double)d;
    *mu = m;
    *sigma = std::sqrt(q / den);
}

// ---------------------------------------------------------------------------
// Standard normal CDF and its inverse (the "ppf" of Alg. 1).
// Phi(z) = erfc(-z / sqrt 2) / 2.  The inverse is found by bisection on z
// until the bracket cannot shrink; no coefficient tables.
// ---------------------------------------------------------------------------
double oracle_norm_cdf(double z) { return 0.5 * std::erfc(-z / std::sqrt(2.0)); }

double oracle_norm_ppf(double p) {
    if (!(p > 0.0)) return -std::numeric_limits<double>::infinity();
    if (!(p < 1.0)) return std::numeric_limits<double>::infinity();
    double lo = -40.0, hi = 40.0;
    for (int it = 0; it < 200; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (mid <= lo || mid >= hi) break;
        if (oracle_norm_cdf(mid) < p) lo = mid; else hi = mid;
    }
    // lo and hi are now adjacent doubles; return the one whose CDF is nearer p
    return (p - oracle_norm_cdf(lo) <= oracle_norm_cdf(hi) - p) ? lo : hi;
}

// ---------------------------------------------------------------------------
// Alg. 1, loop body, for one threshold: the mask |u_i| > thres and its number
// of True values.
// ---------------------------------------------------------------------------
int64_t oracle_count_above(const float* u, int64_t d, double thres) {
    int64_t c = 0;
    for (int64_t i = 0; i < d; ++i)
        if ((double)std::fabs(u[i]) > thres) ++c;
    return c;
}

// ---------------------------------------------------------------------------
// Algorithm 1 up to the end of its loop.  The first threshold is the normal quantile at
// probability 1 - k/d for the vector's own mean and deviation.  Then, at most four times: count
// the magnitudes above the threshold; fewer than two thirds of k halves the threshold, more
// than four thirds of k multiplies it by 1.5 (both tested exactly in integers), anything
// between ends the loop.  The mask that is returned is the one of the last count taken, so
// thr_final and nnz record that round and an adjustment made after it is dropped.
// ---------------------------------------------------------------------------
void oracle_gaussiank_threshold(const float* u, int64_t d, int64_t k, int max_rounds,
                                int unbiased, oracle_stats* st) {
    std::memset(st, 0, sizeof(*st));
    if (k >= d) {  // the probability is <= 0: the quantile is -inf, every element passes
        st->mu = st->sigma = std::numeric_limits<double>::quiet_NaN();
        st->z = st->thres0 = st->thr_final = -std::numeric_limits<double>::infinity();
        st->rounds = 0;
        st->nnz = d;
        return;
    }
    oracle_mean_std(u, d, unbiased, &st->mu, &st->sigma);
    const double p = 1.0 - (double)k / (double)d;
    st->z = oracle_norm_ppf(p);
    double thres = st->mu + st->sigma * st->z;
    st->thres0 = thres;
    if (max_rounds > 4) max_rounds = 4;
    for (int i = 0; i < max_rounds; ++i) {
        const int64_t est = oracle_count_above(u, d, thres);
        st->counts[i] = est;
        st->rounds = i + 1;
        st->thr_final = thres;
        st->nnz = est;
        if (3 * est < 2 * k) thres = 0.5 * thres;
        else if (3 * est > 4 * k) thres = 1.5 * thres;
        else break;
    }
}

// ---------------------------------------------------------------------------
// Alg. 1, final masked assignment, with the compact output form of Section 1 ("with
// corresponding indices"): pairs (i, u_i) with |u_i| > thres, ascending i.
// Returns the number of pairs; writes at most cap of them.
// ---------------------------------------------------------------------------
int64_t oracle_select(const float* u, int64_t d, double thres, int64_t cap,
                      int32_t* idx, float* val) {
    int64_t n = 0;
    for (int64_t i = 0; i < d; ++i) {
        if ((double)std::fabs(u[i]) > thres) {
            if (n < cap) { idx[n] = (int32_t)i; val[n] = u[i]; }
            ++n;
        }
    }
    return n;
}

// ---------------------------------------------------------------------------
// Eq. 2: eps_new = u - Comp(u).  Selected slots hold u_i - u_i = +0, the
// others u_i - 0 = u_i.  idx lists the selected positions.
// ---------------------------------------------------------------------------
void oracle_residual(const float* u, int64_t d, const int32_t* idx, const float* val,
                     int64_t nnz, float* eps_new) {
    std::vector<float> comp((size_t)d, 0.0f);
    for (int64_t j = 0; j < nnz; ++j) comp[(size_t)idx[j]] = val[j];
    for (int64_t i = 0; i < d; ++i) {
        eps_new[i] = u[i] - comp[(size_t)i];
    }
}

// ---------------------------------------------------------------------------
// One whole sparsifier step (Eq. 2 with Comp = Gaussian_k, Alg. 1).
// eps is updated in place.  Pairs beyond cap are not emitted and their slots
// keep u in eps_new, so that Comp(u) + eps_new == u still holds.
// ---------------------------------------------------------------------------
int64_t oracle_gk_sparsify(const float* g, float* eps, int64_t d, int64_t k, int64_t cap,
                           int32_t* idx, float* val, oracle_stats* st) {
    std::vector<float> u((size_t)d);
    oracle_accumulate(g, eps, d, u.data());
    oracle_gaussiank_threshold(u.data(), d, k, 4, 1, st);
    int64_t n = oracle_select(u.data(), d, st->thr_final, cap, idx, val);
    if (n > cap) n = cap;
    oracle_residual(u.data(), d, idx, val, n, eps);
    return n;
}

// ---------------------------------------------------------------------------
// Layer-wise variant: Alg. 1 run independently on each contiguous segment
// [off[s], off[s+1]) with its own k_s.  Indices are global, segments are
// emitted in order.  (The paper states Alg. 1 for the whole vector; the
// segmented form is this repository's workload definition.)
// ---------------------------------------------------------------------------
int64_t oracle_gk_sparsify_segmented(const float* g, float* eps, int64_t d,
                                     const int64_t* off, const int64_t* seg_k, int32_t S,
                                     int64_t cap, int32_t* idx, float* val,
                                     int64_t* seg_nnz, oracle_stats* st /* S entries */) {
    int64_t total = 0;
    for (int32_t s = 0; s < S; ++s) {
        const int64_t lo = off[s], n = off[s + 1] - off[s];
        if (n <= 0) { std::memset(&st[s], 0, sizeof(oracle_stats)); seg_nnz[s] = 0; continue; }
        const int64_t room = cap > total ? cap - total : 0;
        const int64_t m = oracle_gk_sparsify(g + lo, eps + lo, n, seg_k[s], room,
                                             idx + total, val + total, &st[s]);
        for (int64_t j = 0; j < m; ++j) idx[total + j] += (int32_t)lo;
        seg_nnz[s] = m;
        total += m;
    }
    (void)d;
    return total;
}

// ---------------------------------------------------------------------------
// Section 1, definition of Top_k: the k entries of largest absolute value with
// their indices.  Full sort of all d positions by (|u_i| descending, i
// ascending); the first k are kept and re-emitted in ascending index order.
// Magnitudes are compared through their IEEE bit patterns with the sign bit
// cleared, which orders finite non-negative floats exactly as their values
// (so +0 and -0 tie).
// ---------------------------------------------------------------------------
void oracle_topk_exact(const float* u, int64_t d, int64_t k, int32_t* idx, float* val) {
    std::vector<uint64_t> key((size_t)d);
    for (int64_t i = 0; i < d; ++i) {
        uint32_t b;
        std::memcpy(&b, &u[i], 4);
        b &= 0x7fffffffu;
        // larger magnitude first, then lower index first
        key[(size_t)i] = ((uint64_t)(0x7fffffffu - b) << 32) | (uint64_t)(uint32_t)i;
    }
    std::sort(key.begin(), key.end());
    std::vector<int32_t> chosen((size_t)k);
    for (int64_t j = 0; j < k; ++j) chosen[(size_t)j] = (int32_t)(key[(size_t)j] & 0xffffffffu);
    std::sort(chosen.begin(), chosen.end());
    for (int64_t j = 0; j < k; ++j) { idx[j] = chosen[(size_t)j]; val[j] = u[chosen[(size_t)j]]; }
}

// ---------------------------------------------------------------------------
// Eq. 5: ||u - Top_k(u)||^2 / ||u||^2 from the list of kept positions.
// ---------------------------------------------------------------------------
double oracle_error_ratio(const float* u, int64_t d, const int32_t* idx, int64_t nnz) {
    double all = 0.0, kept = 0.0;
    for (int64_t i = 0; i < d; ++i) all += (double)u[i] * (double)u[i];
    for (int64_t j = 0; j < nnz; ++j) kept += (double)u[idx[j]] * (double)u[idx[j]];
    return (all - kept) / all;
}

// ---------------------------------------------------------------------------
// DGC_k, the hierarchical sampling selector the paper compares against.
// Section 3.3 describes it in one sentence: a sample of 0.1 % to 1 % of the
// entries estimates the threshold, and top-k selection runs twice, each time on
// a subset of the vector; Section 4.3 takes a 1 % sample.  The paper gives no
// more than that; the reading taken here:
//   1. the sample is the multiset { |u[s_j]| : j < m } at the positions s_j the
//      caller drew (the random draw is an input, not part of the arithmetic);
//   2. first top-k, on the sample: with k_m = ceil(k * m / d) (the density k/d
//      applied to the sample size), tau = the k_m-th largest sampled magnitude;
//   3. candidates C = { i : |u_i| >= tau } over the whole vector;
//   4. second top-k, on C, only when |C| > k: the k largest magnitudes of C,
//      ties toward the lower index; otherwise all of C is returned (fewer than
//      k entries are accepted, as with any sampled threshold).
// Pairs come out in ascending index.  info: [0] bits of tau, [1] |C|, [2] k_m.
// Returns the number of pairs.
// ---------------------------------------------------------------------------
int64_t oracle_dgck_select(const float* u, int64_t d, int64_t k, const int32_t* sidx, int64_t m,
                           int32_t* idx, float* val, int64_t* info) {
    std::vector<float> v((size_t)m);
    for (int64_t j = 0; j < m; ++j) v[(size_t)j] = std::fabs(u[sidx[j]]);        // step 1
    const int64_t km = (k * m + d - 1) / d;                                       // step 2
    std::sort(v.begin(), v.end(), [](float a, float b) { return a > b; });
    const float tau = v[(size_t)(km - 1)];
    std::vector<int32_t> cand;                                                    // step 3
    for (int64_t i = 0; i < d; ++i)
        if (std::fabs(u[i]) >= tau) cand.push_back((int32_t)i);
    const int64_t n = (int64_t)cand.size();
    uint32_t tb;
    std::memcpy(&tb, &tau, 4);
    info[0] = (int64_t)tb; info[1] = n; info[2] = km;
    if (n > k) {                                                                  // step 4
        std::stable_sort(cand.begin(), cand.end(), [&](int32_t a, int32_t b) {
            return std::fabs(u[a]) > std::fabs(u[b]);   // stable: equal magnitudes keep index order
        });
        cand.resize((size_t)k);
        std::sort(cand.begin(), cand.end());
    }
    for (size_t j = 0; j < cand.size(); ++j) { idx[j] = cand[j]; val[j] = u[cand[j]]; }
    return (int64_t)cand.size();
}

// Eq. 2 with Comp_k = DGC_k: u = g + eps, selection as above, eps <- u - Comp(u).
int64_t oracle_dgck_sparsify(const float* g, float* eps, int64_t d, int64_t k, const int32_t* sidx,
                             int64_t m, int32_t* idx, float* val, int64_t* info) {
    std::vector<float> u((size_t)d);
    oracle_accumulate(g, eps, d, u.data());
    const int64_t n = oracle_dgck_select(u.data(), d, k, sidx, m, idx, val, info);
    oracle_residual(u.data(), d, idx, val, n, eps);
    return n;
}

// ---------------------------------------------------------------------------
// Eq. 2, the update of the model from the exchanged messages:
//     x <- x + alpha * sum_p Comp_k(u^p),      alpha = -eta / P in the paper.
// Rank p's message is the list (idx[p * cap + j], val[p * cap + j]), j < nnz[p]
// (what the sparsifier wrote).  The sum over the workers is taken in rank
// order p = 0, 1, ... in fp32, one IEEE addition per term, starting from the
// first term; then one multiplication by alpha and one addition to x.  Only
// positions that occur in some message are touched.  The paper does not say
// in which order the P terms are added; rank order is this repository's choice.
// ---------------------------------------------------------------------------
void oracle_apply_sparse(float* x, int64_t d, const int32_t* idx, const float* val, const int64_t* nnz,
                         int32_t P, int64_t cap, float alpha) {
    std::vector<float> s((size_t)d, 0.0f);
    std::vector<unsigned char> seen((size_t)d, 0);
    for (int32_t p = 0; p < P; ++p) {
        for (int64_t j = 0; j < nnz[p]; ++j) {
            const int64_t i = idx[(int64_t)p * cap + j];
            const float v = val[(int64_t)p * cap + j];
            if (!seen[(size_t)i]) { s[(size_t)i] = v; seen[(size_t)i] = 1; }
            else s[(size_t)i] = s[(size_t)i] + v;
        }
    }
    for (int64_t i = 0; i < d; ++i) {
        if (seen[(size_t)i]) {
            const float t = alpha * s[(size_t)i];
            x[i] = x[i] + t;
        }
    }
}

// ---------------------------------------------------------------------------
// The histogram of u that the paper's gradient-distribution figures show
// (Section 3.1, Fig. 2, and the cumulative curves of the appendix): nbins equal bins
// over [lo, hi), plus one count below and one above.  Floating point decides
// an integer here, so the rule is fixed in fp32, the vector's own precision:
//     t = (u_i - lo) * inv_w    (one fp32 subtraction, one fp32 multiplication,
//                                inv_w = nbins / (hi - lo) given by the caller)
//     bin = floor(t);  t < 0 -> "below";  t >= nbins (or NaN) -> "above".
// counts: nbins + 2 entries: [0] below, [1 .. nbins] the bins, [nbins + 1] above.
// The cumulative distribution is the running sum of these counts over d.
// ---------------------------------------------------------------------------
void oracle_histogram(const float* u, int64_t d, float lo, float inv_w, int32_t nbins, int64_t* counts) {
    for (int32_t b = 0; b < nbins + 2; ++b) counts[b] = 0;
    for (int64_t i = 0; i < d; ++i) {
        const float diff = u[i] - lo;
        const float t = diff * inv_w;
        if (t < 0.0f) counts[0] += 1;
        else if (!(t < (float)nbins)) counts[nbins + 1] += 1;
        else counts[1 + (int32_t)std::floor(t)] += 1;
    }
}

}  // extern "C"
