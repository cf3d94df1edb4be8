"""Pins for the CPU oracle: every check here compares the oracle with something
that is not the oracle -- closed forms, textbook tables, library routines,
brute force on tiny inputs, invariants the paper states."""
import math
import os

import numpy as np
import pytest
from scipy import stats as sps

from oracle import oracle as orc
from paper_1911_08772_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


# --------------------------------------------------------------------------- Eq. 2: u = g + eps
def test_accumulate_is_one_ieee_add():
    rng = wl.misc_rng(1)
    g = (rng.standard_normal(5000) * 1e-3).astype(np.float32)
    e = (rng.standard_normal(5000) * 1e-2).astype(np.float32)
    # signed zeros, exact cancellation, denormals, large/small mixes
    g[:8] = np.array([0.0, -0.0, -0.0, 1.5, 1e-45, 1e-39, 3e38, 1.0], dtype=np.float32)
    e[:8] = np.array([-0.0, -0.0, 0.0, -1.5, 1e-45, -1e-39, 1e30, 2.0 ** -25], dtype=np.float32)
    u = orc.accumulate(g, e)
    with np.errstate(all="ignore"):
        ref = g + e  # numpy's fp32 add: the IEEE operation itself
    assert np.array_equal(bits(u), bits(ref))
    assert bits(u)[1] == 0x80000000          # -0 + -0 = -0
    assert bits(u)[0] == 0 and bits(u)[2] == 0 and bits(u)[3] == 0  # x + (-x) = +0
    assert u[7] == np.float32(1.0)           # round to nearest even


# --------------------------------------------------------------------------- mean / std
def test_mean_std_closed_forms():
    mu, sg = orc.mean_std(np.array([1, 2, 3, 4], dtype=np.float32))
    assert mu == 2.5 and abs(sg - math.sqrt(5.0 / 3.0)) < 1e-15
    mu, sg = orc.mean_std(np.array([1, 2, 3, 4], dtype=np.float32), unbiased=False)
    assert mu == 2.5 and abs(sg - math.sqrt(5.0 / 4.0)) < 1e-15
    # arithmetic progression 0..n-1: mean (n-1)/2, sample variance n(n+1)/12
    n = 4097
    mu, sg = orc.mean_std(np.arange(n, dtype=np.float32))
    assert mu == (n - 1) / 2 and abs(sg - math.sqrt(n * (n + 1) / 12.0)) < 1e-9
    # constant vector: sigma exactly 0
    mu, sg = orc.mean_std(np.full(1000, 0.75, dtype=np.float32))
    assert mu == 0.75 and sg == 0.0


def test_mean_std_against_numpy_longdouble():
    g = wl.normal(300_001, 1e-3, step=3)
    g += np.float32(2e-3)  # non-zero mean
    mu, sg = orc.mean_std(g)
    x = g.astype(np.longdouble)
    m = x.sum() / x.size
    s = np.sqrt(((x - m) ** 2).sum() / (x.size - 1))
    assert abs(mu - float(m)) <= 1e-13 * abs(float(m))
    assert abs(sg - float(s)) <= 1e-12 * float(s)
    # iid N(0, s^2): sigma/s = 1 +- a few 1/sqrt(2d)
    assert abs(sg / 1e-3 - 1.0) < 6.0 / math.sqrt(2 * g.size)


# --------------------------------------------------------------------------- normal ppf
def _quantile_table():
    rows = []
    with open(os.path.join(GOLDEN, "normal_quantiles.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            p, z = line.split()
            rows.append((float(p), float(z)))
    return rows


def test_ppf_textbook_table():
    rows = _quantile_table()
    assert len(rows) >= 10
    for p, z in rows:
        assert abs(orc.norm_ppf(p) - z) < 6e-7, (p, z)


def test_ppf_against_scipy_and_round_trip():
    ps = [1e-12, 1e-6, 1e-4, 0.01, 0.3, 0.5, 0.7, 0.97, 0.999, 0.9999, 1 - 1e-7, 1 - 1e-10]
    for p in ps:
        z = orc.norm_ppf(p)
        ref = float(sps.norm.ppf(p))
        # allow for the conditioning of the inverse near p -> 1: dz = dp / phi(z)
        slack = 4 * np.finfo(float).eps * max(p, 1 - p) / sps.norm.pdf(ref)
        assert abs(z - ref) <= 1e-13 * max(1.0, abs(ref)) + slack, (p, z, ref)
        back = 0.5 * math.erfc(-z / math.sqrt(2.0))
        assert abs(back - p) <= 4e-16 * max(p, 1e-300) + 2e-16
    for p in [0.001, 0.2, 0.4]:
        assert abs(orc.norm_ppf(1 - p) + orc.norm_ppf(p)) < 1e-12
    assert orc.norm_ppf(0.0) == -math.inf and orc.norm_ppf(1.0) == math.inf
    assert orc.norm_ppf(0.5) == 0.0 or abs(orc.norm_ppf(0.5)) < 1e-16


def test_ppf_at_the_workload_densities():
    for rho, (num, den) in wl.RHO.items():
        for d in [wl.D_RESNET20, wl.D_RESNET50, 1 << 28]:
            k = wl.ceil_k(d, num, den)
            p = 1.0 - k / d
            assert abs(orc.norm_ppf(p) - float(sps.norm.isf(k / d))) < 1e-11
    assert wl.ceil_k(wl.D_RESNET20, 1, 1000) == 270


# --------------------------------------------------------------------------- counts / masks
def test_count_is_strict_and_two_sided():
    u = np.array([0.5, -0.5, 0.25, -1.0, 0.0, -0.0, 0.5000001], dtype=np.float32)
    assert orc.count_above(u, 0.5) == 2           # ties are not above
    assert orc.count_above(u, 0.49999) == 4
    assert orc.count_above(u, -1e-30) == 7        # negative threshold: everything
    assert orc.count_above(u, 0.0) == 5           # zeros are not above zero
    assert orc.count_above(u, 2.0) == 0
    # an fp64 threshold strictly between two neighbouring floats
    a = np.float32(1.0)
    b = np.nextafter(a, np.float32(2.0))
    t = (float(a) + float(b)) / 2
    assert orc.count_above(np.array([a, b], dtype=np.float32), t) == 1
    rng = wl.misc_rng(2)
    x = rng.standard_normal(777).astype(np.float32)
    for t in [0.0, 0.3, 1.7, 2.5]:
        brute = sum(1 for v in x.tolist() if abs(v) > t)
        assert orc.count_above(x, t) == brute


# --------------------------------------------------------------------------- Alg. 1 refinement rule
def _branch_cases():
    out = []
    with open(os.path.join(GOLDEN, "alg1_branch_cases.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, d, k, levels, rounds, counts, fn, fd, nnz = line.split()
            lv = [(int(c), float(v)) for c, v in (x.split(":") for x in levels.split(","))]
            out.append((name, int(d), int(k), lv, int(rounds), [int(c) for c in counts.split(",")],
                        int(fn), int(fd), int(nnz)))
    return out


def _levels_vector(d, levels, seed):
    u = np.zeros(d, dtype=np.float32)
    pos = wl.misc_rng(seed).permutation(d)
    at = 0
    for cnt, v in levels:
        assert cnt % 2 == 0
        u[pos[at:at + cnt // 2]] = v
        u[pos[at + cnt // 2:at + cnt]] = -v
        at += cnt
    return u


@pytest.mark.parametrize("case", _branch_cases(), ids=lambda c: c[0])
def test_alg1_hand_built_branches(case):
    name, d, k, levels, rounds, counts, fn, fd, nnz = case
    u = _levels_vector(d, levels, seed=11)
    st = orc.gaussiank_threshold(u, k)
    var = sum(c * float(np.float32(v)) ** 2 for c, v in levels) / (d - 1)
    z = float(sps.norm.ppf(1.0 - k / d))
    thres0 = z * math.sqrt(var)
    assert abs(st.mu) < 1e-12
    assert abs(st.thres0 - thres0) <= 1e-9 * thres0
    assert st.rounds == rounds
    assert st.counts == counts
    assert st.nnz == nnz
    assert abs(st.thr_final / st.thres0 - fn / fd) < 1e-15
    idx, val, n = orc.select(u, st.thr_final)
    assert n == nnz
    # the selected set is exactly the entries above the hand-computed threshold
    brute = [i for i, v in enumerate(u.tolist()) if abs(v) > thres0 * fn / fd]
    assert idx.tolist() == brute


def test_alg1_max_rounds_is_four_and_exact_edges_break():
    # est == 4k/3 exactly and est == 2k/3 exactly both stop the loop (k = 30: 40 and 20)
    for cnt in (40, 20):
        u = _levels_vector(1000, [(cnt, 1.0)], seed=5)
        st = orc.gaussiank_threshold(u, 30)
        assert st.rounds == 1 and st.nnz == cnt
    for cnt in (42, 18):
        u = _levels_vector(1000, [(cnt, 1.0)], seed=5)
        st = orc.gaussiank_threshold(u, 30)
        assert st.rounds == 4


def _tail_two_sided(dist, t):
    if dist == "normal":
        return 2.0 * sps.norm.sf(t)
    return math.exp(-t)  # Laplace(0,1): P(|x| > t)


# Decision sequences and final outcomes that follow from the tail function of the
# input law alone (u = up x1.5, d = down x0.5, b = break), thresholds in units of sigma.
WORKED = [
    ("normal", "1e-3", "udud", 1.125, 0.508),
    ("normal", "1e-2", "udub", 1.125, 0.887),
    ("normal", "5e-3", "udub", 1.125, 0.752),
    ("normal", "1e-4", "udud", 1.125, 0.287),
    ("laplace", "1e-3", "uudu", 1.125, 7.32),
    ("laplace", "1e-2", "ub", 1.5, 0.719),
    ("laplace", "1e-4", "uudu", 1.125, 26.9),
]


@pytest.mark.parametrize("dist,rho,path,factor,nnz_over_k", WORKED)
def test_alg1_worked_paths_on_large_iid_inputs(dist, rho, path, factor, nnz_over_k):
    d = 1 << 22
    num, den = wl.RHO[rho]
    k = wl.ceil_k(d, num, den)
    w = wl.sweep_point(d, dist)
    u = w.grad(0, None)
    st = orc.gaussiank_threshold(u, k)
    sigma = 1.0 if dist == "normal" else math.sqrt(2.0)
    z = float(sps.norm.isf(k / d))
    # replay from the closed-form tail: expected count at threshold t is d * tail(t)
    t = z * sigma
    seq = ""
    exp_counts = []
    for _ in range(4):
        est = d * _tail_two_sided(dist, t)
        exp_counts.append(est)
        if 3 * est < 2 * k:
            seq += "d"; t_next = 0.5 * t
        elif 3 * est > 4 * k:
            seq += "u"; t_next = 1.5 * t
        else:
            seq += "b"; break
        t_last = t
        t = t_next
    assert seq == path  # the literal in WORKED agrees with the closed form
    assert st.rounds == len(path)
    got = ""
    for i, c in enumerate(st.counts):
        got += "d" if 3 * c < 2 * k else ("u" if 3 * c > 4 * k else "b")
    assert got == path
    assert abs(st.thr_final / st.thres0 - factor) < 1e-12
    for c, e in zip(st.counts, exp_counts):
        assert abs(c - e) <= 0.05 * e + 6 * math.sqrt(e) + 3
    assert abs(st.nnz / k - nnz_over_k) <= 0.08 * nnz_over_k + 6 / math.sqrt(k)
    assert abs(st.sigma / sigma - 1) < 5e-3 and abs(st.mu) < 5e-3


def test_alg1_invariants_on_assorted_inputs():
    cases = [
        (wl.normal(50_000, 1e-3, step=9), 50),
        (wl.laplace(80_001, 1.0, step=9), 800),
        (wl.laplace_mixture(123_457, step=1), 124),
        (wl.student_t3_outliers(200_003, step=1), 1001),
    ]
    allowed = sorted({(0.5 ** a) * (1.5 ** b) for a in range(4) for b in range(4) if a + b <= 3})
    assert len(allowed) == 10
    for u, k in cases:
        st = orc.gaussiank_threshold(u, k)
        ratio = st.thr_final / st.thres0
        assert min(abs(ratio - f) for f in allowed) < 1e-15
        assert 1 <= st.rounds <= 4
        last = st.counts[-1]
        if st.rounds < 4:
            assert 2 * k <= 3 * last <= 4 * k
        for c in st.counts[:-1]:
            assert 3 * c < 2 * k or 3 * c > 4 * k
        assert st.nnz == last == orc.count_above(u, st.thr_final)


def test_alg1_degenerate_sizes():
    u = np.array([3.0, -1.0, 0.0, 2.0], dtype=np.float32)
    st = orc.gaussiank_threshold(u, 4)        # k = d: everything, no statistics
    assert st.rounds == 0 and st.nnz == 4 and st.thr_final == -math.inf
    idx, val, n = orc.select(u, st.thr_final)
    assert idx.tolist() == [0, 1, 2, 3]
    st = orc.gaussiank_threshold(np.zeros(100, dtype=np.float32), 10)   # sigma = 0, all zero
    assert st.sigma == 0.0 and st.thres0 == 0.0 and st.nnz == 0 and st.rounds == 4
    st = orc.gaussiank_threshold(np.array([5.0], dtype=np.float32), 1)  # d = 1
    assert st.rounds == 0 and st.nnz == 1


# --------------------------------------------------------------------------- selection and residual (Eq. 2)
def test_select_and_residual_identity():
    rng = wl.misc_rng(4)
    g = (rng.standard_normal(20_011) * 1e-3).astype(np.float32)
    e = (rng.standard_normal(20_011) * 3e-3).astype(np.float32)
    g[100] = -0.0; e[100] = -0.0          # u = -0.0 must survive in eps_new
    u = g + e
    eps = e.copy()
    idx, val, st = orc.gk_sparsify(g, eps, 40)
    mask = np.abs(u.astype(np.float64)) > st.thr_final       # numpy mask, not the oracle's
    assert np.array_equal(idx, np.nonzero(mask)[0].astype(np.int32))
    assert np.array_equal(bits(val), bits(u[mask]))
    assert np.all(np.diff(idx) > 0) and st.nnz == idx.size
    dense = np.zeros_like(u)
    dense[idx] = val
    # Comp(u) + eps_new == u exactly, and eps_new is +0 on the selected slots, u elsewhere
    assert np.all(bits(eps)[mask] == 0)
    assert np.array_equal(bits(eps)[~mask], bits(u)[~mask])
    assert bits(eps)[100] == 0x80000000
    assert np.array_equal((dense + eps), u)


def test_capacity_truncation_keeps_the_identity():
    u = wl.normal(10_000, 1.0, step=2)
    eps = np.zeros_like(u)
    full_idx, full_val, st = orc.gk_sparsify(u, eps.copy(), 500)
    assert st.nnz > 20
    eps2 = np.zeros_like(u)
    idx, val, st2 = orc.gk_sparsify(u, eps2, 500, cap=20)
    assert idx.size == 20 and np.array_equal(idx, full_idx[:20])
    dense = np.zeros_like(u); dense[idx] = val
    assert np.array_equal(dense + eps2, u)


def test_error_compensation_loop_conserves_mass():
    d, k, T = 30_000, 30, 12
    eps = np.zeros(d, dtype=np.float32)
    sent = np.zeros(d, dtype=np.float64)
    total = np.zeros(d, dtype=np.float64)
    for t in range(T):
        g = wl.normal(d, 1e-3, step=100 + t)
        total += g
        idx, val, st = orc.gk_sparsify(g, eps, k)
        sent[idx] += val
    # sum of gradients = what was sent + what is still held back (up to fp32 rounding of the adds)
    assert np.max(np.abs(total - sent - eps)) < 1e-8


def test_segmented_equals_per_slice_runs():
    part = wl.seeded_partition(40_000, 9, min_size=64, max_weight=2e4)
    g = wl.segmented_normal(part, step=0)
    e0 = wl.normal(part.d, 1e-4, step=77)
    seg_k = part.seg_k(1, 100)
    eps = e0.copy()
    idx, val, seg_nnz, sts = orc.gk_sparsify_segmented(g, eps, part.offsets, seg_k)
    cat_idx, cat_val = [], []
    for s in range(part.S):
        lo, hi = int(part.offsets[s]), int(part.offsets[s + 1])
        es = e0[lo:hi].copy()
        i, v, st = orc.gk_sparsify(g[lo:hi].copy(), es, int(seg_k[s]))
        cat_idx.append(i + lo); cat_val.append(v)
        assert seg_nnz[s] == i.size and sts[s].thr_final == st.thr_final
        assert np.array_equal(bits(es), bits(eps[lo:hi]))
    assert np.array_equal(idx, np.concatenate(cat_idx))
    assert np.array_equal(bits(val), bits(np.concatenate(cat_val)))
    assert np.all(np.diff(idx) > 0)


# --------------------------------------------------------------------------- exact Top_k
def _brute_topk(u, k):
    order = sorted(range(len(u)), key=lambda i: (-abs(float(u[i])), i))
    return sorted(order[:k])


def test_topk_brute_force_with_ties_and_zeros():
    u = np.array([0.5, -2.0, 0.0, 2.0, -0.5, 0.5, -0.0, 1.0, -2.0, 0.25], dtype=np.float32)
    for k in range(1, u.size + 1):
        idx, val = orc.topk_exact(u, k)
        assert idx.tolist() == _brute_topk(u, k)
        assert np.array_equal(bits(val), bits(u[idx]))
    # three entries tie at 2.0: k = 2 keeps the two lowest indices
    assert orc.topk_exact(u, 2)[0].tolist() == [1, 3]
    # +0 and -0 tie: lower index wins
    z = np.array([-0.0, 0.0, -0.0], dtype=np.float32)
    assert orc.topk_exact(z, 2)[0].tolist() == [0, 1]
    rng = wl.misc_rng(6)
    for n in (1, 2, 17, 300):
        x = np.round(rng.standard_normal(n) * 3).astype(np.float32) / 2   # many ties
        for k in sorted({1, n // 3 + 1, n}):
            assert orc.topk_exact(x, k)[0].tolist() == _brute_topk(x, k)


def test_topk_against_numpy_partition():
    u = wl.laplace(1_000_003, 1.0, step=5)
    k = 1001
    idx, val = orc.topk_exact(u, k)
    a = np.abs(u)
    kth = np.partition(a, u.size - k)[u.size - k]
    assert np.all(a[idx] >= kth) and idx.size == k and np.all(np.diff(idx) > 0)
    rest = np.ones(u.size, dtype=bool); rest[idx] = False
    assert a[rest].max() <= kth


def test_topk_contraction_bounds_and_gaussian_closed_form():
    # Eq. 3 / Eq. 10: the (1 - k/d) bound holds for every input
    for u in (wl.laplace_mixture(50_000, step=4), wl.student_t3_outliers(50_000, step=4),
              np.ones(1000, dtype=np.float32), wl.normal(50_000, 2.0, step=1) + np.float32(5.0)):
        for k in (1, 50, u.size // 3):
            idx, _ = orc.topk_exact(u, k)
            assert orc.error_ratio(u, idx) <= (1 - k / u.size) + 1e-12
    # Section 4.2 / Fig. 3 setup: a 100,000-dimensional Gaussian vector.  The exact ratio sits
    # below (1-k/d)^2 and matches 1 - 2(t phi(t) + Q(t)), t = Phi^-1(1 - k/2d).
    d = 100_000
    u = wl.normal(d, 1.0, step=42)
    for rho, expect in (("1e-3", 0.98730), ("1e-2", 0.91551)):
        k = wl.ceil_k(d, *wl.RHO[rho])
        idx, val = orc.topk_exact(u, k)
        r = orc.error_ratio(u, idx)
        t = float(sps.norm.isf(k / (2 * d)))
        closed = 1 - 2 * (t * sps.norm.pdf(t) + sps.norm.sf(t))
        assert abs(closed - expect) < 1e-5
        assert abs(r - closed) < 2.5e-3
        assert r <= (1 - k / d) ** 2 <= (1 - k / d)
        assert abs(np.abs(val).min() / t - 1) < 0.03    # k-th magnitude ~ t sigma


def test_eq5_ratio_from_sorted_normalised_magnitudes():
    # Eq. 5: the ratio equals sum_{i>k} pi_i^2 / sum_i pi_i^2 with pi = sorted |u| / max|u|
    u = wl.laplace(20_000, 3.0, step=8)
    k = 200
    idx, _ = orc.topk_exact(u, k)
    pi = np.sort(np.abs(u.astype(np.float64)) / np.abs(u).max())[::-1]
    ratio = (pi[k:] ** 2).sum() / (pi ** 2).sum()
    assert abs(orc.error_ratio(u, idx) - ratio) < 1e-12


# --------------------------------------------------------------------------- DGC_k (Section 3.3)
def _dgck_brute(u, k, sidx):
    """Pure-Python DGC_k: sampled threshold, candidates, second selection with ties to the
    lower index."""
    d = len(u)
    mags = sorted((abs(float(u[j])) for j in sidx), reverse=True)
    km = -(-k * len(sidx) // d)
    tau = mags[km - 1]
    cand = [i for i in range(d) if abs(float(u[i])) >= tau]
    n = len(cand)
    if n > k:
        cand = sorted(sorted(cand, key=lambda i: (-abs(float(u[i])), i))[:k])
    return cand, tau, n, km


def test_dgck_hand_worked_cases():
    lines = [l.split() for l in open(os.path.join(GOLDEN, "dgck_hand_case.txt")) if not l.startswith("#")]
    u = np.array([float(x) for x in lines[0][1:]], dtype=np.float32)
    for l in lines[1:]:
        assert l[0] == "case"
        k = int(l[l.index("k") + 1])
        s0, t0, i0 = l.index("sample"), l.index("tau"), l.index("idx")
        sidx = np.array([int(x) for x in l[s0 + 1:t0]], dtype=np.int32)
        tau, n, km = float(l[t0 + 1]), int(l[l.index("n") + 1]), int(l[l.index("km") + 1])
        want = np.array([int(x) for x in l[i0 + 1:]], dtype=np.int32)
        idx, val, info = orc.dgck_select(u, k, sidx)
        assert (info.tau, info.n_cand, info.k_m) == (tau, n, km), l[1]
        assert np.array_equal(idx, want) and np.array_equal(val, u[want]), l[1]


def test_dgck_brute_force_small_inputs_with_ties():
    rng = wl.misc_rng(40)
    for trial in range(300):
        d = int(rng.integers(1, 40))
        k = int(rng.integers(1, d + 1))
        m = int(rng.integers(1, 2 * d + 1))
        # few distinct magnitudes, both signs, zeros: ties everywhere
        u = (rng.integers(-4, 5, size=d) * 0.5).astype(np.float32)
        if trial % 3 == 0:
            u = rng.standard_normal(d).astype(np.float32)
        sidx = rng.integers(0, d, size=m).astype(np.int32)
        idx, val, info = orc.dgck_select(u, k, sidx)
        cand, tau, n, km = _dgck_brute(u, k, sidx)
        assert (info.tau, info.n_cand, info.k_m) == (tau, n, km)
        assert idx.tolist() == cand and np.array_equal(bits(val), bits(u[cand]))


def test_dgck_with_the_whole_vector_as_sample_is_exact_topk():
    # sampling every position once makes k_m = k and tau the k-th largest magnitude, so the
    # candidates hold the exact Top_k and the second selection returns it (numpy route)
    rng = wl.misc_rng(41)
    for d, k in [(1000, 1), (1000, 10), (4097, 333), (50_000, 50)]:
        u = rng.standard_normal(d).astype(np.float32)
        u[rng.integers(0, d, size=d // 10)] = np.float32(1.25)  # planted ties
        sidx = rng.permutation(d).astype(np.int32)
        idx, val, info = orc.dgck_select(u, k, sidx)
        order = np.lexsort((np.arange(d), -np.abs(u).astype(np.float64)))  # magnitude desc, index asc
        want = np.sort(order[:k]).astype(np.int32)
        assert info.k_m == k and info.n_cand >= k
        assert np.array_equal(idx, want) and np.array_equal(bits(val), bits(u[want]))


def test_dgck_properties_on_workload_like_inputs():
    d = 1 << 20
    for dist, rho in [("normal", "1e-3"), ("laplace", "1e-2"), ("normal", "1e-2")]:
        w = wl.sweep_point(d, dist)
        u = w.grad(0)
        k = wl.ceil_k(d, *wl.RHO[rho])
        sidx = wl.sample_positions(d, wl.sample_size(d), step=3)
        idx, val, info = orc.dgck_select(u, k, sidx)
        mag = np.abs(u)
        tau = np.float32(info.tau)
        assert info.k_m == -(-k * sidx.size // d)
        # tau is the k_m-th largest sampled magnitude (numpy partition)
        sm = mag[sidx]
        assert tau == np.partition(sm, sm.size - info.k_m)[sm.size - info.k_m]
        assert info.n_cand == int((mag >= tau).sum())
        assert np.all(np.diff(idx) > 0) and np.array_equal(bits(val), bits(u[idx]))
        if info.n_cand <= k:
            assert np.array_equal(idx, np.nonzero(mag >= tau)[0])
        else:
            # more candidates than k: the answer is the exact Top_k of the whole vector
            kth = np.partition(mag, d - k)[d - k]
            assert idx.size == k and mag[idx].min() == kth and int((mag > kth).sum()) <= k
            assert set(np.nonzero(mag > kth)[0]).issubset(set(idx.tolist()))
        # a 1 % sample estimates the density within sampling noise (binomial, k_m entries)
        assert abs(info.n_cand / k - 1.0) < 6.0 / math.sqrt(info.k_m)


def test_dgck_sparsify_identity():
    rng = wl.misc_rng(42)
    d, k = 20_000, 100
    g = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    e = (rng.standard_normal(d) * 2e-3).astype(np.float32)
    sidx = wl.sample_positions(d, 2000, step=5)
    u = g + e
    eps = e.copy()
    idx, val, info = orc.dgck_sparsify(g, eps, k, sidx)
    i2, v2, info2 = orc.dgck_select(u, k, sidx)
    assert np.array_equal(idx, i2) and np.array_equal(bits(val), bits(v2)) and info == info2
    comp = np.zeros(d, dtype=np.float32)
    comp[idx] = val
    assert np.array_equal(bits(comp + eps), bits(u + np.float32(0)))  # Comp(u) + eps_new == u
    assert np.all(eps[idx] == 0) and np.array_equal(bits(np.delete(eps, idx)), bits(np.delete(u, idx)))


# --------------------------------------------------------------------------- Eq. 2: the update from P messages
def _messages(rng, d, P, cap, dense=False):
    idx = np.zeros(P * cap, dtype=np.int32)
    val = np.zeros(P * cap, dtype=np.float32)
    nnz = np.zeros(P, dtype=np.int64)
    for p in range(P):
        n = int(rng.integers(0, cap + 1)) if not dense else cap
        pos = np.sort(rng.choice(d, size=n, replace=False)).astype(np.int32)
        idx[p * cap:p * cap + n] = pos
        val[p * cap:p * cap + n] = rng.standard_normal(n).astype(np.float32)
        nnz[p] = n
    return idx, val, nnz


def test_apply_sparse_single_rank_is_a_scaled_scatter_add():
    rng = wl.misc_rng(50)
    d, cap = 5000, 300
    idx, val, nnz = _messages(rng, d, 1, cap)
    x = rng.standard_normal(d).astype(np.float32)
    want = x.copy()
    n = int(nnz[0])
    alpha = np.float32(-0.125)
    want[idx[:n]] = want[idx[:n]] + alpha * val[:n]     # numpy fp32: one multiply, one add
    orc.apply_sparse(x, idx, val, nnz, cap, float(alpha))
    assert np.array_equal(bits(x), bits(want))


def test_apply_sparse_rank_order_brute_force_and_exact_small_integers():
    rng = wl.misc_rng(51)
    d, P, cap = 400, 5, 120          # dense enough for many positions to occur in several ranks
    idx, val, nnz = _messages(rng, d, P, cap)
    x0 = rng.standard_normal(d).astype(np.float32)
    alpha = np.float32(0.3)
    want = x0.copy()
    for i in range(d):
        s, hit = np.float32(0), False
        for p in range(P):
            lst = idx[p * cap:p * cap + int(nnz[p])]
            j = np.nonzero(lst == i)[0]
            if j.size:
                v = val[p * cap + int(j[0])]
                s = v if not hit else np.float32(s + v)
                hit = True
        if hit:
            want[i] = np.float32(want[i] + np.float32(alpha * s))
    x = x0.copy()
    orc.apply_sparse(x, idx, val, nnz, cap, float(alpha))
    assert np.array_equal(bits(x), bits(want))
    # small integers: every order of additions is exact, so the fp64 scatter-add agrees exactly
    vi = rng.integers(-8, 9, size=P * cap).astype(np.float32)
    x = np.zeros(d, dtype=np.float32)
    orc.apply_sparse(x, idx, vi, nnz, cap, 2.0)
    ref = np.zeros(d)
    for p in range(P):
        n = int(nnz[p])
        np.add.at(ref, idx[p * cap:p * cap + n], 2.0 * vi[p * cap:p * cap + n].astype(np.float64))
    assert np.array_equal(x.astype(np.float64), ref)
    # untouched positions keep their bits (including -0.0)
    x = np.full(d, -0.0, dtype=np.float32)
    orc.apply_sparse(x, idx, val, nnz, cap, 1.0)
    touched = np.zeros(d, dtype=bool)
    for p in range(P):
        touched[idx[p * cap:p * cap + int(nnz[p])]] = True
    assert np.all(bits(x[~touched]) == 0x80000000)


def test_apply_sparse_sums_what_the_workers_selected():
    # P workers sparsify their own vectors; the update applied to x = 0 with alpha = 1 equals
    # the sum of their dense Comp_k(u^p) vectors (fp64 reference, fp32 rounding tolerance)
    rng = wl.misc_rng(52)
    d, P, k = 50_000, 4, 500
    cap = 2 * k
    idx = np.zeros(P * cap, dtype=np.int32); val = np.zeros(P * cap, dtype=np.float32)
    nnz = np.zeros(P, dtype=np.int64)
    dense = np.zeros(d)
    for p in range(P):
        u = (rng.standard_normal(d) * 1e-2).astype(np.float32)
        ti, tv = orc.topk_exact(u, k)
        idx[p * cap:p * cap + k] = ti; val[p * cap:p * cap + k] = tv; nnz[p] = k
        dense[ti] += tv.astype(np.float64)
    x = np.zeros(d, dtype=np.float32)
    orc.apply_sparse(x, idx, val, nnz, cap, 1.0)
    assert np.allclose(x, dense, rtol=1e-6, atol=1e-9)


# --------------------------------------------------------------------------- histogram of u (Section 3.1, Fig. 2)
def test_histogram_on_a_dyadic_grid_equals_numpy():
    # values on a grid of 2^-10 with dyadic bin edges: every fp32 operation of the rule is
    # exact, so numpy's fp64 histogram must agree count for count
    rng = wl.misc_rng(60)
    u = (rng.integers(-3000, 3000, size=200_000) / 1024.0).astype(np.float32)
    lo, hi, nbins = -2.0, 2.0, 64
    counts = orc.histogram(u, lo, nbins / (hi - lo), nbins)
    ref, _ = np.histogram(u.astype(np.float64), bins=nbins, range=(lo, hi))
    # numpy puts x == hi into the last bin; the rule here counts it as "above"
    at_hi = int((u == hi).sum())
    ref[-1] -= at_hi
    assert np.array_equal(counts[1:-1], ref)
    assert counts[0] == int((u < lo).sum()) and counts[-1] == int((u >= hi).sum())
    assert counts.sum() == u.size


def test_histogram_hand_case_and_edges():
    u = np.array([-1.0, -0.5, -0.0, 0.0, 0.25, 0.4999, 0.5, 0.75, 1.0, 7.0, -7.0], dtype=np.float32)
    counts = orc.histogram(u, -1.0, 2.0, 4)   # bins [-1,-.5) [-.5,0) [0,.5) [.5,1)
    assert counts.tolist() == [1, 1, 1, 4, 2, 2]
    assert orc.histogram(np.array([np.nan], dtype=np.float32), 0.0, 1.0, 3).tolist() == [0, 0, 0, 0, 1]


def test_histogram_cdf_of_gaussian_input_matches_the_normal_cdf():
    d = 1 << 21
    u = wl.normal(d, 1e-3, step=9)
    nbins, lo, hi = 200, -5e-3, 5e-3
    counts = orc.histogram(u, np.float32(lo), np.float32(nbins / (hi - lo)), nbins)
    cdf = np.cumsum(counts)[:-1] / d                      # P(u < edge_j), j = 0 .. nbins
    edges = np.linspace(lo, hi, nbins + 1)
    assert np.max(np.abs(cdf - sps.norm.cdf(edges / 1e-3))) < 5.0 / math.sqrt(d)
    # against numpy on the same data: only values within rounding of an edge may move
    ref, _ = np.histogram(u.astype(np.float64), bins=nbins, range=(lo, hi))
    assert np.abs(counts[1:-1] - ref).sum() <= 1e-5 * d
