"""GPU-vs-oracle parity through the C ABI: small sizes element by element (several
tiles and ragged tails), edge cases, and the five workload families at full size."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_1911_08772_b200 import binding as gk
from paper_1911_08772_b200 import workloads as wl

from gpu_util import DeviceStep, bits, check_gk_step, check_segmented_step, check_topk

pytestmark = pytest.mark.gpu

TILE = 8192  # compaction tile of the library, to place sizes around its edges


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    gk.gk_set_capacity(0)
    yield


@pytest.fixture(params=[0, 1, 2], ids=["default", "three_kernel", "persistent"])
def gk_path(request):
    """Run a test once per implementation of gk_sparsify."""
    gk.gk_set_path(request.param)
    yield request.param
    gk.gk_set_path(0)


# ------------------------------------------------------------------ small sizes, every boundary
SMALL_D = [1, 2, 3, 4, 5, 7, 8, 31, 32, 33, 127, 128, 129, 1023, 1024, 1025, 4095, 4096, 4097,
           TILE - 1, TILE, TILE + 1, 2 * TILE + 3, 5 * TILE - 2, 100_003]


@pytest.mark.parametrize("d", SMALL_D)
def test_gk_sparsify_small_sizes(d, gk_path):
    rng = wl.misc_rng(1000 + d)
    g = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    e = (rng.standard_normal(d) * 2e-3).astype(np.float32)
    step = DeviceStep(d)
    for k in sorted({1, max(1, d // 100), max(1, d // 7), d}):
        check_gk_step(step, g, e, k)


def test_gk_sparsify_special_values(gk_path):
    d = 3 * TILE + 1
    rng = wl.misc_rng(7)
    g = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    e = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    g[:6] = np.array([0.0, -0.0, -0.0, 1e-45, 1e-39, 2.5], dtype=np.float32)
    e[:6] = np.array([-0.0, -0.0, 0.0, 1e-45, -1e-39, -2.5], dtype=np.float32)
    step = DeviceStep(d)
    eps_new, st = check_gk_step(step, g, e, 25)
    assert bits(eps_new)[1] == 0x80000000   # -0 + -0 = -0 survives, denormals are not flushed
    assert bits(eps_new)[3] == 2
    # all zeros: sigma = 0, threshold 0, nothing selected
    z = np.zeros(d, dtype=np.float32)
    _, st = check_gk_step(step, z, z, 10)
    assert st.nnz == 0 and st.sigma == 0.0
    # constant vector: sigma = 0 and thres0 = mu, so every element sits exactly on the first
    # threshold.  One rounding of difference in mu (the two sides sum in different orders) moves
    # all d elements across it, so the per-round counts are not compared here; the threshold
    # (1e-6) and the selection at the library's own threshold still are.
    c = np.full(d, 0.375, dtype=np.float32)
    check_gk_step(step, c, z, 10, check_counts=False)
    # large mean relative to the spread
    check_gk_step(step, (g + np.float32(0.5)).astype(np.float32), z, 30)
    # negative threshold: mean far below zero selects everything
    _, st = check_gk_step(step, (g - np.float32(5.0)).astype(np.float32), z, 30)
    assert st.nnz == d


def test_gk_hand_built_branch_cases(gk_path):
    # the same level vectors that pin the oracle's branch sequences
    from test_oracle_pins import _branch_cases, _levels_vector
    for name, d, k, levels, rounds, counts, fn, fd, nnz in _branch_cases():
        u = _levels_vector(d, levels, seed=11)
        step = DeviceStep(d)
        _, st = check_gk_step(step, u, np.zeros(d, np.float32), k)
        assert st.rounds == rounds and st.counts == counts and st.nnz == nnz, name
        assert abs(st.thr_final / st.thres0 - fn / fd) < 1e-15


def test_gk_capacity_truncation(gk_path):
    d = 4 * TILE + 5
    u = wl.normal(d, 1.0, step=2)
    z = np.zeros(d, dtype=np.float32)
    try:
        gk.gk_set_capacity(37)
        step = DeviceStep(d, cap=37)
        eps_new, st = check_gk_step(step, u, z, 500)
        assert st.status & gk.GK_DEV_TRUNCATED and st.emitted == 37 and st.nnz > 37
    finally:
        gk.gk_set_capacity(0)


def test_gk_is_deterministic_and_stateless(gk_path):
    d = 1_000_003
    g = wl.laplace_mixture(d, step=3)
    e = wl.normal(d, 1e-4, step=4)
    step = DeviceStep(d)
    outs = []
    for _ in range(3):
        eps_new, st = check_gk_step(step, g, e, 1001)
        outs.append((bits(eps_new).copy(), st.thr_final, st.mu, st.sigma, st.nnz))
    for o in outs[1:]:
        assert np.array_equal(o[0], outs[0][0]) and o[1:] == outs[0][1:]


def test_gk_on_a_side_stream(gk_path):
    d = 300_007
    g = wl.normal(d, 1e-3, step=11)
    z = np.zeros(d, np.float32)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        step = DeviceStep(d)
        check_gk_step(step, g, z, 301)


# ------------------------------------------------------------------ exact Top_k
@pytest.mark.parametrize("d", [1, 2, 3, 4, 5, 33, 1025, 4096, 4099, TILE, TILE + 1, 3 * TILE + 2, 250_001,
                               1_900_003])
def test_topk_small_sizes(d, gk_path):
    rng = wl.misc_rng(2000 + d)
    u = rng.standard_normal(d).astype(np.float32)
    for k in sorted({1, max(1, d // 1000), max(1, d // 50), max(1, d // 3), d}):
        check_topk(u, k)


def test_topk_ties_across_rows_and_ctas(gk_path):
    """Heavy ties in a vector of several rows per CTA: the supply of keys equal to the k-th one
    runs out in the middle of a CTA's run, in its last row, or in the ragged tail."""
    rng = wl.misc_rng(77)
    d = 1_300_003
    u = (np.round(rng.standard_normal(d) * 4) / 4).astype(np.float32)
    u[1::5] *= -1
    for k in (1, 17, 1300, 40_000, d // 2, d - 2, d - 1, d):
        check_topk(u, k)
    same = np.full(d, 0.75, dtype=np.float32)
    same[2::7] = -0.75
    for k in (1, 4096, 4097, 600_000, d - 3, d - 2, d - 1, d):
        idx, _ = check_topk(same, k)
        assert idx[0] == 0 and idx[-1] == k - 1
    # one large entry in the ragged tail, ties everywhere else
    same[d - 1] = 9.0
    idx, _ = check_topk(same, 5)
    assert idx.tolist() == [0, 1, 2, 3, d - 1]


def test_topk_ties_and_zeros(gk_path):
    rng = wl.misc_rng(5)
    d = 2 * TILE + 77
    u = (np.round(rng.standard_normal(d) * 2) / 2).astype(np.float32)  # heavy ties, many +-0
    u[::3] *= -1
    for k in (1, 10, 500, d // 2, d - 1, d):
        check_topk(u, k)
    z = np.zeros(d, dtype=np.float32)
    z[1::2] = -0.0
    idx, _ = check_topk(z, 100)
    assert idx.tolist() == list(range(100))
    same = np.full(d, -3.5, dtype=np.float32)
    idx, _ = check_topk(same, 1000)
    assert idx.tolist() == list(range(1000))
    tiny = np.array([1e-45, -1e-45, 0.0, 3e-39, -3e38], dtype=np.float32)
    check_topk(tiny, 3)


@pytest.mark.parametrize("d,k", [(3 * TILE + 9, 123), (7, 7), (5, 2), (2_000_003, 2001), (2_000_003, 1_000_000)])
def test_topk_sparsify_matches_eq2_with_exact_topk(d, k, gk_path):
    g = wl.laplace(d, 1.0, step=21)
    e = wl.normal(d, 0.5, step=22)
    dev = torch.device("cuda:0")
    dg, de = torch.from_numpy(g).to(dev), torch.from_numpy(e).to(dev)
    idx = torch.empty(k, dtype=torch.int32, device=dev)
    val = torch.empty(k, dtype=torch.float32, device=dev)
    nnz = torch.zeros(1, dtype=torch.int64, device=dev)
    gk.topk_sparsify(dg, de, k, idx, val, nnz)
    torch.cuda.synchronize()
    u = orc.accumulate(g, e)
    oi, ov = orc.topk_exact(u, k)
    assert int(nnz.item()) == k
    assert np.array_equal(idx.cpu().numpy(), oi) and np.array_equal(bits(val.cpu().numpy()), bits(ov))
    assert np.array_equal(bits(de.cpu().numpy()), bits(orc.residual(u, oi, ov)))


# ------------------------------------------------------------------ error ratio (Eq. 5)
@pytest.mark.parametrize("d,k", [(1, 1), (6, 2), (4099, 40), (250_001, 250), (2_000_003, 20_000)])
def test_error_ratio_after_gaussiank_and_topk(d, k):
    """||u - Comp(u)||^2 / ||u||^2 from the residual and the values sent, against the oracle's
    Eq. 5 evaluated on u and the kept positions, for Gaussian_k and for exact Top_k."""
    g = wl.normal(d, 1.0, step=31)
    e = wl.laplace(d, 0.3, step=32)
    u = orc.accumulate(g, e)
    dev = torch.device("cuda:0")
    for which in ("gaussiank", "topk"):
        dg, de = torch.from_numpy(g).to(dev), torch.from_numpy(e).to(dev)
        idx = torch.empty(d, dtype=torch.int32, device=dev)
        val = torch.empty(d, dtype=torch.float32, device=dev)
        nnz = torch.zeros(1, dtype=torch.int64, device=dev)
        if which == "gaussiank":
            gk.gk_sparsify(dg, de, k, idx, val, nnz)
        else:
            gk.topk_sparsify(dg, de, k, idx, val, nnz)
        ratio, err2, all2 = gk.gk_error_ratio(de, val, nnz)
        n = int(nnz.item())
        kept = idx[:n].cpu().numpy()
        expect = orc.error_ratio(u, kept)
        assert abs(ratio - expect) <= 1e-10, (which, ratio, expect)
        u64 = u.astype(np.float64)
        assert abs(all2 - float(np.dot(u64, u64))) <= 1e-10 * all2
        assert abs(err2 - ratio * all2) <= 1e-10 * all2
        if which == "topk":
            assert ratio <= (1.0 - k / d) + 1e-12           # Eq. 4 holds for every u
    # a zero vector: nothing to lose
    z = torch.zeros(4099, device=dev)
    val = torch.zeros(8, device=dev)
    nnz = torch.zeros(1, dtype=torch.int64, device=dev)
    assert gk.gk_error_ratio(z, val, nnz) == (0.0, 0.0, 0.0)


# ------------------------------------------------------------------ segmented
def _dev_i64(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int64)).to("cuda:0")


def test_segmented_small_and_ragged(gk_path):
    offsets = np.array([0, 1, 1, 3, 10, 64, 65, 1000, 1003, 5000, 5000, 9001, 3 * TILE + 6, 4 * TILE + 1],
                       dtype=np.int64)
    d = int(offsets[-1])
    S = offsets.shape[0] - 1
    rng = wl.misc_rng(31)
    g = (rng.standard_normal(d) * np.repeat(rng.uniform(1e-4, 1e-1, S), np.diff(offsets))).astype(np.float32)
    e = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    sizes = np.diff(offsets)
    step = DeviceStep(d)
    nn = torch.zeros(S, dtype=torch.int64, device="cuda:0")
    for rho_num, rho_den in ((1, 100), (1, 3), (1, 1)):
        seg_k = np.array([max(1, wl.ceil_k(int(n), rho_num, rho_den)) for n in sizes], dtype=np.int64)
        check_segmented_step(step, g, e, offsets, seg_k, _dev_i64(offsets), _dev_i64(seg_k), nn)


def test_segmented_single_segment_equals_whole_vector(gk_path):
    d = 2 * TILE + 11
    g = wl.normal(d, 1e-2, step=5)
    z = np.zeros(d, np.float32)
    offsets = np.array([0, d], dtype=np.int64)
    seg_k = np.array([50], dtype=np.int64)
    step = DeviceStep(d)
    nn = torch.zeros(1, dtype=torch.int64, device="cuda:0")
    eps_a, sts = check_segmented_step(step, g, z, offsets, seg_k, _dev_i64(offsets), _dev_i64(seg_k), nn)
    eps_b, st = check_gk_step(step, g, z, 50)
    assert np.array_equal(bits(eps_a), bits(eps_b))
    assert sts[0].thr_final == st.thr_final or abs(sts[0].thr_final / st.thr_final - 1) < 1e-12


@pytest.mark.parametrize("S,d", [(256, 700_003), (257, 700_003), (200, 5_000), (40, 3_000_001)])
def test_segmented_many_segments_across_rows_and_ctas(S, d, gk_path):
    """Random tables: boundaries inside rows and inside float4 groups, empty segments, segments
    that select everything, runs of several CTAs in one segment and many segments in one row;
    256 segments is the most the single-kernel form takes, 257 goes to the three-kernel form."""
    rng = wl.misc_rng(900 + S)
    cuts = np.sort(rng.integers(0, d + 1, size=S - 1))
    cuts[: S // 10] = np.sort(rng.integers(0, min(d, 6000) + 1, size=S // 10))   # a crowd at the start
    cuts = np.sort(cuts)
    offsets = np.concatenate([[0], cuts, [d]]).astype(np.int64)
    offsets[5] = offsets[4]          # an empty segment
    sizes = np.diff(offsets)
    scale = np.repeat(rng.uniform(1e-4, 1e-1, S), sizes)
    g = (rng.standard_normal(d) * scale).astype(np.float32)
    e = (rng.standard_normal(d) * scale * 0.5).astype(np.float32)
    seg_k = np.array([max(1, wl.ceil_k(int(n), 1, 50)) for n in sizes], dtype=np.int64)
    seg_k[::7] = 10 ** 9             # more than the segment holds: everything is selected there
    step = DeviceStep(d)
    nn = torch.zeros(S, dtype=torch.int64, device="cuda:0")
    eps, _ = check_segmented_step(step, g, e, offsets, seg_k, _dev_i64(offsets), _dev_i64(seg_k), nn)
    check_segmented_step(step, g, eps, offsets, seg_k, _dev_i64(offsets), _dev_i64(seg_k), nn)


def test_segmented_bad_table_is_reported_not_fatal(gk_path):
    d = 20_000
    g = wl.normal(d, 1e-2, step=6)
    offsets = np.array([0, 9000, 8000, d], dtype=np.int64)  # not ascending
    seg_k = np.array([5, 5, 5], dtype=np.int64)
    step = DeviceStep(d)
    step.g.copy_(torch.from_numpy(g))
    step.eps.zero_()
    step.arm()
    nn = torch.zeros(3, dtype=torch.int64, device="cuda:0")
    gk.gk_sparsify_segmented(step.g, step.eps, _dev_i64(offsets), _dev_i64(seg_k), step.idx[:d], step.val[:d],
                             nn, step.nnz[:1])
    idx, val, n = step.outputs()
    sts = gk.gk_last_segment_stats(3)
    assert n == 0 and all(s.status & gk.GK_DEV_BAD_SEGMENTS for s in sts)


# ------------------------------------------------------------------ the workload families, full size
def _ec_loop(w, rho, steps, check_every=1, also=None):
    k = w.k(rho)
    step = DeviceStep(w.d)
    eps = np.zeros(w.d, dtype=np.float32)
    g = np.empty(w.d, dtype=np.float32)
    for t in range(steps):
        w.grad(t, g)
        eps, st = check_gk_step(step, g, eps, k)
        if also is not None:
            also(t, st)
    return eps


def test_workload_resnet20_normal(gk_path):
    w = wl.resnet20_normal()
    assert w.k("1e-3") == 270
    _ec_loop(w, "1e-3", 1 + 10)


def test_workload_vgg16_laplace_mixture_100_steps():
    w = wl.vgg16_laplace_mixture()
    nnzs = []
    _ec_loop(w, "1e-3", 100, also=lambda t, st: nnzs.append(st.nnz))
    assert min(nnzs) > 0


def test_workload_resnet50_three_kernel_path():
    gk.gk_set_path(1)
    try:
        w = wl.resnet50_segmented()
        _ec_loop(w, "1e-3", 5)
        # and the layer-wise call in its three-kernel form
        part = w.partition
        seg_k = part.seg_k(*wl.RHO["1e-3"])
        step = DeviceStep(w.d)
        dev_off, dev_k = _dev_i64(part.offsets), _dev_i64(seg_k)
        nn = torch.zeros(part.S, dtype=torch.int64, device="cuda:0")
        eps = np.zeros(w.d, dtype=np.float32)
        for t in range(3):
            eps, _ = check_segmented_step(step, w.grad(t, None), eps, part.offsets, seg_k, dev_off, dev_k, nn)
    finally:
        gk.gk_set_path(0)


def test_both_paths_agree_bit_for_bit():
    w = wl.vgg16_laplace_mixture()
    g = w.grad(0, None)
    e = wl.normal(w.d, 1e-4, step=9)
    k = w.k("1e-3")
    step = DeviceStep(w.d)
    outs = []
    for path in (0, 1):
        gk.gk_set_path(path)
        try:
            eps_new, st = check_gk_step(step, g, e, k)
        finally:
            gk.gk_set_path(0)
        outs.append((bits(eps_new).copy(), st.thr_final, st.counts, st.nnz))
    assert np.array_equal(outs[0][0], outs[1][0]) and outs[0][2:] == outs[1][2:]
    assert abs(outs[0][1] / outs[1][1] - 1) < 1e-12


@pytest.mark.parametrize("rho", ["1e-3", "1e-2"])
def test_workload_resnet50_global_and_segmented(rho):
    w = wl.resnet50_segmented()
    part = w.partition
    assert part.S == 161 and int(part.sizes().min()) >= 64
    steps = 20
    # global selection
    _ec_loop(w, rho, steps)
    # layer-wise selection
    seg_k = part.seg_k(*wl.RHO[rho])
    step = DeviceStep(w.d)
    dev_off, dev_k = _dev_i64(part.offsets), _dev_i64(seg_k)
    nn = torch.zeros(part.S, dtype=torch.int64, device="cuda:0")
    eps = np.zeros(w.d, dtype=np.float32)
    g = np.empty(w.d, dtype=np.float32)
    for t in range(steps):
        w.grad(t, g)
        eps, _ = check_segmented_step(step, g, eps, part.offsets, seg_k, dev_off, dev_k, nn)


@pytest.mark.parametrize("rho", ["1e-3", "5e-3"])
def test_workload_lstm_student_t(rho):
    w = wl.lstm_student_t()
    eps = _ec_loop(w, rho, 20)
    # exact radix Top_k on the same u (= last eps plus a fresh gradient)
    g = w.grad(20, None)
    u = orc.accumulate(g, eps)
    check_topk(u, w.k(rho))


@pytest.mark.parametrize("dist", ["normal", "laplace"])
@pytest.mark.parametrize("log2d", [20, 22, 24, 26])
def test_workload_sweep(dist, log2d):
    w = wl.sweep_point(1 << log2d, dist)
    g = w.grad(0, None)
    z = np.zeros(w.d, dtype=np.float32)
    step = DeviceStep(w.d)
    for rho in w.rhos:
        check_gk_step(step, g, z, w.k(rho))
    for rho in w.rhos:
        check_topk(g, w.k(rho))


@pytest.mark.parametrize("dist", ["normal", "laplace"])
def test_workload_sweep_largest(dist):
    """d = 2^28 (1 GiB per vector): Gaussian_k against the oracle in full; exact Top_k by
    properties that fix the answer uniquely (count, threshold, tie order), since a full
    CPU sort of 2^28 keys takes most of a minute per case."""
    w = wl.sweep_point(1 << 28, dist)
    g = w.grad(0, None)
    z = np.zeros(w.d, dtype=np.float32)
    step = DeviceStep(w.d)
    for rho in w.rhos:
        check_gk_step(step, g, z, w.k(rho))
    del step
    torch.cuda.empty_cache()
    k = w.k("1e-3")
    dev = torch.device("cuda:0")
    du = torch.from_numpy(g).to(dev)
    idx = torch.empty(k, dtype=torch.int32, device=dev)
    val = torch.empty(k, dtype=torch.float32, device=dev)
    gk.topk_exact(du, k, idx, val)
    torch.cuda.synchronize()
    hi, hv = idx.cpu().numpy(), val.cpu().numpy()
    assert np.all(np.diff(hi) > 0)
    assert np.array_equal(bits(hv), bits(g[hi]))
    kth = np.abs(hv).min()
    # everything strictly above the k-th magnitude is in; nothing below it is
    assert orc.count_above(g, float(kth)) == int((np.abs(hv) > kth).sum())
    below = np.nextafter(kth, np.float32(0))
    assert orc.count_above(g, float(below)) >= k
    # entries equal to the k-th magnitude are the lowest-index ones
    ties_all = np.nonzero(np.abs(g) == kth)[0]
    ties_sel = hi[np.abs(hv) == kth]
    assert np.array_equal(ties_sel, ties_all[:ties_sel.size].astype(np.int32))


def test_gk_half_a_billion_elements_on_the_fused_kernel():
    """d = 2^29 + 3 (the upper end of the paper's operator timing sweep, Section 4.1): 886 rows
    per CTA, eps taken through the ring, one row kept on chip, a ragged tail; against the
    oracle in full."""
    d = (1 << 29) + 3
    k = wl.ceil_k(d, 1, 1000)
    g = wl.normal(d, 1.0, step=11)
    z = np.zeros(d, dtype=np.float32)
    cap = 2 * k
    gk.gk_set_capacity(cap)
    try:
        step = DeviceStep(d, cap=cap)
        before = gk.gk_launch_count()
        check_gk_step(step, g, z, k)
        assert gk.gk_launch_count() - before == 1      # one cooperative kernel, not the three-kernel form
    finally:
        gk.gk_set_capacity(0)
    del step
    torch.cuda.empty_cache()


def test_everything_selected_on_a_vector_of_many_rows(gk_path):
    """A mean far below zero makes every threshold of Algorithm 1 negative, so every element is
    selected: more survivors per CTA than the on-chip list of places holds, which takes the
    write-out of one warp per segment; whole vector and layer-wise."""
    d = 6_000_003
    rng = wl.misc_rng(77)
    g = (rng.standard_normal(d) * 1e-3 - 5.0).astype(np.float32)
    z = np.zeros(d, dtype=np.float32)
    step = DeviceStep(d)
    eps_new, st = check_gk_step(step, g, z, 6000)
    assert st.nnz == d and st.thr_final < 0 and not eps_new.any()
    if gk_path == 0:
        offsets = np.array([0, 1_000_001, 1_000_001, 3_500_000, d], dtype=np.int64)
        seg_k = np.array([1000, 5, 2500, 2500], dtype=np.int64)
        dev_off = torch.from_numpy(offsets).cuda()
        dev_k = torch.from_numpy(seg_k).cuda()
        nn = torch.zeros(4, dtype=torch.int64, device="cuda")
        eps_new, _ = check_segmented_step(step, g, z, offsets, seg_k, dev_off, dev_k, nn)
        assert not eps_new.any()


def test_the_three_implementations_agree_on_a_small_vector():
    # the cluster kernel (default below 589,824 elements), the persistent kernel and the three
    # kernels: same pairs, same residual, same counts
    d = 269_722
    g = wl.normal(d, 1e-3, step=21)
    e = wl.laplace(d, 1e-3, step=22)
    step = DeviceStep(d)
    outs = []
    for path in (0, 1, 2):
        gk.gk_set_path(path)
        try:
            before = gk.gk_launch_count()
            eps_new, st = check_gk_step(step, g, e, 270)
            launches = gk.gk_launch_count() - before
        finally:
            gk.gk_set_path(0)
        assert launches == (3 if path == 1 else 1)
        outs.append((bits(eps_new).copy(), st.counts, st.nnz, st.rounds))
    for o in outs[1:]:
        assert np.array_equal(o[0], outs[0][0]) and o[1:] == outs[0][1:]
