"""GPU-vs-oracle parity of DGC_k (Section 3.3 of the paper) through the C ABI.

Everything here is integer and bit work: the sampled threshold, the candidate count, the
rank taken in the sample and the (index, value) lists must equal the oracle's exactly."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_1911_08772_b200 import binding as gk
from paper_1911_08772_b200 import workloads as wl

from gpu_util import CANARY_F, CANARY_I, GUARD, bits

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    yield


def run_select(u, k, sidx):
    du = torch.from_numpy(u).to(DEV)
    ds = torch.from_numpy(sidx).to(DEV)
    idx = torch.full((k + GUARD,), int(CANARY_I), dtype=torch.int32, device=DEV)
    val = torch.full((k + GUARD,), float(CANARY_F), dtype=torch.float32, device=DEV)
    nnz = torch.full((3,), -99, dtype=torch.int64, device=DEV)
    gk.dgck_select(du, k, ds, idx[:k], val[:k], nnz[:1])
    info = gk.dgck_last_info()
    st = gk.gk_last_stats()
    hn = nnz.cpu().numpy()
    assert hn[1] == -99 and hn[2] == -99
    n = int(hn[0])
    hi, hv = idx.cpu().numpy(), val.cpu().numpy()
    assert np.all(hi[n:] == CANARY_I) and np.all(hv[n:] == CANARY_F), "write past the pairs"
    assert np.array_equal(bits(du.cpu().numpy()), bits(u)), "u modified"
    return hi[:n].copy(), hv[:n].copy(), info, st.status


def check_select(u, k, sidx):
    hi, hv, info, status = run_select(u, k, sidx)
    oi, ov, oinfo = orc.dgck_select(u, k, sidx)
    assert status == 0
    assert info[:3] == (oinfo.tau_bits, oinfo.n_cand, oinfo.k_m), (info, oinfo)
    assert info[3] == oi.size == hi.size
    assert np.array_equal(hi, oi)
    assert np.array_equal(bits(hv), bits(ov))
    return oinfo


def check_sparsify(g, e, k, sidx):
    d = g.shape[0]
    dg, de = torch.from_numpy(g).to(DEV), torch.from_numpy(e).to(DEV)
    ds = torch.from_numpy(sidx).to(DEV)
    idx = torch.full((k + GUARD,), int(CANARY_I), dtype=torch.int32, device=DEV)
    val = torch.full((k + GUARD,), float(CANARY_F), dtype=torch.float32, device=DEV)
    nnz = torch.full((1,), -99, dtype=torch.int64, device=DEV)
    gk.dgck_sparsify(dg, de, k, ds, idx[:k], val[:k], nnz)
    info = gk.dgck_last_info()
    n = int(nnz.item())
    hi, hv = idx.cpu().numpy(), val.cpu().numpy()
    assert np.all(hi[n:] == CANARY_I) and np.all(hv[n:] == CANARY_F)
    oeps = e.copy()
    oi, ov, oinfo = orc.dgck_sparsify(g, oeps, k, sidx)
    assert info[:3] == (oinfo.tau_bits, oinfo.n_cand, oinfo.k_m)
    assert n == oi.size and np.array_equal(hi[:n], oi) and np.array_equal(bits(hv[:n]), bits(ov))
    assert np.array_equal(bits(de.cpu().numpy()), bits(oeps))
    assert np.array_equal(bits(dg.cpu().numpy()), bits(g)), "g modified"
    return de.cpu().numpy()


SMALL_D = [1, 2, 3, 5, 8, 33, 127, 129, 1023, 1025, 4095, 4096, 4097, 8193, 3 * 4096 + 3, 40 * 4096 - 2, 700_001]


@pytest.mark.parametrize("d", SMALL_D)
def test_dgck_select_small_sizes(d):
    rng = wl.misc_rng(3000 + d)
    u = (rng.standard_normal(d) * 1e-3).astype(np.float32)
    for k in sorted({1, max(1, d // 100), max(1, d // 7), d}):
        for m in sorted({1, max(1, d // 100), max(1, d // 3), d, 2 * d + 1}):
            sidx = rng.integers(0, d, size=m).astype(np.int32)
            check_select(u, k, sidx)


def test_dgck_select_ties_and_zeros():
    # few distinct magnitudes across rows and CTAs: tau and the k-th candidate both sit in ties
    rng = wl.misc_rng(3100)
    d = 600 * 4096 + 2
    u = (rng.integers(-3, 4, size=d) * 0.25).astype(np.float32)
    u[rng.integers(0, d, size=50)] = np.float32(-0.0)
    for k, m in [(1, 10), (1000, 5000), (d // 7, d // 50), (d // 2, 1000), (d, 1000)]:
        sidx = rng.integers(0, d, size=m).astype(np.int32)
        info = check_select(u, k, sidx)
    z = np.zeros(d, dtype=np.float32)  # tau = 0: every entry is a candidate
    info = check_select(z, 100, rng.integers(0, d, size=1000).astype(np.int32))
    assert info.n_cand == d and info.tau == 0.0


def test_dgck_both_branches_are_reached():
    # the same vector with a sample that over-estimates tau (fewer than k candidates, returned
    # as they are) and one that under-estimates it (second selection among the candidates)
    rng = wl.misc_rng(3200)
    d, k = 1 << 20, 1000
    u = rng.standard_normal(d).astype(np.float32)
    order = np.argsort(-np.abs(u), kind="stable")
    high = order[:50].astype(np.int32)            # the 50 largest: tau lands far above the k-th magnitude
    low = order[5000:5100].astype(np.int32)       # tau below the k-th magnitude
    few = check_select(u, k, np.concatenate([high, high]))
    assert few.n_cand < k
    many = check_select(u, k, low)
    assert many.n_cand > k
    # the whole vector as the sample reproduces exact Top_k
    hi, hv, info, _ = run_select(u, k, rng.permutation(d).astype(np.int32))
    ti, tv = orc.topk_exact(u, k)
    assert np.array_equal(hi, ti) and np.array_equal(bits(hv), bits(tv))


def test_dgck_sample_larger_than_the_on_chip_cache():
    # more sampled positions per CTA than the shared-memory cache of keys holds
    rng = wl.misc_rng(3300)
    d = 1 << 20
    u = rng.standard_normal(d).astype(np.float32)
    sidx = rng.integers(0, d, size=148 * 45056 + 12345).astype(np.int32)
    check_select(u, 2000, sidx)


def test_dgck_bad_sample_position_is_flagged_not_fatal():
    rng = wl.misc_rng(3400)
    d = 100_000
    u = rng.standard_normal(d).astype(np.float32)
    sidx = rng.integers(0, d, size=1000).astype(np.int32)
    sidx[17] = d + 5
    sidx[400] = -3
    hi, hv, info, status = run_select(u, 100, sidx)
    assert status & gk.GK_DEV_BAD_SAMPLE
    clamped = np.clip(sidx, 0, d - 1)
    oi, ov, _ = orc.dgck_select(u, 100, clamped)
    assert np.array_equal(hi, oi)
    # and the library is still usable
    check_select(u, 100, clamped)


@pytest.mark.parametrize("d", [5, 4097, 300_007, 2_000_003])
def test_dgck_sparsify_error_compensation_loop(d):
    rng = wl.misc_rng(3500 + d % 1000)
    k = max(1, d // 1000)
    m = wl.sample_size(d)
    eps = np.zeros(d, dtype=np.float32)
    for t in range(4):
        g = (rng.standard_normal(d) * 1e-3).astype(np.float32)
        sidx = wl.sample_positions(d, m, step=t)
        eps = check_sparsify(g, eps, k, sidx)


def test_dgck_argument_errors():
    d = 1000
    u = torch.zeros(d, device=DEV)
    s = torch.zeros(10, dtype=torch.int32, device=DEV)
    idx = torch.zeros(d, dtype=torch.int32, device=DEV)
    val = torch.zeros(d, device=DEV)
    nnz = torch.zeros(1, dtype=torch.int64, device=DEV)
    L = gk.load()
    st = torch.cuda.current_stream().cuda_stream
    assert L.dgck_select(u.data_ptr(), d, 0, s.data_ptr(), 10, idx.data_ptr(), val.data_ptr(), nnz.data_ptr(), st) == -3
    assert L.dgck_select(u.data_ptr(), d, d + 1, s.data_ptr(), 10, idx.data_ptr(), val.data_ptr(), nnz.data_ptr(), st) == -3
    assert L.dgck_select(u.data_ptr(), d, 5, s.data_ptr(), 0, idx.data_ptr(), val.data_ptr(), nnz.data_ptr(), st) == -2
    assert L.dgck_select(None, d, 5, s.data_ptr(), 10, idx.data_ptr(), val.data_ptr(), nnz.data_ptr(), st) == -1
    assert L.dgck_sparsify(u.data_ptr(), u.data_ptr(), d, 5, s.data_ptr(), 10, idx.data_ptr(), val.data_ptr(),
                           nnz.data_ptr(), st) == -5


# ------------------------------------------------------------------ the workload families, full size
@pytest.mark.parametrize("name", ["resnet20", "vgg16", "resnet50", "lstm"])
def test_dgck_workloads(name):
    w = {"resnet20": wl.resnet20_normal, "vgg16": wl.vgg16_laplace_mixture,
         "resnet50": wl.resnet50_segmented, "lstm": wl.lstm_student_t}[name]()
    m = wl.sample_size(w.d)
    eps = np.zeros(w.d, dtype=np.float32)
    for t in range(2):
        g = w.grad(t, None)
        for rho in w.rhos[:1]:
            eps_next = check_sparsify(g, eps, w.k(rho), wl.sample_positions(w.d, m, step=t))
        eps = eps_next
    u = orc.accumulate(w.grad(2, None), eps)
    for rho in w.rhos:
        check_select(u, w.k(rho), wl.sample_positions(w.d, m, step=7))


@pytest.mark.parametrize("dist", ["normal", "laplace"])
@pytest.mark.parametrize("log2d", [20, 24, 26])
def test_dgck_sweep(dist, log2d):
    w = wl.sweep_point(1 << log2d, dist)
    u = w.grad(0, None)
    sidx = wl.sample_positions(w.d, wl.sample_size(w.d), step=1)
    for rho in w.rhos:
        check_select(u, w.k(rho), sidx)


def test_dgck_sweep_largest():
    """d = 2^28: the oracle's second selection sorts only the candidates, so the full
    comparison stays affordable."""
    w = wl.sweep_point(1 << 28, "normal")
    u = w.grad(0, None)
    sidx = wl.sample_positions(w.d, wl.sample_size(w.d), step=1)
    check_select(u, w.k("1e-3"), sidx)
