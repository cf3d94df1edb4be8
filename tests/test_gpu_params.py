"""gk_set_params -- the two constants of Algorithm 1 that the paper leaves open to reading (the
divisor of the variance, the number of rounds) -- against the oracle run with the same
settings, on both implementations and on the layer-wise call."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_1911_08772_b200 import binding as gk
from paper_1911_08772_b200 import workloads as wl

from gpu_util import DeviceStep, check_gk_step

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _library():
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    gk.gk_set_capacity(0)
    gk.gk_set_path(0)
    yield
    gk.gk_set_params(True, 4)
    gk.gk_set_path(0)


@pytest.mark.parametrize("path", [0, 1, 2], ids=["default", "three_kernel", "persistent"])
@pytest.mark.parametrize("max_rounds", [1, 2, 3, 4])
@pytest.mark.parametrize("unbiased", [True, False])
def test_rounds_and_divisor(path, max_rounds, unbiased):
    gk.gk_set_path(path)
    gk.gk_set_params(unbiased, max_rounds)
    # a small vector makes the two divisors differ by far more than the tolerance (1 / 2d = 4e-4)
    for d, k, g in ((1_237, 13, wl.normal(1_237, 1e-3, step=40)),
                    (3_000_017, 3001, wl.laplace(3_000_017, 1e-3, step=41))):
        step = DeviceStep(d)
        eps = wl.normal(d, 1e-3, step=42)
        _, st = check_gk_step(step, g, eps, k, max_rounds=max_rounds, unbiased=unbiased)
        assert st.rounds <= max_rounds
    if not unbiased:
        u = orc.accumulate(wl.normal(1_237, 1e-3, step=40), wl.normal(1_237, 1e-3, step=42))
        a, b = orc.gaussiank_threshold(u, 13, unbiased=True), orc.gaussiank_threshold(u, 13, unbiased=False)
        assert abs(a.sigma / b.sigma - 1) > 1e-4     # the test above could tell the two apart


def test_out_of_range_rounds_are_refused():
    L = gk.load()
    assert L.gk_set_params(1, 0) == -2 and L.gk_set_params(1, 5) == -2


def test_segmented_call_follows_the_parameters():
    from gpu_util import check_segmented_step  # noqa: F401  (the default-parameter check lives there)
    d = 400_003
    part = wl.seeded_partition(d, 9)
    g = wl.segmented_normal(part, step=43)
    dev = torch.device("cuda:0")
    seg_k = part.seg_k(1, 100)
    step = DeviceStep(d)
    step.g.copy_(torch.from_numpy(g))
    step.eps.zero_()
    step.arm()
    d_off, d_k = torch.from_numpy(part.offsets).to(dev), torch.from_numpy(seg_k).to(dev)
    seg_nnz = torch.zeros(part.S, dtype=torch.int64, device=dev)
    gk.gk_set_params(False, 2)
    gk.gk_sparsify_segmented(step.g, step.eps, d_off, d_k, step.idx[:d], step.val[:d], seg_nnz, step.nnz[:1])
    idx, val, n = step.outputs()
    sts = gk.gk_last_segment_stats(part.S)
    for s in range(part.S):
        lo, hi = int(part.offsets[s]), int(part.offsets[s + 1])
        ost = orc.gaussiank_threshold(np.ascontiguousarray(g[lo:hi]), int(seg_k[s]), max_rounds=2, unbiased=False)
        assert sts[s].rounds == ost.rounds and sts[s].counts == ost.counts
        assert abs(sts[s].sigma - ost.sigma) <= 1e-6 * ost.sigma
        assert abs(sts[s].thr_final - ost.thr_final) <= 1e-6 * abs(ost.thr_final)
