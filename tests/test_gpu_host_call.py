"""gk_sparsify_host -- the host-buffer entry point behind the end-to-end number -- against the
CPU oracle: pageable and pinned buffers, an error-compensation loop, a step that selects
nothing, a truncated step and k = d."""
import numpy as np
import pytest
import torch

from paper_1911_08772_b200 import binding as gk
from paper_1911_08772_b200 import workloads as wl

from gpu_util import compare_with_oracle

pytestmark = pytest.mark.gpu

CANARY_I = np.int32(-424242)
CANARY_F = np.float32(-3.5)


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    gk.gk_set_capacity(0)
    gk.gk_set_path(0)
    yield
    gk.gk_set_capacity(0)


def _host_step(g, eps, k, cap, pinned):
    """One call on host buffers; returns what check needs.  eps is updated in place."""
    d = g.shape[0]
    if pinned:
        hg = torch.from_numpy(g.copy()).pin_memory()
        he = torch.from_numpy(eps.copy()).pin_memory()
        hi = torch.full((cap + 8,), int(CANARY_I), dtype=torch.int32).pin_memory()
        hv = torch.full((cap + 8,), float(CANARY_F), dtype=torch.float32).pin_memory()
        n, st = gk.gk_sparsify_host(hg, he, k, hi, hv)
        idx, val, eps_new = hi.numpy(), hv.numpy(), he.numpy().copy()
    else:
        hg, he = g.copy(), eps.copy()
        idx = np.full(cap + 8, CANARY_I, dtype=np.int32)
        val = np.full(cap + 8, CANARY_F, dtype=np.float32)
        n, st = gk.gk_sparsify_host(hg, he, k, idx, val)
        eps_new = he
        assert np.array_equal(hg.view(np.uint32), g.view(np.uint32)), "g modified"
    assert 0 <= n <= cap
    assert np.all(idx[n:] == CANARY_I) and np.all(val[n:] == CANARY_F), "write past the reported count"
    return idx[:n].copy(), val[:n].copy(), n, st, eps_new


@pytest.mark.parametrize("pinned", [False, True], ids=["pageable", "pinned"])
@pytest.mark.parametrize("d", [5, 100_003, 2_500_001])
def test_host_call_error_compensation_loop(d, pinned):
    k = max(1, wl.ceil_k(d, 1, 1000))
    eps = np.zeros(d, dtype=np.float32)
    for t in range(3):
        g = wl.normal(d, 1e-3, step=70 + t) if t != 1 else wl.laplace(d, 1e-3, step=70 + t)
        idx, val, n, st, eps_new = _host_step(g, eps, k, d, pinned)
        compare_with_oracle(g, eps, k, idx, val, n, st, eps_new, d)
        eps = eps_new


def test_host_call_selects_nothing_on_a_zero_vector():
    d = 70_001
    z = np.zeros(d, dtype=np.float32)
    idx, val, n, st, eps_new = _host_step(z, z, 7, d, False)
    assert n == 0 and st.nnz == 0 and st.sigma == 0.0
    compare_with_oracle(z, z, 7, idx, val, n, st, eps_new, d)


def test_host_call_truncates_at_the_capacity():
    d = 40_009
    u = wl.normal(d, 1.0, step=75)
    z = np.zeros(d, dtype=np.float32)
    try:
        gk.gk_set_capacity(29)
        idx, val, n, st, eps_new = _host_step(u, z, 400, 29, True)
        assert n == 29 and st.nnz > 29 and st.status & gk.GK_DEV_TRUNCATED
        compare_with_oracle(u, z, 400, idx, val, n, st, eps_new, 29)
    finally:
        gk.gk_set_capacity(0)


def test_host_call_with_k_equal_d_selects_everything():
    d = 12_345
    g = wl.normal(d, 1e-2, step=76)
    e = wl.normal(d, 1e-2, step=77)
    idx, val, n, st, eps_new = _host_step(g, e, d, d, False)
    assert n == d and st.rounds == 0
    compare_with_oracle(g, e, d, idx, val, n, st, eps_new, d)
    assert not eps_new.any()
