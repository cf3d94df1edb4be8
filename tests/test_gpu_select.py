"""gk_select -- Gaussian_k as an operator on a given u (Algorithm 1 as printed) -- against the
oracle's threshold search and selection: small sizes with ragged tails, both implementations,
the hand-built branch cases, truncation, and workload-sized vectors."""
import numpy as np
import pytest

from paper_1911_08772_b200 import binding as gk
from paper_1911_08772_b200 import workloads as wl

from gpu_util import DeviceStep, check_gk_select

pytestmark = pytest.mark.gpu

TILE = 8192
SMALL_D = [1, 2, 3, 4, 5, 7, 8, 31, 32, 33, 127, 128, 129, 1023, 1024, 1025, 4095, 4096, 4097,
           TILE - 1, TILE, TILE + 1, 2 * TILE + 3, 5 * TILE - 2, 100_003]


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    gk.gk_set_capacity(0)
    yield
    gk.gk_set_path(0)
    gk.gk_debug_set(gk.KNOB_PREDICTION, -1)


@pytest.fixture(params=[0, 1, 2], ids=["default", "three_kernel", "persistent"])
def gk_path(request):
    gk.gk_set_path(request.param)
    yield request.param
    gk.gk_set_path(0)


@pytest.mark.parametrize("d", SMALL_D)
def test_gk_select_small_sizes(d, gk_path):
    rng = wl.misc_rng(3000 + d)
    u = (rng.standard_normal(d) * 3e-3).astype(np.float32)
    step = DeviceStep(d)
    for k in sorted({1, max(1, d // 100), max(1, d // 7), d}):
        check_gk_select(step, u, k)


def test_gk_select_hand_built_branch_cases(gk_path):
    from test_oracle_pins import _branch_cases, _levels_vector
    for name, d, k, levels, rounds, counts, fn, fd, nnz in _branch_cases():
        u = _levels_vector(d, levels, seed=11)
        st = check_gk_select(DeviceStep(d), u, k)
        assert st.rounds == rounds and st.counts == counts and st.nnz == nnz, name


def test_gk_select_truncation_and_special_values(gk_path):
    d = 4 * TILE + 5
    u = wl.normal(d, 1.0, step=2)
    u[:4] = np.array([0.0, -0.0, 1e-45, -1e-39], dtype=np.float32)
    try:
        gk.gk_set_capacity(37)
        st = check_gk_select(DeviceStep(d, cap=37), u, 500)
        assert st.status & gk.GK_DEV_TRUNCATED and st.emitted == 37 and st.nnz > 37
    finally:
        gk.gk_set_capacity(0)
    check_gk_select(DeviceStep(d), (u - np.float32(9.0)).astype(np.float32), 30)   # negative threshold: everything
    check_gk_select(DeviceStep(d), np.zeros(d, np.float32), 30)


@pytest.mark.parametrize("mode", [0, 1], ids=["counted_after", "counted_while_streaming"])
def test_gk_select_workload_vectors(mode):
    gk.gk_set_path(0)
    gk.gk_debug_set(gk.KNOB_PREDICTION, mode)
    try:
        for u, k in ((wl.laplace_mixture(6_000_011, step=5), 6001),
                     (wl.normal(9_000_001, 1e-3, step=6), 90_001),
                     (wl.student_t3_outliers(7_000_003, step=7), 7001)):
            check_gk_select(DeviceStep(u.shape[0]), u, k)
    finally:
        gk.gk_debug_set(gk.KNOB_PREDICTION, -1)


def test_gk_select_on_the_benchmark_vector():
    w = wl.resnet50_segmented()
    u = w.grad(0, None)
    for rho in w.rhos:
        check_gk_select(DeviceStep(w.d), u, w.k(rho))
