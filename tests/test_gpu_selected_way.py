"""The persistent kernel's second phase counting only the candidates it expects the rounds of
Algorithm 1 to reach (estimated from the table of cell maxima): whether the expectation is
right, too wide, or wrong -- so that the rounds ask for a candidate left out and the count is
taken again in full -- the statistics, the per-round counts, the pairs and the residual must
equal the oracle's.  gk_debug_set(5, 1) selects thres0 alone, which makes every call with a
second round take the count again; gk_debug_set(5, 0) switches the selection off."""
import numpy as np
import pytest

from paper_1911_08772_b200 import binding as gk
from paper_1911_08772_b200 import workloads as wl

from gpu_util import DeviceStep, check_gk_select, check_gk_step

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    gk.gk_set_capacity(0)
    gk.gk_set_path(2)          # the persistent kernel at every size
    gk.gk_debug_set(gk.KNOB_PREDICTION, 0)
    yield
    gk.gk_debug_set(gk.KNOB_PREDICTION, -1)
    gk.gk_debug_set(gk.KNOB_SELECTED_WAY, -1)
    gk.gk_set_path(0)


@pytest.fixture(params=[-1, 0, 1], ids=["auto", "off", "thres0_alone"])
def selection(request):
    gk.gk_debug_set(gk.KNOB_SELECTED_WAY, request.param)
    yield request.param
    gk.gk_debug_set(gk.KNOB_SELECTED_WAY, -1)


def _data(dist, d, t):
    if dist == "normal":
        return wl.normal(d, 1e-3, step=140 + t)
    if dist == "laplace":
        return wl.laplace(d, 1e-3, step=140 + t)
    if dist == "mixture":
        return wl.laplace_mixture(d, step=140 + t)
    if dist == "uniform":
        return wl.misc_rng(140 + t).uniform(-1.0, 1.0, size=d).astype(np.float32)
    raise ValueError(dist)


@pytest.mark.parametrize("dist", ["normal", "laplace", "mixture", "uniform"])
@pytest.mark.parametrize("d,rho", [(3_000_017, "1e-3"), (3_000_017, "1e-2"), (9_000_001, "1e-3"), (1_200_003, "1e-4")])
def test_every_setting_gives_the_oracles_result(dist, d, rho, selection):
    k = wl.ceil_k(d, *wl.RHO[rho])
    step = DeviceStep(d)
    eps = np.zeros(d, dtype=np.float32)
    for t in range(2):
        eps, st = check_gk_step(step, _data(dist, d, t), eps, k)
        info = gk.gk_last_path_info()
        ctas, selected, recount = info[4], info[5], info[2]
        assert ctas > 0
        if selection == 0:
            assert selected == 0
        if selection == 1 and st.rounds > 1 and selected > 0:
            assert recount == 1        # thres0 alone was counted, the second round asked for more
        if selection == 1 and st.rounds == 1:
            assert recount == 0


def test_the_selection_is_used_and_is_right_on_plain_data():
    # independent values, vectors of a few million elements: nothing is sparse enough for the
    # short way over loud cells, every CTA selects, and the selection covers the rounds
    gk.gk_debug_set(gk.KNOB_SELECTED_WAY, -1)
    d = 8_000_003
    step = DeviceStep(d)
    for dist in ("normal", "laplace"):
        for rho in ("1e-3", "1e-2"):
            k = wl.ceil_k(d, *wl.RHO[rho])
            eps = np.zeros(d, dtype=np.float32)
            for t in range(3):
                eps, st = check_gk_step(step, _data(dist, d, 10 + t), eps, k)
                info = gk.gk_last_path_info()
                assert info[5] == info[4] and info[2] == 0, (dist, rho, t, info)


def test_survivors_that_sit_together_mislead_the_estimate_and_are_found_out():
    # one stretch of the vector a hundred times louder than the rest: the cells that reach a
    # candidate are few, the survivors in them many, and the estimate from the number of loud
    # cells is far too low.  Whatever is selected, the result is the oracle's.
    gk.gk_debug_set(gk.KNOB_SELECTED_WAY, -1)
    d = 6_000_011
    g = wl.normal(d, 1e-3, step=151)
    g[1_000_000:1_400_000] *= np.float32(100.0)
    # and enough loud cells elsewhere that the short way over loud cells is not taken
    g[::97] *= np.float32(40.0)
    step = DeviceStep(d)
    eps = np.zeros(d, dtype=np.float32)
    for k in (wl.ceil_k(d, 1, 1000), wl.ceil_k(d, 1, 100)):
        eps, st = check_gk_step(step, g, eps, k)


def test_operator_form_and_small_vectors(selection):
    for d in (4096 * 3 + 5, 700_001):
        g = wl.laplace(d, 1e-3, step=160)
        check_gk_select(DeviceStep(d), g, wl.ceil_k(d, 1, 100))
