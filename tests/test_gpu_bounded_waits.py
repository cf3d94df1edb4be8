"""Every wait in the kernels is bounded: a grid barrier or a look-back poll that cannot
complete gives up after a fixed number of polls, the call ends with GK_DEV_TIMEOUT in its
status word, and the next call finds clean counters.  The tests make the waits run out the
harmless way -- a barrier that expects one arrival more than there are CTAs, a tile that keeps
its status word to itself -- with the poll limits lowered to a few hundred, so nothing hangs
and nothing faults."""
import numpy as np
import pytest
import torch

from paper_1911_08772_b200 import binding as gk
from paper_1911_08772_b200 import workloads as wl

from gpu_util import DeviceStep, check_gk_step

pytestmark = pytest.mark.gpu

BARRIER_POLLS_DEFAULT = 1 << 24
LOOKBACK_POLLS_DEFAULT = 1 << 22


@pytest.fixture(autouse=True)
def _library():
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    gk.gk_set_capacity(0)
    gk.gk_set_path(0)
    yield
    gk.gk_debug_set(gk.KNOB_BARRIER_POLLS, BARRIER_POLLS_DEFAULT)
    gk.gk_debug_set(gk.KNOB_LOOKBACK_POLLS, LOOKBACK_POLLS_DEFAULT)
    gk.gk_debug_set(gk.KNOB_EXTRA_ARRIVALS, 0)
    gk.gk_debug_set(gk.KNOB_MUTE_TILE, -1)
    gk.gk_set_path(0)


def _raw_call(fn, d, k, g):
    dev = torch.device("cuda:0")
    dg = torch.from_numpy(g).to(dev)
    eps = torch.zeros(d, dtype=torch.float32, device=dev)
    idx = torch.empty(d, dtype=torch.int32, device=dev)
    val = torch.empty(d, dtype=torch.float32, device=dev)
    nnz = torch.zeros(1, dtype=torch.int64, device=dev)
    fn(dg, eps, k, idx, val, nnz)
    torch.cuda.synchronize()
    return gk.gk_last_stats()


@pytest.mark.parametrize("d", [300_007, 9_000_001])
def test_a_grid_barrier_that_cannot_complete_gives_up(d):
    g = wl.normal(d, 1e-3, step=60)
    k = wl.ceil_k(d, 1, 1000)
    gk.gk_set_path(2)           # the persistent kernel at either size (small vectors go to the cluster kernel otherwise)
    gk.gk_debug_set(gk.KNOB_BARRIER_POLLS, 300)
    gk.gk_debug_set(gk.KNOB_EXTRA_ARRIVALS, 1)
    for _ in range(2):     # twice: the counters are reset by the CTAs that gave up
        st = _raw_call(gk.gk_sparsify, d, k, g)
        assert st.status & gk.GK_DEV_TIMEOUT
    gk.gk_debug_set(gk.KNOB_EXTRA_ARRIVALS, 0)
    gk.gk_debug_set(gk.KNOB_BARRIER_POLLS, BARRIER_POLLS_DEFAULT)
    # the next ordinary call is correct
    eps_new, st = check_gk_step(DeviceStep(d), g, np.zeros(d, np.float32), k)
    assert not (st.status & gk.GK_DEV_TIMEOUT)


def test_a_look_back_that_meets_a_silent_tile_gives_up():
    d = 20 * 8192 + 77          # 21 compaction tiles
    g = wl.normal(d, 1e-3, step=61)
    k = wl.ceil_k(d, 1, 100)
    gk.gk_set_path(1)           # the three-kernel form: compaction by decoupled look-back
    gk.gk_debug_set(gk.KNOB_LOOKBACK_POLLS, 100)
    gk.gk_debug_set(gk.KNOB_MUTE_TILE, 5)
    st = _raw_call(gk.gk_sparsify, d, k, g)
    assert st.status & gk.GK_DEV_TIMEOUT
    gk.gk_debug_set(gk.KNOB_MUTE_TILE, -1)
    gk.gk_debug_set(gk.KNOB_LOOKBACK_POLLS, LOOKBACK_POLLS_DEFAULT)
    eps_new, st = check_gk_step(DeviceStep(d), g, np.zeros(d, np.float32), k)
    assert not (st.status & gk.GK_DEV_TIMEOUT)
    gk.gk_set_path(0)
