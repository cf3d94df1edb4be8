"""GPU-vs-oracle parity of the histogram of u (Section 3.1, Fig. 2): integer counts, the
binning decision taken in fp32 on both sides, so the comparison is exact."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_1911_08772_b200 import binding as gk
from paper_1911_08772_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    yield


def check(u, lo, hi, nbins):
    lo32 = np.float32(lo)
    inv_w = np.float32(nbins / (hi - lo))
    want = orc.histogram(u, float(lo32), float(inv_w), nbins)
    du = torch.from_numpy(u).to(DEV)
    out = torch.full((nbins + 2 + 4,), -5, dtype=torch.int64, device=DEV)
    gk.gk_histogram(du, float(lo32), float(inv_w), out[:nbins + 2])
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert np.all(got[nbins + 2:] == -5), "write past the counts"
    assert np.array_equal(got[:nbins + 2], want)
    assert got[:nbins + 2].sum() == u.size
    return got[:nbins + 2]


@pytest.mark.parametrize("d", [1, 3, 4, 5, 1023, 4097, 100_003, 3_000_001])
def test_histogram_small_sizes(d):
    rng = wl.misc_rng(5000 + d % 997)
    u = rng.standard_normal(d).astype(np.float32)
    for nbins in (1, 7, 256, 8192):
        check(u, -3.0, 3.0, nbins)


def test_histogram_special_values_and_edges():
    u = np.array([-1.0, -0.5, -0.0, 0.0, 0.25, 0.4999, 0.5, 0.75, 1.0, 7.0, -7.0, np.nan, np.inf, -np.inf,
                  1e-45, -1e-45], dtype=np.float32)
    got = check(u, -1.0, 1.0, 4)
    # -1e-45 - (-1) rounds to 1.0 in fp32, so by the fp32 rule it lands in the bin that starts at 0
    assert got.tolist() == [2, 1, 1, 6, 2, 4]


@pytest.mark.parametrize("name", ["resnet50", "lstm", "sweep26"])
def test_histogram_workloads(name):
    w = {"resnet50": wl.resnet50_segmented, "lstm": wl.lstm_student_t,
         "sweep26": lambda: wl.sweep_point(1 << 26, "laplace")}[name]()
    u = w.grad(0, None)
    s = float(np.std(u[:1_000_000]))
    check(u, -4 * s, 4 * s, 512)
