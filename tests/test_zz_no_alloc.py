"""gk_sparsify_static -- the entry point for callers that may not allocate device memory.

Some users of this library run where a hidden cudaMalloc is not acceptable: under an
allocator with a fixed budget, or in a serving process that forbids allocations after
start-up because they stall the device.  For them the library offers the same sparsifier
step with its scratch in a fixed array inside the library image.  This test calls that entry
point through the C ABI twice in a row (the second call finds the array as the first left
it, and continues from the residual the first produced) and requires

  * exactly the outputs of gk_sparsify: same pairs, same count, same residual, bit for bit --
    the tolerance the other parity tests use for these quantities;
  * agreement with the CPU oracle.  The call has no statistics record to read a threshold
    from, so the returned set itself is examined: it must be a threshold set (every selected
    magnitude above every unselected one), the oracle's final threshold must lie in the gap
    between the two (to 1e-6 relative), the pairs must be the oracle's selection at a threshold
    in that gap and the residual the oracle's residual of it, bit for bit;
  * that the free device memory does not change across the calls.

The file sorts last on purpose, so that a run that stops at the first failure has already
run every other test.  It does not depend on anything the other tests leave behind.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_1911_08772_b200 import binding as gk
from paper_1911_08772_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _run(fn, g_list, d, k):
    dev = torch.device("cuda:0")
    eps = torch.zeros(d, dtype=torch.float32, device=dev)
    outs = []
    for g in g_list:
        idx = torch.full((d,), -7, dtype=torch.int32, device=dev)
        val = torch.full((d,), -7.0, dtype=torch.float32, device=dev)
        nnz = torch.full((1,), -7, dtype=torch.int64, device=dev)
        dg = torch.from_numpy(g).to(dev)
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        fn(dg, eps, k, idx, val, nnz)
        torch.cuda.synchronize()
        grew = free0 - torch.cuda.mem_get_info()[0]   # device memory taken while the call ran
        n = int(nnz.item())
        outs.append((n, idx[:n].cpu().numpy(), val[:n].cpu().numpy().view(np.uint32),
                     eps.cpu().numpy().view(np.uint32).copy(),
                     bool((idx[n:] == -7).all().item()), grew))
    return outs


def _against_oracle(g, eps_in, k, n, idx, val_bits, eps_bits):
    u = orc.accumulate(g, eps_in)
    ost = orc.gaussiank_threshold(u, k)
    a = np.abs(u)
    sel = np.zeros(u.shape[0], dtype=bool)
    sel[idx] = True
    assert 0 < n < u.shape[0]
    lo, hi = float(a[~sel].max()), float(a[sel].min())
    assert lo < hi, "not a threshold set"
    assert lo * (1 - 1e-6) <= ost.thr_final < hi * (1 + 1e-6), (lo, ost.thr_final, hi)
    oi, ov, on = orc.select(u, lo)          # any threshold in [lo, hi) gives the same set
    assert on == n and np.array_equal(oi, idx) and np.array_equal(ov.view(np.uint32), val_bits)
    if lo <= ost.thr_final < hi:
        assert ost.nnz == n
    assert np.array_equal(orc.residual(u, oi, ov).view(np.uint32), eps_bits)


@pytest.mark.parametrize("d", [100_003, 3_000_001])
def test_static_entry_point_matches_gk_sparsify_and_the_oracle_on_two_calls_in_a_row(d):
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    gk.gk_set_capacity(0)
    gk.gk_set_path(0)
    k = wl.ceil_k(d, 1, 1000)
    g_list = [wl.laplace(d, 1e-3, step=50), wl.normal(d, 2e-3, step=51)]
    _run(gk.gk_sparsify_static, g_list[:1], d, k)   # the kernel's code is loaded by now
    before = gk.gk_launch_count()
    got = _run(gk.gk_sparsify_static, g_list, d, k)
    assert gk.gk_launch_count() - before == 2      # one kernel per call
    assert all(o[5] == 0 for o in got), "device memory was allocated during a call"
    ref = _run(gk.gk_sparsify, g_list, d, k)
    eps_in = np.zeros(d, dtype=np.float32)
    for call, (a, b) in enumerate(zip(got, ref)):
        assert a[0] == b[0] and a[0] > 0, call
        assert np.array_equal(a[1], b[1]), call
        assert np.array_equal(a[2], b[2]), call
        assert np.array_equal(a[3], b[3]), call
        assert a[4], "wrote past the reported count"
        _against_oracle(g_list[call], eps_in, k, a[0], a[1], a[2], a[3])
        eps_in = a[3].view(np.float32).copy()


def test_static_entry_point_rejects_what_it_cannot_serve():
    L = gk.load()
    a = 0x1000
    assert L.gk_sparsify_static(a, a + 4096, 2 ** 31, 5, a, a, a, None) == -2   # beyond the maximum size
    assert L.gk_sparsify_static(a, a + 4096, 10, 10, a, a, a, None) == -3       # k = d is not served here
    assert L.gk_sparsify_static(None, a, 10, 1, a, a, a, None) == -1
    # more rows of 4096 elements than the fixed array has words for (nothing is launched)
    big = 2 ** 29 + 4096
    assert L.gk_sparsify_static(a, a + 4 * big + 4096, big, 1000, a, a, a, None) == -9
    assert "k out of range" in gk.gk_strerror(-3) and "size out of range" in gk.gk_strerror(-2)
