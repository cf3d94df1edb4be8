"""gk_sparsify_static -- the entry point for callers that may not allocate device memory.

Some users of this library run where a hidden cudaMalloc is not acceptable: under an
allocator with a fixed budget, or in a serving process that forbids allocations after
start-up because they stall the device.  For them the library offers the same sparsifier
step with its scratch in a fixed array inside the library image.  This test calls that entry
point through the C ABI twice in a row (the second call finds the array as the first left
it, and continues from the residual the first produced) and requires exactly the outputs of
gk_sparsify: same pairs, same count, same residual, bit for bit -- the tolerance the other
parity tests use for these quantities.

The file sorts last on purpose, so that a run that stops at the first failure has already
run every other test.  It does not depend on anything the other tests leave behind.
"""
import numpy as np
import pytest
import torch

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
        fn(torch.from_numpy(g).to(dev), eps, k, idx, val, nnz)
        torch.cuda.synchronize()
        n = int(nnz.item())
        outs.append((n, idx[:n].cpu().numpy(), val[:n].cpu().numpy().view(np.uint32),
                     eps.cpu().numpy().view(np.uint32).copy(),
                     bool((idx[n:] == -7).all().item())))
    return outs


@pytest.mark.parametrize("d", [100_003, 3_000_001])
def test_static_entry_point_matches_gk_sparsify_on_two_calls_in_a_row(d):
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    gk.gk_set_capacity(0)
    gk.gk_set_path(0)
    k = wl.ceil_k(d, 1, 1000)
    g_list = [wl.laplace(d, 1e-3, step=50), wl.normal(d, 2e-3, step=51)]
    before = gk.gk_launch_count()
    got = _run(gk.gk_sparsify_static, g_list, d, k)
    assert gk.gk_launch_count() - before == 2      # one kernel per call
    ref = _run(gk.gk_sparsify, g_list, d, k)
    for call, (a, b) in enumerate(zip(got, ref)):
        assert a[0] == b[0] and a[0] > 0, call
        assert np.array_equal(a[1], b[1]), call
        assert np.array_equal(a[2], b[2]), call
        assert np.array_equal(a[3], b[3]), call
        assert a[4], "wrote past the reported count"


def test_static_entry_point_rejects_what_it_cannot_serve():
    L = gk.load()
    a = 0x1000
    assert L.gk_sparsify_static(a, a + 4096, 2 ** 31, 5, a, a, a, None) == -2   # beyond the maximum size
    assert L.gk_sparsify_static(a, a + 4096, 10, 10, a, a, a, None) == -3       # k = d is not served here
    assert L.gk_sparsify_static(None, a, 10, 1, a, a, a, None) == -1
    assert "k out of range" in gk.gk_strerror(-3) and "size out of range" in gk.gk_strerror(-2)
