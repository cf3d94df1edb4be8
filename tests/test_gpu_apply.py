"""GPU-vs-oracle parity of the model update from P messages (Eq. 2): bit-exact, since the
order of the fp32 additions is fixed (rank order)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_1911_08772_b200 import binding as gk
from paper_1911_08772_b200 import workloads as wl

from gpu_util import bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _library():
    from paper_1911_08772_b200 import build
    build.build()
    gk.load()
    yield


def messages(rng, d, P, cap, fill):
    idx = np.full(P * cap, -11, dtype=np.int32)
    val = np.full(P * cap, np.float32(777.0), dtype=np.float32)
    nnz = np.zeros(P, dtype=np.int64)
    for p in range(P):
        n = int(cap * fill) if fill >= 0 else int(rng.integers(0, cap + 1))
        pos = np.sort(rng.choice(d, size=n, replace=False)).astype(np.int32)
        idx[p * cap:p * cap + n] = pos
        val[p * cap:p * cap + n] = (rng.standard_normal(n) * 1e-2).astype(np.float32)
        nnz[p] = n
    return idx, val, nnz


def check(d, P, cap, fill, alpha, seed, separate=False):
    rng = wl.misc_rng(seed)
    idx, val, nnz = messages(rng, d, P, cap, fill)
    x0 = rng.standard_normal(d).astype(np.float32)
    want = x0.copy()
    orc.apply_sparse(want, idx, val, nnz, cap, alpha)
    dx = torch.from_numpy(x0).to(DEV)
    dn = torch.from_numpy(nnz).to(DEV)
    if separate:
        il = [torch.from_numpy(idx[p * cap:(p + 1) * cap].copy()).to(DEV) for p in range(P)]
        vl = [torch.from_numpy(val[p * cap:(p + 1) * cap].copy()).to(DEV) for p in range(P)]
        gk.gk_apply_sparse(dx, il, vl, dn, cap, alpha)
    else:
        gk.gk_apply_gathered(dx, torch.from_numpy(idx).to(DEV), torch.from_numpy(val).to(DEV), dn, cap, alpha)
    assert gk.gk_last_stats().status == 0
    assert np.array_equal(bits(dx.cpu().numpy()), bits(want))


@pytest.mark.parametrize("P", [1, 2, 3, 8, 9, 16, 17, 64])
def test_apply_small_dense_overlap(P):
    # few positions, many ranks: almost every position occurs in several messages
    check(d=500, P=P, cap=200, fill=-1, alpha=-0.25, seed=4000 + P)
    check(d=500, P=P, cap=200, fill=-1, alpha=0.3, seed=4100 + P, separate=True)


def test_apply_empty_and_full_lists():
    check(d=1000, P=4, cap=1, fill=0.0, alpha=1.0, seed=4200)       # all lists empty
    check(d=1000, P=4, cap=1000, fill=1.0, alpha=1.0, seed=4201)    # every list holds every position
    check(d=1, P=5, cap=1, fill=1.0, alpha=-1.0, seed=4202)


def test_apply_bad_index_is_skipped_and_flagged():
    rng = wl.misc_rng(4300)
    d, P, cap = 1000, 2, 50
    idx, val, nnz = messages(rng, d, P, cap, 1.0)
    idx[cap - 1] = d + 3            # last entry of rank 0's ascending list
    x0 = rng.standard_normal(d).astype(np.float32)
    dx = torch.from_numpy(x0).to(DEV)
    gk.gk_apply_gathered(dx, torch.from_numpy(idx).to(DEV), torch.from_numpy(val).to(DEV),
                         torch.from_numpy(nnz).to(DEV), cap, 1.0)
    assert gk.gk_last_stats().status & gk.GK_DEV_BAD_INDEX
    good = nnz.copy(); good[0] = cap - 1
    want = x0.copy()
    orc.apply_sparse(want, idx, val, good, cap, 1.0)
    assert np.array_equal(bits(dx.cpu().numpy()), bits(want))


@pytest.mark.parametrize("P", [2, 8, 16])
def test_apply_after_real_sparsifier_steps(P):
    """P workers (emulated on one GPU, one after the other) sparsify their own ResNet-50-sized
    gradients with Gaussian_k; the update of x from their messages equals the oracle's."""
    w = wl.resnet50_segmented()
    d, k = w.d, w.k("1e-3")
    cap = 4 * k
    didx = torch.full((P * cap,), -1, dtype=torch.int32, device=DEV)
    dval = torch.zeros(P * cap, dtype=torch.float32, device=DEV)
    dnnz = torch.zeros(P, dtype=torch.int64, device=DEV)
    gk.gk_set_capacity(cap)
    try:
        for p in range(P):
            g = torch.from_numpy(w.grad(50 + p, None)).to(DEV)
            eps = torch.zeros(d, dtype=torch.float32, device=DEV)
            gk.gk_sparsify(g, eps, k, didx[p * cap:(p + 1) * cap], dval[p * cap:(p + 1) * cap], dnnz[p:p + 1])
            del g, eps
    finally:
        gk.gk_set_capacity(0)
    torch.cuda.synchronize()
    x0 = wl.normal(d, 1.0, step=77)
    want = x0.copy()
    orc.apply_sparse(want, didx.cpu().numpy(), dval.cpu().numpy(), dnnz.cpu().numpy(), cap, -0.1 / P)
    dx = torch.from_numpy(x0).to(DEV)
    gk.gk_apply_gathered(dx, didx, dval, dnnz, cap, -0.1 / P)
    assert np.array_equal(bits(dx.cpu().numpy()), bits(want))
    assert int((want != x0).sum()) > 0


def test_exchange_and_apply_through_nccl_with_one_rank():
    """The wrapper end to end on the GPU: a one-rank NCCL group (one GPU is enough), the
    all-gather of the message, the update kernel; against the oracle."""
    import os
    import socket
    import torch.distributed as dist
    from paper_1911_08772_b200 import exchange

    if dist.is_initialized():
        pytest.skip("a process group already exists in this process")
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device(DEV))
    try:
        rng = wl.misc_rng(4400)
        d, cap = 200_000, 3000
        idx, val, nnz = messages(rng, d, 1, cap, 0.7)
        x0 = rng.standard_normal(d).astype(np.float32)
        want = x0.copy()
        orc.apply_sparse(want, idx, val, nnz, cap, -0.05)
        dx = torch.from_numpy(x0).to(DEV)
        # buffers longer than cap, as a sparsifier's output buffers are
        di = torch.cat([torch.from_numpy(idx), torch.full((100,), -3, dtype=torch.int32)]).to(DEV)
        dv = torch.cat([torch.from_numpy(val), torch.zeros(100)]).to(DEV)
        exchange.exchange_and_apply(dx, di, dv, torch.from_numpy(nnz).to(DEV), cap, -0.05)
        torch.cuda.synchronize()
        assert np.array_equal(bits(dx.cpu().numpy()), bits(want))
    finally:
        dist.destroy_process_group()
