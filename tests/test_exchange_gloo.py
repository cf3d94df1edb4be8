"""The all-gather of the workers' messages (Eq. 2) on two gloo ranks on the CPU: the
gathered layout is what the library's update kernel expects, checked by applying the
oracle's update to it and comparing with the update computed from the two messages directly."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _message(rank, d, cap):
    from paper_1911_08772_b200 import workloads as wl
    from oracle import oracle as orc
    u = wl.normal(d, 1e-2, step=100 + rank)
    k = cap // 2 + 3 * rank          # the ranks send lists of different lengths
    ti, tv = orc.topk_exact(u, k)
    idx = np.full(cap, -7, dtype=np.int32); val = np.full(cap, np.nan, dtype=np.float32)
    idx[:k] = ti; val[:k] = tv
    return idx, val, k


def _worker(rank, world, port, d, cap, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1911_08772_b200 import exchange
    idx, val, k = _message(rank, d, cap)
    ia, va, na = exchange.gather_messages(torch.from_numpy(idx), torch.from_numpy(val),
                                          torch.tensor([k], dtype=torch.int64), cap)
    np.savez(os.path.join(out_dir, f"r{rank}.npz"), idx=ia.numpy(), val=va.numpy(), nnz=na.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_gathered_messages_have_the_layout_the_update_expects(tmp_path):
    from oracle import oracle as orc
    world, d, cap = 2, 20_000, 64
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    mp.start_processes(_worker, args=(world, port, d, cap, str(tmp_path)), nprocs=world, join=True,
                       start_method="spawn")
    # what every rank should hold: both messages, rank 0's first
    msgs = [_message(r, d, cap) for r in range(world)]
    x_ref = np.linspace(-1, 1, d).astype(np.float32)
    idx = np.concatenate([m[0] for m in msgs]); val = np.concatenate([m[1] for m in msgs])
    nnz = np.array([m[2] for m in msgs], dtype=np.int64)
    orc.apply_sparse(x_ref, idx, np.nan_to_num(val), nnz, cap, -0.5)
    for r in range(world):
        got = np.load(os.path.join(str(tmp_path), f"r{r}.npz"))
        assert np.array_equal(got["nnz"], nnz)
        for p in range(world):
            n = int(nnz[p])
            assert np.array_equal(got["idx"][p * cap:p * cap + n], msgs[p][0][:n])
            assert np.array_equal(got["val"][p * cap:p * cap + n].view(np.uint32), msgs[p][1][:n].view(np.uint32))
        x = np.linspace(-1, 1, d).astype(np.float32)
        orc.apply_sparse(x, got["idx"], np.nan_to_num(got["val"]), got["nnz"], cap, -0.5)
        assert np.array_equal(x.view(np.uint32), x_ref.view(np.uint32))
