"""The exchange that follows the sparsifier in Eq. 2 of the paper: every worker's message
(its (index, value) list) goes to every other worker, and each applies
    x <- x + alpha * sum_p Comp_k(u^p)
to its own copy of the model.  The paper names its communication libraries but not the
collective; here it is one all-gather of fixed-capacity buffers through torch.distributed
(NCCL over NVLink on GPUs) followed by the library's gk_apply_gathered kernel.

Plumbing only: the gather is torch.distributed's, the arithmetic is the library's kernel.
"""
from __future__ import annotations

from typing import Optional, Tuple


def gather_messages(idx, val, nnz, cap: int, group=None) -> Tuple["torch.Tensor", "torch.Tensor", "torch.Tensor"]:
    """All-gather the ranks' messages.  idx (int32), val (float32): at least `cap` entries, the
    first nnz[0] of them valid; nnz: one int64.  Returns (idx_all, val_all, nnz_all) with rank
    p's list at [p * cap, p * cap + nnz_all[p]).  Works on whatever device the tensors live on
    (NCCL for CUDA tensors, gloo for CPU tensors)."""
    import torch
    import torch.distributed as dist

    P = dist.get_world_size(group)
    if idx.numel() < cap or val.numel() < cap:
        raise ValueError("idx / val hold fewer than cap entries")
    idx_all = torch.empty(P * cap, dtype=torch.int32, device=idx.device)
    val_all = torch.empty(P * cap, dtype=torch.float32, device=val.device)
    nnz_all = torch.empty(P, dtype=torch.int64, device=nnz.device)
    dist.all_gather_into_tensor(idx_all, idx[:cap].contiguous(), group=group)
    dist.all_gather_into_tensor(val_all, val[:cap].contiguous(), group=group)
    dist.all_gather_into_tensor(nnz_all, nnz[:1].contiguous(), group=group)
    return idx_all, val_all, nnz_all


def exchange_and_apply(x, idx, val, nnz, cap: int, alpha: float, group=None) -> None:
    """One model update of Eq. 2 on this rank's x from all ranks' messages (CUDA tensors)."""
    from . import binding as gk

    idx_all, val_all, nnz_all = gather_messages(idx, val, nnz, cap, group)
    gk.gk_apply_gathered(x, idx_all, val_all, nnz_all, cap, alpha)
