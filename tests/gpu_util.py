"""Helpers of the GPU parity tests: run the CUDA library through its binding on numpy
inputs and compare with the CPU oracle by the acceptance rule below.

Acceptance (floating point decides an integer here -- the mask -- so both sides take that
decision with the same threshold):
  * u and eps are bit-exact;
  * the library's mu, sigma, thres0 and final threshold are within 1e-6 relative of the
    oracle's fp64 values (the summation order differs; fp64 accumulation keeps the
    difference near 1e-12);
  * rounds and per-round counts equal the oracle's;
  * the (index, value) list is bit-exact against the oracle's selection evaluated with the
    library's reported fp64 threshold, and eps_new against the oracle's residual of it.
"""
from __future__ import annotations

import math

import numpy as np
import torch

from oracle import oracle as orc
from paper_1911_08772_b200 import binding as gk

CANARY_I = np.int32(-1234567)
CANARY_F = np.float32(-7.25)
GUARD = 64
REL_TOL = 1e-6


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def rel_close(a, b, tol=REL_TOL):
    if a == b:
        return True
    if math.isinf(a) or math.isinf(b) or math.isnan(a) or math.isnan(b):
        return False
    return abs(a - b) <= tol * max(abs(a), abs(b))


class DeviceStep:
    """Device buffers for repeated calls on vectors of length d (capacity = cap pairs)."""

    def __init__(self, d, cap=None):
        self.d = d
        self.cap = d if cap is None else cap
        dev = torch.device("cuda:0")
        self.g = torch.empty(d, dtype=torch.float32, device=dev)
        self.eps = torch.zeros(d, dtype=torch.float32, device=dev)
        self.idx = torch.empty(self.cap + GUARD, dtype=torch.int32, device=dev)
        self.val = torch.empty(self.cap + GUARD, dtype=torch.float32, device=dev)
        self.nnz = torch.zeros(1 + 2, dtype=torch.int64, device=dev)

    def arm(self):
        self.idx.fill_(int(CANARY_I))
        self.val.fill_(float(CANARY_F))
        self.nnz.fill_(-99)

    def outputs(self):
        torch.cuda.synchronize()
        nnz = self.nnz.cpu().numpy()
        assert nnz[1] == -99 and nnz[2] == -99, "write past nnz_out"
        n = int(nnz[0])
        assert 0 <= n <= self.cap
        idx = self.idx.cpu().numpy()
        val = self.val.cpu().numpy()
        assert np.all(idx[self.cap:] == CANARY_I) and np.all(val[self.cap:] == CANARY_F), "write past capacity"
        assert np.all(idx[n:self.cap] == CANARY_I) and np.all(val[n:self.cap] == CANARY_F), "write past nnz"
        return idx[:n].copy(), val[:n].copy(), n


def compare_with_oracle(g, eps_in, k, idx, val, n, st, eps_new, cap, check_counts=True, max_rounds=4,
                        unbiased=True):
    """One finished sparsifier step (pairs idx/val[:n], record st, residual eps_new, output
    capacity cap) against the oracle, by the acceptance rule in this module's header.

    Two of the tolerances have an absolute alternative, for quantities that can sit at zero,
    where a relative bound says nothing: mu against 1e-9 sigma (the mean of zero-mean data is
    rounding noise around 0), thres0 and the final threshold against 1e-6 sigma (mu + sigma z
    crosses zero for k near d / 2).  z is compared absolutely, 1e-12 on a quantity of order 1:
    at p = 1/2 the oracle's bisection ends one denormal below zero where the library's Newton
    iteration returns 0 exactly."""
    d = g.shape[0]
    u = orc.accumulate(g, eps_in)
    ost = orc.gaussiank_threshold(u, k, max_rounds=max_rounds, unbiased=unbiased)
    assert st.status in (0, gk.GK_DEV_TRUNCATED)
    if k < d:
        assert rel_close(st.mu, ost.mu, 1e-6) or abs(st.mu - ost.mu) <= 1e-9 * ost.sigma
        assert rel_close(st.sigma, ost.sigma)
        assert abs(st.z - ost.z) <= 1e-12 * max(1.0, abs(ost.z))
        assert rel_close(st.thres0, ost.thres0) or abs(st.thres0 - ost.thres0) <= 1e-6 * ost.sigma
        assert rel_close(st.thr_final, ost.thr_final) or abs(st.thr_final - ost.thr_final) <= 1e-6 * ost.sigma, \
            (st, ost)
        if check_counts:
            assert st.rounds == ost.rounds and st.counts == ost.counts, (st, ost)
    else:
        assert st.rounds == 0 and st.thr_final == -math.inf
    # selection with the library's own threshold
    oi, ov, on = orc.select(u, st.thr_final, cap=cap)
    assert st.nnz == on
    assert n == min(on, cap) == st.emitted
    assert (st.status & gk.GK_DEV_TRUNCATED) == (gk.GK_DEV_TRUNCATED if on > cap else 0)
    assert np.array_equal(idx, oi)
    assert np.array_equal(bits(val), bits(ov))
    oeps = orc.residual(u, oi, ov)
    assert np.array_equal(bits(eps_new), bits(oeps))


def check_gk_step(step: DeviceStep, g: np.ndarray, eps_in: np.ndarray, k: int, check_counts=True,
                  call=None, max_rounds=4, unbiased=True):
    """Run one gk_sparsify step (or `call`, an entry point with the same arguments) on the
    device and compare with the oracle.  Returns (eps_new (numpy, from the device), stats)."""
    step.g.copy_(torch.from_numpy(g))
    step.eps.copy_(torch.from_numpy(eps_in))
    step.arm()
    (call or gk.gk_sparsify)(step.g, step.eps, k, step.idx[:step.cap], step.val[:step.cap], step.nnz[:1])
    idx, val, n = step.outputs()
    st = gk.gk_last_stats()
    eps_new = step.eps.cpu().numpy()
    compare_with_oracle(g, eps_in, k, idx, val, n, st, eps_new, step.cap, check_counts, max_rounds, unbiased)
    return eps_new, st


def check_gk_select(step: DeviceStep, u: np.ndarray, k: int, check_counts=True):
    """gk_select on the device against the oracle: Algorithm 1 on u as given, u untouched."""
    step.g.copy_(torch.from_numpy(u))
    step.arm()
    gk.gk_select(step.g, k, step.idx[:step.cap], step.val[:step.cap], step.nnz[:1])
    idx, val, n = step.outputs()
    st = gk.gk_last_stats()
    assert np.array_equal(bits(step.g.cpu().numpy()), bits(u)), "u modified"
    # the operator is the sparsifier's selection with a neutral residual coming in; the residual
    # the oracle would leave is u with the selected entries cleared
    zero = np.full_like(u, -0.0)    # x + (-0) == x for every x, -0 included: the oracle sees u itself
    u_cleared = u.copy()
    u_cleared[idx] = 0.0
    compare_with_oracle(u, zero, k, idx, val, n, st, u_cleared, step.cap, check_counts)
    return st


def check_segmented_step(step: DeviceStep, g, eps_in, offsets, seg_k, dev_off, dev_k, dev_seg_nnz):
    d = g.shape[0]
    S = offsets.shape[0] - 1
    step.g.copy_(torch.from_numpy(g))
    step.eps.copy_(torch.from_numpy(eps_in))
    step.arm()
    dev_seg_nnz.fill_(-5)
    gk.gk_sparsify_segmented(step.g, step.eps, dev_off, dev_k, step.idx[:step.cap], step.val[:step.cap],
                             dev_seg_nnz, step.nnz[:1])
    idx, val, n = step.outputs()
    sts = gk.gk_last_segment_stats(S)
    seg_nnz = dev_seg_nnz.cpu().numpy()
    eps_new = step.eps.cpu().numpy()

    u = orc.accumulate(g, eps_in)
    exp_idx, exp_val = [], []
    for s in range(S):
        lo, hi = int(offsets[s]), int(offsets[s + 1])
        st = sts[s]
        assert st.status == 0
        if hi == lo:
            assert seg_nnz[s] == 0
            continue
        us = np.ascontiguousarray(u[lo:hi])
        ks = min(int(seg_k[s]), hi - lo)
        ost = orc.gaussiank_threshold(us, ks)
        if ks < hi - lo:
            assert rel_close(st.sigma, ost.sigma), (s, st, ost)
            assert rel_close(st.thr_final, ost.thr_final) or \
                abs(st.thr_final - ost.thr_final) <= 1e-6 * ost.sigma, (s, st, ost)
            assert st.rounds == ost.rounds and st.counts == ost.counts, (s, st, ost)
        else:
            assert st.rounds == 0 and st.thr_final == -math.inf
        oi, ov, on = orc.select(us, st.thr_final)
        assert seg_nnz[s] == on == st.nnz, (s, seg_nnz[s], on)
        exp_idx.append(oi + np.int32(lo))
        exp_val.append(ov)
    exp_idx = np.concatenate(exp_idx) if exp_idx else np.zeros(0, np.int32)
    exp_val = np.concatenate(exp_val) if exp_val else np.zeros(0, np.float32)
    assert n == exp_idx.shape[0]
    assert np.array_equal(idx, exp_idx)
    assert np.array_equal(bits(val), bits(exp_val))
    oeps = orc.residual(u, exp_idx, exp_val)
    assert np.array_equal(bits(eps_new), bits(oeps))
    return eps_new, sts


def check_topk(u: np.ndarray, k: int, oracle_result=None):
    d = u.shape[0]
    dev = torch.device("cuda:0")
    du = torch.from_numpy(u).to(dev)
    idx = torch.full((k + GUARD,), int(CANARY_I), dtype=torch.int32, device=dev)
    val = torch.full((k + GUARD,), float(CANARY_F), dtype=torch.float32, device=dev)
    gk.topk_exact(du, k, idx[:k], val[:k])
    torch.cuda.synchronize()
    hi, hv = idx.cpu().numpy(), val.cpu().numpy()
    assert np.all(hi[k:] == CANARY_I) and np.all(hv[k:] == CANARY_F)
    assert np.array_equal(bits(du.cpu().numpy()), bits(u)), "u modified"
    oi, ov = oracle_result if oracle_result is not None else orc.topk_exact(u, k)
    assert np.array_equal(hi[:k], oi)
    assert np.array_equal(bits(hv[:k]), bits(ov))
    return hi[:k], hv[:k]
