"""ctypes access to the C++ CPU oracle (oracle/gk_oracle.cpp).

Test infrastructure only: imported by tests/, by the smoke check and by the
CPU-baseline leg of the benchmark.  The CUDA library and its Python binding
never import this module.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import List, Optional, Tuple

import numpy as np

from . import build as _build


class _Stats(C.Structure):
    _fields_ = [
        ("mu", C.c_double),
        ("sigma", C.c_double),
        ("z", C.c_double),
        ("thres0", C.c_double),
        ("thr_final", C.c_double),
        ("counts", C.c_int64 * 4),
        ("rounds", C.c_int32),
        ("pad", C.c_int32),
        ("nnz", C.c_int64),
    ]


@dataclass
class Stats:
    mu: float
    sigma: float
    z: float
    thres0: float
    thr_final: float
    counts: List[int]
    rounds: int
    nnz: int

    @staticmethod
    def of(s: _Stats) -> "Stats":
        return Stats(s.mu, s.sigma, s.z, s.thres0, s.thr_final,
                     [int(c) for c in s.counts][: max(int(s.rounds), 0)], int(s.rounds), int(s.nnz))


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        fp = C.POINTER(C.c_float)
        ip = C.POINTER(C.c_int32)
        lp = C.POINTER(C.c_int64)
        L.oracle_accumulate.argtypes = [fp, fp, C.c_int64, fp]
        L.oracle_accumulate.restype = None
        L.oracle_mean_std.argtypes = [fp, C.c_int64, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.oracle_mean_std.restype = None
        L.oracle_norm_cdf.argtypes = [C.c_double]
        L.oracle_norm_cdf.restype = C.c_double
        L.oracle_norm_ppf.argtypes = [C.c_double]
        L.oracle_norm_ppf.restype = C.c_double
        L.oracle_count_above.argtypes = [fp, C.c_int64, C.c_double]
        L.oracle_count_above.restype = C.c_int64
        L.oracle_gaussiank_threshold.argtypes = [fp, C.c_int64, C.c_int64, C.c_int, C.c_int, C.POINTER(_Stats)]
        L.oracle_gaussiank_threshold.restype = None
        L.oracle_select.argtypes = [fp, C.c_int64, C.c_double, C.c_int64, ip, fp]
        L.oracle_select.restype = C.c_int64
        L.oracle_residual.argtypes = [fp, C.c_int64, ip, fp, C.c_int64, fp]
        L.oracle_residual.restype = None
        L.oracle_gk_sparsify.argtypes = [fp, fp, C.c_int64, C.c_int64, C.c_int64, ip, fp, C.POINTER(_Stats)]
        L.oracle_gk_sparsify.restype = C.c_int64
        L.oracle_gk_sparsify_segmented.argtypes = [fp, fp, C.c_int64, lp, lp, C.c_int32, C.c_int64, ip, fp, lp,
                                                   C.POINTER(_Stats)]
        L.oracle_gk_sparsify_segmented.restype = C.c_int64
        L.oracle_topk_exact.argtypes = [fp, C.c_int64, C.c_int64, ip, fp]
        L.oracle_topk_exact.restype = None
        L.oracle_error_ratio.argtypes = [fp, C.c_int64, ip, C.c_int64]
        L.oracle_error_ratio.restype = C.c_double
        L.oracle_apply_sparse.argtypes = [fp, C.c_int64, ip, fp, lp, C.c_int32, C.c_int64, C.c_float]
        L.oracle_apply_sparse.restype = None
        L.oracle_histogram.argtypes = [fp, C.c_int64, C.c_float, C.c_float, C.c_int32, lp]
        L.oracle_histogram.restype = None
        L.oracle_dgck_select.argtypes = [fp, C.c_int64, C.c_int64, ip, C.c_int64, ip, fp, lp]
        L.oracle_dgck_select.restype = C.c_int64
        L.oracle_dgck_sparsify.argtypes = [fp, fp, C.c_int64, C.c_int64, ip, C.c_int64, ip, fp, lp]
        L.oracle_dgck_sparsify.restype = C.c_int64
        _lib = L
    return _lib


def _f(a: np.ndarray):
    assert a.dtype == np.float32 and a.flags.c_contiguous
    return a.ctypes.data_as(C.POINTER(C.c_float))


def _i(a: np.ndarray):
    assert a.dtype == np.int32 and a.flags.c_contiguous
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def _l(a: np.ndarray):
    assert a.dtype == np.int64 and a.flags.c_contiguous
    return a.ctypes.data_as(C.POINTER(C.c_int64))


def accumulate(g: np.ndarray, eps: np.ndarray) -> np.ndarray:
    u = np.empty_like(g)
    lib().oracle_accumulate(_f(g), _f(eps), g.shape[0], _f(u))
    return u


def mean_std(u: np.ndarray, unbiased: bool = True) -> Tuple[float, float]:
    mu, sg = C.c_double(), C.c_double()
    lib().oracle_mean_std(_f(u), u.shape[0], int(unbiased), C.byref(mu), C.byref(sg))
    return mu.value, sg.value


def norm_cdf(z: float) -> float:
    return lib().oracle_norm_cdf(z)


def norm_ppf(p: float) -> float:
    return lib().oracle_norm_ppf(p)


def count_above(u: np.ndarray, thres: float) -> int:
    return int(lib().oracle_count_above(_f(u), u.shape[0], thres))


def gaussiank_threshold(u: np.ndarray, k: int, max_rounds: int = 4, unbiased: bool = True) -> Stats:
    st = _Stats()
    lib().oracle_gaussiank_threshold(_f(u), u.shape[0], k, max_rounds, int(unbiased), C.byref(st))
    return Stats.of(st)


def select(u: np.ndarray, thres: float, cap: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray, int]:
    """Pairs (idx, val) with |u| > thres in ascending index; returns (idx, val, true_count)."""
    d = u.shape[0]
    n = count_above(u, thres)
    m = n if cap is None else min(n, cap)
    idx = np.empty(m, dtype=np.int32)
    val = np.empty(m, dtype=np.float32)
    got = lib().oracle_select(_f(u), d, thres, m, _i(idx), _f(val))
    assert got == n
    return idx, val, n


def residual(u: np.ndarray, idx: np.ndarray, val: np.ndarray) -> np.ndarray:
    out = np.empty_like(u)
    lib().oracle_residual(_f(u), u.shape[0], _i(idx), _f(val), idx.shape[0], _f(out))
    return out


def gk_sparsify(g: np.ndarray, eps: np.ndarray, k: int, cap: Optional[int] = None):
    """One step of Eq. 2 with Gaussian_k.  eps is updated IN PLACE.
    Returns (idx, val, stats)."""
    d = g.shape[0]
    cap = d if cap is None else cap
    idx = np.empty(cap, dtype=np.int32)
    val = np.empty(cap, dtype=np.float32)
    st = _Stats()
    n = lib().oracle_gk_sparsify(_f(g), _f(eps), d, k, cap, _i(idx), _f(val), C.byref(st))
    return idx[:n].copy(), val[:n].copy(), Stats.of(st)


def gk_sparsify_segmented(g: np.ndarray, eps: np.ndarray, offsets: np.ndarray, seg_k: np.ndarray,
                          cap: Optional[int] = None):
    """Layer-wise Gaussian_k.  eps updated IN PLACE.  Returns (idx, val, seg_nnz, [stats])."""
    d = g.shape[0]
    S = offsets.shape[0] - 1
    cap = d if cap is None else cap
    idx = np.empty(cap, dtype=np.int32)
    val = np.empty(cap, dtype=np.float32)
    seg_nnz = np.zeros(S, dtype=np.int64)
    st = (_Stats * S)()
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    seg_k = np.ascontiguousarray(seg_k, dtype=np.int64)
    n = lib().oracle_gk_sparsify_segmented(_f(g), _f(eps), d, _l(offsets), _l(seg_k), S, cap,
                                           _i(idx), _f(val), _l(seg_nnz), st)
    return idx[:n].copy(), val[:n].copy(), seg_nnz, [Stats.of(s) for s in st]


def topk_exact(u: np.ndarray, k: int) -> Tuple[np.ndarray, np.ndarray]:
    idx = np.empty(k, dtype=np.int32)
    val = np.empty(k, dtype=np.float32)
    lib().oracle_topk_exact(_f(u), u.shape[0], k, _i(idx), _f(val))
    return idx, val


def error_ratio(u: np.ndarray, idx: np.ndarray) -> float:
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    return lib().oracle_error_ratio(_f(u), u.shape[0], _i(idx), idx.shape[0])


@dataclass
class DgcInfo:
    tau_bits: int   # fp32 pattern of the sampled threshold
    n_cand: int     # entries of the vector at or above it
    k_m: int        # rank taken in the sample

    @property
    def tau(self) -> float:
        return float(np.array([self.tau_bits], dtype=np.uint32).view(np.float32)[0])


def dgck_select(u: np.ndarray, k: int, sample_idx: np.ndarray):
    """DGC_k on a given vector.  Returns (idx, val, DgcInfo)."""
    d = u.shape[0]
    sample_idx = np.ascontiguousarray(sample_idx, dtype=np.int32)
    idx = np.empty(d, dtype=np.int32)
    val = np.empty(d, dtype=np.float32)
    info = np.zeros(3, dtype=np.int64)
    n = lib().oracle_dgck_select(_f(u), d, k, _i(sample_idx), sample_idx.shape[0], _i(idx), _f(val), _l(info))
    return idx[:n].copy(), val[:n].copy(), DgcInfo(int(info[0]), int(info[1]), int(info[2]))


def dgck_sparsify(g: np.ndarray, eps: np.ndarray, k: int, sample_idx: np.ndarray):
    """One step of Eq. 2 with DGC_k.  eps is updated IN PLACE.  Returns (idx, val, DgcInfo)."""
    d = g.shape[0]
    sample_idx = np.ascontiguousarray(sample_idx, dtype=np.int32)
    idx = np.empty(d, dtype=np.int32)
    val = np.empty(d, dtype=np.float32)
    info = np.zeros(3, dtype=np.int64)
    n = lib().oracle_dgck_sparsify(_f(g), _f(eps), d, k, _i(sample_idx), sample_idx.shape[0], _i(idx), _f(val),
                                   _l(info))
    return idx[:n].copy(), val[:n].copy(), DgcInfo(int(info[0]), int(info[1]), int(info[2]))


def apply_sparse(x: np.ndarray, idx: np.ndarray, val: np.ndarray, nnz: np.ndarray, cap: int, alpha: float) -> None:
    """x += alpha * (sum over ranks of their messages), IN PLACE (Eq. 2).  idx, val: P * cap
    entries, rank p's list at [p * cap, p * cap + nnz[p])."""
    P = nnz.shape[0]
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    val = np.ascontiguousarray(val, dtype=np.float32)
    nnz = np.ascontiguousarray(nnz, dtype=np.int64)
    assert idx.shape[0] == P * cap and val.shape[0] == P * cap
    lib().oracle_apply_sparse(_f(x), x.shape[0], _i(idx), _f(val), _l(nnz), P, cap, alpha)


def histogram(u: np.ndarray, lo: float, inv_w: float, nbins: int) -> np.ndarray:
    """Counts of u in nbins equal bins from lo (bin width 1 / inv_w): [below, bins..., above]."""
    counts = np.zeros(nbins + 2, dtype=np.int64)
    lib().oracle_histogram(_f(u), u.shape[0], lo, inv_w, nbins, _l(counts))
    return counts
