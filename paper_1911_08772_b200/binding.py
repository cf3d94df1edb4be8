"""Python binding of the C ABI in include/gk.h.

Argument marshalling only: every function takes torch CUDA tensors (device
memory) or numpy arrays (the host call), hands raw pointers and the current
CUDA stream to libgk_b200.so, and returns.  There is no CPU fallback: if the
library is missing or no CUDA device is present the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libgk_b200.so")

GK_DEV_TRUNCATED = 1
GK_DEV_TIMEOUT = 2
GK_DEV_BAD_SEGMENTS = 4
GK_DEV_BAD_SAMPLE = 8
GK_DEV_BAD_INDEX = 16

EXPORTS = [
    "gk_sparsify", "gk_sparsify_segmented", "topk_exact", "topk_sparsify", "gk_sparsify_host",
    "gk_sparsify_static", "gk_set_capacity", "gk_set_path", "gk_reserve", "gk_workspace_bytes", "gk_last_stats", "gk_last_segment_stats",
    "gk_stage_timing", "gk_last_stage_ms", "gk_last_cta_trace", "gk_launch_count", "gk_strerror", "gk_last_cuda_error", "gk_version",
    "gk_error_ratio", "dgck_select", "dgck_sparsify", "dgck_last_info",
    "gk_apply_sparse", "gk_apply_gathered", "gk_histogram", "gk_debug_set", "gk_last_path_info", "gk_select", "gk_set_params",
]


class GkStats(C.Structure):
    _fields_ = [
        ("mu", C.c_double), ("sigma", C.c_double), ("z", C.c_double), ("thres0", C.c_double),
        ("thr_final", C.c_double), ("counts", C.c_int64 * 4), ("rounds", C.c_int32),
        ("status", C.c_int32), ("nnz", C.c_int64), ("emitted", C.c_int64),
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
    status: int
    nnz: int
    emitted: int

    @staticmethod
    def of(s: GkStats) -> "Stats":
        return Stats(s.mu, s.sigma, s.z, s.thres0, s.thr_final, [int(c) for c in s.counts][: max(int(s.rounds), 0)],
                     int(s.rounds), int(s.status), int(s.nnz), int(s.emitted))


class GkError(RuntimeError):
    pass


_lib: Optional[C.CDLL] = None


def load() -> C.CDLL:
    """Load libgk_b200.so (built by paper_1911_08772_b200/build.py).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise GkError(f"{LIB_PATH} not found: run `python -m paper_1911_08772_b200.build` first "
                      "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int32
    L.gk_sparsify.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp]
    L.gk_select.argtypes = [vp, i64, i64, vp, vp, vp, vp]
    L.gk_select.restype = C.c_int
    L.gk_sparsify_static.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp]
    L.gk_sparsify_static.restype = C.c_int
    L.gk_error_ratio.argtypes = [vp, i64, vp, vp, vp, C.POINTER(C.c_double)]
    L.gk_error_ratio.restype = C.c_int
    L.gk_apply_sparse.argtypes = [vp, i64, C.POINTER(vp), C.POINTER(vp), vp, i32, i64, C.c_float, vp]
    L.gk_apply_sparse.restype = C.c_int
    L.gk_apply_gathered.argtypes = [vp, i64, vp, vp, vp, i32, i64, C.c_float, vp]
    L.gk_apply_gathered.restype = C.c_int
    L.gk_histogram.argtypes = [vp, i64, C.c_float, C.c_float, i32, vp, vp]
    L.gk_histogram.restype = C.c_int
    L.dgck_select.argtypes = [vp, i64, i64, vp, i64, vp, vp, vp, vp]
    L.dgck_select.restype = C.c_int
    L.dgck_sparsify.argtypes = [vp, vp, i64, i64, vp, i64, vp, vp, vp, vp]
    L.dgck_sparsify.restype = C.c_int
    L.dgck_last_info.argtypes = [vp, C.POINTER(i64)]
    L.dgck_last_info.restype = C.c_int
    L.gk_sparsify_segmented.argtypes = [vp, vp, i64, vp, vp, i32, vp, vp, vp, vp, vp]
    L.topk_exact.argtypes = [vp, i64, i64, vp, vp, vp]
    L.topk_sparsify.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp]
    L.gk_sparsify_host.argtypes = [vp, vp, i64, i64, vp, vp, vp, C.POINTER(GkStats)]
    L.gk_set_capacity.argtypes = [i64]
    L.gk_set_path.argtypes = [C.c_int]
    L.gk_reserve.argtypes = [i64, i32, vp]
    L.gk_workspace_bytes.argtypes = [i64, i32]
    L.gk_workspace_bytes.restype = i64
    L.gk_last_stats.argtypes = [vp, C.POINTER(GkStats)]
    L.gk_last_segment_stats.argtypes = [vp, i32, C.POINTER(GkStats)]
    L.gk_stage_timing.argtypes = [C.c_int]
    L.gk_stage_timing.restype = C.c_int
    L.gk_last_stage_ms.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int)]
    L.gk_last_stage_ms.restype = C.c_int
    L.gk_last_cta_trace.argtypes = [vp, C.POINTER(C.c_uint64), C.POINTER(C.c_int)]
    L.gk_last_cta_trace.restype = C.c_int
    L.gk_launch_count.argtypes = []
    L.gk_launch_count.restype = i64
    L.gk_strerror.argtypes = [C.c_int]
    L.gk_strerror.restype = C.c_char_p
    L.gk_last_cuda_error.argtypes = []
    L.gk_last_cuda_error.restype = C.c_char_p
    L.gk_version.argtypes = []
    L.gk_last_path_info.argtypes = [vp, C.POINTER(i64)]
    L.gk_last_path_info.restype = C.c_int
    L.gk_set_params.argtypes = [C.c_int, C.c_int]
    L.gk_set_params.restype = C.c_int
    L.gk_debug_set.argtypes = [C.c_int, i64]
    L.gk_debug_set.restype = C.c_int
    for name in ("gk_sparsify", "gk_sparsify_segmented", "topk_exact", "topk_sparsify", "gk_sparsify_host",
                 "gk_set_capacity", "gk_set_path", "gk_reserve", "gk_last_stats", "gk_last_segment_stats", "gk_version"):
        getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _check(rc: int) -> None:
    if rc != 0:
        L = load()
        msg = L.gk_strerror(rc).decode()
        if rc == -6:
            msg += ": " + L.gk_last_cuda_error().decode()
        raise GkError(f"gk error {rc}: {msg}")


def _stream() -> int:
    import torch
    return int(torch.cuda.current_stream().cuda_stream)


def _dev(t, dtype) -> int:
    import torch
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise GkError("expected a CUDA tensor")
    if t.dtype != dtype or not t.is_contiguous():
        raise GkError(f"expected a contiguous {dtype} tensor, got {t.dtype}")
    return t.data_ptr()


def gk_sparsify(g, eps, k: int, idx_out, val_out, nnz_out) -> None:
    """Enqueue one Gaussian_k error-compensated step on the current stream (see gk.h)."""
    import torch
    d = g.numel()
    _check(load().gk_sparsify(_dev(g, torch.float32), _dev(eps, torch.float32), d, k,
                              _dev(idx_out, torch.int32), _dev(val_out, torch.float32),
                              _dev(nnz_out, torch.int64), _stream()))


def gk_select(u, k: int, idx_out, val_out, nnz_out) -> None:
    """Gaussian_k as an operator on a given vector u, which is not modified (see gk.h)."""
    import torch
    _check(load().gk_select(_dev(u, torch.float32), u.numel(), k, _dev(idx_out, torch.int32),
                            _dev(val_out, torch.float32), _dev(nnz_out, torch.int64), _stream()))


def gk_sparsify_static(g, eps, k: int, idx_out, val_out, nnz_out) -> None:
    """gk_sparsify without any device allocation: the scratch is a fixed array inside the
    library (see gk.h for who needs this and for the limits)."""
    import torch
    d = g.numel()
    _check(load().gk_sparsify_static(_dev(g, torch.float32), _dev(eps, torch.float32), d, k,
                                     _dev(idx_out, torch.int32), _dev(val_out, torch.float32),
                                     _dev(nnz_out, torch.int64), _stream()))


def gk_error_ratio(eps, val, nnz):
    """(ratio, ||u - Comp(u)||^2, ||u||^2) of the step that left `eps` as its residual and wrote
    the values `val[:nnz]` (Eq. 5 of the paper).  Synchronises the stream."""
    import torch
    out = (C.c_double * 3)()
    _check(load().gk_error_ratio(_dev(eps, torch.float32), eps.numel(), _dev(val, torch.float32),
                                 _dev(nnz, torch.int64), _stream(), out))
    return float(out[0]), float(out[1]), float(out[2])


def gk_sparsify_segmented(g, eps, seg_offsets, seg_k, idx_out, val_out, seg_nnz_out, nnz_out) -> None:
    import torch
    d = g.numel()
    S = seg_offsets.numel() - 1
    _check(load().gk_sparsify_segmented(
        _dev(g, torch.float32), _dev(eps, torch.float32), d, _dev(seg_offsets, torch.int64),
        _dev(seg_k, torch.int64), S, _dev(idx_out, torch.int32), _dev(val_out, torch.float32),
        None if seg_nnz_out is None else _dev(seg_nnz_out, torch.int64), _dev(nnz_out, torch.int64), _stream()))


def topk_exact(u, k: int, idx_out, val_out) -> None:
    import torch
    _check(load().topk_exact(_dev(u, torch.float32), u.numel(), k, _dev(idx_out, torch.int32),
                             _dev(val_out, torch.float32), _stream()))


def topk_sparsify(g, eps, k: int, idx_out, val_out, nnz_out) -> None:
    import torch
    _check(load().topk_sparsify(_dev(g, torch.float32), _dev(eps, torch.float32), g.numel(), k,
                                _dev(idx_out, torch.int32), _dev(val_out, torch.float32),
                                _dev(nnz_out, torch.int64), _stream()))


def dgck_select(u, k: int, sample_idx, idx_out, val_out, nnz_out) -> None:
    """DGC_k on a given vector (see gk.h): sampled threshold, then the k largest candidates."""
    import torch
    _check(load().dgck_select(_dev(u, torch.float32), u.numel(), k, _dev(sample_idx, torch.int32),
                              sample_idx.numel(), _dev(idx_out, torch.int32), _dev(val_out, torch.float32),
                              _dev(nnz_out, torch.int64), _stream()))


def dgck_sparsify(g, eps, k: int, sample_idx, idx_out, val_out, nnz_out) -> None:
    """One error-compensated step with DGC_k as the compressor (see gk.h)."""
    import torch
    _check(load().dgck_sparsify(_dev(g, torch.float32), _dev(eps, torch.float32), g.numel(), k,
                                _dev(sample_idx, torch.int32), sample_idx.numel(), _dev(idx_out, torch.int32),
                                _dev(val_out, torch.float32), _dev(nnz_out, torch.int64), _stream()))


def dgck_last_info():
    """(tau_bits, n_candidates, k_m, pairs_written) of the last dgck_* call on the current
    stream.  Synchronises the stream."""
    out = (C.c_int64 * 4)()
    _check(load().dgck_last_info(_stream(), out))
    return int(out[0]), int(out[1]), int(out[2]), int(out[3])


def gk_apply_gathered(x, idx, val, nnz, cap: int, alpha: float) -> None:
    """x += alpha * (sum over the P = nnz.numel() messages), list p at [p * cap, p * cap + nnz[p])
    of idx / val (Eq. 2; see gk.h)."""
    import torch
    P = nnz.numel()
    if idx.numel() < P * cap or val.numel() < P * cap:
        raise GkError("idx / val hold fewer than P * cap entries")
    _check(load().gk_apply_gathered(_dev(x, torch.float32), x.numel(), _dev(idx, torch.int32),
                                    _dev(val, torch.float32), _dev(nnz, torch.int64), P, cap, alpha, _stream()))


def gk_apply_sparse(x, idx_lists, val_lists, nnz, cap: int, alpha: float) -> None:
    """The same with one tensor per message (each may live in a peer GPU's memory)."""
    import torch
    P = len(idx_lists)
    ip = (C.c_void_p * P)(*[_dev(t, torch.int32) for t in idx_lists])
    vp_ = (C.c_void_p * P)(*[_dev(t, torch.float32) for t in val_lists])
    _check(load().gk_apply_sparse(_dev(x, torch.float32), x.numel(), ip, vp_, _dev(nnz, torch.int64), P, cap,
                                  alpha, _stream()))


def gk_histogram(u, lo: float, inv_w: float, counts_out) -> None:
    """Histogram of u over nbins = counts_out.numel() - 2 equal bins from lo (width 1 / inv_w);
    counts_out (int64): [below, bins..., above] (see gk.h).  Enqueued on the current stream."""
    import torch
    _check(load().gk_histogram(_dev(u, torch.float32), u.numel(), lo, inv_w, counts_out.numel() - 2,
                               _dev(counts_out, torch.int64), _stream()))


def gk_sparsify_host(g, eps, k: int, idx_out, val_out):
    """Host-buffer step.  g, eps, idx_out, val_out: numpy arrays or CPU torch tensors
    (pinned for speed).  eps is updated in place.  Returns (nnz, Stats)."""
    def ptr(a):
        return a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data
    d = g.numel() if hasattr(g, "numel") else g.size
    nnz = C.c_int64(0)
    st = GkStats()
    _check(load().gk_sparsify_host(ptr(g), ptr(eps), d, k, ptr(idx_out), ptr(val_out),
                                   C.addressof(nnz), C.byref(st)))
    return int(nnz.value), Stats.of(st)


def gk_set_capacity(cap: int) -> None:
    _check(load().gk_set_capacity(cap))


def gk_set_params(unbiased_std: bool = True, max_rounds: int = 4) -> None:
    """Divisor of the variance (d - 1 or d) and number of rounds of Algorithm 1 (see gk.h)."""
    _check(load().gk_set_params(int(bool(unbiased_std)), max_rounds))


def gk_set_path(path: int) -> None:
    """0: cluster kernel for small vectors, else the persistent cooperative kernel (default);
    1: three kernels with look-back; 2: the persistent kernel at every size."""
    _check(load().gk_set_path(path))


def gk_reserve(d: int, S: int = 1) -> None:
    _check(load().gk_reserve(d, S, _stream()))


def gk_workspace_bytes(d: int, S: int = 1) -> int:
    return int(load().gk_workspace_bytes(d, S))


def gk_last_stats() -> Stats:
    st = GkStats()
    _check(load().gk_last_stats(_stream(), C.byref(st)))
    return Stats.of(st)


def gk_last_segment_stats(S: int) -> List[Stats]:
    arr = (GkStats * S)()
    _check(load().gk_last_segment_stats(_stream(), S, arr))
    return [Stats.of(s) for s in arr]


def gk_stage_timing(enable: bool) -> None:
    _check(load().gk_stage_timing(int(enable)))


def gk_last_stage_ms() -> List[float]:
    """Durations (ms) of the stages of the last call on the current stream; needs
    gk_stage_timing(True) before that call.  Synchronises the stream."""
    ms = (C.c_float * 8)()
    n = C.c_int(0)
    _check(load().gk_last_stage_ms(_stream(), ms, C.byref(n)))
    return [float(ms[i]) for i in range(n.value)]


def gk_last_cta_trace():
    """Per-CTA timestamps (ns) of the last fused call on the current stream: list of 8-tuples."""
    buf = (C.c_uint64 * (512 * 8))()
    n = C.c_int(0)
    _check(load().gk_last_cta_trace(_stream(), buf, C.byref(n)))
    return [tuple(int(buf[i * 8 + j]) for j in range(8)) for i in range(n.value)]


KNOB_BARRIER_POLLS, KNOB_LOOKBACK_POLLS, KNOB_EXTRA_ARRIVALS, KNOB_MUTE_TILE, KNOB_PREDICTION, KNOB_SELECTED_WAY = range(6)


def gk_debug_set(key: int, value: int) -> None:
    """Test hooks (see gk.h): poll limits of the bounded waits, and switches that force either
    side of the library's run-time decisions."""
    _check(load().gk_debug_set(key, value))


def gk_last_path_info():
    """(CTAs with a prediction, CTAs whose bands held, second count needed, cells left to the
    second phase, CTAs launched, CTAs that counted a selection of the candidates) of the last
    fused gk_sparsify / gk_select call on the current stream.  Synchronises the stream."""
    out = (C.c_int64 * 6)()
    _check(load().gk_last_path_info(_stream(), out))
    return tuple(int(v) for v in out)


def gk_launch_count() -> int:
    return int(load().gk_launch_count())


def gk_version() -> int:
    return int(load().gk_version())


def gk_strerror(code: int) -> str:
    return load().gk_strerror(code).decode()
