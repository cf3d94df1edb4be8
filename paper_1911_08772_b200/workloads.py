"""Seeded synthetic gradient generators.

This module only produces input bytes.  It holds none of the sparsifier's
arithmetic and imports neither the CUDA binding nor the CPU oracle; both are
fed the arrays made here, so generator arithmetic never enters a comparison.

The paper's gradients come from training runs on data sets that are not
available offline.  The generators below stand in for them: the vector sizes
follow Table 1 and Section 3.3 (ResNet-20, VGG-16, ResNet-50, LSTM-PTB), the
value distributions follow the paper's description of accumulated gradients in
Section 3.1 (bell shaped, most coordinates near zero, wider tails once
residuals accumulate), and the sweep mirrors the operator-timing experiment of
Section 4.3 (Fig. 4).

Every stream is counter based: element chunk ``c`` of step ``t`` of workload
``w`` is drawn from Philox keyed by ``(seed, w)`` with counter ``(0, 0, c, t)``,
so chunks are independent of the thread that draws them and of each other.
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

MASTER_SEED = 0x1911_08772
CHUNK = 1 << 20  # elements per independently keyed chunk

# workload tags (second Philox key word)
TAG_NORMAL = 1
TAG_LAPLACE_MIX = 2
TAG_SEGMENTED = 3
TAG_STUDENT_T = 4
TAG_SWEEP_NORMAL = 5
TAG_SWEEP_LAPLACE = 6
TAG_PARTITION = 7
TAG_MISC = 8
TAG_SAMPLE = 9


def ceil_k(d: int, num: int, den: int) -> int:
    """k = ceil(rho * d) for rho = num/den, in integers."""
    return (d * num + den - 1) // den


RHO = {
    "1e-4": (1, 10000),
    "1e-3": (1, 1000),
    "5e-3": (5, 1000),
    "1e-2": (1, 100),
}


def _rng(tag: int, chunk: int, step: int, seed: int) -> np.random.Generator:
    bg = np.random.Philox(counter=[0, 0, chunk, step], key=[seed & (2**64 - 1), tag])
    return np.random.Generator(bg)


def _n_threads() -> int:
    return max(1, min(32, os.cpu_count() or 1))


def _fill_chunks(d: int, fn: Callable[[np.ndarray, int, int], None], out: Optional[np.ndarray]) -> np.ndarray:
    """Call fn(view, chunk_index, start) for every CHUNK-sized slice of out."""
    if out is None:
        out = np.empty(d, dtype=np.float32)
    assert out.dtype == np.float32 and out.shape == (d,)
    n_chunks = (d + CHUNK - 1) // CHUNK

    def job(c: int) -> None:
        lo = c * CHUNK
        hi = min(d, lo + CHUNK)
        fn(out[lo:hi], c, lo)

    if n_chunks <= 1 or _n_threads() == 1:
        for c in range(n_chunks):
            job(c)
    else:
        with ThreadPoolExecutor(max_workers=_n_threads()) as pool:
            list(pool.map(job, range(n_chunks)))
    return out


def normal(d: int, sigma: float, step: int = 0, tag: int = TAG_NORMAL,
           seed: int = MASTER_SEED, out: Optional[np.ndarray] = None) -> np.ndarray:
    """iid N(0, sigma^2), fp32."""
    s = np.float32(sigma)

    def fn(view: np.ndarray, c: int, lo: int) -> None:
        _rng(tag, c, step, seed).standard_normal(out=view, dtype=np.float32)
        view *= s

    return _fill_chunks(d, fn, out)


def _laplace_unit(rng: np.random.Generator, n: int) -> Tuple[np.ndarray, np.ndarray]:
    """Unit Laplace draws as (magnitude ~ Exp(1), raw 32-bit words for sign / mixing)."""
    mag = rng.standard_exponential(n, dtype=np.float32)
    bits = rng.integers(0, 2**32, size=n, dtype=np.uint32)
    return mag, bits


def laplace(d: int, b: float, step: int = 0, tag: int = TAG_SWEEP_LAPLACE,
            seed: int = MASTER_SEED, out: Optional[np.ndarray] = None) -> np.ndarray:
    """iid Laplace(0, b), fp32: an Exp(1) magnitude with a random sign."""
    bb = np.float32(b)

    def fn(view: np.ndarray, c: int, lo: int) -> None:
        mag, bits = _laplace_unit(_rng(tag, c, step, seed), view.shape[0])
        np.multiply(mag, bb, out=mag)
        np.negative(mag, out=mag, where=(bits & 1).astype(bool))
        view[:] = mag

    return _fill_chunks(d, fn, out)


def laplace_mixture(d: int, step: int = 0, w_wide: float = 0.1, b_narrow: float = 1e-4,
                    b_wide: float = 1e-2, seed: int = MASTER_SEED,
                    out: Optional[np.ndarray] = None) -> np.ndarray:
    """Per-element mixture: Laplace(0, b_wide) w.p. w_wide, else Laplace(0, b_narrow)."""
    cut = np.uint32(int(w_wide * 2**31))

    def fn(view: np.ndarray, c: int, lo: int) -> None:
        mag, bits = _laplace_unit(_rng(TAG_LAPLACE_MIX, c, step, seed), view.shape[0])
        wide = (bits >> 1) < cut
        scale = np.where(wide, np.float32(b_wide), np.float32(b_narrow))
        np.multiply(mag, scale, out=mag)
        np.negative(mag, out=mag, where=(bits & 1).astype(bool))
        view[:] = mag

    return _fill_chunks(d, fn, out)


def student_t3_outliers(d: int, step: int = 0, scale: float = 1e-3, p_out: float = 1e-4,
                        seed: int = MASTER_SEED, out: Optional[np.ndarray] = None) -> np.ndarray:
    """scale * t_3 (as Z / sqrt((Z1^2+Z2^2+Z3^2)/3)); each entry independently
    replaced w.p. p_out by +-U(0.1, 1)."""
    sc = np.float32(scale)

    def fn(view: np.ndarray, c: int, lo: int) -> None:
        rng = _rng(TAG_STUDENT_T, c, step, seed)
        n = view.shape[0]
        z = rng.standard_normal(n, dtype=np.float32)
        chi = np.zeros(n, dtype=np.float32)
        for _ in range(3):
            w = rng.standard_normal(n, dtype=np.float32)
            chi += w * w
        chi *= np.float32(1.0 / 3.0)
        np.sqrt(chi, out=chi)
        np.maximum(chi, np.float32(1e-20), out=chi)
        z /= chi
        z *= sc
        hit = rng.random(n, dtype=np.float32) < np.float32(p_out)
        m = int(hit.sum())
        if m:
            mag = (0.1 + 0.9 * rng.random(m, dtype=np.float32)).astype(np.float32)
            sgn = rng.integers(0, 2, size=m).astype(np.float32) * 2.0 - 1.0
            z[hit] = mag * sgn.astype(np.float32)
        view[:] = z

    return _fill_chunks(d, fn, out)


@dataclass
class Partition:
    """Contiguous layer-wise partition of a length-d vector."""
    d: int
    offsets: np.ndarray  # int64, S+1, offsets[0] = 0, offsets[S] = d
    sigmas: np.ndarray   # float64, S

    @property
    def S(self) -> int:
        return int(self.offsets.shape[0] - 1)

    def sizes(self) -> np.ndarray:
        return np.diff(self.offsets)

    def seg_k(self, num: int, den: int) -> np.ndarray:
        return np.array([ceil_k(int(n), num, den) for n in self.sizes()], dtype=np.int64)


def seeded_partition(d: int, S: int, min_size: int = 64, max_weight: float = 2.4e6,
                     seed: int = MASTER_SEED) -> Partition:
    """S contiguous segments: weights exp(U(ln min_size, ln max_weight)) scaled to
    sum d, floored, every size >= min_size, the remainder given to the largest.
    Per-segment sigma is log-uniform in [1e-5, 1e-2]."""
    assert d >= S * min_size
    rng = _rng(TAG_PARTITION, 0, S, seed)
    w = np.exp(rng.uniform(math.log(min_size), math.log(max_weight), size=S))
    sizes = np.floor(w * (d / w.sum())).astype(np.int64)
    sizes = np.maximum(sizes, min_size)
    big = int(np.argmax(sizes))
    sizes[big] += d - int(sizes.sum())
    assert sizes[big] >= min_size and int(sizes.sum()) == d
    offsets = np.zeros(S + 1, dtype=np.int64)
    np.cumsum(sizes, out=offsets[1:])
    sigmas = np.exp(rng.uniform(math.log(1e-5), math.log(1e-2), size=S))
    return Partition(d=d, offsets=offsets, sigmas=sigmas)


def segmented_normal(part: Partition, step: int = 0, seed: int = MASTER_SEED,
                     out: Optional[np.ndarray] = None) -> np.ndarray:
    """Segment s is iid N(0, sigma_s^2)."""
    out = normal(part.d, 1.0, step=step, tag=TAG_SEGMENTED, seed=seed, out=out)
    for s in range(part.S):
        lo, hi = int(part.offsets[s]), int(part.offsets[s + 1])
        out[lo:hi] *= np.float32(part.sigmas[s])
    return out


# ---------------------------------------------------------------------------
# The five workload families
# ---------------------------------------------------------------------------

D_RESNET20 = 269_722
D_VGG16 = 14_728_266
D_RESNET50 = 25_557_032
D_LSTM_PTB = 66_034_000
S_RESNET50 = 161
SWEEP_D = [1 << 20, 1 << 22, 1 << 24, 1 << 26, 1 << 28]


@dataclass
class Workload:
    name: str
    d: int
    rhos: List[str]
    steps: int
    grad: Callable[[int, Optional[np.ndarray]], np.ndarray]  # (step, out) -> g
    partition: Optional[Partition] = None
    note: str = ""

    def k(self, rho: str) -> int:
        num, den = RHO[rho]
        return ceil_k(self.d, num, den)


def resnet20_normal(d: int = D_RESNET20) -> Workload:
    return Workload("resnet20_normal", d, ["1e-3"], 10,
                    lambda t, out=None: normal(d, 1e-3, step=t, out=out),
                    note="g ~ iid N(0, 1e-3^2)")


def vgg16_laplace_mixture(d: int = D_VGG16) -> Workload:
    return Workload("vgg16_laplace_mixture", d, ["1e-3"], 100,
                    lambda t, out=None: laplace_mixture(d, step=t, out=out),
                    note="0.9 Laplace(0,1e-4) + 0.1 Laplace(0,1e-2)")


def resnet50_segmented(d: int = D_RESNET50, S: int = S_RESNET50) -> Workload:
    part = seeded_partition(d, S)
    return Workload("resnet50_segmented", d, ["1e-3", "1e-2"], 20,
                    lambda t, out=None: segmented_normal(part, step=t, out=out),
                    partition=part,
                    note="161 segments, N(0, sigma_s^2), sigma_s log-uniform [1e-5,1e-2]")


def lstm_student_t(d: int = D_LSTM_PTB) -> Workload:
    return Workload("lstm_student_t", d, ["1e-3", "5e-3"], 20,
                    lambda t, out=None: student_t3_outliers(d, step=t, out=out),
                    note="1e-3 * t_3 with 1e-4 of entries +-U(0.1,1)")


def sweep_point(d: int, dist: str) -> Workload:
    if dist == "normal":
        fn = lambda t, out=None: normal(d, 1.0, step=t, tag=TAG_SWEEP_NORMAL, out=out)
    elif dist == "laplace":
        fn = lambda t, out=None: laplace(d, 1.0, step=t, tag=TAG_SWEEP_LAPLACE, out=out)
    else:
        raise ValueError(dist)
    return Workload(f"sweep_{dist}_2^{d.bit_length() - 1}", d, ["1e-4", "1e-3", "1e-2"], 1, fn,
                    note=f"iid {dist}(0,1)")


def misc_rng(stream: int) -> np.random.Generator:
    """Generator for small hand-shaped test vectors."""
    return _rng(TAG_MISC, 0, stream, MASTER_SEED)


def sample_positions(d: int, m: int, step: int = 0, seed: int = MASTER_SEED) -> np.ndarray:
    """m positions drawn uniformly from [0, d) with replacement (int32): the random sample a
    sampling selector such as DGC_k takes.  The draw is an input of the method, so it is made
    here and handed to whoever needs it."""
    rng = _rng(TAG_SAMPLE, 0, step, seed)
    return rng.integers(0, d, size=m, dtype=np.int64).astype(np.int32)


def sample_size(d: int, num: int = 1, den: int = 100) -> int:
    """Sample size ceil(d * num / den); the default is the 1 % sample of Section 4.3."""
    return max(1, (d * num + den - 1) // den)
