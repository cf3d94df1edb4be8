#!/usr/bin/env python
"""Benchmark of the error-compensated Gaussian_k sparsifier on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload NAME] [--path 0|1] [--loop-only] [--sweep]

One "step" is one whole pass of the hot path -- gk_sparsify(g, eps, d, k, ...) -- over one
synthetic gradient vector with the residual eps carried from step to step.  The default
workload is the ResNet-50-sized vector (d = 25,557,032, rho = 1e-3, whole-vector
selection).  The metric is throughput in GB/s of ALGORITHMIC bytes:
    bytes/step = (16 + 4 r) * d + 12 * nnz,   r = count passes over u that the step ran
(read g and eps, write u over eps, one read of u per count pass, one read of u for the
compaction, 8 bytes per emitted pair and 4 per cleared residual slot).  r = 1 when all ten
candidate thresholds are counted in one pass after the statistics; r = 0 when the counts were
taken while the vector streamed in (the kernel reports which, see gk_last_path_info).

With a small --steps K the K-step region is repeated until about 0.3 s have been timed and
the median region is reported, so that a short run and a long one measure the same thing.

Printed: one JSON line.  With --impl reference the CPU oracle
is timed instead, on the host cores, on the same workload.  With N > 1 (torchrun) every rank
runs an independent replica on its own GPU: the method has no exchange inside this path.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1911_08772_b200 import workloads as wl  # noqa: E402

METRIC = "GaussianK sparsify GB/s (% HBM peak) at d=25.6M, rho=1e-3; speedup vs exact Top_k"
UNIT = "GB/s"
L2_BYTES = 126 * 1024 * 1024
N_ROTATE = 20   # distinct gradients: the workload's 20 error-compensation iterations, then again
EPISODE = 20    # steps that share one residual buffer (eps starts at zero)
FUSED_PROFILE = os.path.join(ROOT, "profiles", "k_gk_fused_resnet50_ncu_full.txt")
# files whose contents decide what k_gk_fused does: the ncu figures hold only for these
FUSED_SOURCES = ["gk_fused.cu", "gk_coop.cuh", "gk_count.cuh", "gk_alg1.cuh", "gk_common.cuh"]
MIN_TIMED_MS = 300.0   # the timed region is repeated until this much has been timed
MAX_EPS = 256   # residual buffers kept, one per episode of a timed region (memory permitting); all are zeroed
                # again before every region, outside the timing


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    return 6650.0, "fallback (earlier measurement on this pool)"


def algorithmic_bytes(d: int, nnz: float, r: float = 1.0) -> float:
    """(16 + 4 r) d + 12 nnz: r = count passes over u (1: one pass for all ten candidates)."""
    return (16.0 + 4.0 * r) * d + 12.0 * nnz


def fused_source_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in FUSED_SOURCES:
        with open(os.path.join(ROOT, "paper_1911_08772_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(d: int):
    """DRAM bytes per launch of k_gk_fused from the committed ncu summary, or None when that
    capture was of another size or of other kernel sources."""
    try:
        rec = {}
        with open(FUSED_PROFILE) as f:
            for line in f:
                if ":" in line:
                    key, _, v = line.partition(":")
                    rec[key.strip()] = v.strip()
        if int(rec["capture_d"]) != d or rec["kernel_source_sha256_16"] != fused_source_hash():
            return None
        return int(rec["dram_bytes_per_launch"])
    except Exception:
        return None


def pick_workload(name: str):
    table = {
        "resnet50": (wl.resnet50_segmented, "1e-3"),
        "resnet20": (wl.resnet20_normal, "1e-3"),
        "vgg16": (wl.vgg16_laplace_mixture, "1e-3"),
        "lstm": (wl.lstm_student_t, "1e-3"),
    }
    if name in table:
        f, rho = table[name]
        return f(), rho
    if name.startswith("sweep_"):
        _, dist, lg = name.split("_")
        return wl.sweep_point(1 << int(lg), dist), "1e-3"
    raise SystemExit(f"unknown workload {name}")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while a region runs (read only)."""

    def __init__(self, index: int, period_s: float = 0.005):
        self.index = index
        self.period = period_s
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonHwPowerBrakeSlowdown: "hw_power_brake_slowdown",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, nm in names.items():
                    if r & bit:
                        self.reasons.add(nm)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()

    def summary(self):
        return {
            "sm_mhz": (statistics.median(self.samples) if self.samples else None),
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


def cpu_oracle_rate(w, rho, steps: int, warmup: int = 0):
    """Time the CPU oracle (single thread, as it stands) on `steps` steps of the workload."""
    from oracle import oracle as orc

    k = w.k(rho)
    eps = np.zeros(w.d, dtype=np.float32)
    g = np.empty(w.d, dtype=np.float32)
    total_t, total_b, nnz_last = 0.0, 0.0, 0
    for t in range(warmup + steps):
        w.grad(t, g)
        t0 = time.perf_counter()
        idx, val, st = orc.gk_sparsify(g, eps, k)
        dt = time.perf_counter() - t0
        if t >= warmup:
            total_t += dt
            total_b += algorithmic_bytes(w.d, idx.size, st.rounds)   # the oracle reads u once per round
        nnz_last = idx.size
    return total_b / total_t / 1e9, total_t / steps, nnz_last


def workload_string(w, rho) -> str:
    return f"{w.name} d={w.d} rho={rho} k={w.k(rho)} whole-vector selection, eps carried over"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w, rho = pick_workload(args.workload)
    # each oracle step at d = 25.6M takes ~0.5 s on one core: bound the run to a few minutes
    steps = max(1, min(args.steps, 60))
    warm = max(0, min(args.warmup, 20))
    gbs, s_per_step, nnz = cpu_oracle_rate(w, rho, steps, warm)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": s_per_step * 1e3, "steps_per_s": 1.0 / s_per_step,
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_string(w, rho),
                   "note": "CPU oracle (oracle/gk_oracle.cpp), one thread"},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"{steps} full steps of the workload (requested {args.steps})"},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def time_region(torch, fn, steps):
    """CUDA-event time (ms) of `steps` calls of fn(t) on the current stream."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for t in range(steps):
        fn(t)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b)


def max_over_ranks(ms: float, world: int, device) -> float:
    """Slowest rank's time: the job is as fast as its slowest replica."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(world: int, bytes_per_step: float, steps: int, ms: float) -> float:
    """Aggregate over all replicas: every rank processed `steps` vectors in `ms`."""
    return world * bytes_per_step * steps / (ms * 1e-3) / 1e9


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_1911_08772_b200 import binding as gk
    from paper_1911_08772_b200 import build as lib_build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        lib_build.build()
    if world > 1:
        dist.barrier()
    gk.load()
    gk.gk_set_path(args.path)

    w, rho = pick_workload(args.workload)
    d, k = w.d, w.k(rho)
    K, W = args.steps, max(args.warmup, 3)

    # inputs resident in HBM: the gradients of N_ROTATE steps (a different seed per rank), and
    # one zeroed residual per episode of EPISODE steps, as in the workload's EC loop
    n_rot = N_ROTATE if 4 * d * (N_ROTATE + 8) < 60e9 else 4
    if args.rotate:
        n_rot = args.rotate
    gs = []
    buf = np.empty(d, dtype=np.float32)
    for j in range(n_rot):
        gs.append(torch.from_numpy(w.grad(1000 * rank + j, buf)).to(dev))
    # every episode of a region gets a residual buffer of its own (zeroed before the region), as far
    # as 60 GB go; with fewer, later episodes continue from an earlier episode's residual
    episodes = (max(K, W) + EPISODE - 1) // EPISODE
    n_eps = max(1, min(MAX_EPS, episodes, int((60e9 - 4.0 * d * n_rot) // (4.0 * d))))
    if args.rotate:
        n_eps = min(n_eps, 2)   # profiler captures: little memory
    epss = [torch.zeros(d, dtype=torch.float32, device=dev) for _ in range(n_eps)]

    def fresh_episodes():
        for e_ in epss:
            e_.zero_()
    eps = epss[0]
    idx = torch.empty(d, dtype=torch.int32, device=dev)
    val = torch.empty(d, dtype=torch.float32, device=dev)
    nnz = torch.zeros(1, dtype=torch.int64, device=dev)
    gk.gk_reserve(d, 1)

    def step(t):
        gk.gk_sparsify(gs[t % n_rot], epss[(t // EPISODE) % n_eps], k, idx, val, nnz)

    if args.call != "gk":
        # a capture of one of the other entry points: the same loop, nothing else (--loop-only)
        if args.call == "segmented":
            part = w.partition
            d_off = torch.from_numpy(part.offsets).to(dev)
            d_k = torch.from_numpy(part.seg_k(*wl.RHO[rho])).to(dev)
            seg_nnz = torch.zeros(part.S, dtype=torch.int64, device=dev)

            def step(t):  # noqa: F811
                gk.gk_sparsify_segmented(gs[t % n_rot], epss[(t // EPISODE) % n_eps], d_off, d_k, idx, val,
                                         seg_nnz, nnz)
        elif args.call == "topk_sparsify":
            def step(t):  # noqa: F811
                gk.topk_sparsify(gs[t % n_rot], epss[(t // EPISODE) % n_eps], k, idx, val, nnz)
        elif args.call in ("dgck_sparsify", "dgck_select"):
            smp = torch.from_numpy(wl.sample_positions(d, wl.sample_size(d), step=0)).to(dev)
            if args.call == "dgck_sparsify":
                def step(t):  # noqa: F811
                    gk.dgck_sparsify(gs[t % n_rot], epss[(t // EPISODE) % n_eps], k, smp, idx, val, nnz)
            else:
                def step(t):  # noqa: F811
                    gk.dgck_select(gs[t % n_rot], k, smp, idx, val, nnz)
        elif args.call == "gk_select":
            def step(t):  # noqa: F811
                gk.gk_select(gs[t % n_rot], k, idx, val, nnz)
        else:
            def step(t):  # noqa: F811
                gk.topk_exact(gs[t % n_rot], k, idx, val)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for t in range(W):
        step(t)
    fresh_episodes()
    barrier()
    # the K-step region, repeated until MIN_TIMED_MS have been timed (the same number of
    # repeats on every rank); the median region is the one reported
    launches0 = gk.gk_launch_count()
    sampler = ClockSampler(local)
    regions = []
    with sampler:
        first = max_over_ranks(time_region(torch, step, K), world, dev)
        regions.append(first)
        if args.repeats > 0:
            repeats = args.repeats
        else:
            repeats = 1 if args.loop_only else max(1, min(2000, int(MIN_TIMED_MS / max(first, 1e-3)) + 1))
        for rep in range(1, repeats):
            fresh_episodes()   # every region starts its episodes from eps = 0 (not timed)
            barrier()
            regions.append(max_over_ranks(time_region(torch, step, K), world, dev))
    barrier()
    launches = (gk.gk_launch_count() - launches0) // len(regions)
    ms = statistics.median(regions)
    nnz_mean = float(nnz.item())  # of the last step; 12 * nnz is ~0.03 % of the bytes
    # how the last step took its counts: r = 0 when every CTA counted while streaming
    info = gk.gk_last_path_info() if args.call == "gk" and args.path == 0 else (0, 0, 0, 0, 0, 0)
    r_passes = (0.0 if info[4] > 0 and info[1] == info[4] else 1.0) + (1.0 if info[2] else 0.0)
    bytes_step = algorithmic_bytes(d, nnz_mean, r_passes)
    value = whole_job_gbs(world, bytes_step, K, ms)
    peak, peak_src = measured_peaks()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    if args.loop_only:
        print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
                          "warmup": W, "ms_per_step": ms / K, "path": args.path, "loop_only": True,
                          "count_passes": r_passes, "path_info": info}))
        return

    # ---- per-kernel durations (CUDA events recorded by the library around its kernels)
    Ks = min(K, 200)

    def stage_means(n_stage):
        acc = np.zeros(n_stage)
        fresh_episodes()
        gk.gk_stage_timing(True)
        for t in range(Ks):
            step(t)
            acc += np.array(gk.gk_last_stage_ms()[:n_stage])
        gk.gk_stage_timing(False)
        return acc / Ks

    fused = stage_means(7)
    fused_ms = float(fused[0])
    traffic = recorded_traffic(d)
    roof = {
        "bound": "hbm", "kernel": "k_gk_fused", "achieved": bytes_step / (fused_ms * 1e-3) / 1e9,
        "peak": peak, "unit": "GB/s", "peak_source": peak_src,
        "frac": bytes_step / (fused_ms * 1e-3) / 1e9 / peak,
        "frac_of_nominal_8TBs": bytes_step / (fused_ms * 1e-3) / 1e9 / 8000.0,
        "traffic": traffic,
        "traffic_source": "dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of k_gk_fused at this d "
                          "(profiles/k_gk_fused_resnet50_ncu_full.txt); null when the kernel's sources have "
                          "changed since that capture",
        "kernel_ms": fused_ms,
        "kernel_ms_source": "mean over %d launches of CUDA events the library records around the kernel on its "
                            "stream, one launch at a time (a second loop right after the headline loop, whose "
                            "back-to-back launches overlap their ends and starts: ms_per_step is smaller)" % Ks,
        "phase_ms": {"accumulate_stats+barrier": fused[1], "count_loop": fused[2], "barrier2": fused[3],
                     "replay_rounds": fused[4], "compact": fused[5], "last_cta_exit": fused[6]},
        "bytes_per_launch": bytes_step,
        "bytes_model": f"(16 + 4 r) d + 12 nnz with r = {r_passes:g} count passes over u",
        # what DRAM really moved, against both peaks: the counts and most of the compaction are
        # served from shared memory and L2, so this is below the algorithmic rate
        "dram": None if traffic is None else {
            "bytes_per_launch": traffic, "gbs": traffic / (fused_ms * 1e-3) / 1e9,
            "frac_of_measured_copy": traffic / (fused_ms * 1e-3) / 1e9 / peak,
            "frac_of_nominal_8TBs": traffic / (fused_ms * 1e-3) / 1e9 / 8000.0},
        "floor": {"bytes": 12.0 * d + 12.0 * nnz_mean,
                  "note": "read g and eps once, write u once, the pairs and the cleared slots: what no "
                          "implementation of the step can avoid moving",
                  "gbs": (12.0 * d + 12.0 * nnz_mean) / (fused_ms * 1e-3) / 1e9,
                  "frac_of_measured_copy": (12.0 * d + 12.0 * nnz_mean) / (fused_ms * 1e-3) / 1e9 / peak,
                  "frac_of_nominal_8TBs": (12.0 * d + 12.0 * nnz_mean) / (fused_ms * 1e-3) / 1e9 / 8000.0},
    }
    # the three-kernel path (look-back compaction) on the same steps, stage by stage
    gk.gk_set_path(1)
    for t in range(3):
        step(t)
    fresh_episodes()
    ms3 = time_region(torch, step, Ks) / Ks
    stage = stage_means(3)
    gk.gk_set_path(0)
    three = {
        "ms_per_step": ms3, "gbs": bytes_step / ms3 / 1e6,
        "stage_ms": {"accumulate_stats": stage[0], "count_candidates": stage[1], "compact": stage[2]},
        "stage_gbs": {"accumulate_stats(12d)": 12.0 * d / stage[0] / 1e6,
                      "count_candidates(4d)": 4.0 * d / stage[1] / 1e6,
                      "compact(4d+12nnz)": (4.0 * d + 12 * nnz_mean) / stage[2] / 1e6},
    }

    # ---- cold-L2 variant: a 2 x L2 write between steps, each step timed by its own events
    flush = torch.empty(2 * L2_BYTES // 4, dtype=torch.float32, device=dev)
    cold = []
    for t in range(min(K, 50)):
        flush.fill_(float(t))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); step(t); b.record()
        torch.cuda.synchronize()
        cold.append(a.elapsed_time(b))
    del flush

    # ---- exact Top_k on the same data: operator (given u) and sparsifier (Eq. 2 with Top_k),
    # as one cooperative kernel (path 0) and as histogram passes + look-back compaction (path 1)
    Kt = min(K, 100)
    us = [epss[j] for j in range(min(4, n_eps))]   # residual buffers of the loop above serve as u, in rotation
    tk_idx = torch.empty(k, dtype=torch.int32, device=dev)
    tk_val = torch.empty(k, dtype=torch.float32, device=dev)
    eps2 = torch.zeros_like(epss[0])
    topk = {}
    for path, name in ((0, "fused"), (1, "multi_kernel")):
        gk.gk_set_path(path)
        for t in range(3):
            gk.topk_exact(us[t % len(us)], k, tk_idx, tk_val)
        ms_op = time_region(torch, lambda t: gk.topk_exact(us[t % len(us)], k, tk_idx, tk_val), Kt) / Kt
        eps2.zero_()
        for t in range(3):
            gk.topk_sparsify(gs[t % n_rot], eps2, k, tk_idx, tk_val, nnz)
        ms_sp = time_region(torch, lambda t: gk.topk_sparsify(gs[t % n_rot], eps2, k, tk_idx, tk_val, nnz),
                            Kt) / Kt
        rec = {"topk_exact_ms": ms_op, "topk_sparsify_ms": ms_sp,
               "topk_exact_gbs_12B_per_elem": 12.0 * d / ms_op / 1e6,
               "topk_sparsify_gbs_20B_per_elem": 20.0 * d / ms_sp / 1e6}
        if path == 0:
            gk.gk_stage_timing(True)
            acc_op, acc_sp = np.zeros(8), np.zeros(8)
            for t in range(20):
                gk.topk_exact(us[t % len(us)], k, tk_idx, tk_val)
                acc_op += np.array(gk.gk_last_stage_ms()[:8])
                gk.topk_sparsify(gs[t % n_rot], eps2, k, tk_idx, tk_val, nnz)
                acc_sp += np.array(gk.gk_last_stage_ms()[:8])
            gk.gk_stage_timing(False)
            names = ["kernel", "pass1", "barrier1+digit", "pass2+barrier2+digit", "pass3+barrier3+digit",
                     "count+barrier4", "offsets+emit", "last_cta_exit"]
            rec["phase_ms_operator"] = dict(zip(names, (acc_op / 20).tolist()))
            rec["phase_ms_sparsifier"] = dict(zip(names, (acc_sp / 20).tolist()))
        topk[name] = rec
    gk.gk_set_path(0)
    ms_topk, ms_topk_sp = topk["fused"]["topk_exact_ms"], topk["fused"]["topk_sparsify_ms"]
    # Gaussian_k as an operator on the same given vectors (Fig. 4 compares the operators)
    for t in range(3):
        gk.gk_select(us[t % len(us)], k, idx, val, nnz)
    ms_gk_op = time_region(torch, lambda t: gk.gk_select(us[t % len(us)], k, idx, val, nnz), Kt) / Kt

    # ---- DGC_k (the paper's third operator, Section 4.3: a 1 % sample) on the same data, as
    # operator and as sparsifier; a fresh seeded sample per step, resident on the device
    smps = [torch.from_numpy(wl.sample_positions(d, wl.sample_size(d), step=j)).to(dev) for j in range(4)]
    for t in range(3):
        gk.dgck_select(us[t % len(us)], k, smps[t % 4], tk_idx, tk_val, nnz)
    ms_dg_op = time_region(torch, lambda t: gk.dgck_select(us[t % len(us)], k, smps[t % 4], tk_idx, tk_val, nnz),
                           Kt) / Kt
    eps2.zero_()
    for t in range(3):
        gk.dgck_sparsify(gs[t % n_rot], eps2, k, smps[t % 4], tk_idx, tk_val, nnz)
    ms_dg_sp = time_region(torch, lambda t: gk.dgck_sparsify(gs[t % n_rot], eps2, k, smps[t % 4], tk_idx, tk_val,
                                                             nnz), Kt) / Kt
    gk.gk_stage_timing(True)
    acc_op, acc_sp = np.zeros(8), np.zeros(8)
    for t in range(20):
        gk.dgck_select(us[t % len(us)], k, smps[t % 4], tk_idx, tk_val, nnz)
        acc_op += np.array(gk.gk_last_stage_ms()[:8])
        gk.dgck_sparsify(gs[t % n_rot], eps2, k, smps[t % 4], tk_idx, tk_val, nnz)
        acc_sp += np.array(gk.gk_last_stage_ms()[:8])
    gk.gk_stage_timing(False)
    dg_info = gk.dgck_last_info()
    dg_names = ["kernel", "sample_threshold", "stream", "barrier+count", "second_selection", "count+barrier",
                "offsets+emit", "last_cta_exit"]
    m_s = int(smps[0].numel())
    dgck = {"sample": f"{m_s} positions (1 % of d), uniform with replacement, seeded",
            "dgck_select_ms": ms_dg_op, "dgck_sparsify_ms": ms_dg_sp,
            "dgck_select_gbs_4B_per_elem": (4.0 * d + 32.0 * m_s + 8.0 * k) / ms_dg_op / 1e6,
            "dgck_sparsify_gbs_12B_per_elem": (12.0 * d + 64.0 * m_s + 12.0 * k) / ms_dg_sp / 1e6,
            "vs_gaussiank_sparsify": ms_dg_sp / (ms / K), "vs_topk_sparsify": ms_dg_sp / ms_topk_sp,
            "vs_gaussiank_select": ms_dg_op / ms_gk_op, "vs_topk_exact": ms_dg_op / ms_topk,
            "candidates_last": dg_info[1], "k_m": dg_info[2], "pairs_last": dg_info[3],
            "phase_ms_operator": dict(zip(dg_names, (acc_op / 20).tolist())),
            "phase_ms_sparsifier": dict(zip(dg_names, (acc_sp / 20).tolist())),
            "note": "algorithmic bytes: one pass over the vector (4 d, or 12 d with the add and the store of "
                    "u), one 32-byte sector per sampled position and operand, 8 bytes per pair (+4 per "
                    "cleared slot)"}
    del eps2, us, smps

    # ---- the model update of Eq. 2 from P workers' messages (P workers emulated one after the
    # other on this GPU, each with its own gradient; messages = exact Top_k lists of k pairs)
    upd = {}
    x_model = torch.zeros(d, dtype=torch.float32, device=dev)
    eps4 = torch.zeros_like(epss[0])
    for P_w in (8, 16):
        m_idx = torch.empty(P_w * k, dtype=torch.int32, device=dev)
        m_val = torch.empty(P_w * k, dtype=torch.float32, device=dev)
        m_nnz = torch.zeros(P_w, dtype=torch.int64, device=dev)
        for p_w in range(P_w):
            eps4.zero_()
            gk.topk_sparsify(gs[p_w % n_rot], eps4, k, m_idx[p_w * k:(p_w + 1) * k], m_val[p_w * k:(p_w + 1) * k],
                             m_nnz[p_w:p_w + 1])
        for t in range(3):
            gk.gk_apply_gathered(x_model, m_idx, m_val, m_nnz, k, -0.01 / P_w)
        ms_up = time_region(torch, lambda t: gk.gk_apply_gathered(x_model, m_idx, m_val, m_nnz, k, -0.01 / P_w),
                            Kt) / Kt
        upd[f"P={P_w}"] = {"ms": ms_up, "entries": P_w * k,
                           "entries_per_s": P_w * k / (ms_up * 1e-3),
                           "list_gbs_8B_per_entry": 8.0 * P_w * k / ms_up / 1e6}
        del m_idx, m_val, m_nnz
    upd["note"] = ("gk_apply_gathered: x += alpha * sum_p Comp_k(u^p), rank order, one kernel; messages resident "
                   "(no all-gather in this number)")
    del x_model, eps4

    # ---- the layer-wise (segmented) call on the same data, where the workload has segments:
    # episodes of 4 steps from eps = 0
    seg = None
    if w.partition is not None:
        part = w.partition
        seg = {}
        d_off = torch.from_numpy(part.offsets).to(dev)
        seg_nnz = torch.zeros(part.S, dtype=torch.int64, device=dev)
        eps5 = torch.zeros_like(epss[0])
        gk.gk_reserve(d, part.S)
        for rho_s in ("1e-3", "1e-2"):
            d_k = torch.from_numpy(part.seg_k(*wl.RHO[rho_s])).to(dev)

            def seg_step(t, d_k=d_k):
                gk.gk_sparsify_segmented(gs[t % n_rot], eps5, d_off, d_k, idx, val, seg_nnz, nnz)

            eps5.zero_()
            for t in range(4):
                seg_step(t)
            ms_seg, n_seg = 0.0, 0
            for e in range(10):
                eps5.zero_()
                ms_seg += time_region(torch, seg_step, 4)
                n_seg += 4
            ms_seg /= n_seg
            nz = float(nnz.item())
            seg[f"rho={rho_s}"] = {"ms": ms_seg, "nnz_last": nz, "gbs": algorithmic_bytes(d, nz) / ms_seg / 1e6,
                                   "frac_of_measured_hbm": algorithmic_bytes(d, nz) / ms_seg / 1e6 / peak}
        seg["segments"] = part.S
        seg["call"] = "gk_sparsify_segmented, one cooperative kernel, k_s = ceil(rho * d_s)"
        del eps5

    # ---- the error ratio of Eq. 5 for one Gaussian_k step and one Top_k step from eps = 0
    diag = {"bound_eq4_1_minus_k_over_d": 1.0 - k / d, "bound_theorem1_squared": (1.0 - k / d) ** 2}
    eps3 = torch.zeros_like(epss[0])
    for name, fn in (("gaussiank", gk.gk_sparsify), ("topk", gk.topk_sparsify)):
        eps3.zero_()
        fn(gs[0], eps3, k, idx, val, nnz)
        gk.gk_stage_timing(True)
        acc = 0.0
        for _ in range(10):
            r = gk.gk_error_ratio(eps3, val, nnz)
            acc += gk.gk_last_stage_ms()[0]
        gk.gk_stage_timing(False)
        diag[name] = {"error_ratio": r[0], "nnz": int(nnz.item()), "ms": acc / 10,
                      "gbs_4B_per_elem": 4.0 * d / (acc / 10) / 1e6}
    # the histogram of u (Section 3.1): 512 bins over +-4 sigma of one step's u (eps3 holds it, minus
    # the selected entries)
    hcnt = torch.zeros(514, dtype=torch.int64, device=dev)
    sig = float(eps3[:1_000_000].std().item()) or 1.0
    for _ in range(3):
        gk.gk_histogram(eps3, -4 * sig, 512 / (8 * sig), hcnt)
    ms_h = time_region(torch, lambda t: gk.gk_histogram(eps3, -4 * sig, 512 / (8 * sig), hcnt), 20) / 20
    diag["histogram"] = {"bins": 512, "ms": ms_h, "gbs_4B_per_elem": 4.0 * d / ms_h / 1e6,
                         "inside": int(hcnt[1:-1].sum().item()), "outside": int(hcnt[0].item() + hcnt[-1].item())}
    del eps3, hcnt

    # ---- end to end through the host-buffer entry point (pinned host memory)
    hg = [torch.from_numpy(w.grad(j, None)).pin_memory() for j in range(2)]
    heps = torch.zeros(d, dtype=torch.float32).pin_memory()
    hidx = torch.empty(d, dtype=torch.int32).pin_memory()
    hval = torch.empty(d, dtype=torch.float32).pin_memory()
    Ke = max(3, min(K, 20))
    for t in range(2):
        gk.gk_sparsify_host(hg[t % 2], heps, k, hidx, hval)
    t0 = time.perf_counter()
    e_nnz = 0
    for t in range(Ke):
        n, _ = gk.gk_sparsify_host(hg[t % 2], heps, k, hidx, hval)
        e_nnz += n
    e_s = (time.perf_counter() - t0) / Ke
    e_nnz /= Ke
    e2e = {"value": algorithmic_bytes(d, e_nnz) / e_s / 1e9, "unit": UNIT,
           "h2d_bytes_per_step": 8 * d, "d2h_bytes_per_step": int(4 * d + 8 * e_nnz + 8 + 96),
           "ms_per_step": e_s * 1e3, "steps": Ke,
           "call": "gk_sparsify_host (pinned host g, eps, idx, val; copies inside the call)"}
    del hg, heps, hidx, hval

    # ---- CPU oracle on a bounded sample of the same workload (~10-30 s on one core)
    cpu_steps = 16
    cpu_gbs, cpu_s, _ = cpu_oracle_rate(w, rho, cpu_steps)
    cpu = {"value": cpu_gbs, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"{cpu_steps} full steps of the workload, single thread ({cpu_s * 1e3:.0f} ms/step); "
                     f"host has {os.cpu_count()} cores"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "repeats": len(regions), "steps_per_s": K / (ms * 1e-3) * world,
        "gbs_at_20_bytes_per_element": whole_job_gbs(world, algorithmic_bytes(d, nnz_mean, 1.0), K, ms),
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": workload_string(w, rho),
            "l2": f"inputs per step g+eps = {8 * d / 1e6:.0f} MB > {L2_BYTES / 1e6:.0f} MB L2; "
                  f"{n_rot} gradient buffers in rotation, {n_eps} residual buffers for the {episodes} episodes of "
                  f"{EPISODE} steps of a region, every episode from eps = 0 (buffers zeroed before each region, "
                  f"outside the timing); no flush in the headline loop",
            "path": "fused cooperative kernel (1 launch per step)",
            "bytes_per_step": bytes_step, "nnz_last_step": nnz_mean,
            "bytes_model": f"(16 + 4 r) d + 12 nnz, r = {r_passes:g} count passes over u in the last step",
            "counting": {"ctas": info[4], "ctas_with_prediction": info[0], "ctas_whose_bands_held": info[1],
                         "second_full_count": info[2], "cells_left_to_second_phase": info[3],
                         "ctas_that_counted_a_selection": info[5],
                         "cells": (d // 4096) * 32},
            "timed": f"{len(regions)} repeats of the {K}-step region, median reported "
                     f"(min {min(regions) / K * 1e3:.2f} us, max {max(regions) / K * 1e3:.2f} us per step)",
            "parallelism": "replicas only" if world > 1 else "single GPU",
        },
        "pct_of_hbm_peak": {"measured_copy": value / world / peak, "nominal_8TBs": value / world / 8000.0},
        "elements_per_s": world * d * K / (ms * 1e-3),
        "roofline": roof, "three_kernel_path": three,
        "cold_l2": {"ms_per_step": statistics.median(cold), "gbs": bytes_step / statistics.median(cold) / 1e6,
                    "note": "256 MB written between steps; per-step CUDA events"},
        "topk": {"topk_exact_ms": ms_topk, "topk_sparsify_ms": ms_topk_sp, "gaussiank_select_ms": ms_gk_op,
                 "speedup_operator": ms_topk / ms_gk_op,
                 "speedup_sparsifier": ms_topk_sp / (ms / K),
                 "note": "operator against operator (gk_select vs topk_exact on a given u, the comparison of "
                         "Fig. 4) and sparsifier against sparsifier (gk_sparsify vs topk_sparsify)",
                 "fused": topk["fused"], "multi_kernel": topk["multi_kernel"],
                 "paper_context": "paper: exact Top_k 0.4 s at this d on one V100 (Section 3.3)"},
        "segmented": seg, "dgck": dgck, "update_from_messages": upd, "diagnostics": diag, "e2e": e2e, "cpu_baseline": cpu, "gpu_launches": int(launches),
        "clocks": sampler.summary(),
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Every workload family at 1 GPU: Gaussian_k (fused kernel), the segmented call where the
    workload has segments, and exact Top_k, each timed with CUDA events over a few EC steps
    with fresh gradients; one JSON object per line on stdout."""
    import torch

    from paper_1911_08772_b200 import binding as gk
    from paper_1911_08772_b200 import build as lib_build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    lib_build.build()
    gk.load()
    peak, peak_src = measured_peaks()
    points = [(wl.resnet20_normal(), ["1e-3"]), (wl.vgg16_laplace_mixture(), ["1e-3"]),
              (wl.resnet50_segmented(), ["1e-3", "1e-2"]), (wl.lstm_student_t(), ["1e-3", "5e-3"])]
    for lg in (20, 22, 24, 26, 28):
        for dist in ("normal", "laplace"):
            points.append((wl.sweep_point(1 << lg, dist), ["1e-4", "1e-3", "1e-2"]))
    n_grad = 4
    for w, rhos in points:
        d = w.d
        gs = [torch.from_numpy(w.grad(j, None)).to(dev) for j in range(n_grad)]
        eps = torch.zeros(d, dtype=torch.float32, device=dev)
        idx = torch.empty(d, dtype=torch.int32, device=dev)
        val = torch.empty(d, dtype=torch.float32, device=dev)
        nnz = torch.zeros(1, dtype=torch.int64, device=dev)
        gk.gk_reserve(d, 161)
        reps = 40 if d <= (1 << 26) else 12
        for rho in rhos:
            k = w.k(rho)

            def timed(fn):
                # EC episodes of n_grad steps from eps = 0, as many as fit `reps` steps
                for t in range(3):
                    fn(t)
                ms = 0.0
                for e in range(max(1, reps // n_grad)):
                    eps.zero_()
                    ms += time_region(torch, fn, n_grad)
                return ms / (max(1, reps // n_grad) * n_grad)

            ms_gk = timed(lambda t: gk.gk_sparsify(gs[t % n_grad], eps, k, idx, val, nnz))
            n_gk = int(nnz.item())
            st = gk.gk_last_stats()
            rec = {"workload": w.name, "d": d, "rho": rho, "k": k, "gaussiank_ms": ms_gk,
                   "gaussiank_gbs": algorithmic_bytes(d, n_gk) / ms_gk / 1e6,
                   "gaussiank_elements_per_s": d / (ms_gk * 1e-3),
                   "frac_of_measured_hbm": algorithmic_bytes(d, n_gk) / ms_gk / 1e6 / peak,
                   "frac_of_nominal_8TBs": algorithmic_bytes(d, n_gk) / ms_gk / 1e6 / 8000.0,
                   "nnz_last": n_gk, "rounds_last": st.rounds}
            if w.partition is not None:
                part = w.partition
                off = torch.from_numpy(part.offsets).to(dev)
                sk = torch.from_numpy(part.seg_k(*wl.RHO[rho])).to(dev)
                snn = torch.zeros(part.S, dtype=torch.int64, device=dev)
                ms_seg = timed(lambda t: gk.gk_sparsify_segmented(gs[t % n_grad], eps, off, sk, idx, val, snn, nnz))
                rec["segmented_ms"] = ms_seg
                rec["segmented_gbs"] = algorithmic_bytes(d, int(nnz.item())) / ms_seg / 1e6
            u = gs[0]
            for _ in range(3):
                gk.gk_select(u, k, idx, val, nnz)
            ms_gko = time_region(torch, lambda t: gk.gk_select(u, k, idx, val, nnz), 10) / 10
            rec["gaussiank_select_ms"] = ms_gko
            tk_i = torch.empty(k, dtype=torch.int32, device=dev)
            tk_v = torch.empty(k, dtype=torch.float32, device=dev)
            for _ in range(3):
                gk.topk_exact(u, k, tk_i, tk_v)
            ms_tk = time_region(torch, lambda t: gk.topk_exact(u, k, tk_i, tk_v), 10) / 10
            ms_tks = timed(lambda t: gk.topk_sparsify(gs[t % n_grad], eps, k, tk_i, tk_v, nnz))
            smp = torch.from_numpy(wl.sample_positions(d, wl.sample_size(d), step=0)).to(dev)
            for _ in range(3):
                gk.dgck_select(u, k, smp, tk_i, tk_v, nnz)
            ms_dg = time_region(torch, lambda t: gk.dgck_select(u, k, smp, tk_i, tk_v, nnz), 10) / 10
            ms_dgs = timed(lambda t: gk.dgck_sparsify(gs[t % n_grad], eps, k, smp, tk_i, tk_v, nnz))
            rec.update({"topk_exact_ms": ms_tk, "topk_sparsify_ms": ms_tks,
                        "speedup_vs_topk_sparsify": ms_tks / ms_gk,
                        "speedup_select_vs_topk_exact": ms_tk / ms_gko,
                        "topk_exact_gbs_12B_per_elem": 12.0 * d / ms_tk / 1e6,
                        "dgck_select_ms": ms_dg, "dgck_sparsify_ms": ms_dgs,
                        "dgck_candidates_last": gk.dgck_last_info()[1]})
            print(json.dumps(rec), flush=True)
        del gs, eps, idx, val
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50")
    ap.add_argument("--path", type=int, default=0, choices=[0, 1],
                    help="0: fused cooperative kernel, 1: three kernels with look-back")
    ap.add_argument("--rotate", type=int, default=0,
                    help="number of gradient buffers kept on the device (default 20; small for captures)")
    ap.add_argument("--repeats", type=int, default=0,
                    help="times the timed K-step region is run (0: until about 0.3 s have been timed)")
    ap.add_argument("--loop-only", action="store_true",
                    help="run only warm-up and the timed loop (for profiler captures)")
    ap.add_argument("--call", default="gk", choices=["gk", "gk_select", "segmented", "topk_exact", "topk_sparsify", "dgck_select", "dgck_sparsify"],
                    help="entry point the timed loop calls (other than gk: with --loop-only, for captures)")
    ap.add_argument("--sweep", action="store_true",
                    help="time every workload family (Gaussian_k, segmented, exact Top_k) and print one line each")
    args = ap.parse_args()
    if args.call != "gk" and not args.loop_only:
        ap.error("--call other than gk needs --loop-only")
    if args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
