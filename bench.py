#!/usr/bin/env python
"""Benchmark of the distance-transform hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl ours|reference]

A step is one full transform (every pass plus the fused epilogue) of one seeded synthetic workload.
Prints ONE JSON line.  `value` is Gvoxel/s with the mask already resident in device memory; `e2e` is
the same metric through the host-buffer entry point (pinned host memory, copies inside the timed
region).  With N > 1 (torchrun) every rank transforms its own copy of the workload on its own GPU --
the images of a batch are independent, so there is no data-path collective -- and the time is the
maximum over ranks.  `--impl reference` times the CPU oracle instead (a deliberately plain program).
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import sys
import threading
import time
import zlib

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "edt_gvoxels_per_s"
UNIT = "Gvoxel/s"
NOMINAL_HBM_GBS = 8000.0  # HBM3e figure of the part's data sheet, reported beside the measured copy bandwidth
_L2_FALLBACK = 126 * 1024 * 1024


def l2_bytes(dev=None) -> int:
    """L2 size of the device, read from its properties."""
    try:
        import torch

        return int(torch.cuda.get_device_properties(dev if dev is not None else torch.cuda.current_device()).L2_cache_size)
    except Exception:
        return _L2_FALLBACK
REASON_BITS = {
    0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
    0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
    0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
}


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, torch_device_index: int, period_s: float = 0.01):
        self.period = period_s
        self.samples = []
        self._stop = threading.Event()
        self._thread = None
        self.ok = False
        self.max_mhz = None
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as exc:  # pragma: no cover - depends on the box
            self.err = repr(exc)

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    rs = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    rs = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                self.samples.append((time.perf_counter(), mhz, rs))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.ok:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self, t0: float, t1: float):
        if not self.ok:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable"}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        if not inside and self.samples:  # region shorter than a sampling period: nearest samples
            inside = sorted(self.samples, key=lambda s: abs(s[0] - 0.5 * (t0 + t1)))[:3]
        bits = 0
        for s in inside:
            bits |= s[2]
        reasons = [name for bit, name in REASON_BITS.items() if bits & bit and name != "gpu_idle"]
        return {
            "sm_mhz": statistics.median([s[1] for s in inside]) if inside else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": reasons,
            "samples": len(inside),
        }


def dist_env():
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Largest `value` over all ranks (the process group must exist when world > 1)."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist

    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, seconds_max: float) -> float:
    """Aggregate rate of a weak-scaling job: every rank did `units_per_rank` in at most `seconds_max`."""
    return units_per_rank * world / seconds_max


def sample_images(w, max_voxels: int):
    """First images of the workload, as many as fit in max_voxels (at least one)."""
    B, C = w.mask.shape[:2]
    per = w.voxels // (B * C)
    flat = w.mask.reshape((B * C, 1) + w.mask.shape[2:])
    k = max(1, min(B * C, max_voxels // per))
    return flat[:k], k, B * C


def time_oracle(w, max_voxels: int, repeats: int = 1, threads: int = 0):
    """The oracle on the first images of the workload; threads = 0 keeps its own thread count (all cores)."""
    import oracle

    sub, k, total = sample_images(w, max_voxels)
    before = oracle.threads()
    if threads > 0:
        oracle.set_threads(threads)
    try:
        used = oracle.threads()
        best = None
        for _ in range(repeats):
            t0 = time.perf_counter()
            oracle.sep(sub, w.sampling, want_idx=w.want_idx)
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
    finally:
        if threads > 0:
            oracle.set_threads(before)
    what = "%d of %d images (%d voxels), full oracle incl. index decode" % (k, total, sub.size)
    if sub.shape[2:] != w.mask.shape[2:]:
        what = "part of one image (%d voxels)" % sub.size
    return sub.size / best / 1e9, best, what, used


def time_oracle_single_thread(w, seconds_all_cores: float, voxels_all_cores: int, cores: int):
    """One oracle thread (the protocol of the paper's CPU column) on a sample sized for about ten seconds."""
    per_voxel = seconds_all_cores * max(cores, 1) / max(voxels_all_cores, 1)
    want = int(10.0 / max(per_voxel, 1e-12))
    one = w.voxels // (w.mask.shape[0] * w.mask.shape[1])
    if want >= one:
        return time_oracle(w, want, threads=1)
    # less than one image: the leading slices of the first image along spatial axis 0
    import copy

    keep = max(2, int(w.mask.shape[2] * want / one))
    part = copy.copy(w)
    part.mask = np.ascontiguousarray(w.mask.reshape((-1, 1) + w.mask.shape[2:])[:1, :, :keep])
    return time_oracle(part, part.mask.size, threads=1)


def run_reference(args, w, world, rank):
    """The CPU oracle as the reference arm: rank 0 only, bounded sample per step."""
    if rank != 0:
        return
    import oracle

    # size the per-step sample so that the whole run stays near a minute
    one, _, total = sample_images(w, 1)
    t0 = time.perf_counter()
    oracle.sep(one, w.sampling, want_idx=w.want_idx)
    t_img = max(time.perf_counter() - t0, 1e-6)
    budget_imgs = int(60.0 / (args.steps + args.warmup) / t_img)
    sub, k, total = sample_images(w, min(args.ref_voxels, max(1, budget_imgs) * one.size))
    what = "%d of %d images per step" % (k, total)
    if budget_imgs < 1 and sub.shape[2] > 2:
        # even one image per step would run for minutes: take the leading part of its first spatial axis
        keep = max(2, int(sub.shape[2] * 90.0 / ((args.steps + args.warmup) * t_img)))
        if keep < sub.shape[2]:
            sub = np.ascontiguousarray(sub[:, :, :keep])
            what = "first %d of %d slices along spatial axis 0 of one image per step" % (keep, w.mask.shape[2])
    for _ in range(args.warmup):
        oracle.sep(sub, w.sampling, want_idx=w.want_idx)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.sep(sub, w.sampling, want_idx=w.want_idx)
    dt = time.perf_counter() - t0
    val = sub.size * args.steps / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64" if w.sampling is not None else "int64", "data": "synthetic",
        "config": {"workload": w.name, "voxels_per_step": int(sub.size)},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": what},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def load_traffic(workload_number: int, kernel_label: str = None):
    """DRAM bytes per launch from the committed ncu summary (profiles/traffic.txt): of one kernel, or -- without a
    kernel label -- summed over all kernels of the workload's path.  None if the summary has no such line."""
    try:
        total, found = 0, False
        name = kernel_label.split(":", 1)[1] if kernel_label else None
        with open(os.path.join(ROOT, "profiles", "traffic.txt")) as fh:
            for line in fh:
                parts = line.split()
                if len(parts) == 3 and parts[0] == "C%d" % workload_number and (name is None or parts[1] == name):
                    total += int(parts[2])
                    found = True
        return total if found else None
    except Exception:
        return None


def measure_device(w, steps, warmup, profile_steps, dev, world, sampler=None):
    """Device-timed throughput of one workload plus per-kernel event times (inputs resident in HBM)."""
    import torch

    from paper_2608_24738_b200 import binding

    # buffers: rotate over enough independent sets that one lap exceeds twice the L2
    io = w.io_bytes()
    sets = max(2, min(16, -(-2 * l2_bytes(dev) // io)))
    host_mask = torch.from_numpy(w.mask)
    shape = tuple(w.mask.shape)
    calls = []
    for _ in range(sets):
        m = host_mask.to(dev)
        d = torch.empty(shape, dtype=torch.float32, device=dev) if w.want_dist else None
        s = torch.empty(shape, dtype=torch.int64, device=dev) if w.want_sq else None
        xshape = shape if w.flat_index else shape[:2] + (w.ndim,) + shape[2:]
        x = torch.empty(xshape, dtype=torch.int64, device=dev) if w.want_idx else None
        calls.append(binding.PreparedCall(m, w.sampling, d, s, x, flags=binding.FLAG_FLAT_INDEX if w.flat_index else 0))
    stream = torch.cuda.current_stream()
    sp = ctypes.c_void_p(stream.cuda_stream)
    for i in range(warmup):
        calls[i % sets](sp)
    launches_per_step = binding.tm_edt_last_launch_count()
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist

        dist.barrier()
        torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    ev0.record(stream)
    for i in range(steps):
        calls[i % sets](sp)
    ev1.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
        torch.cuda.synchronize()
    t1 = time.perf_counter()
    seconds = max_over_ranks(ev0.elapsed_time(ev1) / 1e3, world, dev)
    clocks = sampler.summary(t0, t1) if sampler is not None else None
    value = whole_job_rate(w.voxels * steps, world, seconds) / 1e9

    # every repetition timed by itself (rotating buffers: cold L2), then one buffer set over and over (warm L2)
    def each(reps, pick):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for i, (a, b) in enumerate(evs):
            a.record(stream)
            calls[pick(i)](sp)
            b.record(stream)
        torch.cuda.synchronize()
        return sorted(a.elapsed_time(b) for a, b in evs)
    reps = max(30, min(steps, 200))
    cold = each(reps, lambda i: i % sets)
    each(3, lambda i: 0)
    warm = each(reps, lambda i: 0)
    spread = {"repetitions": reps, "ms_median": statistics.median(cold), "ms_min": cold[0],
              "warm_l2_ms_median": statistics.median(warm), "warm_l2_ms_min": warm[0],
              "note": "each repetition between its own pair of events; warm = the same buffer set every time"}

    # per-kernel times (events between launches), same buffers, right after the timed region
    ksum, korder = {}, []
    for i in range(max(1, profile_steps)):
        c = calls[i % sets]
        _, ks = binding.tm_edt_profile(c.mask, w.sampling, distances=c.d, sqdist=c.s, indices=c.x, workspace=c.ws,
                                       return_distances=w.want_dist, return_sqdist=w.want_sq,
                                       return_indices=w.want_idx, flags=c.flags)
        for j, (name, ms, nbytes) in enumerate(ks):
            key = (j, name)
            if key not in ksum:
                ksum[key] = [0.0, nbytes, 0]
                korder.append(key)
            ksum[key][0] += ms
            ksum[key][2] += 1
    peak, peak_kind = measured_peak_gbs()
    kernels = []
    for key in korder:
        tot, nbytes, cnt = ksum[key]
        avg_ms = tot / cnt
        kernels.append({"kernel": "%d:%s" % key, "avg_ms": avg_ms, "bytes": nbytes,
                        "gbs": nbytes / (avg_ms * 1e-3) / 1e9 if avg_ms > 0 else None})
    dom = max(kernels, key=lambda k: k["avg_ms"])
    # Roofline of the path: the bytes the method cannot avoid (mask in, requested outputs out) over the time of one
    # whole transform, against the measured copy bandwidth; the kernel with the largest share is reported beside it
    # with the same algorithmic bytes over its own duration and with its own compulsory bytes (inputs + outputs of
    # that launch, intermediates included).
    path_gbs = io * steps * 1.0 / seconds / 1e9
    traffic = load_traffic(w.number)
    roofline = {
        "bound": "hbm", "achieved": path_gbs, "peak": peak, "unit": "GB/s", "frac": path_gbs / peak,
        "peak_kind": peak_kind + " copy bandwidth", "frac_of_nominal_8TBs": path_gbs / NOMINAL_HBM_GBS,
        "algorithmic_bytes_per_step": io, "bytes_per_voxel": io / w.voxels,
        "traffic": traffic, "traffic_over_algorithmic": (traffic / io) if traffic else None,
        "traffic_kind": "dram read + write bytes of every kernel of the path, ncu (profiles/traffic.txt)",
        "dominant": {"kernel": dom["kernel"], "avg_ms": dom["avg_ms"], "share": dom["avg_ms"] / sum(k["avg_ms"] for k in kernels),
                     "algorithmic_gbs": io / (dom["avg_ms"] * 1e-3) / 1e9, "algorithmic_frac": io / (dom["avg_ms"] * 1e-3) / 1e9 / peak,
                     "own_bytes": dom["bytes"], "own_gbs": dom["gbs"], "own_frac": dom["gbs"] / peak,
                     "traffic": load_traffic(w.number, dom["kernel"])},
        "kernels": kernels,
    }
    del calls
    torch.cuda.empty_cache()
    return {"io": io, "shape": shape, "host_mask": host_mask, "value": value, "seconds": seconds, "clocks": clocks,
            "roofline": roofline, "launches_per_step": launches_per_step, "sets": sets, "spread": spread}


MORPH_CASES = {
    # name: (image shape (B, C, spatial...), element shape, kind); sizes follow the paper's morphology table (2-D 256^2
    # and 1024^2 images, batched) plus one 3-D volume; inputs are larger than L2 or rotated over several buffer sets
    "grey_erosion_2d_1024": ((64, 1, 1024, 1024), (3, 3), "grey"),
    "grey_dilation_2d_1024": ((64, 1, 1024, 1024), (3, 3), "grey_dilation"),
    "grey_erosion_2d_256": ((512, 1, 256, 256), (3, 3), "grey"),
    "grey_erosion_3d_256": ((4, 1, 256, 256, 256), (3, 3, 3), "grey"),
    "binary_erosion_2d_1024": ((64, 1, 1024, 1024), (3, 3), "binary"),
    "binary_dilation_2d_1024": ((64, 1, 1024, 1024), (3, 3), "binary_dilation"),
}


def run_morph(args):
    """Measurement of the fused erosion / dilation kernel (a later row of the scope, not the headline metric):
    one JSON line with throughput in Gvoxel/s per case, the fraction of the HBM roofline (unavoidable bytes: input +
    output once) and the numpy oracle timed on a bounded sample."""
    import numpy as np
    import torch

    from oracle import morph_oracle as mo
    from paper_2608_24738_b200 import binding, buildlib

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    buildlib.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peak_gbs()
    peak_kind += " copy bandwidth"
    stream = torch.cuda.current_stream()
    cases = []
    for name, (shape, fps, kind) in MORPH_CASES.items():
        if args.morph_case and name != args.morph_case:
            continue
        rng = np.random.default_rng(zlib.crc32(name.encode()))
        binary = kind.startswith("binary")
        fp = np.ones(fps, dtype=bool)
        per_voxel = 2 if binary else 8
        nvox = int(np.prod(shape))
        sets = max(2, -(-2 * l2_bytes(dev) // (nvox * per_voxel)))
        if binary:
            ins = [torch.from_numpy((rng.random(shape) < 0.8).astype(np.uint8)).to(dev) for _ in range(sets)]
        else:
            ins = [torch.from_numpy(rng.normal(size=shape).astype(np.float32)).to(dev) for _ in range(sets)]
        outs = [torch.empty_like(t) for t in ins]
        op = "dilation" if kind.endswith("dilation") else "erosion"
        # arguments marshalled once per buffer set: the loop below only enqueues
        prepared = [binding.PreparedMorph(ins[i], fp, None, op=op, mode="reflect", out=outs[i]) for i in range(sets)]
        sp = ctypes.c_void_p(stream.cuda_stream)
        call = lambda i: prepared[i](sp)
        for i in range(max(3, args.warmup)):
            call(i % sets)
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        steps = max(10, args.steps // 4)
        ev0.record(stream)
        for i in range(steps):
            call(i % sets)
        ev1.record(stream)
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1) / steps
        gbs = nvox * per_voxel / (ms * 1e-3) / 1e9
        # the oracle on one image of the same workload
        one = ins[0][:1].cpu().numpy()
        t0 = time.perf_counter()
        (mo.binary_erosion(one, fp) if binary else mo.grey_erosion(one, fp, None, "reflect")) if op == "erosion" else (
            mo.binary_dilation(one, fp) if binary else mo.grey_dilation(one, fp, None, "reflect"))
        cpu_s = time.perf_counter() - t0
        cases.append({"case": name, "shape": list(shape), "element": list(fps), "ms_per_step": ms,
                      "value": nvox / (ms * 1e-3) / 1e9, "unit": "Gvoxel/s", "inputs_per_ms": shape[0] * shape[1] / ms,
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                                   "peak_kind": peak_kind, "bytes_per_voxel": per_voxel},
                      "cpu_baseline": {"value": one.size / cpu_s / 1e9, "unit": "Gvoxel/s", "cores": 1, "kind": "oracle",
                                       "sample": "1 image"},
                      "l2": "rotating %d buffer sets" % sets})
    head = cases[0]
    print(json.dumps({"metric": "morph_gvoxels_per_s", "value": head["value"], "unit": "Gvoxel/s", "n_gpus": 1,
                      "steps": max(10, args.steps // 4), "warmup": max(3, args.warmup), "ms_per_step": head["ms_per_step"],
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": head["case"], "shape": head["shape"], "element": head["element"]},
                      "gpu_launches": max(10, args.steps // 4), "roofline": head["roofline"],
                      "cpu_baseline": head["cpu_baseline"], "cases": cases}), flush=True)


def run_cdt(args):
    """Measurement of tm_cdt and tm_bfdt (later rows of the scope, their own metric): disks as in workload C2 at the
    paper's 2-D sizes; HBM roofline = mask in + int32 out once (5 B/voxel); the brute-force transform is quadratic and
    reported in voxel-site pairs per second."""
    import numpy as np
    import torch

    from oracle import cdt_oracle as co
    from paper_2608_24738_b200 import binding, buildlib, workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    buildlib.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peak_gbs()
    peak_kind += " copy bandwidth"
    stream = torch.cuda.current_stream()
    steps = max(10, args.steps // 4)

    def timed(call, sets):
        for i in range(max(3, args.warmup)):
            call(i % sets)
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for i in range(steps):
            call(i % sets)
        ev1.record(stream)
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1) / steps

    cases = []
    for size, batch in ((1024, 64), (256, 512)):
        base = workloads.config2(batch=8, size=size, disks=20 * (size // 512) ** 2 if size >= 512 else 5).mask
        mask = np.concatenate([base] * (batch // 8), axis=0)
        nvox = mask.size
        sets = max(2, -(-2 * l2_bytes(dev) // (nvox * 5)))
        ins = [torch.from_numpy(mask).to(dev) for _ in range(sets)]
        outs = [torch.empty(mask.shape, dtype=torch.int32, device=dev) for _ in range(sets)]
        for metric in ("chessboard", "taxicab"):
            ms = timed(lambda i: binding.tm_cdt(ins[i], metric, out=outs[i]), sets)
            t0 = time.perf_counter()
            co.separable(mask[:1], metric)
            cpu_s = time.perf_counter() - t0
            gbs = nvox * 5 / (ms * 1e-3) / 1e9
            cases.append({"case": "cdt_%s_2d_%d" % (metric, size), "shape": list(mask.shape), "ms_per_step": ms,
                          "value": nvox / (ms * 1e-3) / 1e9, "unit": "Gvoxel/s", "inputs_per_ms": batch / ms,
                          "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                                       "peak_kind": peak_kind, "bytes_per_voxel": 5},
                          "cpu_baseline": {"value": mask[:1].size / cpu_s / 1e9, "unit": "Gvoxel/s", "cores": 1,
                                           "kind": "oracle", "sample": "1 image"},
                          "l2": "rotating %d buffer sets" % sets})
    # brute force: 64 images of 128^2 (about 6000 background voxels each)
    bmask = workloads.config2(batch=64, size=128, disks=6).mask
    t = torch.from_numpy(bmask).to(dev)
    o = torch.empty(bmask.shape, dtype=torch.float32, device=dev)
    sites = int((bmask == 0).sum()) // bmask.shape[0]
    for metric in ("euclidean", "chessboard"):
        ms = timed(lambda i: binding.tm_bfdt(t, None, metric, out=o), 1)
        pairs = bmask.size * sites
        cases.append({"case": "bfdt_%s_2d_128" % metric, "shape": list(bmask.shape), "ms_per_step": ms,
                      "value": bmask.size / (ms * 1e-3) / 1e9, "unit": "Gvoxel/s", "inputs_per_ms": bmask.shape[0] / ms,
                      "pairs_per_s": pairs / (ms * 1e-3), "background_voxels_per_image": sites})
    head = cases[0]
    print(json.dumps({"metric": "cdt_gvoxels_per_s", "value": head["value"], "unit": "Gvoxel/s", "n_gpus": 1, "steps": steps,
                      "warmup": max(3, args.warmup), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
                      "config": {"workload": head["case"], "shape": head["shape"]}, "gpu_launches": 2 * steps,
                      "roofline": head["roofline"], "cpu_baseline": head["cpu_baseline"], "cases": cases}), flush=True)


def run_ex(args):
    """Measurement of the tm_edt_ex variants (a later row of the scope): flat index output on workload C4, float64
    distances, a strided (z-fastest) mask gathered by the library and the virtual-background convention on workload
    C3, each beside the default call on the same mask.  HBM roofline = the unavoidable bytes of the variant."""
    import numpy as np
    import torch

    from paper_2608_24738_b200 import binding, buildlib, workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    buildlib.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peak_gbs()
    stream = torch.cuda.current_stream()
    steps = max(20, args.steps // 2)

    def timed(call):
        for _ in range(max(3, args.warmup)):
            call()
        torch.cuda.synchronize()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in evs:
            a.record(stream)
            call()
            b.record(stream)
        torch.cuda.synchronize()
        return statistics.median(a.elapsed_time(b) for a, b in evs)

    c3, c4 = workloads.config3(), workloads.config4()
    m3, m4 = torch.from_numpy(c3.mask).to(dev), torch.from_numpy(c4.mask).to(dev)
    n3, n4 = c3.mask.size, c4.mask.size
    cases = []

    def add(name, mask_t, nvox, bpv, ms, base_ms, note):
        gbs = nvox * bpv / (ms * 1e-3) / 1e9
        cases.append({"case": name, "shape": list(mask_t.shape), "ms_per_step": ms, "default_call_ms": base_ms,
                      "value": nvox / (ms * 1e-3) / 1e9, "unit": "Gvoxel/s", "note": note,
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                                   "peak_kind": peak_kind + " copy bandwidth", "bytes_per_voxel": bpv}})

    # workload C4: coordinate planes (the default) against one linear index per voxel
    d4 = torch.empty(c4.mask.shape, dtype=torch.float32, device=dev)
    x4 = torch.empty(c4.mask.shape[:2] + (4,) + c4.mask.shape[2:], dtype=torch.int64, device=dev)
    f4 = torch.empty(c4.mask.shape, dtype=torch.int64, device=dev)
    base4 = timed(lambda: binding.tm_edt(m4, None, distances=d4, indices=x4, return_indices=True))
    ms = timed(lambda: binding.tm_edt(m4, None, distances=d4, indices=f4, return_indices=True, flat_index=True))
    add("c4_flat_index", m4, n4, 13, ms, base4, "dist f32 + one int64 linear index per voxel")
    del x4, f4
    # workload C3: float64 distances, a z-fastest mask, the virtual-background convention
    d3 = torch.empty(c3.mask.shape, dtype=torch.float32, device=dev)
    base3 = timed(lambda: binding.tm_edt(m3, c3.sampling, distances=d3))
    d64 = torch.empty(c3.mask.shape, dtype=torch.float64, device=dev)
    ms = timed(lambda: binding.tm_edt(m3, c3.sampling, distances=d64, dist_f64=True))
    add("c3_dist_f64", m3, n3, 9, ms, base3, "float64 distances recomputed from the sites")
    zfast = m3.permute(0, 1, 4, 3, 2).contiguous().permute(0, 1, 4, 3, 2)  # same values, z varies fastest in memory
    ms = timed(lambda: binding.tm_edt(zfast, c3.sampling, distances=d3, keep_strides=True))
    add("c3_strided_z_fastest", m3, n3, 5, ms, base3, "byte strides passed, gathered by the library")
    vb = m3.clone()
    vb[-1, -1] = 1  # one image without background
    ms = timed(lambda: binding.tm_edt(vb, c3.sampling, distances=d3, virtual_background=True))
    add("c3_virtual_background", m3, n3, 5, ms, base3, "one of 16 images without background")
    head = cases[0]
    print(json.dumps({"metric": "edt_ex_gvoxels_per_s", "value": head["value"], "unit": "Gvoxel/s", "n_gpus": 1,
                      "steps": steps, "warmup": max(3, args.warmup), "ms_per_step": head["ms_per_step"],
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": head["case"], "shape": head["shape"]}, "gpu_launches": binding.tm_edt_last_launch_count() * steps,
                      "roofline": head["roofline"], "cases": cases}), flush=True)


def run_long(args):
    """Measurement of the paths for extents beyond 128 (wide-key and long-line kernels; a later row of the scope, its
    own line): the paper's 2-D 1024^2 row at B = 8, one 4096^2 image and one 512^3 volume; blob masks (disks / balls as
    in workload C2, radii 0.02 .. 0.12 of the extent), unit sampling (and one case with decimal sampling), float32 distances.  HBM roofline = mask in +
    distances out once (5 B/voxel); the oracle is timed on a bounded sample of each case."""
    import numpy as np
    import torch

    import oracle
    from paper_2608_24738_b200 import binding, buildlib, workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    buildlib.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peak_gbs()
    stream = torch.cuda.current_stream()
    sp = ctypes.c_void_p(stream.cuda_stream)
    steps = max(30, args.steps // 4)

    def blobs(seed, shape, count):
        rng = np.random.default_rng(24738 + seed)
        grids = np.meshgrid(*[np.arange(n, dtype=np.float32) for n in shape], indexing="ij", sparse=True)
        fg = np.zeros(shape, dtype=bool)
        for _ in range(count):
            c = [rng.uniform(0, n) for n in shape]
            r = rng.uniform(0.02, 0.12) * min(shape)
            fg |= sum((g - ci) ** 2 for g, ci in zip(grids, c)) <= r * r
        if fg.all():
            fg.flat[0] = False
        return fg.astype(np.uint8)

    specs = [("edt_2d_1024_b8", (8, 1, 1024, 1024), 20, None), ("edt_2d_4096_b1", (1, 1, 4096, 4096), 40, None),
             ("edt_3d_512_b1", (1, 1, 512, 512, 512), 24, None),
             ("edt_3d_512_b1_sampling_2.5_0.8_1", (1, 1, 512, 512, 512), 24, (2.5, 0.8, 1.0))]
    cases = []
    for k, (name, shape, count, samp) in enumerate(specs):
        imgs = [blobs(100 * k + i, shape[2:], count) for i in range(shape[0])]
        mask = np.stack(imgs)[:, None]
        nvox = mask.size
        io = 5 * nvox
        sets = max(2, min(8, -(-2 * l2_bytes(dev) // io)))
        calls = [binding.PreparedCall(torch.from_numpy(mask).to(dev), samp,
                                      torch.empty(mask.shape, dtype=torch.float32, device=dev), None, None)
                 for _ in range(sets)]
        for i in range(max(3, args.warmup)):
            calls[i % sets](sp)
        launches = binding.tm_edt_last_launch_count()
        torch.cuda.synchronize()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i, (a, b) in enumerate(evs):
            a.record(stream)
            calls[i % sets](sp)
            b.record(stream)
        torch.cuda.synchronize()
        times = sorted(a.elapsed_time(b) for a, b in evs)
        ms = statistics.median(times)
        c0 = calls[0]
        _, ks = binding.tm_edt_profile(c0.mask, samp, distances=c0.d, workspace=c0.ws, return_distances=True)
        # the oracle on the first image (its leading rows if the image alone would take minutes)
        one = mask[:1]
        rows = one.shape[2]
        t0 = time.perf_counter()
        oracle.sep(np.ascontiguousarray(one[:, :, : max(2, rows // 8)]), samp, want_idx=False)
        t_part = time.perf_counter() - t0
        keep = rows if t_part * 8 < 20 else max(2, int(rows / 8 * 20 / (t_part * 8)))
        part = np.ascontiguousarray(one[:, :, :keep])
        t0 = time.perf_counter()
        oracle.sep(part, samp, want_idx=False)
        cpu_s = time.perf_counter() - t0
        gbs = io / (ms * 1e-3) / 1e9
        cases.append({"case": name, "shape": list(mask.shape), "sampling": samp, "ms_per_step": ms, "ms_min": times[0],
                      "value": nvox / (ms * 1e-3) / 1e9, "unit": UNIT, "inputs_per_ms": shape[0] / ms,
                      "gpu_launches_per_step": launches,
                      "kernels": [(n, round(t, 4)) for n, t, _ in ks],
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                                   "peak_kind": peak_kind + " copy bandwidth", "bytes_per_voxel": 5},
                      "cpu_baseline": {"value": part.size / cpu_s / 1e9, "unit": UNIT, "cores": oracle.threads(),
                                       "kind": "oracle", "sample": "first %d of %d rows of one image" % (keep, rows)},
                      "l2": "rotating %d buffer sets" % sets})
        del calls
        torch.cuda.empty_cache()
    head = cases[0]
    print(json.dumps({"metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": 1, "steps": steps,
                      "warmup": max(3, args.warmup), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
                      "config": {"workload": head["case"], "shape": head["shape"], "outputs": ["dist_f32"]},
                      "gpu_launches": head["gpu_launches_per_step"] * steps, "roofline": head["roofline"],
                      "cpu_baseline": head["cpu_baseline"], "cases": cases}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=4, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-voxels", type=int, default=8 << 20, help="voxels per step of the reference arm")
    ap.add_argument("--cpu-voxels", type=int, default=64 << 20, help="sample size of the cpu_baseline leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-all-configs", action="store_true", help="skip the short runs of the other four workloads")
    ap.add_argument("--profile-steps", type=int, default=20)
    ap.add_argument("--unit-sampling", action="store_true", help="override the workload's sampling with 1.0 per axis")
    ap.add_argument("--outputs", default=None, help="override the requested outputs, e.g. dist,idx or dist,sq,idx")
    ap.add_argument("--flat-index", action="store_true",
                    help="index output as one linear index per voxel (variant of tm_edt_ex; not the headline layout)")
    ap.add_argument("--workload", default="edt", choices=["edt", "morph", "cdt", "long", "ex"],
                    help="edt: the headline benchmark; long: the same transform on extents beyond 128 (1024^2, 4096^2, 512^3); ex: the tm_edt_ex variants (flat index, float64 distances, strided mask, virtual background); morph / cdt: the erosion-dilation kernels and the taxicab / chessboard / brute-force transforms (their own metrics)")
    ap.add_argument("--morph-case", default=None, help="with --workload morph: run only this case (profiling aid)")
    ap.add_argument("--images", type=int, default=0, help="use only the first K images of the workload (profiling aid)")
    args = ap.parse_args()
    if args.workload == "morph":
        run_morph(args)
        return
    if args.workload == "ex":
        run_ex(args)
        return
    if args.workload == "cdt":
        run_cdt(args)
        return
    if args.workload == "long":
        run_long(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    world, rank, local = dist_env()

    from paper_2608_24738_b200 import workloads

    w = workloads.CONFIGS[args.config]()
    if args.unit_sampling:
        w.sampling = None
        w.name += " (unit sampling)"
    if args.images > 0:
        B, C = w.mask.shape[:2]
        flat = w.mask.reshape((B * C, 1) + w.mask.shape[2:])
        w.mask = flat[: args.images].copy()
        w.name += " (first %d images)" % args.images
    if args.outputs:
        want = set(args.outputs.split(","))
        w.want_dist, w.want_sq, w.want_idx = "dist" in want, "sq" in want, "idx" in want
        w.name += " (outputs %s)" % args.outputs
    if args.flat_index:
        w.flat_index = True
        w.name += " (flat index)"
    if args.impl == "reference":
        run_reference(args, w, world, rank)
        return

    import torch

    from paper_2608_24738_b200 import binding, buildlib

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the transform has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
        if local == 0:
            buildlib.build()  # one rank per node compiles (a no-op when the library is up to date)
        dist.barrier()
    else:
        buildlib.build()
    binding.lib()

    stream = torch.cuda.current_stream()
    sampler = ClockSampler(local)
    sampler.start()
    m = measure_device(w, args.steps, args.warmup, args.profile_steps, dev, world, sampler)
    io, shape, host_mask = m["io"], m["shape"], m["host_mask"]
    value, seconds, clocks, roofline = m["value"], m["seconds"], m["clocks"], m["roofline"]
    launches_per_step, sets = m["launches_per_step"], m["sets"]

    # ---- end to end: host buffers in, host buffers out, through tm_edt_host ----
    e2e = None
    if not args.no_e2e and not w.flat_index:  # the host entry point has the headline index layout only
        hm = host_mask.pin_memory()
        hd = torch.empty(shape, dtype=torch.float32, pin_memory=True) if w.want_dist else None
        hs = torch.empty(shape, dtype=torch.int64, pin_memory=True) if w.want_sq else None
        hx = torch.empty(shape[:2] + (w.ndim,) + shape[2:], dtype=torch.int64, pin_memory=True) if w.want_idx else None
        e2e_steps = max(3, min(args.steps, int(2e9 // max(io, 1)) or 3))
        kw = dict(return_distances=w.want_dist, return_sqdist=w.want_sq, return_indices=w.want_idx,
                  distances=hd, sqdist=hs, indices=hx)
        for _ in range(3):
            binding.tm_edt_host(hm, w.sampling, **kw)
            torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            binding.tm_edt_host(hm, w.sampling, **kw)
            stream.synchronize()  # the caller reads the host result every step
        e1.record(stream)
        torch.cuda.synchronize()
        es = max_over_ranks(e0.elapsed_time(e1) / 1e3, world, dev)
        e2e = {"value": whole_job_rate(w.voxels * e2e_steps, world, es) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": w.voxels, "d2h_bytes_per_step": io - w.voxels, "steps": e2e_steps}
    sampler.stop()

    others = None
    if world == 1 and not args.no_all_configs and not args.unit_sampling and not args.outputs and not args.images and not args.flat_index:
        others = []
        for num in (1, 2, 3, 4, 5):
            if num == args.config:
                continue
            wo = workloads.CONFIGS[num]()
            mo = measure_device(wo, 40, 5, 5, dev, world)
            others.append({"workload": wo.name, "value": mo["value"], "unit": UNIT, "ms_per_step": mo["seconds"] / 40 * 1e3,
                           "ms_median": mo["spread"]["ms_median"], "ms_min": mo["spread"]["ms_min"],
                           "warm_l2_ms_median": mo["spread"]["warm_l2_ms_median"],
                           "roofline_frac": mo["roofline"]["frac"], "dominant": mo["roofline"]["dominant"]["kernel"],
                           "kernels": [(k["kernel"], round(k["avg_ms"], 4)) for k in mo["roofline"]["kernels"]]})

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle

        v, secs, what, used = time_oracle(w, args.cpu_voxels)
        nvox = min(w.voxels, max(args.cpu_voxels, w.voxels // (w.mask.shape[0] * w.mask.shape[1])))
        v1, secs1, what1, _ = time_oracle_single_thread(w, secs, nvox, used)
        cpu = {"value": v, "unit": UNIT, "cores": used, "kind": "oracle", "sample": what, "seconds": secs,
               "single_thread": {"value": v1, "unit": UNIT, "cores": 1, "sample": what1, "seconds": secs1}}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": seconds / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "shape": list(shape), "sampling": w.sampling,
                       "outputs": [n for n, f in (("dist_f32", w.want_dist), ("sqdist_i64", w.want_sq),
                                                   ("indices_i64", w.want_idx)) if f],
                       "voxels_per_step": w.voxels,
                       "l2": "rotating %d buffer sets, %d MB per set, L2 %d MB" % (sets, io >> 20, l2_bytes(dev) >> 20),
                       "sha256": w.sha256()[:16]},
            "timing": m["spread"],
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "cpu_baseline": cpu, "other_configs": others,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
