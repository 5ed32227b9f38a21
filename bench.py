#!/usr/bin/env python
"""Benchmark of libfsoftmax: last-dimension softmax, achieved HBM GB/s against the roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5] [--impl reference] [--all]

A step is one fs_softmax call (dispatcher -> one kernel) over one batch of the headline workload:
the largest of the five configurations, the fp32 causal-masked matrix of 32768 x 32768 (cfg5, 4 GiB in,
4 GiB out). Inputs are seeded synthetic data already resident in HBM; where a workload is smaller
than eight times the L2 cache, successive steps rotate over enough independent (x, y) buffer
pairs (8 x L2 in total) that every step reads and writes DRAM. Timing is on the device with CUDA events recorded on the
launching stream around exactly K launches (a "train"); the train is repeated (30 times, fewer when
a train is long) and the median train is reported, so that the figure does not depend on K; the
slowest rank counts.

One JSON line goes to stdout (rank 0). Beyond the base keys it carries
  roofline      algorithmic bytes (read x once + write y once) per launch / average launch time,
                against the measured copy bandwidth of this GPU pool (MEASURED_PEAKS.json); DRAM
                traffic per launch from the ncu capture recorded in profiles/dram_traffic.txt
  per_config    all five configurations, each timed the same way: time, GB/s, fractions of the
                measured and of the nominal peak, the library's own copy over the same bytes, the
                input's 64-bit checksum
  e2e           the same metric through fs_softmax_host: pinned host buffers, H2D and D2H copies
                inside the timed region
  cpu_baseline  the fp64 oracle, as it stands, on the host cores over a bounded sample of the
                headline workload; `cpu_baselines` has the same for every configuration (all cores
                and one core)
  fixed_cost    time = t0 + bytes / B fitted over 1x..16x the rows of the two short configurations,
                for fs_softmax and for the library's copy
  workloads     the widened entry points (causal, router, log_softmax, backward, masked, norms)
With N > 1 (launched by torch.distributed.run) every rank runs the same per-GPU workload on its
own GPU: rows are independent, so there is no collective on the data path ("weak" scaling).

--impl reference times the CPU oracle instead (rank 0 only), on a bounded sample per step.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2607_24762_b200 import workloads as W  # noqa: E402

METRIC = "softmax achieved HBM GB/s (min read+write bytes/time)"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.txt")


def ncu_traffic():
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum, averaged over eight consecutive
    launches on rotating buffers, so that the write-back of one launch's output is counted while the next runs)
    per workload, as recorded in profiles/dram_traffic.txt by `python -m paper_2607_24762_b200.traffic`."""
    from paper_2607_24762_b200 import traffic
    try:
        return traffic.read(TRAFFIC_FILE)
    except Exception:
        return {}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index          # nvidia-smi -i accepts an index or a GPU UUID
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def n_samples(self) -> int:
        if not self.file:
            return 0
        try:
            with open(self.file.name) as f:
                return sum(1 for _ in f)
        except Exception:
            return 0

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if not self.proc:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            with open(self.file.name) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) >= 8:
                        rows.append(parts)
            os.unlink(self.file.name)
        except Exception:
            pass
        sm = []
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for p in rows:
            try:
                sm.append(float(p[0]))
                out["sm_max_mhz"] = float(p[1])
            except ValueError:
                continue
            for name, v in zip(names, p[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out["sm_mhz"] = statistics.median(sm)
        out["reasons"] = sorted(reasons)
        out["samples"] = len(sm)
        return out


# ---------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------

def device_buffers(w: W.Workload, n_pairs: int, threads: int, checksum: list | None = None):
    """n_pairs independent (x, y) device buffer pairs holding the workload's seeded input. With `checksum`
    (a list), the 64-bit checksum of the input is appended to it (computed slab by slab on the host)."""
    import torch
    tdtype = torch.float32 if w.dtype == W.FP32 else torch.int16
    slab = max(1, (64 << 20) // (w.cols * w.elem_size))
    x0 = torch.empty((w.rows, w.cols), dtype=tdtype, device="cuda")
    cs = W.Checksum() if checksum is not None else None
    for r0 in range(0, w.rows, slab):
        r1 = min(w.rows, r0 + slab)
        h = W.generate_rows(w, r0, r1, threads=threads)
        if cs is not None:
            cs.update(h)
        x0[r0:r1].copy_(torch.from_numpy(h.view(np.int16) if w.dtype != W.FP32 else h))
    if cs is not None:
        checksum.append(cs.value())
    xs = [x0] + [x0.clone() for _ in range(n_pairs - 1)]
    ys = [torch.empty_like(x0) for _ in range(n_pairs)]
    return xs, ys


def run_trains(launch, steps: int, stream, barrier=None, n_trains: int = 30, budget_ms: float = 3000.0):
    """Times trains of exactly `steps` launches, one CUDA event pair (on the launching stream) around each train.
    30 trains, fewer (at least 3) when 30 would exceed budget_ms of device time. Returns the list of train times in ms."""
    import torch
    out = []
    i = 0
    while len(out) < n_trains:
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        if barrier:
            barrier()
        start.record(stream)
        for _ in range(steps):
            launch(i)
            i += 1
        stop.record(stream)
        torch.cuda.synchronize()
        if barrier:
            barrier()
        out.append(start.elapsed_time(stop))
        if len(out) >= 3 and sum(out) + out[-1] > budget_ms:
            break
    return out


def train_stats(trains, steps: int):
    each = sorted(t / steps for t in trains)
    return {"n_trains": len(each), "median": round(statistics.median(each), 6), "min": round(each[0], 6),
            "max": round(each[-1], 6), "first": round(trains[0] / steps, 6)}


def time_device(w: W.Workload, steps: int, warmup: int, l2_bytes: int, sampler: ClockSampler | None = None,
                barrier=None, min_clock_samples: int = 0, causal_q=None, extras: bool = False, n_trains: int = 30,
                causal_too: bool = False):
    """Times trains of `steps` fs_softmax (or, with causal_q, fs_softmax_causal) launches with CUDA events on
    the launching stream (run_trains); ms_per_step is the median train divided by `steps`.
    With `extras`, the same buffers are then timed two more ways: the library's own copy kernel over
    the same bytes (the ceiling this device gives a kernel that only moves the data), and the same
    launches one at a time, an event pair around each (that figure includes the launch gap)."""
    import torch

    import paper_2607_24762_b200 as fs
    free, _ = torch.cuda.mem_get_info()
    pair_bytes = w.min_bytes
    want = max(1, math.ceil(8 * l2_bytes / pair_bytes))     # 8 x L2: at 4 x, a fifth of cfg3's reads still hit L2 (ncu)
    n_pairs = int(max(1, min(want, 256, (free * 0.6) // pair_bytes)))
    csum = []
    xs, ys = device_buffers(w, n_pairs, threads=min(8, os.cpu_count() or 1), checksum=csum)
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream
    lib = fs.binding.lib()
    ptrs = [(x.data_ptr(), y.data_ptr()) for x, y in zip(xs, ys)]
    scale = w.scale_f32

    def launch(i):
        xp, yp = ptrs[i % n_pairs]
        if causal_q is None:
            st = lib.fs_softmax(xp, yp, w.rows, w.cols, w.dtype, scale, sh)
        else:
            st = lib.fs_softmax_causal(xp, yp, w.rows, w.cols, causal_q, w.dtype, scale, sh)
        if st != 0:
            raise RuntimeError(f"fs_softmax failed: {fs.fs_strerror(st)}")

    for i in range(max(3, warmup)):
        launch(i)
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
        time.sleep(0.12)
    trains = run_trains(launch, steps, stream, barrier=barrier, n_trains=n_trains)
    launches = len(trains) * steps
    extension_s = 0.0
    if sampler and min_clock_samples:
        # the timed region can be shorter than nvidia-smi's sampling period: keep the same loop
        # running (untimed) until enough clock samples were taken under load
        t0 = time.time()
        i = 0
        while sampler.n_samples() < min_clock_samples + 3 and time.time() - t0 < 3.0:
            for _ in range(8 if w.min_bytes > (1 << 30) else 64):
                launch(i)
                i += 1
            torch.cuda.synchronize()
        extension_s = time.time() - t0
    clocks = sampler.stop() if sampler else None
    if clocks is not None:
        clocks["sampled_over"] = "timed trains" + (f" + {extension_s:.1f} s of the same launches" if extension_s else "")
    status = fs.fs_device_status()
    if status != 0:
        raise RuntimeError(f"device status: {fs.fs_strerror(status)}")
    kernel = fs.fs_kernel_name(fs.fs_select_kernel(w.rows, w.cols, w.dtype))
    stats = train_stats(trains, steps)
    extra = {}
    if extras:
        nbytes = w.rows * w.cols * w.elem_size
        if nbytes % 16 == 0:
            def copy(i):
                lib.fs_copy(ptrs[i % n_pairs][0], ptrs[i % n_pairs][1], nbytes, sh)
            for i in range(3):
                copy(i)
            copy_ms = statistics.median(run_trains(copy, steps, stream, n_trains=n_trains)) / steps
            extra["own_copy"] = {"ms_per_step": round(copy_ms, 6), "GB/s": round(w.min_bytes / (copy_ms * 1e-3) / 1e9, 1),
                                 "softmax_over_copy_time": round(stats["median"] / copy_ms, 4)}
        n1 = min(100, max(steps, 20))
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n1)]
        for i, (a, b) in enumerate(pairs):
            a.record(stream)
            launch(i)
            b.record(stream)
        torch.cuda.synchronize()
        each = sorted(a.elapsed_time(b) for a, b in pairs)
        extra["single_launch_ms"] = {"median": round(statistics.median(each), 6), "best": round(each[0], 6), "n": n1,
                                     "note": "event pair around each launch: includes the launch gap"}
    if causal_too:
        # fs_softmax_causal(q_offset = 0) over the same buffers: the masked part of x is never read
        def causal(i):
            xp, yp = ptrs[i % n_pairs]
            st = lib.fs_softmax_causal(xp, yp, w.rows, w.cols, 0, w.dtype, scale, sh)
            if st != 0:
                raise RuntimeError(f"fs_softmax_causal failed: {fs.fs_strerror(st)}")
        for i in range(3):
            causal(i)
        extra["causal_ms_per_step"] = statistics.median(run_trains(causal, steps, stream, n_trains=min(n_trains, 10))) / steps
    del xs, ys
    torch.cuda.empty_cache()
    return {"ms_per_step": statistics.median(trains) / steps, "trains": stats, "launches": launches, "n_pairs": n_pairs,
            "kernel": kernel, "clocks": clocks, "checksum": f"{csum[0]:016x}", **extra}


def fit_fixed_cost(w: W.Workload, l2_bytes: int, steps: int = 200):
    """time = t0 + bytes / B over 1x, 2x, 4x, 8x, 16x the rows of a short workload, for fs_softmax and for the library's
    copy over the same buffers (least squares; device-seeded data of the workload's shape and dtype)."""
    import torch

    import paper_2607_24762_b200 as fs
    lib = fs.binding.lib()
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream
    tdt = {W.FP32: torch.float32, W.BF16: torch.bfloat16, W.FP16: torch.float16}[w.dtype]
    g = torch.Generator(device="cuda").manual_seed(7)
    pts = {"softmax": [], "copy": []}
    for mult in (1, 2, 4, 8, 16):
        rows = w.rows * mult
        nbytes = rows * w.cols * w.elem_size
        n_pairs = int(max(1, min(16, math.ceil(4 * l2_bytes / (2 * nbytes)))))
        xs = [(torch.randn((rows, w.cols), generator=g, device="cuda") * 2.0).to(tdt) for _ in range(n_pairs)]
        ys = [torch.empty_like(x) for x in xs]

        def soft(i):
            lib.fs_softmax(xs[i % n_pairs].data_ptr(), ys[i % n_pairs].data_ptr(), rows, w.cols, w.dtype, w.scale_f32, sh)

        def copy(i):
            lib.fs_copy(xs[i % n_pairs].data_ptr(), ys[i % n_pairs].data_ptr(), nbytes, sh)

        for name, fn in (("softmax", soft), ("copy", copy)):
            for i in range(5):
                fn(i)
            k = max(20, steps // mult)
            ms = statistics.median(run_trains(fn, k, stream, n_trains=9, budget_ms=400.0)) / k
            pts[name].append((2.0 * nbytes, ms * 1e3))
        del xs, ys
        torch.cuda.empty_cache()
    out = {"workload": w.name, "rows_multiples": [1, 2, 4, 8, 16]}
    for name, p in pts.items():
        bx = np.array([b for b, _ in p])
        ty = np.array([t for _, t in p])
        slope, t0 = np.polyfit(bx, ty, 1)
        out[name] = {"t0_us": round(float(t0), 3), "GB/s_marginal": round(1e-3 / float(slope), 1),
                     "us": [round(float(t), 3) for t in ty]}
    return out


def time_static(w: W.Workload, steps: int, l2_bytes: int):
    """fs_softmax_static against fs_softmax on device-seeded data of the workload's shape: the same kernels, the
    scratch in the library's fixed device array instead of allocated memory."""
    import torch

    import paper_2607_24762_b200 as fs
    lib = fs.binding.lib()
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream
    tdt = {W.FP32: torch.float32, W.BF16: torch.bfloat16, W.FP16: torch.float16}[w.dtype]
    n_pairs = int(max(1, min(8, math.ceil(8 * l2_bytes / w.min_bytes))))
    g = torch.Generator(device="cuda").manual_seed(11)
    xs = [(torch.randn((w.rows, w.cols), generator=g, device="cuda") * 3.0).to(tdt) for _ in range(n_pairs)]
    ys = [torch.empty_like(x) for x in xs]
    out = {"what": f"fs_softmax_static on {w.name} ({w.rows} x {w.cols} {W.DTYPE_NAME[w.dtype]})", "steps": steps}
    for name, fn in (("static", lib.fs_softmax_static), ("allocating", lib.fs_softmax)):
        def launch(i):
            st = fn(xs[i % n_pairs].data_ptr(), ys[i % n_pairs].data_ptr(), w.rows, w.cols, w.dtype, 1.0, sh)
            if st != 0:
                raise RuntimeError(fs.fs_strerror(st))
        for i in range(5):
            launch(i)
        ms = statistics.median(run_trains(launch, steps, stream, n_trains=9, budget_ms=1000.0)) / steps
        out[name + "_ms_per_step"] = round(ms, 6)
        out[name + "_GB/s"] = round(w.min_bytes / (ms * 1e-3) / 1e9, 1)
    if fs.fs_static_status() != 0:
        raise RuntimeError("fs_static_status reported an expired wait")
    return out


def time_router(w: W.Workload, k: int, steps: int, warmup: int, l2_bytes: int):
    """fs_router_topk on the router workload: reads x once, writes k weights and k columns per row."""
    import torch

    import paper_2607_24762_b200 as fs
    alg = w.rows * w.cols * w.elem_size + w.rows * k * 8
    n_pairs = int(max(1, min(16, math.ceil(4 * l2_bytes / alg))))
    xs, _ = device_buffers(w, n_pairs, threads=min(8, os.cpu_count() or 1))
    ws = [torch.empty((w.rows, k), dtype=torch.float32, device="cuda") for _ in range(n_pairs)]
    ids = [torch.empty((w.rows, k), dtype=torch.int32, device="cuda") for _ in range(n_pairs)]
    stream = torch.cuda.current_stream()
    lib = fs.binding.lib()

    def launch(i):
        j = i % n_pairs
        st = lib.fs_router_topk(xs[j].data_ptr(), ws[j].data_ptr(), ids[j].data_ptr(), w.rows, w.cols, k, w.dtype,
                                w.scale_f32, 1, stream.cuda_stream)
        if st != 0:
            raise RuntimeError(fs.fs_strerror(st))

    for i in range(max(3, warmup)):
        launch(i)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record(stream)
    for i in range(steps):
        launch(i)
    stop.record(stream)
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / steps
    peak, _ = measured_peak()
    gbs = alg / (ms * 1e-3) / 1e9
    return {"what": f"fs_router_topk(k={k}, renormalize) on cfg3: reads x, writes {k} weights + {k} columns per row",
            "steps": steps, "ms_per_step": round(ms, 6), "algorithmic_bytes": alg, "GB/s": round(gbs, 1),
            "rows_per_s": round(w.rows / (ms * 1e-3), 1), "frac_of_measured_copy": round(gbs / peak, 4)}


def time_log_softmax(w: W.Workload, steps: int, warmup: int, l2_bytes: int, eager: bool = True):
    """fs_log_softmax on a softmax workload's data: reads x once, writes y once."""
    import torch

    import paper_2607_24762_b200 as fs
    n_pairs = int(max(1, min(16, math.ceil(4 * l2_bytes / w.min_bytes))))
    xs, ys = device_buffers(w, n_pairs, threads=min(8, os.cpu_count() or 1))
    stream = torch.cuda.current_stream()
    lib = fs.binding.lib()

    def launch(i):
        j = i % n_pairs
        st = lib.fs_log_softmax(xs[j].data_ptr(), ys[j].data_ptr(), w.rows, w.cols, w.dtype, w.scale_f32, stream.cuda_stream)
        if st != 0:
            raise RuntimeError(fs.fs_strerror(st))

    tdt = {W.FP32: torch.float32, W.BF16: torch.bfloat16, W.FP16: torch.float16}[w.dtype]

    def eager_launch(i):
        torch.log_softmax(xs[i % n_pairs].view(tdt).view(w.rows, w.cols) * w.scale_f32, dim=-1)

    def timed(fn, k):
        for i in range(max(3, warmup)):
            fn(i)
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record(stream)
        for i in range(k):
            fn(i)
        stop.record(stream)
        torch.cuda.synchronize()
        return start.elapsed_time(stop) / k

    ms = timed(launch, steps)
    peak, _ = measured_peak()
    gbs = w.min_bytes / (ms * 1e-3) / 1e9
    out = {"what": f"fs_log_softmax on {w.name}", "steps": steps, "ms_per_step": round(ms, 6), "algorithmic_bytes": w.min_bytes,
           "GB/s": round(gbs, 1), "frac_of_measured_copy": round(gbs / peak, 4), "n_pairs": n_pairs}
    if eager:
        out["torch_eager_ms"] = round(timed(eager_launch, max(5, steps // 4)), 6)
    return out


def time_softmax_f32out(w: W.Workload, steps: int, warmup: int, l2_bytes: int, eager: bool = True):
    """fs_softmax_f32out on a 16-bit softmax workload: reads 2 bytes and writes 4 per element."""
    import torch

    import paper_2607_24762_b200 as fs
    if w.dtype == W.FP32:
        raise ValueError("fs_softmax_f32out takes bf16/fp16 input")
    alg = w.rows * w.cols * 6
    n_pairs = int(max(1, min(16, math.ceil(4 * l2_bytes / alg))))
    xs, _ = device_buffers(w, n_pairs, threads=min(8, os.cpu_count() or 1))
    ys = [torch.empty((w.rows, w.cols), dtype=torch.float32, device="cuda") for _ in range(n_pairs)]
    stream = torch.cuda.current_stream()
    lib = fs.binding.lib()
    tdt = torch.bfloat16 if w.dtype == W.BF16 else torch.float16

    def launch(i):
        j = i % n_pairs
        st = lib.fs_softmax_f32out(xs[j].data_ptr(), ys[j].data_ptr(), w.rows, w.cols, w.dtype, w.scale_f32, stream.cuda_stream)
        if st != 0:
            raise RuntimeError(fs.fs_strerror(st))

    def eager_launch(i):
        torch.softmax(xs[i % n_pairs].view(tdt).view(w.rows, w.cols) * w.scale_f32, dim=-1, dtype=torch.float32)

    def timed(fn, k):
        for i in range(max(3, warmup)):
            fn(i)
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record(stream)
        for i in range(k):
            fn(i)
        stop.record(stream)
        torch.cuda.synchronize()
        return start.elapsed_time(stop) / k

    ms = timed(launch, steps)
    peak, _ = measured_peak()
    gbs = alg / (ms * 1e-3) / 1e9
    out = {"what": f"fs_softmax_f32out on {w.name}: 16-bit in, float32 out", "steps": steps, "ms_per_step": round(ms, 6),
           "algorithmic_bytes": alg, "GB/s": round(gbs, 1), "frac_of_measured_copy": round(gbs / peak, 4), "n_pairs": n_pairs}
    if eager:
        out["torch_eager_ms"] = round(timed(eager_launch, max(5, steps // 4)), 6)
    return out


def time_softmax_masked(w: W.Workload, steps: int, warmup: int, l2_bytes: int, heads: int = 8, eager: bool = True):
    """fs_softmax_masked on a softmax workload's data viewed as (batch 1, `heads`, rows/heads queries) with a
    causal mask shared by the heads; algorithmic bytes = x + y + the mask once."""
    import torch

    import paper_2607_24762_b200 as fs
    q = w.rows // heads
    alg = w.min_bytes + q * w.cols * w.elem_size
    n_pairs = int(max(1, min(16, math.ceil(4 * l2_bytes / alg))))
    xs, ys = device_buffers(w, n_pairs, threads=min(8, os.cpu_count() or 1))
    tdt = {W.FP32: torch.float32, W.BF16: torch.bfloat16, W.FP16: torch.float16}[w.dtype]
    mask = torch.full((q, w.cols), float("-inf"), device="cuda", dtype=torch.float32).triu(1 + w.cols - q).to(tdt).contiguous()
    stream = torch.cuda.current_stream()
    lib = fs.binding.lib()

    def launch(i):
        j = i % n_pairs
        st = lib.fs_softmax_masked(xs[j].data_ptr(), mask.data_ptr(), ys[j].data_ptr(), w.rows, w.cols, q, heads, w.dtype,
                                   w.scale_f32, stream.cuda_stream)
        if st != 0:
            raise RuntimeError(fs.fs_strerror(st))

    def eager_launch(i):
        s = xs[i % n_pairs].view(tdt).view(1, heads, q, w.cols)
        torch.softmax(s * w.scale_f32 + mask, dim=-1)

    def timed(fn, k):
        for i in range(max(3, warmup)):
            fn(i)
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record(stream)
        for i in range(k):
            fn(i)
        stop.record(stream)
        torch.cuda.synchronize()
        return start.elapsed_time(stop) / k

    ms = timed(launch, steps)
    peak, _ = measured_peak()
    gbs = alg / (ms * 1e-3) / 1e9
    out = {"what": f"fs_softmax_masked on {w.name} as 1 x {heads} x {q} x {w.cols}, causal mask shared by the heads", "steps": steps,
           "ms_per_step": round(ms, 6), "algorithmic_bytes": alg, "GB/s": round(gbs, 1), "frac_of_measured_copy": round(gbs / peak, 4),
           "n_pairs": n_pairs}
    if eager:
        out["torch_eager_ms"] = round(timed(eager_launch, max(5, steps // 4)), 6)
    return out


def time_softmax_backward(w: W.Workload, steps: int, warmup: int, l2_bytes: int):
    """fs_softmax_backward on a softmax workload's shape: y = the library's forward output, dy seeded on
    the device; reads dy and y once, writes dx once (3 elements of traffic per element)."""
    import torch

    import paper_2607_24762_b200 as fs
    alg = 3 * w.rows * w.cols * w.elem_size
    n_sets = int(max(1, min(12, math.ceil(4 * l2_bytes / alg))))
    xs, ys = device_buffers(w, n_sets, threads=min(8, os.cpu_count() or 1))
    stream = torch.cuda.current_stream()
    lib = fs.binding.lib()
    tdt = {W.FP32: torch.float32, W.BF16: torch.bfloat16, W.FP16: torch.float16}[w.dtype]
    g = torch.Generator(device="cuda").manual_seed(99)
    for j in range(n_sets):                                   # y_j = softmax(x_j); x_j then becomes dy_j
        st = lib.fs_softmax(xs[j].data_ptr(), ys[j].data_ptr(), w.rows, w.cols, w.dtype, w.scale_f32, stream.cuda_stream)
        if st != 0:
            raise RuntimeError(fs.fs_strerror(st))
        torch.cuda.synchronize()
        xs[j].view(tdt).copy_(torch.randn((w.rows, w.cols), generator=g, device="cuda", dtype=torch.float32))
    dxs = [torch.empty_like(x) for x in xs]

    def launch(i):
        j = i % n_sets
        st = lib.fs_softmax_backward(xs[j].data_ptr(), ys[j].data_ptr(), dxs[j].data_ptr(), w.rows, w.cols, w.dtype, w.scale_f32,
                                     stream.cuda_stream)
        if st != 0:
            raise RuntimeError(fs.fs_strerror(st))

    for i in range(max(3, warmup)):
        launch(i)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record(stream)
    for i in range(steps):
        launch(i)
    stop.record(stream)
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / steps
    peak, _ = measured_peak()
    gbs = alg / (ms * 1e-3) / 1e9
    return {"what": f"fs_softmax_backward on {w.name}'s shape: reads dy and y, writes dx", "steps": steps, "ms_per_step": round(ms, 6),
            "algorithmic_bytes": alg, "GB/s": round(gbs, 1), "frac_of_measured_copy": round(gbs / peak, 4), "n_sets": n_sets}


# Normalisation workloads (synthetic, seeded on the device): the shapes of the two operators the paper
# reports for Stable Diffusion 3.5 Medium (Sec. IV-C): layer_norm over the transformer's hidden size
# (1536) for 4 x 4096 tokens, and the VAE decoder's 32-group group_norm at three resolutions.
NORM_WORKLOADS = {
    "ln_sd35": ("layer", dict(rows=16384, cols=1536, dtype=W.BF16)),
    "ln_4096_f32": ("layer", dict(rows=8192, cols=4096, dtype=W.FP32)),
    "ln_4096_bf16": ("layer", dict(rows=16384, cols=4096, dtype=W.BF16)),
    "gn_c512_128": ("group", dict(n=1, channels=512, spatial=128 * 128, groups=32, dtype=W.BF16)),
    "gn_c256_256": ("group", dict(n=1, channels=256, spatial=256 * 256, groups=32, dtype=W.BF16)),
    "gn_c128_512": ("group", dict(n=1, channels=128, spatial=512 * 512, groups=32, dtype=W.BF16)),
    "gn_c128_1024": ("group", dict(n=1, channels=128, spatial=1024 * 1024, groups=32, dtype=W.BF16)),
    "gn_c512_128_b8": ("group", dict(n=8, channels=512, spatial=128 * 128, groups=32, dtype=W.BF16)),
    "gn_c256_256_b8": ("group", dict(n=8, channels=256, spatial=256 * 256, groups=32, dtype=W.BF16)),
}


def time_norm(name: str, steps: int, warmup: int, l2_bytes: int, eager: bool = True):
    """fs_layer_norm / fs_group_norm on one NORM_WORKLOADS entry: reads x once, writes y once."""
    import torch

    import paper_2607_24762_b200 as fs
    kind, c = NORM_WORKLOADS[name]
    tdt = {W.FP32: torch.float32, W.BF16: torch.bfloat16, W.FP16: torch.float16}[c["dtype"]]
    esz = W.ELEM_SIZE[c["dtype"]]
    shape = (c["rows"], c["cols"]) if kind == "layer" else (c["n"], c["channels"], c["spatial"])
    nelem = int(np.prod(shape))
    alg = 2 * nelem * esz
    n_pairs = int(max(1, min(16, math.ceil(4 * l2_bytes / alg))))
    g = torch.Generator(device="cuda").manual_seed(1234)
    xs = [(torch.randn(shape, generator=g, device="cuda") * 1.5 + 0.25).to(tdt) for _ in range(n_pairs)]
    ys = [torch.empty_like(x) for x in xs]
    na = c["cols"] if kind == "layer" else c["channels"]
    gamma = (torch.randn(na, generator=g, device="cuda") * 0.2 + 1.0).to(tdt)
    beta = (torch.randn(na, generator=g, device="cuda") * 0.1).to(tdt)
    stream = torch.cuda.current_stream()
    lib = fs.binding.lib()

    def launch(i):
        j = i % n_pairs
        if kind == "layer":
            st = lib.fs_layer_norm(xs[j].data_ptr(), gamma.data_ptr(), beta.data_ptr(), ys[j].data_ptr(), c["rows"], c["cols"],
                                   c["dtype"], 1e-5, stream.cuda_stream)
        else:
            st = lib.fs_group_norm(xs[j].data_ptr(), gamma.data_ptr(), beta.data_ptr(), ys[j].data_ptr(), c["n"], c["channels"],
                                   c["spatial"], c["groups"], c["dtype"], 1e-5, stream.cuda_stream)
        if st != 0:
            raise RuntimeError(fs.fs_strerror(st))

    def eager_launch(i):
        j = i % n_pairs
        if kind == "layer":
            torch.nn.functional.layer_norm(xs[j], (c["cols"],), gamma, beta, 1e-5)
        else:
            torch.nn.functional.group_norm(xs[j], c["groups"], gamma, beta, 1e-5)

    def timed(fn, k):
        for i in range(max(3, warmup)):
            fn(i)
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record(stream)
        for i in range(k):
            fn(i)
        stop.record(stream)
        torch.cuda.synchronize()
        return start.elapsed_time(stop) / k

    ms = timed(launch, steps)
    peak, _ = measured_peak()
    gbs = alg / (ms * 1e-3) / 1e9
    out = {"what": f"fs_{kind}_norm {name} {list(shape)} {W.DTYPE_NAME[c['dtype']]}, gamma and beta, eps 1e-5", "steps": steps,
           "ms_per_step": round(ms, 6), "algorithmic_bytes": alg, "GB/s": round(gbs, 1),
           "frac_of_measured_copy": round(gbs / peak, 4), "n_pairs": n_pairs}
    if eager:
        out["torch_eager_ms"] = round(timed(eager_launch, max(5, steps // 4)), 6)
    return out


def time_e2e(w: W.Workload, steps: int, warmup: int):
    """The same metric through fs_softmax_host: pinned host buffers in, pinned host buffers out."""
    import torch

    import paper_2607_24762_b200 as fs
    rows = w.rows
    tdtype = torch.float32 if w.dtype == W.FP32 else torch.int16
    h = W.generate_rows(w, 0, rows, threads=min(8, os.cpu_count() or 1))
    xh = torch.from_numpy(h.view(np.int16) if w.dtype != W.FP32 else h).pin_memory()
    yh = torch.empty((rows, w.cols), dtype=tdtype).pin_memory()
    for _ in range(max(1, warmup)):
        fs.fs_softmax_host(xh, yh, rows, w.cols, w.dtype, w.scale_f32)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        fs.fs_softmax_host(xh, yh, rows, w.cols, w.dtype, w.scale_f32)     # blocks until y_host is complete
    dt = (time.perf_counter() - t0) / steps
    nbytes = rows * w.cols * w.elem_size
    fs.fs_release()
    return {"value": round(2 * nbytes / dt / 1e9, 2), "unit": UNIT, "ms_per_step": round(dt * 1e3, 4),
            "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": nbytes,
            "api": "fs_softmax_host (pinned host buffers, 8 MiB chunks pipelined over copy-in, kernel and copy-out streams)"}


# ---------------------------------------------------------------------------------------------
# CPU oracle arm (reported baseline; also --impl reference)
# ---------------------------------------------------------------------------------------------

def oracle_sample(w: W.Workload, target_cpu_seconds: float):
    """A bounded sample of the workload: evenly spaced row blocks, sized for ~target_cpu_seconds."""
    ns_per_elem = 30.0 if w.index == 5 else 11.0
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    rows = int(target_cpu_seconds * 1e9 / ns_per_elem / w.cols)
    rows = max(cores, min(w.rows, rows))
    rows -= rows % cores if rows >= 2 * cores else 0
    stride = max(1, w.rows // rows)
    idx = [min(w.rows - 1, i * stride) for i in range(rows)]
    x = np.concatenate([W.generate_rows(w, i, i + 1) for i in idx]) if stride > 1 else W.generate_rows(w, 0, rows)
    return x, cores, f"{rows} of {w.rows} rows (every {stride}th), all {w.cols} columns"


def run_oracle(w: W.Workload, x: np.ndarray, cores: int) -> float:
    """Seconds for the single-threaded oracle run on `cores` threads over a row partition of x."""
    from oracle import fso
    parts = [p for p in np.array_split(np.arange(x.shape[0]), cores) if len(p)]
    outs = [None] * len(parts)

    def work(k):
        outs[k] = fso.softmax_f64(x[parts[k][0]:parts[k][-1] + 1], w.dtype, w.scale_f32)

    ths = [threading.Thread(target=work, args=(k,)) for k in range(len(parts))]
    t0 = time.perf_counter()
    for t in ths:
        t.start()
    for t in ths:
        t.join()
    return time.perf_counter() - t0


def cpu_baseline(w: W.Workload, target_cpu_seconds: float = 16.0):
    """The oracle, as it stands, over a bounded sample of the workload: on all host cores (rows partitioned over
    threads, each running the single-threaded oracle) and on one core. `target_cpu_seconds` is the CPU work of one
    pass over the sample, summed over cores; a workload smaller than that is passed over several times."""
    from oracle import fso
    fso.build()
    x, cores, what = oracle_sample(w, target_cpu_seconds)
    run_oracle(w, x[:cores], cores)                        # load the library, touch the code
    est = x.size * 11e-9
    passes = int(max(1, min(200, round(0.6 * target_cpu_seconds / max(est, 1e-3)))))
    dt = sum(run_oracle(w, x, cores) for _ in range(passes)) / passes
    nbytes = 2 * x.size * w.elem_size
    if passes > 1:
        what += f", mean of {passes} passes"
    if x.shape[0] < w.rows:
        what += "; the workload's figure is extrapolated from this sample"
    # the same oracle on one core, over the head of the same sample
    n1 = int(max(1, min(x.shape[0], 0.125 * target_cpu_seconds / 11e-9 // w.cols)))
    dt1 = run_oracle(w, x[:n1], 1)
    one = {"value": round(2 * n1 * w.cols * w.elem_size / dt1 / 1e9, 4), "unit": UNIT, "cores": 1,
           "sample": f"the first {n1} rows of the sample", "seconds": round(dt1, 4)}
    return {"value": round(nbytes / dt / 1e9, 4), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": what, "seconds": round(dt, 4), "rows_per_s": round(x.shape[0] / dt, 1), "one_core": one}


def reference_arm(args, w: W.Workload):
    """--impl reference: the oracle, as it stands, on the host cores; a step is one bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import fso
    fso.build()
    x, cores, what = oracle_sample(w, 4.0)
    for _ in range(max(1, min(args.warmup, 2))):
        run_oracle(w, x, cores)
    steps = max(1, min(args.steps, 20))
    t0 = time.perf_counter()
    for _ in range(steps):
        run_oracle(w, x, cores)
    dt = (time.perf_counter() - t0) / steps
    value = round(2 * x.size * w.elem_size / dt / 1e9, 4)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": args.warmup, "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "shape": [w.rows, w.cols], "storage_dtype": W.DTYPE_NAME[w.dtype],
                       "step": "the fp64 oracle over a bounded sample of the workload: " + what},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# main
# ---------------------------------------------------------------------------------------------

def smi_id(props, local_rank: int) -> str:
    """The GPU's UUID (CUDA_VISIBLE_DEVICES may renumber indices), else its index."""
    try:
        u = str(props.uuid)
        return u if u.startswith("GPU-") else "GPU-" + u
    except Exception:
        return str(local_rank)


def roofline_obj(w: W.Workload, ms_per_step: float, kernel: str):
    peak, which = measured_peak()
    achieved = w.min_bytes / (ms_per_step * 1e-3) / 1e9
    t = ncu_traffic().get(w.name)
    return {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
            "frac": round(achieved / peak, 4), "peak_source": f"of {which} (copy bandwidth)",
            "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
            "traffic": t["bytes_per_launch"] if t else None,
            "traffic_over_algorithmic": round(t["bytes_per_launch"] / w.min_bytes, 4) if t else None,
            "traffic_source": t["note"] if t else "no capture recorded in profiles/dram_traffic.txt",
            "algorithmic_bytes_per_launch": w.min_bytes, "kernel": kernel}


def per_config_entry(w: W.Workload, r: dict):
    peak, _ = measured_peak()
    gbs = w.min_bytes / (r["ms_per_step"] * 1e-3) / 1e9
    t = ncu_traffic().get(w.name)
    e = {"shape": [w.rows, w.cols], "dtype": W.DTYPE_NAME[w.dtype], "kernel": r["kernel"], "ms_per_step": round(r["ms_per_step"], 6),
         "GB/s": round(gbs, 1), "rows_per_s": round(w.rows / (r["ms_per_step"] * 1e-3), 1),
         "frac_of_measured": round(gbs / peak, 4), "frac_of_nominal": round(gbs / NOMINAL_HBM_GBS, 4),
         "steps": r.get("steps"), "trains": r["trains"], "n_pairs": r["n_pairs"], "checksum": r["checksum"],
         "traffic_over_algorithmic": round(t["bytes_per_launch"] / w.min_bytes, 4) if t else None}
    if "own_copy" in r:
        e["own_copy_ms"] = r["own_copy"]["ms_per_step"]
        e["softmax_over_copy_time"] = r["own_copy"]["softmax_over_copy_time"]
    if "single_launch_ms" in r:
        e["single_launch_ms"] = r["single_launch_ms"]["median"]
    return e


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="cfg5", choices=sorted(W.WORKLOADS))
    ap.add_argument("--trains", type=int, default=30, help="how many times the train of --steps launches is timed (median reported)")
    ap.add_argument("--impl", default="fsoftmax", choices=["fsoftmax", "reference"])
    ap.add_argument("--rows", type=int, default=0,
                    help="use only the first ROWS rows of the workload (small cases for profiler captures)")
    ap.add_argument("--cols", type=int, default=0,
                    help="give the workload's rows this many columns instead (same value distribution; profiler captures of "
                         "the kernels the five workloads do not reach)")
    ap.add_argument("--all", dest="all_workloads", action="store_true", default=None,
                    help="also time the other workloads (default: on at --gpus 1)")
    ap.add_argument("--no-all", dest="all_workloads", action="store_false")
    ap.add_argument("--norm-workload", default="ln_sd35", choices=sorted(NORM_WORKLOADS), help="with --op norm")
    ap.add_argument("--op", default="softmax", choices=["softmax", "causal", "router", "norm", "log_softmax", "backward", "masked", "f32out"],
                    help="time only fs_softmax_causal (q_offset 0) or fs_router_topk (k=8, renormalised) on the "
                         "workload and print a short line (profiler captures of those kernels)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the cpu_baseline leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end leg")
    ap.add_argument("--no-clocks", action="store_true", help="do not sample nvidia-smi clocks (profiler captures)")
    args = ap.parse_args()
    w = W.WORKLOADS[args.workload]
    if args.rows:
        import dataclasses
        w = dataclasses.replace(w, rows=min(w.rows, args.rows), note=w.note + f" (first {args.rows} rows)")
    if args.cols:
        import dataclasses
        w = dataclasses.replace(w, cols=args.cols, name=f"{w.name}_cols{args.cols}", note=w.note + f" (rows of {args.cols} columns instead)")

    if args.impl == "reference":
        reference_arm(args, w)
        return

    import torch

    import __graft_entry__ as entry
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libfsoftmax has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        import contextlib
        with contextlib.redirect_stdout(sys.stderr):      # stdout carries the one JSON line only
            entry.build()
    if dist:
        dist.barrier()
    import paper_2607_24762_b200 as fs
    fs.binding.lib()

    def barrier():
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    props = torch.cuda.get_device_properties(local_rank)
    l2 = int(getattr(props, "L2_cache_size", 126 << 20))
    sampler = ClockSampler(smi_id(props, local_rank)) if rank == 0 and not args.no_clocks else None
    if args.op != "softmax":
        if args.op == "causal":
            r = time_device(w, args.steps, args.warmup, l2, causal_q=0, n_trains=args.trains)
            kept = sum(min(w.cols, i + 1) for i in range(w.rows))
            alg = (kept + w.rows * w.cols) * w.elem_size
            r = {"ms_per_step": round(r["ms_per_step"], 6), "algorithmic_bytes": alg,
                 "GB/s": round(alg / (r["ms_per_step"] * 1e-3) / 1e9, 1)}
        elif args.op == "log_softmax":
            r = time_log_softmax(w, args.steps, args.warmup, l2, eager=not args.no_cpu)
        elif args.op == "f32out":
            r = time_softmax_f32out(w, args.steps, args.warmup, l2, eager=not args.no_cpu)
        elif args.op == "masked":
            r = time_softmax_masked(w, args.steps, args.warmup, l2, eager=not args.no_cpu)
        elif args.op == "backward":
            r = time_softmax_backward(w, args.steps, args.warmup, l2)
        elif args.op == "norm":
            r = time_norm(args.norm_workload, args.steps, args.warmup, l2, eager=not args.no_cpu)
        else:
            r = time_router(w, 8, args.steps, args.warmup, l2)
        if rank == 0:
            print(json.dumps({"metric": METRIC, "op": args.op, "unit": UNIT, "value": r["GB/s"], "n_gpus": world,
                              "steps": args.steps, "warmup": max(3, args.warmup), "higher_is_better": True,
                              "config": {"workload": w.name, "shape": [w.rows, w.cols]}, **r}), flush=True)
        if dist:
            dist.barrier()
            dist.destroy_process_group()
        return
    res = time_device(w, args.steps, args.warmup, l2, sampler=sampler, barrier=barrier, min_clock_samples=8,
                      extras=world == 1, n_trains=args.trains,
                      causal_too=world == 1 and w.name == "cfg5" and not args.rows and not args.cols and args.all_workloads is not False)
    from paper_2607_24762_b200 import sharding
    ms = sharding.max_over_ranks(res["ms_per_step"], device="cuda")          # as slow as the slowest rank
    value = sharding.aggregate_throughput(w.min_bytes, ms * 1e-3, world) / 1e9

    res["steps"] = args.steps
    line = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": round(ms, 6), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "what": w.note, "shape": [w.rows, w.cols],
                       "storage_dtype": W.DTYPE_NAME[w.dtype], "scale": w.scale_f32, "kernel": res["kernel"],
                       "parallelism": f"rows independent: {world} replica(s) of the per-GPU workload, no collective",
                       "l2": f"rotating over {res['n_pairs']} independent (x,y) buffer pairs = "
                             f"{res['n_pairs'] * w.min_bytes / 2**20:.0f} MiB, L2 is {l2 / 2**20:.0f} MiB",
                       "timing": f"median of {res['trains']['n_trains']} trains of {args.steps} launches, one CUDA event pair per train",
                       "input_checksum": res["checksum"],
                       "rows_per_s": round(world * w.rows / (ms * 1e-3), 1)},
            "roofline": roofline_obj(w, ms, res["kernel"]),
            "gpu_launches": res["launches"],
            "clocks": res["clocks"]}
    line["roofline"]["trains_ms_per_step"] = res["trains"]
    for key in ("own_copy", "single_launch_ms"):           # the trains above are the headline; these explain it
        if key in res:
            line["roofline"][key] = res[key]

    if rank == 0 and world == 1:
        full = args.all_workloads is None or args.all_workloads
        per = {w.name: per_config_entry(w, res)}
        results = {w.name: res}
        if full:
            for name, ow in W.WORKLOADS.items():
                if name in per:
                    continue
                free, _ = torch.cuda.mem_get_info()
                if free < ow.min_bytes * 1.3:
                    per[name] = {"skipped": "not enough free device memory"}
                    continue
                k = max(20, min(1000, int(0.02 / max(ow.min_bytes / 6.0e12, 4e-6))))
                r = time_device(ow, k, 10, l2, extras=True, n_trains=args.trains, causal_too=name == "cfg5")
                r["steps"] = k
                results[name] = r
                per[name] = per_config_entry(ow, r)
        line["per_config"] = {k: per[k] for k in sorted(per)}
        if not args.no_e2e:
            line["e2e"] = time_e2e(w, steps=max(3, min(args.steps, 5 if w.min_bytes > (1 << 30) else 20)), warmup=1 if w.min_bytes > (1 << 30) else 2)
        if not args.no_cpu:
            line["cpu_baseline"] = cpu_baseline(w)
            if full:
                line["cpu_baselines"] = {name: (line["cpu_baseline"] if name == w.name else cpu_baseline(ow, 4.0))
                                         for name, ow in sorted(W.WORKLOADS.items())}
        if full:
            try:
                line["fixed_cost"] = {n: fit_fixed_cost(W.WORKLOADS[n], l2) for n in ("cfg2", "cfg3")}
            except Exception as exc:                       # never lose the main line to an extra
                line["fixed_cost"] = {"error": str(exc)[:200]}
            others = {}
            # the causal entry point on the causal workload: the masked half of x is never read
            if "causal_ms_per_step" in results.get("cfg5", {}):
                ow = W.WORKLOADS["cfg5"]
                cms = results["cfg5"]["causal_ms_per_step"]
                read_b = ow.rows * (ow.rows + 1) // 2 * ow.elem_size
                alg = read_b + ow.rows * ow.cols * ow.elem_size
                gbs = alg / (cms * 1e-3) / 1e9
                peak, which = measured_peak()
                others["cfg5_causal"] = {"what": "fs_softmax_causal(q_offset=0) on cfg5: reads only columns j <= i, writes every column",
                                         "kernel": "cluster", "ms_per_step": round(cms, 6),
                                         "algorithmic_bytes": alg, "GB/s": round(gbs, 1),
                                         "frac_of_measured_copy": round(gbs / peak, 4),
                                         "speedup_vs_cfg5": round(results["cfg5"]["ms_per_step"] / cms, 3)}
            # the entry point that allocates nothing, on the vocabulary-sized workload (the split-row kernel with its
            # status word in the fixed device array) and on rows beyond a cluster's shared memory (two kernels, the
            # pairs between them in the same array)
            try:
                others["cfg4_static"] = time_static(W.WORKLOADS["cfg4"], 300, l2)
                import dataclasses
                others["long_rows_static"] = time_static(dataclasses.replace(W.WORKLOADS["cfg4"], name="16 rows of 8 MiB", rows=16,
                                                                             cols=1 << 22), 100, l2)
            except Exception as exc:
                others["cfg4_static"] = {"error": str(exc)[:200]}
            # the router step (softmax over experts + top-8, renormalised) on the router workload
            rw = W.WORKLOADS["cfg3"]
            try:
                others["cfg3_router_top8"] = time_router(rw, 8, 500, 10, l2)
            except Exception as exc:                       # never lose the main line to an extra
                others["cfg3_router_top8"] = {"error": str(exc)[:200]}
            # log_softmax on the vocabulary-sized and the attention-score workloads
            for lname in ("cfg4", "cfg2"):
                try:
                    others[lname + "_log_softmax"] = time_log_softmax(W.WORKLOADS[lname], 300, 10, l2)
                except Exception as exc:
                    others[lname + "_log_softmax"] = {"error": str(exc)[:200]}
            try:
                others["cfg2_f32out"] = time_softmax_f32out(W.WORKLOADS["cfg2"], 300, 10, l2)
            except Exception as exc:
                others["cfg2_f32out"] = {"error": str(exc)[:200]}
            try:
                others["cfg2_masked"] = time_softmax_masked(W.WORKLOADS["cfg2"], 300, 10, l2)
            except Exception as exc:
                others["cfg2_masked"] = {"error": str(exc)[:200]}
            for bname in ("cfg2", "cfg4"):
                try:
                    others[bname + "_backward"] = time_softmax_backward(W.WORKLOADS[bname], 300, 10, l2)
                except Exception as exc:
                    others[bname + "_backward"] = {"error": str(exc)[:200]}
            # the normalisation entry points on the shapes of the paper's second workload family
            for nname in NORM_WORKLOADS:
                try:
                    others[nname] = time_norm(nname, 200, 10, l2)
                except Exception as exc:
                    others[nname] = {"error": str(exc)[:200]}
            line["workloads"] = others
    elif rank == 0:
        line["e2e"] = None
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
