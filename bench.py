#!/usr/bin/env python
"""Benchmark of the B200 FFT / SAR library.

Metric: batched FFT effective GB/s = (bytes in + bytes out) / time, cold cache
(every batch is far larger than the 126 MB L2), on the workload
"N=4096, batch=32768 complex64, contiguous, forward". One step = one
fft_execute over the whole batch. Also reported in the same JSON line: the other
workloads (N=8192/16384 in fp32 and fp16 storage, 4096^2 column and 2-D
transforms, the 4096^2 range-Doppler SAR image in ms), the end-to-end number
with host buffers, the roofline fraction of the dominant kernel, and the CPU
oracle timed on this machine.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--only main]

For N > 1 launch under torch.distributed.run; every rank processes its own
batch of the same size (weak scaling, no data-path collective).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_32237_b200 import inputs, metrics, multi  # noqa: E402

MAIN = dict(n=4096, batch=32768, seed=1, dtype=0)
WORKLOAD = "N=4096 batch=32768 complex64 forward, contiguous rows (1 GiB in + 1 GiB out)"


# ----------------------------------------------------------------------------- helpers
def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons while the timed region
    runs: NVML from a polling thread every 2 ms, or nvidia-smi every 100 ms if NVML is not
    importable. Reading only; no setting is changed."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.samples = []          # (time, sm_mhz, reasons bitmask)
        self.window = [None, None]  # timed region, time.monotonic()
        self.max_mhz = None
        self.nvml = None
        self.stop_flag = False

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            idx = self.index
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            if vis:
                try:
                    idx = int(vis.split(",")[self.index])
                except (ValueError, IndexError):
                    idx = self.index
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nvml = pynvml
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _poll(self):
        n = self.nvml
        while not self.stop_flag:
            try:
                mhz = float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM))
                try:
                    rs = int(n.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                except Exception:
                    rs = int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                self.samples.append((time.monotonic(), mhz, rs))
            except Exception:
                pass
            time.sleep(0.002)

    def mark_begin(self):
        self.window[0] = time.monotonic()

    def mark_end(self):
        self.window[1] = time.monotonic()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.monotonic(), line.strip()))

    def stop(self):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        if self.nvml is not None:
            self.stop_flag = True
            self.thread.join(timeout=1)
            n = self.nvml
            bits = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
            t0, t1 = self.window
            inside = [(m, rs) for t, m, rs in self.samples if (t0 is None or t >= t0) and (t1 is None or t <= t1)]
            if not inside and self.samples:      # a region shorter than one poll: the nearest sample
                mid = 0.5 * ((t0 or 0.0) + (t1 or 0.0))
                t, m, rs = min(self.samples, key=lambda x: abs(x[0] - mid))
                inside = [(m, rs)]
            reasons = sorted(k for k, b in bits.items() if any(rs & b for _, rs in inside))
            sm = [m for m, _ in inside]
            return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": self.max_mhz,
                    "sm_min_mhz": float(min(sm)) if sm else None, "reasons": reasons, "samples": len(sm),
                    "source": "nvml, 2 ms polling during the timed region"}
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["clock sampling unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        t0, t1 = self.window
        lines = [ln for t, ln in self.lines if (t0 is None or t >= t0 - 0.1) and (t1 is None or t <= t1 + 0.1)]
        if not lines:
            lines = [ln for _, ln in self.lines]
        for ln in lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for nm, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm), "source": "nvidia-smi -lms 100"}


def run_landscape(args):
    """Throughput against transform size, N = 8 ... 2^20 (the paper's Figure "landscape", our
    kernels only): cold on a 1 GiB footprint (512 MiB in + 512 MiB out, a 512 MiB scratch write
    before every sample), the same number of points cold with fp16 storage (half the bytes), and
    hot on a 32 MiB footprint that stays in the 126 MB L2."""
    import torch
    torch.cuda.set_device(0)
    from paper_2609_32237_b200 import binding as B
    peak, _ = measured_peak_gbs()
    stream = torch.cuda.current_stream()
    scratch = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    big = torch.randn(1 << 26, 2, device="cuda")
    big_out = torch.empty_like(big)
    rows = []
    for lg in range(3, 21):
        n = 1 << lg
        row = {"n": n}
        for label, points, cold, dtype in (("cold_1gib", 1 << 26, True, 0), ("cold_fp16_storage", 1 << 26, True, 1),
                                           ("hot_32mib", 1 << 21, False, 0)):
            batch = points // n
            plan = B.fft_plan_create(n, batch, 1, n, -1, dtype)
            need = B.fft_plan_workspace_bytes(plan)
            ws = None
            if need:
                ws = torch.empty(need, dtype=torch.uint8, device="cuda")
                B.fft_plan_set_workspace(plan, ws.data_ptr(), need)
            call = lambda: B.fft_execute(plan, big.data_ptr(), big_out.data_ptr(), torch.cuda.current_stream().cuda_stream)
            for _ in range(3):
                call()
            torch.cuda.synchronize()
            nb = metrics.fft_bytes(n, batch, dtype)
            if cold:
                per = []
                for _ in range(9):
                    flush_l2(torch, scratch)
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(stream)
                    call()
                    b.record(stream)
                    torch.cuda.synchronize()
                    per.append(a.elapsed_time(b))
                ms = float(np.median(per))
            else:
                reps = 200
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for _ in range(reps):
                    call()
                b.record(stream)
                torch.cuda.synchronize()
                ms = min(a.elapsed_time(b) / reps, hot_graph_ms(torch, call, reps))   # the faster of stream and graph replay
            B.fft_plan_destroy(plan)
            del ws
            row[label] = {"batch": batch, "us": ms * 1e3, "gbs": nb / ms / 1e6,
                          "gflops": metrics.fft_gflops(n, batch, ms * 1e-3)}
        rows.append(row)
    print(json.dumps({"landscape": "forward rows, N = 8 ... 2^20", "hbm_peak_gbs": peak, "rows": rows}))
    return 0


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# ----------------------------------------------------------------------------- reference arm (CPU oracle)
def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return 0
    import oracle
    n = MAIN["n"]
    # size the per-step sample so that the whole run takes about half a minute
    probe = inputs.gaussian_complex64((256, n), MAIN["seed"]).astype(np.complex128)
    oracle.fft_rows(probe[:32])
    t0 = time.perf_counter()
    oracle.fft_rows(probe)
    per_transform = (time.perf_counter() - t0) / 256
    budget = 30.0 / max(1, args.steps + args.warmup)
    sample = int(max(16, min(MAIN["batch"], budget / per_transform)))
    x = inputs.gaussian_complex64((sample, n), MAIN["seed"]).astype(np.complex128)
    for _ in range(args.warmup):
        oracle.fft_rows(x)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.fft_rows(x)
    dt = (time.perf_counter() - t0) / args.steps
    gbs = metrics.fft_bytes(n, sample, 0) / dt / 1e9
    cores = oracle.num_threads()
    line = {
        "impl": "reference", "metric": "batched FFT effective GB/s", "value": gbs, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOAD, "sample": f"{sample} of 32768 transforms per step (bounded CPU sample)"},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle",
                         "sample": f"{sample} transforms of N={n} per step (float64 recursive radix-2)"},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- GPU arm
def time_calls(torch, fn, steps, warmup, stream):
    """Device time of `steps` calls of fn() on `stream`, warm-up first; returns
    (total ms, per-call ms list)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        a.record(stream)
        fn()
        b.record(stream)
    torch.cuda.synchronize()
    per = [a.elapsed_time(b) for a, b in evs]
    return sum(per), per


def flush_l2(torch, scratch):
    scratch.zero_()


def flush_l2_clean(torch, scratch):
    """The scratch write, then a read of half of it: L2 ends up holding clean lines, so the timed kernel
    does not also pay for writing back the dirty lines the flush itself left behind (up to ~120 MB, which
    is a large share of a workload that moves 256 MiB)."""
    scratch.zero_()
    scratch[: scratch.numel() // 2].view(torch.int64).sum()


def time_cold(torch, fn, stream, scratch, steps, warmup, clean=False):
    """Device time of fn(), one sample per step, each after an L2 flush outside the event pair."""
    per = []
    for i in range(warmup + steps):
        (flush_l2_clean if clean else flush_l2)(torch, scratch)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        torch.cuda.synchronize()
        if i >= warmup:
            per.append(a.elapsed_time(b))
    return per


def strips_one_rank(torch, B, sc, rd, dtype, world, stream, scratch, steps, whole_ms):
    desc = B.sar_desc_from_scene(sc, dtype)
    shards = [B.sar_rda_shard_create(desc, r, world) for r in range(world)]
    geo = [B.sar_rda_shard_get_geometry(s) for s in shards]
    ws = [torch.empty(int(g.workspace_bytes), dtype=torch.uint8, device="cuda") for g in geo]
    for s_, w, g in zip(shards, ws, geo):
        B.sar_rda_shard_set_workspace(s_, w.data_ptr(), int(g.workspace_bytes))
    ptrs = [w.data_ptr() for w in ws]
    strip = torch.empty(sc.n_azimuth, int(geo[0].bins), 2, device="cuda")
    for r, (s_, g) in enumerate(zip(shards, geo)):          # every strip filled once, so that step 2 runs on real data
        B.sar_rda_shard_range_compress(s_, rd[g.first_pulse:g.first_pulse + g.pulses].data_ptr(), ptrs, stream.cuda_stream)
    torch.cuda.synchronize()
    g0 = geo[0]
    rows0 = rd[g0.first_pulse:g0.first_pulse + g0.pulses]
    t1 = time_cold(torch, lambda: B.sar_rda_shard_range_compress(shards[0], rows0.data_ptr(), ptrs, stream.cuda_stream),
                   stream, scratch, steps, 2)
    def step2():
        B.sar_rda_shard_azimuth(shards[0], strip.data_ptr(), stream.cuda_stream)
        # the forward transform runs in place on the strip buffer: refill it outside the timed call
    t2 = []
    for i in range(steps + 2):
        for r, (s_, g) in enumerate(zip(shards, geo)):
            B.sar_rda_shard_range_compress(s_, rd[g.first_pulse:g.first_pulse + g.pulses].data_ptr(), ptrs, stream.cuda_stream)
        flush_l2(torch, scratch)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        step2()
        b.record(stream)
        torch.cuda.synchronize()
        if i >= 2:
            t2.append(a.elapsed_time(b))
    for s_ in shards:
        B.sar_rda_shard_destroy(s_)
    rc_ms, az_ms = float(np.median(t1)), float(np.median(t2))
    return {"range_compression_ms": rc_ms, "azimuth_steps_ms": az_ms, "sum_ms": rc_ms + az_ms,
            "whole_image_on_one_device_ms": whole_ms, "ratio_to_whole": (rc_ms + az_ms) / whole_ms,
            "halo_bins": [int(g0.halo_left), int(g0.halo_right)], "strip_bins": int(g0.bins),
            "note": "one rank's two steps per image, all strip buffers on this device; the inter-device stores and "
                    "the barrier between the steps are not in these numbers"}


def bench_fft(torch, B, n, batch, dtype, seed, steps, warmup, layout="rows", direction=-1, cold_flush=None,
              options=None, also_clean=False):
    stream = torch.cuda.current_stream()
    if layout == "rows":
        x = inputs.gaussian_complex64((batch, n), seed)
        plan = B.fft_plan_create(n, batch, 1, n, direction, dtype)
    else:
        x = inputs.uniform_complex64((n, batch), seed)
        plan = B.fft_plan_create(n, batch, batch, 1, direction, dtype)
    for key, value in (options or {}).items():
        B.fft_plan_set_option(plan, key, value)
    if dtype == 0:
        d_in = torch.from_numpy(x).cuda()
    else:
        d_in = torch.from_numpy(inputs.to_half_storage(x)).cuda()
    del x
    d_out = torch.empty_like(d_in)
    need = B.fft_plan_workspace_bytes(plan)
    ws = None
    if need:
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        B.fft_plan_set_workspace(plan, ws.data_ptr(), need)

    def call():
        B.fft_execute(plan, d_in.data_ptr(), d_out.data_ptr(), stream.cuda_stream)

    clean_per = None
    if cold_flush is None:
        total, per = time_calls(torch, call, steps, warmup, stream)
    else:
        per = time_cold(torch, call, stream, cold_flush, steps, warmup)
        total = sum(per)
        if also_clean:
            clean_per = time_cold(torch, call, stream, cold_flush, steps, 1, clean=True)
    B.fft_plan_destroy(plan)
    return total, per, clean_per


def issue_roofline(key, ms):
    """For the workloads bound by instruction issue: the warp instructions of one launch (from the ncu capture
    summarised under profiles/) against what the GPU can issue in the measured time at its maximum clock."""
    inst = metrics.NCU_WARP_INSTRUCTIONS[key]
    floor_ms = metrics.issue_roof_seconds(inst) * 1e3
    return {"bound": "alu", "unit": "warp instructions/s", "achieved": inst / (ms * 1e-3),
            "peak": 148 * 4 * 1.965e9, "frac": floor_ms / ms, "warp_instructions": inst, "ms_at_peak": floor_ms,
            "note": "peak = 148 SMs x 4 schedulers x 1.965 GHz, one warp instruction per scheduler and cycle"}


def summarize(per_ms, nbytes, peak):
    med = float(np.median(per_ms))
    q1, q3 = np.percentile(per_ms, [25, 75])
    gbs = nbytes / (med * 1e-3) / 1e9
    return {"ms_median": med, "ms_min": float(min(per_ms)), "ms_iqr": float(q3 - q1),
            "gbs": gbs, "frac_of_peak": gbs / peak}


def run_gpu(args):
    import torch
    rank, world, local = dist_env()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    from paper_2609_32237_b200 import binding as B   # fails loudly if the CUDA library is missing
    peak, peak_kind = measured_peak_gbs()
    stream = torch.cuda.current_stream()
    n, batch, dtype = MAIN["n"], MAIN["batch"], MAIN["dtype"]
    nbytes = metrics.fft_bytes(n, batch, dtype)

    # ---- main workload: inputs resident in HBM ---------------------------------
    x = inputs.gaussian_complex64((batch, n), multi.rank_seed(MAIN["seed"], rank))
    h_in = torch.from_numpy(x).pin_memory()
    h_out = torch.empty_like(h_in).pin_memory()
    d_in = h_in.cuda()
    d_out = torch.empty_like(d_in)
    plan = B.fft_plan_create(n, batch, 1, n, -1, dtype)

    def step():
        B.fft_execute(plan, d_in.data_ptr(), d_out.data_ptr(), stream.cuda_stream)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()                  # polls from before the warm-up; only samples inside the timed window count
    scratch = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(max(args.warmup, 3)):
        flush_l2(torch, scratch)
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    launches0 = B.launch_count()
    torch.cuda.synchronize()
    # Cold protocol: before every timed sample a 512 MiB scratch buffer is written on the same stream
    # (four times the 126 MB L2); one event pair brackets exactly one fft_execute; one sample per step.
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    sampler.mark_begin()
    for e0, e1 in evs:
        flush_l2(torch, scratch)
        e0.record(stream)
        step()
        e1.record(stream)
    torch.cuda.synchronize()
    sampler.mark_end()
    per = [e0.elapsed_time(e1) for e0, e1 in evs]
    launches = B.launch_count() - launches0
    if world > 1:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    q1, q3 = np.percentile(per, [25, 75])
    local_ms_per_step = float(np.median(per))
    value, ms_per_step = multi.aggregate_throughput(nbytes, local_ms_per_step, world, device="cuda")
    kernel_gbs = nbytes / (local_ms_per_step * 1e-3) / 1e9   # one launch per step: launch duration = step time

    # the same launches back to back (no scratch write in between): context beside the cold figure
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    hot_steps = max(args.steps, 20)
    e0.record(stream)
    for _ in range(hot_steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    hot_ms = e0.elapsed_time(e1) / hot_steps
    del scratch

    # the same kernel for at least two seconds of back-to-back launches: the board settles at its power cap
    # and the SM clock drops; clocks are sampled inside the window (read only), and the rate is also given
    # scaled to the maximum clock so that the clock dependence shows without touching any clock
    sustained = None
    if rank == 0 and not args.only_main:
        s2 = ClockSampler(local)
        s2.start()
        count = int(max(200, 2.2 / (hot_ms * 1e-3)))
        torch.cuda.synchronize()
        s2.mark_begin()
        e0.record(stream)
        for _ in range(count):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        s2.mark_end()
        c2 = s2.stop()
        sus_ms = e0.elapsed_time(e1) / count
        sus_gbs = nbytes / (sus_ms * 1e-3) / 1e9
        sustained = {"launches": count, "seconds": sus_ms * count * 1e-3, "ms_per_launch": sus_ms, "gbs": sus_gbs,
                     "frac_of_peak": sus_gbs / peak, "clocks": c2}
        if c2 and c2.get("sm_mhz") and c2.get("sm_max_mhz"):
            sustained["gbs_scaled_to_max_clock"] = sus_gbs * c2["sm_max_mhz"] / c2["sm_mhz"]

    # ---- end to end: host buffers, copies inside the timed region ------------------
    def step_host():
        B.fft_execute_host(plan, h_in.data_ptr(), h_out.data_ptr(), d_in.data_ptr(), d_out.data_ptr(),
                           stream.cuda_stream)

    e2e_steps = max(2, min(args.steps, 5))
    step_host()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        step_host()
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    e2e_value, _ = multi.aggregate_throughput(nbytes, e2e_ms / e2e_steps, world, device="cuda")
    checksum = float(h_out.view(torch.float32)[:8].abs().sum())
    B.fft_plan_destroy(plan)
    del d_in, d_out, h_in, h_out, x
    torch.cuda.empty_cache()

    line = {
        "metric": "batched FFT effective GB/s", "value": value, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD,
                   "cold_cache": "512 MiB scratch write before every timed launch (L2 flush), one event pair per "
                                 "fft_execute, value = bytes / median; inputs are larger than L2 as well",
                   "parallelism": f"replicas x{world}" if world > 1 else "1 gpu"},
        "ms_min": float(min(per)), "ms_iqr": float(q3 - q1),
        "hot": {"ms_per_step": hot_ms, "gbs": nbytes / (hot_ms * 1e-3) / 1e9, "steps": hot_steps,
                "note": "back-to-back launches between one event pair, no scratch write"},
        "pct_of_hbm_peak": 100.0 * kernel_gbs / peak, "gflops": metrics.fft_gflops(n, batch, ms_per_step * 1e-3) * world,
        "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": nbytes // 2, "d2h_bytes_per_step": nbytes // 2,
                "steps": e2e_steps, "checksum": checksum},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": kernel_gbs, "peak": peak, "unit": "GB/s",
                     "frac": kernel_gbs / peak, "traffic": metrics.NCU_TRAFFIC_BYTES.get("fft_rows_4096_c64"),
                     "peak_kind": f"of {peak_kind}", "algorithmic_bytes": nbytes,
                     "kernel": "fft_kernel<N=4096, rows, c64>"},
    }

    if rank == 0 and not args.only_main:
        line["others"] = run_others(torch, B, args, peak)
        line["others"]["fft_n4096_sustained"] = sustained
    if rank == 0:
        line["cpu_baseline"] = cpu_baseline(n)
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def run_others(torch, B, args, peak):
    """Every other workload, each timed cold (a 512 MiB scratch write before each
    sample, outside the event pair) with its own warm-up."""
    steps, warmup = max(5, min(args.steps, 15)), 3
    scratch = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    out = {}

    def clean_summary(per, nbytes):
        med = float(np.median(per))
        return {"ms_median": med, "gbs": nbytes / (med * 1e-3) / 1e9, "frac_of_peak": nbytes / (med * 1e-3) / 1e9 / peak,
                "note": "L2 flushed by the scratch write followed by a read, so that it holds no dirty lines"}

    def fft_case(name, n, batch, dtype, seed, layout="rows", direction=-1, options=None, also_clean=False):
        _, per, clean = bench_fft(torch, B, n, batch, dtype, seed, steps, warmup, layout, direction, cold_flush=scratch,
                                  options=options, also_clean=also_clean)
        s = summarize(per, metrics.fft_bytes(n, batch, dtype), peak)
        s["gflops"] = metrics.fft_gflops(n, batch, s["ms_median"] * 1e-3)
        if clean:
            s["clean_l2"] = clean_summary(clean, metrics.fft_bytes(n, batch, dtype))
        out[name] = s
        torch.cuda.empty_cache()

    # the copy rate of this very device in this very run, beside the stored peak (context only:
    # the roofline denominators stay the stored measurements)
    stream = torch.cuda.current_stream()
    src = torch.empty(1 << 30, dtype=torch.uint8, device="cuda").fill_(1)
    dst = torch.empty_like(src)
    per = []
    for i in range(warmup + steps):
        flush_l2(torch, scratch)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        dst.copy_(src)
        b.record(stream)
        torch.cuda.synchronize()
        if i >= warmup:
            per.append(a.elapsed_time(b))
    out["device_copy_1gib"] = summarize(per, 2 << 30, peak)
    out["device_copy_1gib"]["note"] = "device-to-device copy of 1 GiB (1 GiB read + 1 GiB written), same protocol"
    del src, dst
    torch.cuda.empty_cache()

    fft_case("fft_n4096_b32768_c64_inverse", 4096, 32768, 0, 1, direction=1)
    fft_case("fft_n8192_b16384_c64", 8192, 16384, 0, 2)
    fft_case("fft_n16384_b8192_c64", 16384, 8192, 0, 2)
    fft_case("fft_n8192_b16384_c32h", 8192, 16384, 1, 2)
    fft_case("fft_n16384_b8192_c32h", 16384, 8192, 1, 2)
    for name, key in (("fft_n8192_b16384_c32h", "fft_rows_8192_b16384_c32h"), ("fft_n16384_b8192_c32h", "fft_rows_16384_b8192_c32h")):
        out[name]["issue_roofline"] = issue_roofline(key, out[name]["ms_median"])
    fft_case("fft_n1024_b256_c64", 1024, 256, 0, 0)

    # block floating point on fp16 storage (one exponent per transform): the cost of the maximum search
    h = torch.from_numpy(inputs.to_half_storage(inputs.gaussian_complex64((16384, 8192), 2))).cuda()
    ho = torch.empty_like(h)
    ex = torch.zeros(16384, dtype=torch.int32, device="cuda")
    pb = B.fft_plan_create(8192, 16384, 1, 8192, -1, 1)
    per = []
    for i in range(warmup + steps):
        flush_l2(torch, scratch)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        B.fft_execute_bfp(pb, h.data_ptr(), 0, ho.data_ptr(), ex.data_ptr(), stream.cuda_stream)
        b.record(stream)
        torch.cuda.synchronize()
        if i >= warmup:
            per.append(a.elapsed_time(b))
    B.fft_plan_destroy(pb)
    out["fft_n8192_b16384_c32h_block_floating_point"] = summarize(per, metrics.fft_bytes(8192, 16384, 1), peak)
    del h, ho, ex
    torch.cuda.empty_cache()
    fft_case("fft_cols_4096x4096_c64", 4096, 4096, 0, 3, layout="cols", also_clean=True)
    fft_case("fft_cols_4096x4096_c64_plain_kernel", 4096, 4096, 0, 3, layout="cols", options={"stream": 0, "cluster": 1})
    out["fft_cols_4096x4096_c64_plain_kernel"]["note"] = "the non-persistent 4-column kernel (plain loads and stores), for comparison"
    fft_case("fft_cols_4096x16384_c64", 4096, 16384, 0, 3, layout="cols")
    fft_case("fft_cols_4096x4096_c32h", 4096, 4096, 1, 3, layout="cols")
    fft_case("fft_n65536_b2048_c64_four_step", 65536, 2048, 0, 5)
    fft_case("fft_cols_4096x4096_c64_via_transpose", 4096, 4096, 0, 3, layout="cols", options={"via_transpose": 1})
    out["fft_cols_4096x4096_c64_via_transpose"]["note"] = ("the paper's four-pass form as a comparison: transpose, row "
                                                           "transforms, transpose back (three passes; bytes counted once)")
    out["fft_n65536_b2048_c64_four_step"]["note"] = "two passes: algorithmic bytes counted once (16 B/point)"

    # 2-D: rows then columns, in place
    stream = torch.cuda.current_stream()
    m = torch.from_numpy(inputs.uniform_complex64((4096, 4096), 3)).cuda()
    pr = B.fft_plan_create(4096, 4096, 1, 4096, -1, 0)
    pc = B.fft_plan_create(4096, 4096, 4096, 1, -1, 0)
    def two_d():
        B.fft_execute(pr, m.data_ptr(), m.data_ptr(), stream.cuda_stream)
        B.fft_execute(pc, m.data_ptr(), m.data_ptr(), stream.cuda_stream)

    per = time_cold(torch, two_d, stream, scratch, steps, warmup)
    clean = time_cold(torch, two_d, stream, scratch, steps, 1, clean=True)
    B.fft_plan_destroy(pr)
    B.fft_plan_destroy(pc)
    out["fft2d_4096x4096_c64"] = summarize(per, 2 * metrics.fft_bytes(4096, 4096, 0), peak)
    out["fft2d_4096x4096_c64"]["clean_l2"] = clean_summary(clean, 2 * metrics.fft_bytes(4096, 4096, 0))
    del m

    # SAR: the chain, each step on its own, the variants kept for comparison, and end to end from host buffers
    sc = inputs.x_band_scene()
    raw = inputs.simulate_raw(sc, seed=4)
    h_raw = torch.from_numpy(raw).pin_memory()
    h_img = torch.empty_like(h_raw).pin_memory()
    rd = h_raw.cuda()
    img = torch.empty_like(rd)
    variants = {"": {}, "_slab_layout": {"layout": 1, "tile_columns": 4}, "_fused_step2": {"fused_rcmc": 1},
                "_via_transpose": {"layout": 2}}
    for dtype, base in ((0, "sar_4096x4096_fp32_intermediates"), (1, "sar_4096x4096_fp16_intermediates")):
        for suffix, opts in variants.items():
            p = B.sar_rda_params_create(B.sar_desc_from_scene(sc, dtype))
            for key, value in opts.items():
                B.sar_rda_set_option(p, key, value)
            need = B.sar_rda_workspace_bytes(p)
            ws = torch.empty(need, dtype=torch.uint8, device="cuda")
            B.sar_rda_set_workspace(p, ws.data_ptr(), need)

            def chain():
                B.sar_rda_form_image(rd.data_ptr(), p, img.data_ptr(), stream.cuda_stream)

            per = time_cold(torch, chain, stream, scratch, steps, warmup)
            r = summarize(per, metrics.sar_bytes(4096, 4096, dtype), peak)
            r["ms_per_image"] = r["ms_median"]
            r["options"] = opts
            if not suffix:
                r["issue_roofline"] = issue_roofline("sar_4096x4096_fp32" if dtype == 0 else "sar_4096x4096_fp16", r["ms_median"])
            per_step = [time_cold(torch, (lambda s=s: B.sar_rda_run_step(rd.data_ptr(), p, img.data_ptr(), s, stream.cuda_stream)),
                                  stream, scratch, steps, 1) for s in range(3)]
            r["passes_ms"] = {"range_compression": float(np.median(per_step[0])),
                              "azimuth_fft": float(np.median(per_step[1])),
                              "rcmc_filter_ifft": float(np.median(per_step[2]))}
            if not suffix:
                clean = time_cold(torch, chain, stream, scratch, steps, 1, clean=True)
                r["clean_l2"] = clean_summary(clean, metrics.sar_bytes(4096, 4096, dtype))
                # end to end: raw data in pinned host memory, image back to pinned host memory
                def host_chain():
                    B.sar_rda_form_image_host(h_raw.data_ptr(), p, h_img.data_ptr(), rd.data_ptr(), img.data_ptr(),
                                              stream.cuda_stream)
                e2e = time_cold(torch, host_chain, stream, scratch, 3, 1)
                r["e2e"] = {"ms_per_image": float(np.median(e2e)), "h2d_bytes_per_image": raw.nbytes,
                            "d2h_bytes_per_image": raw.nbytes, "checksum": float(h_img.view(torch.float32)[:8].abs().sum())}
            B.sar_rda_params_destroy(p)
            out[base + suffix] = r
            if not suffix:
                default_ms = r["ms_median"]
            del ws
        # Column-strip decomposition: what ONE rank of `world` does per image (its pulses' range compression,
        # scattered into all strips, and the azimuth steps on its own strip), timed on this one device with
        # every strip buffer local. The exchange between devices is not in these numbers.
        for world in (2, 8):
            out[f"{base}_column_strips_one_rank_of_{world}"] = strips_one_rank(torch, B, sc, rd, dtype, world, stream, scratch,
                                                                                steps, default_ms)
    return out


def run_case(args):
    """One workload on its own (small JSON line): for profiling a single kernel.
    --case rows:N:BATCH:c64|c32h[:inverse] | cols:N:BATCH:c64|c32h | sar:c64|c32h | sarstrips:c64|c32h"""
    import torch
    torch.cuda.set_device(0)
    from paper_2609_32237_b200 import binding as B
    peak, _ = measured_peak_gbs()
    parts = args.case.split(":")
    kind = parts[0]
    dt = {"c64": 0, "c32h": 1}
    stream = torch.cuda.current_stream()
    if kind in ("rows", "cols"):
        n, batch, dtype = int(parts[1]), int(parts[2]), dt[parts[3]]
        direction = 1 if (len(parts) > 4 and parts[4] == "inverse") else -1
        options = dict((kv.split("=")[0], int(kv.split("=")[1])) for kv in args.option)
        _, per, _ = bench_fft(torch, B, n, batch, dtype, 2, args.steps, args.warmup, kind, direction, options=options)
        out = summarize(per, metrics.fft_bytes(n, batch, dtype), peak)
    elif kind == "sar":
        dtype = dt[parts[1]]
        sc = inputs.x_band_scene()
        rd = torch.from_numpy(inputs.simulate_raw(sc, seed=4)).cuda()
        img = torch.empty_like(rd)
        p = B.sar_rda_params_create(B.sar_desc_from_scene(sc, dtype))
        for kv in args.option:
            B.sar_rda_set_option(p, kv.split("=")[0], int(kv.split("=")[1]))
        need = B.sar_rda_workspace_bytes(p)
        ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        B.sar_rda_set_workspace(p, ws.data_ptr(), need)
        _, per = time_calls(torch, lambda: B.sar_rda_form_image(rd.data_ptr(), p, img.data_ptr(), stream.cuda_stream),
                            args.steps, args.warmup, stream)
        out = summarize(per, metrics.sar_bytes(4096, 4096, dtype), peak)
        # each step on its own, cold (a 512 MiB scratch write before every sample)
        scratch = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
        cold = {}
        for label, fn in [("chain", lambda: B.sar_rda_form_image(rd.data_ptr(), p, img.data_ptr(), stream.cuda_stream))] + [
                (f"step{s}", (lambda s=s: B.sar_rda_run_step(rd.data_ptr(), p, img.data_ptr(), s, stream.cuda_stream)))
                for s in range(3)]:
            ts = []
            for i in range(9):
                flush_l2(torch, scratch)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            cold[label] = round(float(np.median(ts[2:])) * 1e3, 1)
        out["cold_us"] = cold
        B.sar_rda_params_destroy(p)
    elif kind == "sarstrips":
        # The column-strip image formation on real devices, one process per GPU (torch.distributed.run sets
        # RANK / LOCAL_RANK / WORLD_SIZE; without them: a process group of one). Per image: this rank's range
        # compression with its stores into every rank's strip, a barrier, the azimuth steps on its strip, a barrier;
        # device time per image, maximum over ranks.
        import torch.distributed as dist
        from paper_2609_32237_b200 import multi
        dtype = dt[parts[1]]
        rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
        local = int(os.environ.get("LOCAL_RANK", "0"))
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", local))
        sc = inputs.x_band_scene()
        job = multi.SarStripRank(B.sar_desc_from_scene(sc, dtype), host_barrier=any(o == "host_barrier=1" for o in args.option))
        g = job.geometry
        raw = inputs.simulate_raw(sc, seed=4)[g.first_pulse:g.first_pulse + g.pulses]
        rows = torch.from_numpy(np.ascontiguousarray(raw)).cuda()
        stream = torch.cuda.current_stream()
        scratch = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
        per = []
        for i in range(args.warmup + args.steps):
            flush_l2(torch, scratch)
            dist.barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            job.form(rows)
            b.record(stream)
            torch.cuda.synchronize()
            if i >= args.warmup:
                per.append(multi.max_over_ranks(a.elapsed_time(b), device="cuda"))
        out = summarize(per, metrics.sar_bytes(4096, 4096, dtype), peak)
        out["n_gpus"] = world
        out["strip"] = {"bins": int(g.bins), "halo": [int(g.halo_left), int(g.halo_right)], "pulses": int(g.pulses)}
        job.close()
        dist.destroy_process_group()
        if rank != 0:
            return 0
    else:
        raise SystemExit(f"unknown case {args.case}")
    out["case"] = args.case
    print(json.dumps(out))
    return 0


def hot_graph_ms(torch, call, reps):
    """Device time per launch of `reps` back-to-back launches replayed from a CUDA graph, so that the rate
    at which the host can issue launches (a few microseconds per call through the Python binding) does not
    bound short kernels. `call` must launch on torch's current stream."""
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        call()
        side.synchronize()
        with torch.cuda.graph(g, stream=side):
            for _ in range(reps):
                call()
        g.replay()
        side.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(side)
        g.replay()
        b.record(side)
        side.synchronize()
    return a.elapsed_time(b) / reps


def run_sweep(args):
    """Hot versus cold throughput of the N=4096 kernel against the batch footprint (the
    paper's Table "One 4096-Point Kernel vs. Batch Size"): hot = back-to-back launches on
    the same buffers, cold = a 512 MiB scratch write before every launch."""
    import torch
    torch.cuda.set_device(0)
    from paper_2609_32237_b200 import binding as B
    peak, _ = measured_peak_gbs()
    stream = torch.cuda.current_stream()
    scratch = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    n, rows = 4096, []
    for batch in (16, 64, 148, 296, 592, 1184, 2048, 4096, 8192, 16384, 32768):
        x = torch.randn(batch, n, 2, device="cuda")
        y = torch.empty_like(x)
        plan = B.fft_plan_create(n, batch, 1, n, -1, 0)
        call = lambda: B.fft_execute(plan, x.data_ptr(), y.data_ptr(), torch.cuda.current_stream().cuda_stream)
        reps = max(20, min(2000, (256 << 20) // (batch * n * 16)))
        for _ in range(5):
            call()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            call()
        b.record(stream)
        torch.cuda.synchronize()
        hot_ms = a.elapsed_time(b) / reps
        graph_ms = hot_graph_ms(torch, call, min(reps, 200))
        cold = []
        for _ in range(9):
            scratch.zero_()
            a.record(stream)
            call()
            b.record(stream)
            torch.cuda.synchronize()
            cold.append(a.elapsed_time(b))
        cold_ms = float(np.median(cold))
        B.fft_plan_destroy(plan)
        nb = metrics.fft_bytes(n, batch, 0)
        rows.append({"batch": batch, "footprint_mib": nb / 2 ** 20, "hot_gbs": nb / hot_ms / 1e6,
                     "cold_gbs": nb / cold_ms / 1e6, "hot_us": hot_ms * 1e3, "cold_us": cold_ms * 1e3,
                     "hot_graph_us": graph_ms * 1e3, "hot_graph_gbs": nb / graph_ms / 1e6,
                     "hot_gflops": metrics.fft_gflops(n, batch, min(hot_ms, graph_ms) * 1e-3)})
    print(json.dumps({"sweep": "N=4096 c64 forward, hot vs cold", "hbm_peak_gbs": peak, "rows": rows}))
    return 0


def cpu_baseline(n):
    """The oracle as it stands, timed on this machine's host cores on a bounded sample."""
    import oracle
    sample = 8192
    x = inputs.gaussian_complex64((sample, n), MAIN["seed"]).astype(np.complex128)
    oracle.fft_rows(x[:64])
    t0 = time.perf_counter()
    oracle.fft_rows(x)
    dt = time.perf_counter() - t0
    return {"value": metrics.fft_bytes(n, sample, 0) / dt / 1e9, "unit": "GB/s", "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": dt,
            "sample": f"{sample} of 32768 transforms of N={n} (float64 recursive radix-2, OpenMP over transforms)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--only-main", dest="only_main", action="store_true",
                    help="time only the headline workload (skip the other workloads)")
    ap.add_argument("--case", default=None,
                    help="run one workload only, e.g. rows:16384:8192:c64, cols:4096:4096:c64, sar:c64")
    ap.add_argument("--option", action="append", default=[],
                    help="with --case rows/cols: plan option KEY=VALUE (repeatable), e.g. cluster=4")
    ap.add_argument("--landscape", action="store_true", help="throughput against N = 8 ... 2^20, cold 1 GiB and hot 32 MiB")
    ap.add_argument("--sweep", action="store_true", help="hot vs cold throughput against the batch footprint")
    args = ap.parse_args()
    if args.sweep:
        return run_sweep(args)
    if args.landscape:
        return run_landscape(args)
    if args.case:
        return run_case(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
