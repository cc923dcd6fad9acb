#!/usr/bin/env python
"""Benchmark of the fused Sampling-VT operator on B200.

A *step* is one pass of the whole operator (stage matrices -> project -> validity -> bilinear
weights -> per-z normalisation -> gather/accumulate -> store) over one batch of FRAMES
independent synthetic frames of the chosen workload, each frame one call of
``flashbev_sampling_vt`` through the C ABI on its own device-resident inputs.  The frames of a
step together exceed the L2 cache several times over, so every launch starts L2-cold without an
explicit flush.  The launches of a step are replayed from a CUDA graph so that the number is the
GPU's, not the Python launch loop's (``--no-graph`` times direct launches instead).

Prints ONE JSON line.  ``value`` is whole-job sample-channels/s (all B*N*X*Y*Z*C candidate
sample-channels of every frame on every rank / device time, max over ranks).

``--impl reference`` times the fp64 CPU oracle (a deliberately plain program) on the host cores
for the same workload and metric.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_10071_b200 import workloads as wl  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
MIN_LAUNCHES_PER_STEP = 64
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel (bytes), from ncu captures of single
# launches taken from the middle of a step of rotating frames -- the regime that is timed -- summarised under
# profiles/vt_tiled_kernel_<workload>.md.  The output of a launch is still partly in the 126 MB L2 when its kernel
# ends, so these figures can lie below the algorithmic bytes: see `traffic_note` in the JSON line.
NCU_DRAM_TRAFFIC = {"tiny": 0.342e6, "representative": 4.78e6, "half_taller": 8.20e6, "long_range": 41.00e6, "high_res": 21.45e6}
TRAFFIC_NOTE = ("dram__bytes_read.sum + dram__bytes_write.sum of one launch captured in the middle of a rotating-frame "
                "step (ncu, one pass); part of a launch's output is written back from L2 after its kernel ends, so the "
                "figure can be below the algorithmic bytes")
FALLBACK_HBM_GBS = 6650.0
METRIC = "fused_sampling_vt_throughput"
UNIT = "sample-channels/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def whole_job_value(total_ms_local: float, units_per_rank: float, world: int, reduce_max=None) -> tuple:
    """Weak-scaling aggregate: every rank processes `units_per_rank`; the job's time is the slowest
    rank's device time.  `reduce_max(x)` returns the maximum of x over ranks (identity if None)."""
    total_ms = float(reduce_max(total_ms_local)) if (reduce_max is not None and world > 1) else float(total_ms_local)
    return world * units_per_rank / (total_ms * 1e-3), total_ms


def frames_for(w: wl.Workload, min_bytes: int) -> int:
    """Frames per step: their inputs and outputs together exceed `min_bytes` (L2-cold launches without a flush), and
    there are enough launches for the timed region of a step to be milliseconds long."""
    return max(MIN_LAUNCHES_PER_STEP, -(-min_bytes // w.unique_bytes))


def oracle_throughput(w: wl.Workload, seconds_budget: float, max_frames: int):
    """Time the oracle as it stands on the host cores over whole frames of the workload."""
    from oracle import flashbev_oracle as orc
    orc.build()
    inp = wl.make_inputs(w)
    t0 = time.perf_counter()
    frames = 0
    while frames < max_frames and (frames == 0 or time.perf_counter() - t0 < seconds_budget):
        orc.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, w.reduce)
        frames += 1
    dt = time.perf_counter() - t0
    # one thread, best of three frames (about a second for the benchmark workload)
    one = []
    for _ in range(3):
        t1 = time.perf_counter()
        orc.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, w.reduce, threads=1)
        one.append(time.perf_counter() - t1)
    return {"value": frames * w.sample_channels / dt, "unit": UNIT, "cores": orc.max_threads(), "kind": "oracle",
            "sample": f"{frames} whole frame(s) of the '{w.name}' workload, {dt / frames * 1e3:.1f} ms each",
            "ms_per_frame": dt / frames * 1e3, "one_thread_ms_per_frame": min(one) * 1e3,
            "one_thread_value": w.sample_channels / min(one)}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import flashbev_oracle as orc
    orc.build()
    inp = wl.make_inputs(w)
    frames_per_step = 1
    for _ in range(args.warmup):
        orc.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, w.reduce)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.sampling_vt(inp.features, inp.lidar2img, w.img_hw, w.bev_range, w.grid, w.reduce)
    dt = time.perf_counter() - t0
    value = args.steps * frames_per_step * w.sample_channels / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "frames_per_step": frames_per_step, "note": "fp64 CPU oracle on the host cores"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.max_threads(), "kind": "oracle",
                         "sample": f"{frames_per_step} whole frame of '{w.name}' per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


class DeviceFrames:
    """FRAMES independent frames of one workload, resident on the device, with their parameter structs."""

    def __init__(self, w, frames, device, rank, kernel=0, tune=(0, 0, 0, 0)):
        import torch
        from paper_2607_10071_b200 import binding as fb
        self.w, self.frames = w, frames
        X, Y, Z = w.grid
        self.feats, self.mats, self.outs, self.params = [], [], [], []
        base = wl.make_inputs(w, stream=1000 * rank)
        g = torch.Generator(device=device).manual_seed(2607_10071 + rank)
        for i in range(frames):
            if i == 0:
                f = torch.from_numpy(base.features).to(device)
            else:  # same shape and distribution, different values (standard normal, seeded, drawn on the device)
                f = torch.randn(base.features.shape, generator=g, dtype=torch.float32, device=device)
            if w.dtype == "bf16":
                f = f.to(torch.bfloat16)
            self.feats.append(f.contiguous())
            self.mats.append(torch.from_numpy(base.lidar2img).to(device))
            self.outs.append(torch.empty((w.B, X, Y, w.C), dtype=torch.float32, device=device))
            self.params.append(fb.make_params(
                self.feats[-1].data_ptr(), fb.BF16 if w.dtype == "bf16" else fb.F32, self.mats[-1].data_ptr(),
                w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range, w.grid, w.reduce, self.outs[-1].data_ptr(),
                None, kernel, tune))
        self.fb = fb

    def launch_all(self, stream_ptr):
        n = 0
        for p in self.params:
            self.fb.flashbev_sampling_vt(p, stream_ptr)
            n += self.fb.flashbev_last_launch_count()
        return n


def time_steps(torch, step_fn, steps, warmup, dist_barrier):
    """Device time of `steps` steps: per-step CUDA events on the current stream."""
    for _ in range(warmup):
        step_fn()
    torch.cuda.synchronize()
    dist_barrier()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    t_all0, t_all1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_all0.record()
    for a, b in evs:
        a.record()
        step_fn()
        b.record()
    t_all1.record()
    torch.cuda.synchronize()
    dist_barrier()
    torch.cuda.synchronize()
    per = [a.elapsed_time(b) for a, b in evs]
    return t_all0.elapsed_time(t_all1), per


def measure_workload(torch, w, args, device, rank, dist_barrier, steps, warmup, kernel=0, tune=(0, 0, 0, 0)):
    frames = args.frames or frames_for(w, 3 * L2_BYTES)
    df = DeviceFrames(w, frames, device, rank, kernel, tune)
    stream = torch.cuda.Stream(device)
    launches_per_step = frames
    with torch.cuda.stream(stream):
        sp = stream.cuda_stream
        df.launch_all(sp)  # first call: module load
        torch.cuda.synchronize()
        if args.no_graph:
            def step_fn():
                df.launch_all(sp)
        else:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                df.launch_all(torch.cuda.current_stream().cuda_stream)

            def step_fn():
                graph.replay()
        total_ms, per = time_steps(torch, step_fn, steps, warmup, dist_barrier)
    kname = df.fb.flashbev_last_kernel_name()
    return {"frames": frames, "total_ms": total_ms, "per_step_ms": per, "launches_per_step": launches_per_step,
            "kernel": kname, "df": df}


def measure_regimes(torch, df, device):
    """Secondary figures of one workload, from the frames already on the device: warm-L2 latency (the same frame
    back to back in a graph), the latency of single launches without a graph (events around each launch, frames
    rotating, so L2-cold), and the number of valid samples (from the kernel's own count output)."""
    fb = df.fb
    w = df.w
    X, Y, Z = w.grid
    stream = torch.cuda.Stream(device)
    reps = 20
    with torch.cuda.stream(stream):
        sp = stream.cuda_stream
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for _ in range(reps):
                fb.flashbev_sampling_vt(df.params[0], torch.cuda.current_stream().cuda_stream)
        _, per = time_steps(torch, graph.replay, 10, 3, lambda: None)
        warm = statistics.median(per) / reps
        singles = []
        for _ in range(3):
            for p in df.params:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                fb.flashbev_sampling_vt(p, sp)
                b.record()
                singles.append((a, b))
        torch.cuda.synchronize()
        single = statistics.median(a.elapsed_time(b) for a, b in singles[len(df.params):])
        cnt = torch.zeros((w.B, X, Y), dtype=torch.int32, device=device)
        pc = fb.make_params(df.feats[0].data_ptr(), fb.BF16 if w.dtype == "bf16" else fb.F32, df.mats[0].data_ptr(),
                            w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range, w.grid, w.reduce, df.outs[0].data_ptr(),
                            cnt.data_ptr())
        fb.flashbev_sampling_vt(pc, sp)
        torch.cuda.synchronize()
    return {"warm_l2_latency_ms": round(warm, 5), "single_launch_no_graph_latency_ms": round(single, 5),
            "valid_samples": int(cnt.sum().item())}


def measure_backward(torch, w, args, device, steps, warmup, dist_barrier):
    """Latency of flashbev_sampling_vt_backward (memset + scatter kernel) per frame, L2-cold frames."""
    from paper_2607_10071_b200 import binding as fb
    X, Y, Z = w.grid
    Hf, Wf = w.feat_hw
    per_frame = w.output_bytes + w.B * w.N * Hf * Wf * w.C * 4
    frames = max(4, -(-3 * L2_BYTES // per_frame))
    base = wl.make_inputs(w)
    mats = torch.from_numpy(base.lidar2img).to(device)
    g = torch.Generator(device="cpu").manual_seed(99)
    gouts = [torch.randn((w.B, X, Y, w.C), generator=g, dtype=torch.float32).to(device) for _ in range(frames)]
    gfeats = [torch.empty((w.B, w.N, Hf, Wf, w.C), dtype=torch.float32, device=device) for _ in range(frames)]
    ps = [fb.make_backward_params(go.data_ptr(), mats.data_ptr(), w.B, w.N, w.C, w.feat_hw, w.img_hw, w.bev_range,
                                  w.grid, w.reduce, gf.data_ptr()) for go, gf in zip(gouts, gfeats)]
    stream = torch.cuda.Stream(device)
    with torch.cuda.stream(stream):
        for p in ps:
            fb.flashbev_sampling_vt_backward(p, stream.cuda_stream)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for p in ps:
                fb.flashbev_sampling_vt_backward(p, torch.cuda.current_stream().cuda_stream)
        total_ms, per = time_steps(torch, graph.replay, steps, warmup, dist_barrier)
    return statistics.mean(per) / frames


def measure_tensorized(torch, w, device, iters=5):
    """Latency and peak memory of the PyTorch tensorised baseline (paper Alg. 1) on the same GPU: context."""
    from paper_2607_10071_b200 import tensorized_baseline as tb
    if w.dtype != "f32":
        return None
    inp = wl.make_inputs(w)
    feats = torch.from_numpy(inp.features).to(device)
    mats = torch.from_numpy(inp.lidar2img).to(device)
    for _ in range(2):
        tb.sampling_vt_tensorized(feats, mats, w.img_hw, w.bev_range, w.grid, w.reduce)
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats()
    base = torch.cuda.memory_allocated()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(iters):
        tb.sampling_vt_tensorized(feats, mats, w.img_hw, w.bev_range, w.grid, w.reduce)
    b.record()
    torch.cuda.synchronize()
    return {"latency_ms": a.elapsed_time(b) / iters, "peak_mb": (torch.cuda.max_memory_allocated() - base) / 1e6}


def measure_sca(torch, device, P, iters=10, chunk_records=0, bf16=False):
    """Latency of the fused spatial cross-attention at BEVFormer-base sizes (inputs ~350 MB+ per call: L2-cold)."""
    from paper_2607_10071_b200 import binding as fb
    c = wl.make_sca_inputs(P=P)
    t = {k: torch.from_numpy(c[k]).to(device) for k in ("value", "lidar2img", "offsets", "weights")}
    if bf16:
        t["value"] = t["value"].to(torch.bfloat16)
    out = torch.empty((1, c["grid"][0] * c["grid"][1], 256), dtype=torch.float32, device=device)
    call = lambda: fb.sca(t["value"], c["level_hw"], t["lidar2img"], t["offsets"], t["weights"], c["img_hw"],
                          c["bev_range"], c["grid"], out=out, chunk_records=chunk_records)
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(iters):
        call()
    b.record()
    torch.cuda.synchronize()
    bytes_unique = sum(v.numel() * v.element_size() for v in t.values()) + out.numel() * 4
    ms = a.elapsed_time(b) / iters
    return {"latency_ms": ms, "unique_mb": bytes_unique / 1e6, "hbm_roofline_frac_of_measured":
            bytes_unique / (ms * 1e-3) / 1e9 / measured_peaks()[0]}


def measure_e2e(torch, w, args, device, steps, warmup, dist_barrier):
    """Same metric through flashbev_sampling_vt_host: pinned host inputs, host output, copies timed."""
    from paper_2607_10071_b200 import binding as fb
    frames = max(2, min(args.frames or frames_for(w, 3 * L2_BYTES), 8))
    X, Y, Z = w.grid
    inp = wl.make_inputs(w)
    if w.dtype == "bf16":
        hf = torch.from_numpy(inp.features_bf16.view(np.int16)).pin_memory()
    else:
        hf = torch.from_numpy(inp.features).pin_memory()
    hm = torch.from_numpy(inp.lidar2img).pin_memory()
    houts = [torch.empty((w.B, X, Y, w.C), dtype=torch.float32).pin_memory() for _ in range(frames)]
    ps = [fb.make_params(hf.data_ptr(), fb.BF16 if w.dtype == "bf16" else fb.F32, hm.data_ptr(), w.B, w.N, w.C,
                         w.feat_hw, w.img_hw, w.bev_range, w.grid, w.reduce, ho.data_ptr()) for ho in houts]
    need = fb.flashbev_host_staging_bytes(ps[0])
    stagings = [torch.empty(need, dtype=torch.uint8, device=device) for _ in range(frames)]
    stream = torch.cuda.Stream(device)
    # frames go round-robin over three worker streams so that the upload of one frame, the kernel of
    # another and the download of a third overlap (the calls are asynchronous); the timing stream
    # forks to the workers at the start of a step and joins them at its end
    workers = [torch.cuda.Stream(device) for _ in range(3)]
    fork = torch.cuda.Event()
    joins = [torch.cuda.Event() for _ in workers]

    def step_fn():
        fork.record(stream)
        for wk in workers:
            wk.wait_event(fork)
        for i, (p, st) in enumerate(zip(ps, stagings)):
            fb.flashbev_sampling_vt_host(p, st.data_ptr(), need, workers[i % 3].cuda_stream)
        for wk, ev in zip(workers, joins):
            ev.record(wk)
            stream.wait_event(ev)

    with torch.cuda.stream(stream):
        total_ms, _ = time_steps(torch, step_fn, steps, warmup, dist_barrier)
    return {"value_per_rank": steps * frames * w.sample_channels / (total_ms * 1e-3), "frames": frames,
            "h2d": frames * (w.feature_bytes + w.matrix_bytes), "d2h": frames * w.output_bytes, "total_ms": total_ms}


def measure_capacity(torch, device, base_ms: float, base_mb: float):
    """Deployment capacity in the manner of the paper's Table 5, on this GPU and at the paper's reference shape: the
    largest number of height bins and the largest square BEV grid the fused operator handles within the latency of
    the tensorised baseline (Z = 8, 200 x 200), and the largest grid within the baseline's peak memory."""
    from paper_2607_10071_b200 import binding as fb
    wp = wl.get("paper_shape")
    inp = wl.make_inputs(wp)
    feats = torch.from_numpy(inp.features).to(device)
    mats = torch.from_numpy(inp.lidar2img).to(device)
    cell = (wp.bev_range[1] - wp.bev_range[0]) / wp.grid[0]

    def latency_ms(X, Z):
        half = X * cell / 2.0
        rng = (-half, half, -half, half, wp.bev_range[4], wp.bev_range[5])
        out = torch.empty((wp.B, X, X, wp.C), dtype=torch.float32, device=device)
        call = lambda: fb.sampling_vt(feats, mats, wp.img_hw, rng, (X, X, Z), wp.reduce, out=out)
        for _ in range(2):
            call()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 5
        a.record()
        for _ in range(reps):
            call()
        b.record()
        torch.cuda.synchronize()
        del out
        return a.elapsed_time(b) / reps

    def largest(fits, lo, hi):
        """Largest n in [lo, hi] with fits(n), assuming monotonicity and fits(lo)."""
        while lo < hi:
            mid = (lo + hi + 1) // 2
            if fits(mid):
                lo = mid
            else:
                hi = mid - 1
        return lo

    res = {"budget_latency_ms": base_ms, "budget_memory_mb": base_mb,
           "grid_rule": "cell size and height range of the paper's shape kept; the grid grows around the ego"}
    if latency_ms(wp.grid[0], wp.grid[2]) <= base_ms:
        res["max_height_bins_within_latency"] = largest(lambda z: latency_ms(wp.grid[0], z) <= base_ms, wp.grid[2], 4096)
        res["max_grid_within_latency"] = largest(lambda x: latency_ms(x, wp.grid[2]) <= base_ms, wp.grid[0], 6000)
    # memory of the fused operator = its inputs and its output (it has no workspace): solve for the grid
    budget = base_mb * 1e6 - wp.feature_bytes - wp.matrix_bytes
    g = int((budget / (wp.C * 4.0)) ** 0.5)
    ms = latency_ms(g, wp.grid[2])       # and run it once at that size
    res["max_grid_within_memory"] = g
    res["latency_ms_at_max_grid_within_memory"] = ms
    res["paper_rtx_a6000"] = {"max_height_bins_within_latency": 58, "max_grid_within_latency": 529,
                              "max_grid_within_memory": 1992, "source": "Table 5"}
    return res


def full_block(torch, w, args, device, rank, barrier, steps, warmup, world, reduce_max, kernel=0, tune=(0, 0, 0, 0),
               clock_sampler=None, cpu_seconds=12.0):
    """Everything the JSON line carries for one workload: device-resident throughput, roofline, end to end, memory,
    CPU baseline."""
    from paper_2607_10071_b200 import binding as fb
    if clock_sampler is not None and rank == 0:
        clock_sampler.start()
    m = measure_workload(torch, w, args, device, rank, barrier, steps, warmup, kernel, tune)
    clocks = clock_sampler.stop() if (clock_sampler is not None and rank == 0) else None
    frames = m["frames"]
    value, total_ms = whole_job_value(m["total_ms"], steps * frames * w.sample_channels, world, reduce_max)
    launch_ms = statistics.mean(m["per_step_ms"]) / frames  # average duration of one launch (one frame)

    # peak memory of one call: nothing may be allocated
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    torch.cuda.reset_peak_memory_stats()
    a0 = torch.cuda.max_memory_allocated()
    fb.flashbev_sampling_vt(m["df"].params[0], torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    workspace = (torch.cuda.max_memory_allocated() - a0) + max(0, free0 - torch.cuda.mem_get_info()[0])
    m.pop("df")
    torch.cuda.empty_cache()

    e2e_steps = max(3, steps // 4)
    e2e = measure_e2e(torch, w, args, device, e2e_steps, 3, barrier)
    e2e_value, _ = whole_job_value(e2e["total_ms"], e2e_steps * e2e["frames"] * w.sample_channels, world, reduce_max)

    peak, peak_kind = measured_peaks()
    achieved = w.unique_bytes / (launch_ms * 1e-3) / 1e9
    blk = {
        "value": value, "ms_per_step": total_ms / steps, "latency_ms": launch_ms,
        "latency_ms_median": statistics.median(m["per_step_ms"]) / frames,
        "latency_ms_min": min(m["per_step_ms"]) / frames,
        "config": {"workload": w.name, "B": w.B, "N": w.N, "C": w.C, "feat_hw": list(w.feat_hw), "img_hw": list(w.img_hw),
                   "grid": list(w.grid), "bev_range": list(w.bev_range), "reduce": w.reduce, "frames_per_step": frames,
                   "l2": "inputs and outputs of a step total %.0f MB (> 3x the 126 MB L2), no flush" % (frames * w.unique_bytes / 1e6),
                   "launch": "direct" if args.no_graph else "cuda graph replay of the step's launches",
                   "kernel": m["kernel"]},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "traffic": NCU_DRAM_TRAFFIC.get(w.name), "traffic_note": TRAFFIC_NOTE,
                     "algorithmic_bytes_per_launch": w.unique_bytes, "frac_of_8TBs_nominal": achieved / 8000.0,
                     "target_frac": 0.5, "target_met": bool(achieved / peak >= 0.5),
                     "what_binds": "not HBM: a cached gather (features stay in L2); instruction issue and the L1 data "
                                   "pipe set the time, see profiles/"},
        "peak_mb": {"workspace_allocated_by_call": workspace / 1e6, "output": w.output_bytes / 1e6,
                    "inputs_plus_output": w.unique_bytes / 1e6},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                "frames_per_step": e2e["frames"],
                "api": "flashbev_sampling_vt_host (pinned host buffers, frames round-robin over 3 streams)"},
        "gpu_launches": steps * m["launches_per_step"],
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1 and rank == 0:
        blk["cpu_baseline"] = oracle_throughput(w, cpu_seconds, 200)
    return blk


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long_range", choices=list(wl.WORKLOADS),
                    help="headline workload (default: the largest configuration by unique bytes and outputs)")
    ap.add_argument("--frames", type=int, default=0, help="frames per step (0: at least 64, and enough to exceed 3x L2)")
    ap.add_argument("--no-graph", action="store_true", help="time direct launches instead of a CUDA graph replay")
    ap.add_argument("--no-table", action="store_true", help="skip the per-configuration table, the second full block and the context")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel", type=int, default=0, help="0 auto, 1 per-output, 2 tiled")
    ap.add_argument("--tune", type=str, default="0,0,0,0")
    ap.add_argument("--backward-only", action="store_true",
                    help="time flashbev_sampling_vt_backward on the workload's shape with fp32 gradients and print its own line "
                         "(one GPU; what the backward profile under profiles/ was captured with)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = wl.get(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2607_10071_b200 import binding as fb
    from paper_2607_10071_b200 import build as fbuild

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the operator has no CPU path")
    if rank == 0 and fbuild.needs_build():
        fbuild.build()
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

        def barrier():
            dist.barrier()
    else:
        def barrier():
            pass
    barrier()
    fb.lib()
    tune = tuple(int(t, 0) for t in args.tune.split(","))
    if args.backward_only:
        wb = wl.get(args.workload, dtype="f32")
        lat = measure_backward(torch, wb, args, device, args.steps, args.warmup, barrier)
        if rank == 0:
            print(json.dumps({"metric": "sampling_vt_backward_latency", "value": lat, "unit": "ms", "higher_is_better": False,
                              "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "dtype": "f32", "data": "synthetic",
                              "config": {"workload": wb.name, "C": wb.C, "grid": list(wb.grid), "feat_hw": list(wb.feat_hw),
                                         "launch": "cuda graph replay, memset + scatter kernel per frame"},
                              "gpu_launches": args.steps * max(4, -(-3 * L2_BYTES // (wb.output_bytes + wb.B * wb.N * wb.feat_hw[0] * wb.feat_hw[1] * wb.C * 4)))}))
        if world > 1:
            dist.destroy_process_group()
        return

    # max over ranks of the device time of the K steps
    def reduce_max(x):
        t = torch.tensor([x], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    head = full_block(torch, w, args, device, rank, barrier, args.steps, args.warmup, world, reduce_max, args.kernel, tune,
                      ClockSampler(local_rank))

    table, context, second = {}, {}, {}
    side_steps = max(3, args.steps // 4)
    if not args.no_table and world == 1:
        # the configuration with the most samples (64 height bins) gets a full block of its own
        other = "high_res" if w.name != "high_res" else "long_range"
        second[other] = full_block(torch, wl.get(other), args, device, rank, barrier, side_steps, 3, world, reduce_max,
                                   cpu_seconds=6.0)
        from oracle import flashbev_oracle as orc   # (CPU baseline leg: the oracle as it stands, timed beside the GPU)
        orc.build()
        for name in wl.CONFIG_ORDER:
            wi = wl.get(name)
            mi = measure_workload(torch, wi, args, device, rank, barrier, side_steps, 3)
            extra = measure_regimes(torch, mi.pop("df"), device)
            torch.cuda.empty_cache()
            lat = statistics.mean(mi["per_step_ms"]) / mi["frames"]
            peak, _ = measured_peaks()
            row = {"latency_ms": round(lat, 5), "sample_channels_per_s": wi.sample_channels / (lat * 1e-3),
                   "latency_ms_median": round(statistics.median(mi["per_step_ms"]) / mi["frames"], 5),
                   "latency_ms_min": round(min(mi["per_step_ms"]) / mi["frames"], 5),
                   "valid_sample_channels_per_s": extra["valid_samples"] * wi.C / (lat * 1e-3), **extra,
                   "hbm_roofline_frac_of_measured": wi.unique_bytes / (lat * 1e-3) / 1e9 / peak,
                   "hbm_roofline_frac_of_8TBs": wi.unique_bytes / (lat * 1e-3) / 1e9 / 8000.0,
                   "unique_mb": round(wi.unique_bytes / 1e6, 3), "output_mb": round(wi.output_bytes / 1e6, 3),
                   "kernel": mi["kernel"], "frames_per_step": mi["frames"], "reduce": wi.reduce}
            if not args.no_cpu_baseline:
                inp = wl.make_inputs(wi)
                t0 = time.perf_counter()
                orc.sampling_vt(inp.features, inp.lidar2img, wi.img_hw, wi.bev_range, wi.grid, wi.reduce)
                row["cpu_oracle_ms_per_frame"] = (time.perf_counter() - t0) * 1e3
                row["cpu_oracle_cores"] = orc.max_threads()
                if name in ("tiny", "representative"):
                    t0 = time.perf_counter()
                    orc.sampling_vt(inp.features, inp.lidar2img, wi.img_hw, wi.bev_range, wi.grid, wi.reduce, threads=1)
                    row["cpu_oracle_one_thread_ms_per_frame"] = (time.perf_counter() - t0) * 1e3
            if wi.reduce == wl.REDUCE_MEAN_OVER_VALID:
                # the paper's own normalisation (Eq. 1) on the same shape
                me = measure_workload(torch, wl.get(name, reduce=wl.REDUCE_CAMERA_MEAN_Z_SUM), args, device, rank, barrier,
                                      side_steps, 3)
                me.pop("df")
                row["latency_ms_eq1_mode"] = round(statistics.mean(me["per_step_ms"]) / me["frames"], 5)
            table[name] = row

        # the paper's own reference shape (Sec. 4.1: C=128 fp32, 56x100 maps, 200x200x8, Eq. 1), forward and
        # backward, next to the paper's figures on its hardware -- context, not a target
        wp = wl.get("paper_shape")
        mf = measure_workload(torch, wp, args, device, rank, barrier, side_steps, 3)
        mf.pop("df")
        torch.cuda.empty_cache()
        context["paper_shape"] = {
            "forward_latency_ms": statistics.mean(mf["per_step_ms"]) / mf["frames"],
            "backward_latency_ms": measure_backward(torch, wp, args, device, side_steps, 3, barrier),
            "paper_forward_ms": 1.77, "paper_backward_ms": 3.27, "paper_hardware": "RTX A6000, FP32 (Table 4)",
            "paper_trt_forward_ms": 1.128, "paper_trt_hardware": "RTX 4070 Ti SUPER, TensorRT FP32 (Table 6)"}
        tens = measure_tensorized(torch, wp, device)
        context["paper_shape"]["tensorized_pytorch_baseline_on_this_gpu"] = tens
        context["paper_shape"]["paper_tensorized_forward"] = {"latency_ms": 9.18, "peak_mb": 1971.94,
                                                              "hardware": "RTX A6000 (Table 4)"}
        if tens:
            context["paper_shape"]["deployment_capacity"] = measure_capacity(torch, device, tens["latency_ms"], tens["peak_mb"])
        context["representative_tensorized_pytorch_baseline"] = measure_tensorized(torch, wl.get("representative"), device)
        context["flashsca_bevformer_base"] = {
            f"P={P}": dict(measure_sca(torch, device, P), paper_flashsca_ms=ms, paper_bevformer_sca_ms=base,
                           paper_hardware="RTX 4070 Ti SUPER, TensorRT FP32 (Table 7)")
            for P, ms, base in ((8, 5.27, 8.96), (16, 8.16, 15.81), (32, 13.90, 29.27))}
        context["flashsca_bevformer_base"]["P=8, bf16 values"] = measure_sca(torch, device, 8, bf16=True)
        context["representative_backward_latency_ms"] = measure_backward(torch, wl.get("representative"), args, device,
                                                                          side_steps, 3, barrier)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if w.dtype == "f32" else "bf16 features, f32 accumulate", "data": "synthetic",
        "config": head["config"], "latency_ms": head["latency_ms"], "roofline": head["roofline"], "peak_mb": head["peak_mb"],
        "e2e": head["e2e"], "gpu_launches": head["gpu_launches"], "clocks": head["clocks"],
        "cpu_baseline": head.get("cpu_baseline"),
    }
    if second:
        line["also_measured"] = second
    if table:
        line["configs"] = table
    if context:
        line["context"] = context
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
