#!/usr/bin/env python
"""Benchmark of the row-operator library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one launch of the headline operator (LayerNorm fp32 [4096, 4096], the
second benchmark configuration) through the C ABI on inputs already resident in
HBM; successive steps rotate over four buffer pairs so the working set (512 MiB)
exceeds L2.  The one JSON line printed by rank 0 carries the headline number,
the same figure for every configuration (`per_config`) and for the operators
over a non-last axis (`axis_rows`) and the fused residual add + normalisation
(`fused_rows`), the gated activations (`act_rows`) and arg-max / cumulative operators
(`reduction_rows`), the roofline fraction, the end-to-end figure
with host buffers, and the fp64 CPU oracle's timing.

With N > 1 (launched by torch.distributed.run) every rank runs the same
per-GPU workload on its own seed: rows are independent, there is no collective
on the data path ("weak" scaling, replicas).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2512_23424_b200 import workloads as wl  # noqa: E402

METRIC = "achieved HBM GB/s (fraction of B200 peak) and rows/s per op and shape"
HEADLINE = 2
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 * 1000 * 1000


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def profiled_traffic(name: str):
    """DRAM bytes per launch from the committed ncu summary, if one exists."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        with open(path) as fh:
            return json.load(fh).get(name)
    except Exception:
        return None


# --------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML in a background thread."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake", 0x2: "applications_clocks_setting"}

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self, note: str):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0,
                    "note": "NVML unavailable"}
        return {"sm_mhz": int(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples), "note": note}


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------
class DeviceWorkload:
    """A workload resident in HBM, with `pairs` rotating (x, y) buffer pairs."""

    def __init__(self, w: wl.Workload, pairs: int):
        import torch
        from paper_2512_23424_b200 import binding
        self.w, self.binding, self.torch = w, binding, torch
        tdt = {wl.F32: torch.float32, wl.BF16: torch.bfloat16, wl.F16: torch.float16}[w.dtype]

        def dev(a):
            if a is None:
                return None
            if w.dtype in (wl.F32, wl.F16):
                return torch.from_numpy(a).cuda()
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)

        x0 = dev(w.x)
        self.xs = [x0] + [x0.clone() for _ in range(pairs - 1)]
        self.ys = [torch.empty((w.rows, w.cols), dtype=tdt, device="cuda") for _ in range(pairs)]
        self.gamma, self.beta = dev(w.gamma), dev(w.beta)
        self.mask = binding.make_mask(x0, causal=w.causal_period > 0, causal_period=max(w.causal_period, 1))
        # arguments marshalled once per buffer pair: a step is then one C-ABI call
        self.calls = [binding.prepare(w.op, x, y, gamma=self.gamma, beta=self.beta, eps=w.eps,
                                      mask=self.mask) for x, y in zip(self.xs, self.ys)]
        self.i = 0

    def launch(self):
        call = self.calls[self.i % len(self.calls)]
        self.i += 1
        return call.launch()


class AxisDeviceWorkload:
    """A non-last-axis workload x[outer, reduce, inner] resident in HBM, rotating buffer pairs."""

    def __init__(self, w: wl.AxisWorkload, pairs: int):
        import torch
        from paper_2512_23424_b200 import binding
        self.w, self.binding, self.torch = w, binding, torch

        def dev(a):
            if a is None:
                return None
            if w.dtype == wl.F32:
                return torch.from_numpy(a).cuda()
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)

        x0 = dev(w.x)
        self.xs = [x0] + [x0.clone() for _ in range(pairs - 1)]
        self.ys = [torch.empty_like(x0) for _ in range(pairs)]
        self.gamma, self.beta = dev(w.gamma), dev(w.beta)
        self.i = 0

    def launch(self):
        k = self.i % len(self.xs)
        self.i += 1
        return self.binding.rowop_axis(self.w.op, self.xs[k], out=self.ys[k], gamma=self.gamma, beta=self.beta,
                                       eps=self.w.eps)


class FusedDeviceWorkload:
    """A fused residual add + normalisation workload resident in HBM, rotating buffer sets."""

    def __init__(self, w: wl.FusedWorkload, sets: int):
        import torch
        from paper_2512_23424_b200 import binding
        self.w, self.binding, self.torch = w, binding, torch

        def dev(a):
            if a is None:
                return None
            if w.dtype == wl.F32:
                return torch.from_numpy(a).cuda()
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)

        x0, r0 = dev(w.x), dev(w.res)
        self.xs = [x0] + [x0.clone() for _ in range(sets - 1)]
        self.rs = [r0] + [r0.clone() for _ in range(sets - 1)]
        self.ys = [torch.empty_like(x0) for _ in range(sets)]
        self.ss = [torch.empty_like(x0) for _ in range(sets)]
        self.gamma, self.beta = dev(w.gamma), dev(w.beta)
        self.i = 0

    def launch(self):
        k = self.i % len(self.xs)
        self.i += 1
        return self.binding.add_norm(self.w.op, self.xs[k], self.rs[k], gamma=self.gamma, beta=self.beta,
                                     eps=self.w.eps, out=self.ys[k], sum_out=self.ss[k])


class ActDeviceWorkload:
    """A gated-activation workload x[rows, 2 d] resident in HBM, rotating buffer pairs."""

    def __init__(self, w: wl.ActWorkload, pairs: int):
        import torch
        from paper_2512_23424_b200 import binding
        self.w, self.binding, self.torch = w, binding, torch
        if w.dtype == wl.F32:
            x0 = torch.from_numpy(w.x).cuda()
        else:
            x0 = torch.from_numpy(w.x.view(np.int16)).cuda().view(torch.bfloat16)
        self.xs = [x0] + [x0.clone() for _ in range(pairs - 1)]
        self.ys = [torch.empty((x0.shape[0], x0.shape[1] // 2), dtype=x0.dtype, device="cuda") for _ in range(pairs)]
        self.i = 0

    def launch(self):
        k = self.i % len(self.xs)
        self.i += 1
        return self.binding.act_mul(self.w.act, self.xs[k], out=self.ys[k])


def pairs_for(w) -> int:
    one = (w.algorithmic_bytes() if isinstance(w, (wl.AxisWorkload, wl.FusedWorkload, wl.ActWorkload, wl.ReductionWorkload))
           else 2 * w.rows * w.cols * w.itemsize)
    if one >= 3 * L2_BYTES:
        return 1
    return max(2, int(np.ceil(4 * L2_BYTES / one)))


def time_launches(dw: DeviceWorkload, steps: int, warmup: int, barrier=None):
    """Device time of `steps` back-to-back launches (CUDA events on the launch stream)."""
    torch = dw.torch
    for _ in range(max(warmup, 3)):
        dw.launch()
    torch.cuda.synchronize()
    if barrier is not None:
        barrier()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record()
    for _ in range(steps):
        dw.launch()
    stop.record()
    torch.cuda.synchronize()
    if barrier is not None:
        barrier()
    return start.elapsed_time(stop) * 1e-3          # seconds


def e2e_steps(w: wl.Workload, steps: int, warmup: int):
    """Same operator through the C ABI's host-buffer entry point: every step uploads the
    inputs from pinned host memory, runs the kernels and downloads the result, all inside
    the timed region (chunked and pipelined by the library over a caller-owned workspace)."""
    import torch
    from paper_2512_23424_b200 import binding
    tdt = torch.float32 if w.dtype == wl.F32 else torch.bfloat16

    def host(a):
        if a is None:
            return None
        t = torch.from_numpy(a if w.dtype == wl.F32 else a.view(np.int16))
        return (t if w.dtype == wl.F32 else t.view(torch.bfloat16)).pin_memory()

    host_x, gamma, beta = host(w.x), host(w.gamma), host(w.beta)
    host_y = torch.empty((w.rows, w.cols), dtype=tdt).pin_memory()
    ws = torch.empty(binding.host_workspace_bytes(w.rows, w.cols, tdt, gamma is not None, beta is not None),
                     dtype=torch.uint8, device="cuda")

    def step():
        binding.rowop_host(w.op, host_x, host_y, ws, gamma=gamma, beta=beta, eps=w.eps,
                           causal_period=w.causal_period)

    for _ in range(max(1, min(warmup, 3))):
        step()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        step()
    stop.record()
    torch.cuda.synchronize()
    secs = start.elapsed_time(stop) * 1e-3
    vec = sum(v.numel() * v.element_size() for v in (gamma, beta) if v is not None)
    nbytes = w.rows * w.cols * w.itemsize
    return secs / steps, nbytes + vec, nbytes

def graph_launch_us(w: wl.Workload, launches: int = 256, replays: int = 20) -> float:
    """Device time per launch when `launches` calls are captured in one CUDA graph
    (separates the kernel from the host's launch overhead for tiny problems)."""
    import torch
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        dw = DeviceWorkload(w, 2)                      # calls are bound to `stream`
        for _ in range(3):
            dw.launch()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for _ in range(launches):
                dw.launch()
        graph.replay()
        stream.synchronize()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(stream)
        for _ in range(replays):
            graph.replay()
        stop.record(stream)
        stream.synchronize()
    return start.elapsed_time(stop) * 1e3 / (launches * replays)


def oracle_baseline(w: wl.Workload, budget_s: float = 12.0):
    """Time the fp64 oracle, as it stands, on a bounded row sample of the workload."""
    import oracle
    cores = os.cpu_count() or 1

    def run(rows):
        sub = wl.Workload(w.name, w.op, w.dtype, rows, w.cols, w.x[:rows], eps=w.eps, gamma=w.gamma,
                          beta=w.beta, causal_period=w.causal_period)
        t0 = time.perf_counter()
        if w.op in ("softmax", "log_softmax"):
            mask = oracle.Mask(causal=True, causal_period=w.causal_period) if w.causal_period else None
            getattr(oracle, w.op)(sub.x, mask=mask, nthreads=cores)
        elif w.op == "layernorm":
            oracle.layernorm(sub.x, w.gamma, w.beta, eps=float(np.float32(w.eps)), nthreads=cores)
        else:
            oracle.rmsnorm(sub.x, w.gamma, eps=float(np.float32(w.eps)), nthreads=cores)
        return time.perf_counter() - t0, sub.algorithmic_bytes()

    probe_rows = max(1, min(w.rows, max(cores, (1 << 22) // w.cols)))
    run(probe_rows)                                           # page-in / thread start-up
    t_probe, _ = run(probe_rows)
    rows = int(min(w.rows, max(probe_rows, probe_rows * budget_s / max(t_probe, 1e-4))))
    # the sample is repeated until about budget_s of CPU time has been spent
    passes, secs, nbytes = 0, 0.0, 0
    while passes == 0 or (secs < budget_s and passes < 5000):
        t, b = run(rows)
        secs, nbytes, passes = secs + t, nbytes + b, passes + 1
    return {"value": nbytes / secs / 1e9, "unit": "GB/s", "cores": oracle.last_threads(),
            "kind": "oracle", "seconds": round(secs, 3), "rows_per_s": rows * passes / secs,
            "sample": f"first {rows} of {w.rows} rows of {w.name}, {passes} passes, OpenMP over rows"}


def slowest_rank(seconds: float, world: int, device: str) -> float:
    """Max over ranks of a per-rank time (the job is as slow as its slowest rank)."""
    if world == 1:
        return seconds
    import torch
    import torch.distributed as dist
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(bytes_per_rank: int, world: int, seconds: float) -> float:
    """GB/s of the whole job: every rank moves bytes_per_rank in `seconds` (weak scaling)."""
    return bytes_per_rank * world / seconds / 1e9


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2512_23424_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    dev = torch.cuda.current_device()
    binding.lib()                                             # fail loudly if the library is missing

    def barrier():
        if world > 1:
            dist.barrier()

    def max_over_ranks(v: float) -> float:
        return slowest_rank(v, world, "cuda")

    peak, peak_kind = measured_peak()
    w = wl.make_config(HEADLINE, seed_offset=rank)
    dw = DeviceWorkload(w, pairs_for(w))
    sampler = ClockSampler(dev)
    sampler.start()
    secs = max_over_ranks(time_launches(dw, args.steps, args.warmup, barrier))
    note = "timed region"
    if len(sampler.samples) < 5:                             # short region: keep the same kernel running
        t_end = time.perf_counter() + 0.25
        while time.perf_counter() < t_end:
            for _ in range(50):
                dw.launch()
            torch.cuda.synchronize()
        note = "timed region plus 0.25 s of the same launches"
    sampler.stop()
    kernel = binding.last_kernel()
    per_step = secs / args.steps
    nbytes = w.algorithmic_bytes()
    gbs_one = nbytes / per_step / 1e9
    value = whole_job_value(nbytes, world, per_step)

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.CONFIG_NAMES[HEADLINE], "op": w.op, "rows": w.rows, "cols": w.cols,
                   "io_dtype": "f32", "rows_per_s": w.rows * world / per_step, "kernel": kernel,
                   "l2": f"rotating {len(dw.xs)} buffer pairs ({len(dw.xs) * 2 * w.rows * w.cols * w.itemsize >> 20} MiB > L2)",
                   "parallelism": f"replicas x{world}, no collective"},
        "gpu_launches": args.steps,
        "clocks": sampler.summary(note),
    }
    if rank == 0 and world == 1:
        line["roofline"] = {"bound": "hbm", "achieved": gbs_one, "peak": peak, "unit": "GB/s",
                            "frac": gbs_one / peak, "frac_nominal": gbs_one / NOMINAL_HBM_GBS,
                            "peak_kind": peak_kind, "traffic": profiled_traffic(wl.CONFIG_NAMES[HEADLINE]),
                            "algorithmic_bytes": nbytes, "kernel": kernel}
    # end to end with host buffers
    e2e_k = max(3, min(args.steps, 20))
    t_e2e, h2d, d2h = e2e_steps(w, e2e_k, args.warmup)
    t_e2e = max_over_ranks(t_e2e)
    line["e2e"] = {"value": nbytes * world / t_e2e / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": d2h, "ms_per_step": t_e2e * 1e3, "steps": e2e_k}
    del dw
    torch.cuda.empty_cache()

    if rank == 0 and world == 1 and not args.headline_only:
        table = []
        for k in (1, 2, 3, 4, 5):
            wk = w if k == HEADLINE else wl.make_config(k)
            dwk = DeviceWorkload(wk, pairs_for(wk))
            # launches per configuration at the default --steps 1000; fewer steps scale them down
            full = {1: 2000, 2: 1000, 3: 300, 4: 300, 5: 100}[k]
            reps = max(10, min(full, full * args.steps // 1000))
            sk = time_launches(dwk, reps, 10) / reps
            bk = wk.algorithmic_bytes()
            row = {"workload": wl.CONFIG_NAMES[k], "kernel": binding.last_kernel(), "us": sk * 1e6,
                   "rows_per_s": wk.rows / sk, "launches": reps}
            if k == 1:
                row["note"] = ("latency-bound (0.5 MiB, L2-resident); GB/s not meaningful; 'us' is paced by the "
                               "host's launch rate, 'graph_us' is one launch inside a CUDA graph of 256")
                row["graph_us"] = graph_launch_us(wk, replays=max(2, min(20, args.steps // 50)))
            else:
                row.update({"gbs": bk / sk / 1e9, "frac_measured": bk / sk / 1e9 / peak,
                            "frac_nominal": bk / sk / 1e9 / NOMINAL_HBM_GBS, "algorithmic_bytes": bk,
                            "traffic": profiled_traffic(wl.CONFIG_NAMES[k])})
            table.append(row)
            del dwk, wk
            torch.cuda.empty_cache()
        line["per_config"] = table
        # configurations 3 and 5 stored as IEEE half (the paper's float16 regime)
        halves = []
        for k in (3, 5):
            wk = wl.as_f16(wl.make_config(k))
            dwk = DeviceWorkload(wk, pairs_for(wk))
            reps = max(10, min(100, 100 * args.steps // 1000))
            sk = time_launches(dwk, reps, 5) / reps
            bk = wk.algorithmic_bytes()
            halves.append({"workload": wk.name, "kernel": binding.last_kernel(), "us": sk * 1e6, "gbs": bk / sk / 1e9,
                           "frac_measured": bk / sk / 1e9 / peak, "algorithmic_bytes": bk, "launches": reps,
                           "rows_per_s": wk.rows / sk})
            del dwk, wk
            torch.cuda.empty_cache()
        line["fp16_rows"] = halves
        # the operators over a non-last axis (the layout of the paper's RMSNorm sketch)
        axis = []
        for name in wl.AXIS_CONFIGS:
            wa = wl.make_axis(name)
            dwa = AxisDeviceWorkload(wa, pairs_for(wa))
            reps = max(10, min(100, 100 * args.steps // 1000))
            sa = time_launches(dwa, reps, 5) / reps
            ba = wa.algorithmic_bytes()
            axis.append({"workload": name, "kernel": binding.last_kernel(), "us": sa * 1e6, "gbs": ba / sa / 1e9,
                         "frac_measured": ba / sa / 1e9 / peak, "algorithmic_bytes": ba, "launches": reps,
                         "traffic": profiled_traffic(name)})
            del dwa, wa
            torch.cuda.empty_cache()
        line["axis_rows"] = axis
        # fused residual add + normalisation (x and the residual in, y and the sum out)
        fused = []
        for name in wl.FUSED_CONFIGS:
            wf = wl.make_fused(name)
            dwf = FusedDeviceWorkload(wf, pairs_for(wf))
            reps = max(10, min(100, 100 * args.steps // 1000))
            sf = time_launches(dwf, reps, 5) / reps
            bf = wf.algorithmic_bytes()
            fused.append({"workload": name, "kernel": binding.last_kernel(), "us": sf * 1e6, "gbs": bf / sf / 1e9,
                          "frac_measured": bf / sf / 1e9 / peak, "algorithmic_bytes": bf, "launches": reps,
                          "rows_per_s": wf.x.shape[0] / sf, "traffic": profiled_traffic(name)})
            del dwf, wf
            torch.cuda.empty_cache()
        # configuration 5 with its 1/sqrt(128) given to the call instead of baked into the input
        ws = wl.make_scaled_causal()
        xs0 = torch.from_numpy(ws.x.view(np.int16)).cuda().view(torch.bfloat16)
        ys0 = torch.empty_like(xs0)
        mask = binding.make_mask(xs0, causal=True, causal_period=ws.causal_period)

        class _Scaled:
            def launch(self):
                return binding.softmax_scaled(xs0, ws.extra["scale"], out=ys0, mask=mask)

        _Scaled.torch = torch
        reps = max(10, min(100, 100 * args.steps // 1000))
        ss_ = time_launches(_Scaled(), reps, 5) / reps
        bs_ = ws.algorithmic_bytes()
        fused.append({"workload": ws.name, "kernel": binding.last_kernel(), "us": ss_ * 1e6, "gbs": bs_ / ss_ / 1e9,
                      "frac_measured": bs_ / ss_ / 1e9 / peak, "algorithmic_bytes": bs_, "launches": reps,
                      "rows_per_s": ws.rows / ss_, "scale": ws.extra["scale"], "traffic": None})
        del xs0, ys0, ws
        torch.cuda.empty_cache()
        line["fused_rows"] = fused
        # gated activations (gate and factor in, product out)
        acts = []
        for name in wl.ACT_CONFIGS:
            wa = wl.make_act(name)
            dwa = ActDeviceWorkload(wa, pairs_for(wa))
            reps = max(10, min(100, 100 * args.steps // 1000))
            sa = time_launches(dwa, reps, 5) / reps
            ba = wa.algorithmic_bytes()
            acts.append({"workload": name, "kernel": binding.last_kernel(), "us": sa * 1e6, "gbs": ba / sa / 1e9,
                         "frac_measured": ba / sa / 1e9 / peak, "algorithmic_bytes": ba, "launches": reps,
                         "rows_per_s": wa.x.shape[0] / sa, "traffic": profiled_traffic(name)})
            del dwa, wa
            torch.cuda.empty_cache()
        line["act_rows"] = acts
        # arg-max / arg-min and cumulative sum / product over the last axis
        reds = []
        for name in wl.REDUCTION_CONFIGS:
            wr = wl.make_reduction(name)
            fn = getattr(binding, wr.op)
            n_buf = pairs_for(wr)
            if wr.dtype == wl.F32:
                x0 = torch.from_numpy(wr.x).cuda()
            else:
                x0 = torch.from_numpy(wr.x.view(np.int16)).cuda().view(torch.bfloat16)
            rxs = [x0] + [x0.clone() for _ in range(n_buf - 1)]
            routs = [fn(x) for x in rxs]

            class _Red:
                i = 0

                def launch(self):
                    k = self.i % len(rxs)
                    self.i += 1
                    return fn(rxs[k], out=routs[k])

            _Red.torch = torch
            reps = max(10, min(100, 100 * args.steps // 1000))
            sr = time_launches(_Red(), reps, 5) / reps
            br = wr.algorithmic_bytes()
            reds.append({"workload": name, "kernel": binding.last_kernel(), "us": sr * 1e6, "gbs": br / sr / 1e9,
                         "frac_measured": br / sr / 1e9 / peak, "algorithmic_bytes": br, "launches": reps,
                         "rows_per_s": wr.x.shape[0] / sr, "traffic": profiled_traffic(name)})
            del rxs, routs, x0, wr
            torch.cuda.empty_cache()
        line["reduction_rows"] = reds
        # BatchNorm-style column normalisation (two kernels; x is read twice, the second time from
        # L2 while it fits: `gbs` counts one read and one write, `gbs_three_streams` all three)
        colrows = []
        for name in wl.COLNORM_CONFIGS:
            wc = wl.make_colnorm(name)
            cdt = torch.float32 if wc.dtype == wl.F32 else torch.bfloat16

            def cdev(a):
                if wc.dtype == wl.F32:
                    return torch.from_numpy(a).cuda()
                return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)

            cx0 = cdev(wc.x)
            n_buf = 2 if 2 * cx0.numel() * cx0.element_size() >= 2 * L2_BYTES else 3
            cxs = [cx0] + [cx0.clone() for _ in range(n_buf - 1)]
            cys = [torch.empty_like(cx0) for _ in range(n_buf)]
            cg, cb = cdev(wc.gamma), cdev(wc.beta)
            cws = torch.empty(binding.colnorm_workspace_bytes(wc.rows, wc.cols) or 8, dtype=torch.uint8, device="cuda")

            class _Col:
                i = 0

                def launch(self):
                    k = self.i % len(cxs)
                    self.i += 1
                    return binding.colnorm(cxs[k], cg, cb, eps=wc.eps, out=cys[k], workspace=cws)

            _Col.torch = torch
            binding.colnorm(cxs[0], cg, cb, eps=wc.eps, out=cys[0], workspace=cws)      # sets the ctypes signatures
            reps = max(10, min(100, 100 * args.steps // 1000))
            sc = time_launches(_Col(), reps, 5) / reps
            bc = 2 * wc.rows * wc.cols * wc.itemsize
            colrows.append({"workload": name, "kernel": binding.last_kernel(), "us": sc * 1e6, "gbs": bc / sc / 1e9,
                            "frac_measured": bc / sc / 1e9 / peak, "gbs_three_streams": 1.5 * bc / sc / 1e9,
                            "algorithmic_bytes": bc, "launches": 2 * reps, "rows_per_s": wc.rows / sc})
            del cxs, cys, cx0, wc
            torch.cuda.empty_cache()
        line["colnorm_rows"] = colrows
    if rank == 0 and world == 1:
        line["cpu_baseline"] = oracle_baseline(w)
    assert binding.device_status() == 0, "a device-side bounded wait expired"
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------
# reference arm: the fp64 oracle on the host cores
# --------------------------------------------------------------------------------------------
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    import oracle
    w = wl.make_config(HEADLINE, rows=256)                   # bounded sample of the workload per step
    cores = os.cpu_count() or 1
    eps = float(np.float32(w.eps))

    def step():
        oracle.layernorm(w.x, w.gamma, w.beta, eps=eps, nthreads=cores)

    for _ in range(max(args.warmup, 1)):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    per_step = (time.perf_counter() - t0) / args.steps
    gbs = w.algorithmic_bytes() / per_step / 1e9
    sample = f"first 256 of 4096 rows of {wl.CONFIG_NAMES[HEADLINE]} per step, OpenMP over rows"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": wl.CONFIG_NAMES[HEADLINE], "op": w.op, "rows": w.rows, "cols": w.cols,
                   "io_dtype": "f32", "sample": sample},
        "gpu_launches": 0,
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": oracle.last_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_profile(args):
    """Bare launches of one configuration (for a profiler): warm-up + steps launches of
    the operator on resident inputs, nothing else.  --profile-rows truncates the rows."""
    import torch
    from paper_2512_23424_b200 import binding
    torch.cuda.set_device(0)
    if args.profile_act:
        w = wl.make_act(args.profile_act, rows=args.profile_rows)
        dw = ActDeviceWorkload(w, pairs_for(w) if args.profile_rows is None else 1)
        secs = time_launches(dw, args.steps, args.warmup)
        print(json.dumps({"profile": args.profile_act, "shape": list(w.x.shape), "kernel": binding.last_kernel(),
                          "us_per_launch": secs / args.steps * 1e6, "launches": args.steps + max(args.warmup, 3),
                          "algorithmic_bytes": w.algorithmic_bytes()}))
        return
    if args.profile_fused:
        w = wl.make_fused(args.profile_fused, rows=args.profile_rows)
        dw = FusedDeviceWorkload(w, pairs_for(w) if args.profile_rows is None else 1)
        secs = time_launches(dw, args.steps, args.warmup)
        print(json.dumps({"profile": args.profile_fused, "shape": list(w.x.shape), "kernel": binding.last_kernel(),
                          "us_per_launch": secs / args.steps * 1e6, "launches": args.steps + max(args.warmup, 3),
                          "algorithmic_bytes": w.algorithmic_bytes()}))
        return
    if args.profile_axis:
        w = wl.make_axis(args.profile_axis, outer=args.profile_rows)
        for item in filter(None, args.tune.split(",")):
            key, _, val = item.partition("=")
            binding.set_tuning(key, int(val))
        dw = AxisDeviceWorkload(w, pairs_for(w) if args.profile_rows is None else 1)
        secs = time_launches(dw, args.steps, args.warmup)
        print(json.dumps({"profile": args.profile_axis, "shape": list(w.x.shape), "kernel": binding.last_kernel(),
                          "us_per_launch": secs / args.steps * 1e6, "launches": args.steps + max(args.warmup, 3),
                          "algorithmic_bytes": w.algorithmic_bytes()}))
        return
    w = wl.make_config(args.profile, rows=args.profile_rows)
    if args.variant:
        binding.set_variant(args.variant)
    for item in filter(None, args.tune.split(",")):
        key, _, val = item.partition("=")
        binding.set_tuning(key, int(val))
    dw = DeviceWorkload(w, pairs_for(w) if args.profile_rows is None else 1)
    secs = time_launches(dw, args.steps, args.warmup)
    print(json.dumps({"profile": wl.CONFIG_NAMES[args.profile], "rows": w.rows, "kernel": binding.last_kernel(),
                      "us_per_launch": secs / args.steps * 1e6, "launches": args.steps + max(args.warmup, 3),
                      "algorithmic_bytes": w.algorithmic_bytes()}))


SWEEP_COLS = (256, 512, 768, 1024, 1280, 1536, 2048, 2560, 3072, 4096, 5120, 6144, 7168, 8192, 12288, 16384,
              20480, 32000, 32768, 50304, 65536, 128256, 131072, 151936, 262144)


def run_sweep(args):
    """Width sweep of the four operators (fp32 and bf16; 2^26 elements per call, rows = 2^26 / cols;
    seeded normal inputs, unit gamma / beta): fraction of the measured copy peak and the kernel the
    planner chose, one JSON line per (dtype, cols).  Not part of the bench line."""
    import torch
    from paper_2512_23424_b200 import binding
    torch.cuda.set_device(0)
    peak = measured_peak()[0]
    gen = torch.Generator(device="cuda").manual_seed(2512)
    for tdt, dname in ((torch.float32, "f32"), (torch.bfloat16, "bf16")):
        for cols in SWEEP_COLS:
            rows = (1 << 26) // cols
            sets = max(2, (1 << 30) // (rows * cols * 4))              # rotate over > L2 worth of buffers
            xs = [torch.randn((rows, cols), device="cuda", dtype=torch.float32, generator=gen).to(tdt)
                  for _ in range(sets)]
            ys = [torch.empty_like(x) for x in xs]
            g = torch.ones(cols, device="cuda", dtype=tdt)
            b = torch.zeros(cols, device="cuda", dtype=tdt)
            calls = {"softmax": lambda i: binding.softmax(xs[i], out=ys[i]),
                     "log_softmax": lambda i: binding.log_softmax(xs[i], out=ys[i]),
                     "layernorm": lambda i: binding.layernorm(xs[i], g, b, out=ys[i]),
                     "rmsnorm": lambda i: binding.rmsnorm(xs[i], g, out=ys[i])}
            line = {"dtype": dname, "rows": rows, "cols": cols}
            for op, call in calls.items():
                for i in range(sets):
                    call(i)
                torch.cuda.synchronize()
                start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                start.record()
                for k in range(args.steps):
                    call(k % sets)
                stop.record()
                torch.cuda.synchronize()
                secs = start.elapsed_time(stop) * 1e-3 / args.steps
                gbs = 2 * rows * cols * xs[0].element_size() / secs / 1e9
                line[op] = {"frac": round(gbs / peak, 3), "us": round(secs * 1e6, 1), "kernel": binding.last_kernel()}
            print(json.dumps(line), flush=True)
            del xs, ys


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--headline-only", action="store_true",
                    help="skip the per-configuration table (the headline line is unchanged)")
    ap.add_argument("--profile", type=int, default=0, metavar="K",
                    help="only launch configuration K (1..5) warmup+steps times, for use under ncu")
    ap.add_argument("--profile-axis", default="", metavar="NAME",
                    help="as --profile, for a non-last-axis configuration (workloads.AXIS_CONFIGS)")
    ap.add_argument("--profile-act", default="", metavar="NAME",
                    help="as --profile, for a gated-activation configuration (workloads.ACT_CONFIGS)")
    ap.add_argument("--profile-fused", default="", metavar="NAME",
                    help="as --profile, for a fused residual add + normalisation configuration (workloads.FUSED_CONFIGS)")
    ap.add_argument("--profile-rows", type=int, default=None,
                    help="truncate the rows of --profile (the outer axis of --profile-axis)")
    ap.add_argument("--variant", default="", help="force a kernel family in --profile mode")
    ap.add_argument("--tune", default="", help="--profile mode: key=value[,key=value] launch-geometry overrides")
    ap.add_argument("--sweep", action="store_true",
                    help="width sweep of the four operators (one JSON line per dtype and width) instead of the bench line")
    args = ap.parse_args()
    if args.sweep:
        if args.steps == 1000:
            args.steps = 20
        run_sweep(args)
        return
    if args.profile or args.profile_axis or args.profile_fused or args.profile_act:
        run_profile(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
