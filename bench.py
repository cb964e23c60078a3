#!/usr/bin/env python
"""Benchmark of the row-operator library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one launch of the headline operator - the causally masked bf16 softmax
[32 x 4096, 4096], the largest of the five benchmark configurations - through the
C ABI on inputs already resident in HBM (its 2 GiB working set exceeds L2 many
times over).  The one JSON line printed by rank 0 carries the headline number and,
inside `roofline`, one row per benchmark configuration (`per_config`) and per
widened operator (`next_rows`: non-last axis, fused residual add + normalisation,
gated activations, arg-max / cumulative operators, column normalisation, fp16
storage).  Every row is timed three ways over at least 50 launches whatever
--steps is: all launches back to back inside one event pair (`us`, the average
duration of a launch over a timed region, the protocol of the headline number;
consecutive launches overlap their ramp-up and drain through programmatic
dependent launch, so it is a steady-state figure), each launch inside its own CUDA
event pair (`us_median`, `us_min`: one isolated launch with its ramp-up and drain
exposed), and
a few launches each preceded by a 256 MiB fill that empties L2 (`us_cold_median`).
`frac` is algorithmic bytes / us / the measured copy peak; `frac_single_launch` the
same from us_median.  Beside them the line carries the end-to-end figure with
host buffers and the fp64 CPU oracle's timing.

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
HEADLINE = 5
HEADLINE_DTYPE = "bf16 I/O, fp32 accumulate"
MIN_LAUNCHES = 50
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


def measure_row(obj, nbytes: int, peak: float, launches: int = MIN_LAUNCHES, warmup: int = 20, cold: int = 8):
    """Three timings of `obj.launch()` (see the module docstring), as one table row."""
    torch = obj.torch
    launches = max(launches, MIN_LAUNCHES)
    pipelined = time_launches(obj, launches, warmup) / launches
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(launches)]
    for a, b in pairs:                                   # one event pair per launch: no overlap between launches
        a.record()
        obj.launch()
        b.record()
    torch.cuda.synchronize()
    each = np.array([a.elapsed_time(b) for a, b in pairs]) * 1e3
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    cold_pairs = pairs[:cold]
    for a, b in cold_pairs:
        flush.fill_(1)                                    # 256 MiB of stores: nothing of the inputs stays in L2
        a.record()
        obj.launch()
        b.record()
    torch.cuda.synchronize()
    cold_us = np.array([a.elapsed_time(b) for a, b in cold_pairs]) * 1e3
    del flush
    single = float(np.median(each))
    us = pipelined * 1e6
    return {"us": us, "gbs": nbytes / us / 1e3, "frac": nbytes / us / 1e3 / peak,
            "frac_nominal": nbytes / us / 1e3 / NOMINAL_HBM_GBS,
            "us_median": single, "us_min": float(each.min()), "frac_single_launch": nbytes / single / 1e3 / peak,
            "us_cold_median": float(np.median(cold_us)), "launches": launches, "algorithmic_bytes": nbytes}


def launch_floor_us(launches: int = 256, replays: int = 20) -> float:
    """Device time per launch of the library's smallest call (one 4-element row) inside a CUDA
    graph: what any launch costs on this stream before it moves a byte."""
    import torch
    from paper_2512_23424_b200 import binding
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        x = torch.zeros((1, 4), device="cuda")
        call = binding.prepare("rmsnorm", x, torch.empty_like(x), eps=1e-6)
        for _ in range(3):
            call.launch()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for _ in range(launches):
                call.launch()
        graph.replay()
        stream.synchronize()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(stream)
        for _ in range(replays):
            graph.replay()
        stop.record(stream)
        stream.synchronize()
    return start.elapsed_time(stop) * 1e3 / (launches * replays)


def e2e_steps(w: wl.Workload, steps: int, warmup: int):
    """Same operator through the C ABI's host-buffer entry point: every step uploads the
    inputs from pinned host memory, runs the kernels and downloads the result, all inside
    the timed region (chunked and pipelined by the library over a caller-owned workspace)."""
    import torch
    from paper_2512_23424_b200 import binding
    tdt = torch.float32 if w.dtype == wl.F32 else torch.bfloat16
    assert w.dtype in (wl.F32, wl.BF16)

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
    up, down = binding.last_host_copy_bytes()              # what the call copied (the library counts its copies)
    return secs / steps, up, down

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
    if w.causal_period > 0:                                   # whole causal periods: every live length equally often
        rows = min(w.rows, max(w.causal_period, rows // w.causal_period * w.causal_period))
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


def _dev(a, dtype):
    """Host array (float32 / float16, or uint16 bf16 bits) -> device tensor of the same bits."""
    import torch
    if a is None:
        return None
    if dtype in (wl.F32, wl.F16):
        return torch.from_numpy(a).cuda()
    return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)


class _Rotating:
    """`launch()` calls fn(k) for k cycling over n buffer sets."""

    def __init__(self, torch, n, fn):
        self.torch, self.n, self.fn, self.i = torch, n, fn, 0

    def launch(self):
        k = self.i % self.n
        self.i += 1
        return self.fn(k)


def next_rows_table(peak: float):
    """One row per widened operator (the "next" rows): same three timings as the five configurations."""
    import torch
    from paper_2512_23424_b200 import binding
    rows = []

    def add(name, obj, nbytes, **more):
        row = {"workload": name}
        row.update(measure_row(obj, nbytes, peak))
        row["kernel"] = binding.last_kernel()
        row["traffic"] = profiled_traffic(name)
        row.update(more)
        rows.append(row)
        torch.cuda.empty_cache()

    # configurations 3 and 5 stored as IEEE half (the paper's float16 regime)
    for k in (3, 5):
        wk = wl.as_f16(wl.make_config(k))
        add(wk.name, DeviceWorkload(wk, pairs_for(wk)), wk.algorithmic_bytes())
        del wk
    # the operators over a non-last axis (the layout of the paper's RMSNorm sketch)
    for name in wl.AXIS_CONFIGS:
        wa = wl.make_axis(name)
        add(name, AxisDeviceWorkload(wa, pairs_for(wa)), wa.algorithmic_bytes())
        del wa
    # fused residual add + normalisation (x and the residual in, y and the sum out)
    for name in wl.FUSED_CONFIGS:
        wf = wl.make_fused(name)
        add(name, FusedDeviceWorkload(wf, pairs_for(wf)), wf.algorithmic_bytes())
        del wf
    # configuration 5 with its 1/sqrt(128) given to the call instead of baked into the input
    ws = wl.make_scaled_causal()
    xs0 = _dev(ws.x, ws.dtype)
    ys0 = torch.empty_like(xs0)
    mask = binding.make_mask(xs0, causal=True, causal_period=ws.causal_period)
    scale = ws.extra["scale"]
    add(ws.name, _Rotating(torch, 1, lambda k: binding.softmax_scaled(xs0, scale, out=ys0, mask=mask)),
        ws.algorithmic_bytes(), scale=scale)
    del xs0, ys0, ws
    # gated activations (gate and factor in, product out)
    for name in wl.ACT_CONFIGS:
        wa = wl.make_act(name)
        add(name, ActDeviceWorkload(wa, pairs_for(wa)), wa.algorithmic_bytes())
        del wa
    # arg-max / arg-min and cumulative sum / product over the last axis
    for name in wl.REDUCTION_CONFIGS:
        wr = wl.make_reduction(name)
        fn = getattr(binding, wr.op)
        x0 = _dev(wr.x, wr.dtype)
        rxs = [x0] + [x0.clone() for _ in range(pairs_for(wr) - 1)]
        routs = [fn(x) for x in rxs]
        add(name, _Rotating(torch, len(rxs), lambda k: fn(rxs[k], out=routs[k])), wr.algorithmic_bytes())
        del rxs, routs, x0, wr
    # BatchNorm-style column normalisation: two kernels, x is read twice (the second time from L2
    # while it fits), so the bound is three streams and `frac` counts three; `frac_two_streams`
    # counts one read and one write
    for name in wl.COLNORM_CONFIGS:
        wc = wl.make_colnorm(name)
        cx0 = _dev(wc.x, wc.dtype)
        n_buf = 2 if 2 * cx0.numel() * cx0.element_size() >= 2 * L2_BYTES else 3
        cxs = [cx0] + [cx0.clone() for _ in range(n_buf - 1)]
        cys = [torch.empty_like(cx0) for _ in range(n_buf)]
        cg, cb = _dev(wc.gamma, wc.dtype), _dev(wc.beta, wc.dtype)
        cws = torch.empty(binding.colnorm_workspace_bytes(wc.rows, wc.cols) or 8, dtype=torch.uint8, device="cuda")
        eps = wc.eps
        two = 2 * wc.rows * wc.cols * wc.itemsize
        add(name, _Rotating(torch, n_buf, lambda k: binding.colnorm(cxs[k], cg, cb, eps=eps, out=cys[k], workspace=cws)),
            two * 3 // 2, bound="hbm, three streams (x read twice)", kernels_per_call=3)
        rows[-1]["frac_two_streams"] = rows[-1]["frac"] * 2 / 3
        del cxs, cys, cx0, wc
    return rows


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
    working_set = len(dw.xs) * 2 * w.rows * w.cols * w.itemsize

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": HEADLINE_DTYPE, "data": "synthetic",
        "config": {"workload": wl.CONFIG_NAMES[HEADLINE], "op": w.op, "rows": w.rows, "cols": w.cols,
                   "io_dtype": "bf16", "causal_period": w.causal_period,
                   "rows_per_s": w.rows * world / per_step, "kernel": kernel,
                   "l2": f"{len(dw.xs)} buffer pair(s), working set {working_set >> 20} MiB > L2",
                   "timing": "steps launched back to back (consecutive launches overlap through programmatic "
                             "dependent launch); per-launch figures in roofline.per_config",
                   "parallelism": f"replicas x{world}, no collective"},
        "gpu_launches": args.steps,
        "clocks": sampler.summary(note),
    }
    detail = rank == 0 and world == 1
    if detail:
        line["roofline"] = {"bound": "hbm", "achieved": gbs_one, "peak": peak, "unit": "GB/s",
                            "frac": gbs_one / peak, "frac_nominal": gbs_one / NOMINAL_HBM_GBS,
                            "peak_kind": peak_kind, "traffic": profiled_traffic(wl.CONFIG_NAMES[HEADLINE]),
                            "algorithmic_bytes": nbytes, "kernel": kernel,
                            "note": "achieved / frac: algorithmic bytes / average launch duration over the timed "
                                    "region (launches back to back), here and in per_config / next_rows; "
                                    "frac_single_launch: from the median of isolated launches, each in its own "
                                    "event pair (ramp-up and drain of the grid exposed)"}
    # end to end with host buffers
    e2e_k = max(3, min(args.steps, 20))
    t_e2e, h2d, d2h = e2e_steps(w, e2e_k, args.warmup)
    t_e2e = max_over_ranks(t_e2e)
    line["e2e"] = {"value": nbytes * world / t_e2e / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": d2h, "ms_per_step": t_e2e * 1e3, "steps": e2e_k,
                   "copied_gbs": (h2d + d2h) * world / t_e2e / 1e9,
                   "note": "value counts the algorithmic bytes (live reads + writes); copied_gbs counts the bytes "
                           "that crossed PCIe (masked columns of causal rows are not uploaded: a chunk carries the "
                           "columns up to its last row's live length)"}
    del dw
    torch.cuda.empty_cache()

    if detail and not args.headline_only:
        table = []
        for k in (1, 2, 3, 4, 5):
            wk = w if k == HEADLINE else wl.make_config(k)
            dwk = DeviceWorkload(wk, pairs_for(wk))
            row = {"workload": wl.CONFIG_NAMES[k]}
            row.update(measure_row(dwk, wk.algorithmic_bytes(), peak, launches=200 if k <= 2 else MIN_LAUNCHES))
            row.update({"kernel": binding.last_kernel(), "rows_per_s": wk.rows / (row["us"] * 1e-6),
                        "traffic": profiled_traffic(wl.CONFIG_NAMES[k])})
            if k == 1:
                for key in ("gbs", "frac", "frac_nominal", "frac_single_launch"):
                    row.pop(key)
                row["graph_us"] = graph_launch_us(wk, replays=10)
                row["launch_floor_graph_us"] = launch_floor_us(replays=10)
                row["note"] = ("latency-bound (0.5 MiB, L2-resident): no bandwidth figure; 'us' is paced by "
                               "the host's launch rate, 'graph_us' is one launch inside a CUDA graph of 256, "
                               "'launch_floor_graph_us' the same for a one-vector call of this library")
            table.append(row)
            del dwk, wk
            torch.cuda.empty_cache()
        line["roofline"]["per_config"] = table
        large = [r for r in table if "frac" in r]
        line["roofline"]["min_frac"] = min(r["frac"] for r in large)
        line["roofline"]["min_frac_workload"] = min(large, key=lambda r: r["frac"])["workload"]
        line["roofline"]["next_rows"] = next_rows_table(peak)
    if detail:
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
    full = wl.config_shape(HEADLINE)[0]
    w = wl.make_config(HEADLINE, rows=4096)                  # one whole causal period (one head) per step
    cores = os.cpu_count() or 1
    mask = oracle.Mask(causal=True, causal_period=w.causal_period)

    def step():
        oracle.softmax(w.x, mask=mask, nthreads=cores)

    for _ in range(max(args.warmup, 1)):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    per_step = (time.perf_counter() - t0) / args.steps
    gbs = w.algorithmic_bytes() / per_step / 1e9
    sample = (f"first {w.rows} of {full} rows (one whole causal period) of {wl.CONFIG_NAMES[HEADLINE]} per step, "
              "OpenMP over rows")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": wl.CONFIG_NAMES[HEADLINE], "op": w.op, "rows": w.rows, "cols": w.cols,
                   "io_dtype": "bf16", "causal_period": w.causal_period, "sample": sample},
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
    if args.profile_next:
        # one of the arg-max / cumulative / column-normalisation rows (workloads.REDUCTION_CONFIGS, COLNORM_CONFIGS)
        name = args.profile_next
        for item in filter(None, args.tune.split(",")):
            key, _, val = item.partition("=")
            binding.set_tuning(key, int(val))
        if name in wl.REDUCTION_CONFIGS:
            wr = wl.make_reduction(name, rows=args.profile_rows)
            fn = getattr(binding, wr.op)
            x0 = _dev(wr.x, wr.dtype)
            rxs = [x0] + [x0.clone() for _ in range(pairs_for(wr) - 1)]
            routs = [fn(x) for x in rxs]
            obj = _Rotating(torch, len(rxs), lambda k: fn(rxs[k], out=routs[k]))
            nbytes, shape = wr.algorithmic_bytes(), list(wr.x.shape)
        else:
            wc = wl.make_colnorm(name, rows=args.profile_rows)
            cx0 = _dev(wc.x, wc.dtype)
            cxs = [cx0, cx0.clone()]
            cys = [torch.empty_like(cx0) for _ in cxs]
            cg, cb = _dev(wc.gamma, wc.dtype), _dev(wc.beta, wc.dtype)
            cws = torch.empty(binding.colnorm_workspace_bytes(wc.rows, wc.cols) or 8, dtype=torch.uint8, device="cuda")
            obj = _Rotating(torch, 2, lambda k: binding.colnorm(cxs[k], cg, cb, eps=wc.eps, out=cys[k], workspace=cws))
            nbytes, shape = 3 * wc.rows * wc.cols * wc.itemsize, [wc.rows, wc.cols]
        secs = time_launches(obj, args.steps, args.warmup)
        print(json.dumps({"profile": name, "shape": shape, "kernel": binding.last_kernel(),
                          "us_per_launch": secs / args.steps * 1e6, "launches": args.steps + max(args.warmup, 3),
                          "algorithmic_bytes": nbytes,
                          "frac_of_copy_peak": nbytes / (secs / args.steps) / 1e9 / measured_peak()[0]}))
        return
    if args.profile_shape:
        op, dname, rows, cols = args.profile_shape.split(":")
        dtype = {"f32": wl.F32, "bf16": wl.BF16, "f16": wl.F16}[dname]
        w = wl.make_random(op, dtype, int(rows), int(cols), seed=2512, loc=0.5, eps=1e-5)
        name = w.name
    else:
        w = wl.make_config(args.profile, rows=args.profile_rows)
        name = wl.CONFIG_NAMES[args.profile]
    if args.variant:
        binding.set_variant(args.variant)
    for item in filter(None, args.tune.split(",")):
        key, _, val = item.partition("=")
        binding.set_tuning(key, int(val))
    dw = DeviceWorkload(w, pairs_for(w) if args.profile_rows is None else 1)
    secs = time_launches(dw, args.steps, args.warmup)
    print(json.dumps({"profile": name, "rows": w.rows, "kernel": binding.last_kernel(),
                      "frac_of_copy_peak": w.algorithmic_bytes() / (secs / args.steps) / 1e9 / measured_peak()[0],
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
            # arguments marshalled once per buffer set, as in the bench rows (a launch is one C call)
            prepared = {"softmax": [binding.prepare("softmax", xs[i], ys[i]) for i in range(sets)],
                        "log_softmax": [binding.prepare("log_softmax", xs[i], ys[i]) for i in range(sets)],
                        "layernorm": [binding.prepare("layernorm", xs[i], ys[i], gamma=g, beta=b) for i in range(sets)],
                        "rmsnorm": [binding.prepare("rmsnorm", xs[i], ys[i], gamma=g, eps=1e-5) for i in range(sets)]}
            line = {"dtype": dname, "rows": rows, "cols": cols}
            for op, pcs in prepared.items():
                call = lambda i, pcs=pcs: pcs[i].launch()
                for _ in range(3):
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
    ap.add_argument("--profile-next", default="", metavar="NAME",
                    help="as --profile, for an arg-max / cumulative / column-normalisation row of the bench "
                         "(workloads.REDUCTION_CONFIGS, COLNORM_CONFIGS)")
    ap.add_argument("--profile-shape", default="", metavar="OP:DTYPE:ROWS:COLS",
                    help="as --profile, for a seeded random matrix, e.g. layernorm:bf16:512:131072")
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
    if args.profile or args.profile_axis or args.profile_fused or args.profile_act or args.profile_shape or args.profile_next:
        run_profile(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
