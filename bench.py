#!/usr/bin/env python
"""Benchmark of the GDWS convolution forward (Section 3.1 of arXiv 2110.14871) on B200.

A "step" is one pass of the whole hot path (plan already built, weights already
packed: GDW stage, PW stage, bias) over one synthetic batch of the workload.  The
default workload is the CIFAR-shaped VGG-16 middle layer (N=256, C=D=256, 8x8, k=3,
g_c ~ U[1,9], bf16 NHWC).  Timing follows the paper's FPS protocol (Appendix A.1:
warm-up, then successive inferences between two CUDA events, no host I/O in the timed
region), adapted to one layer and a batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--config C] [--layer L] [--path fused|unfused] [--no-graph] [--chain]

A timed region is exactly K steps; it is repeated (--repeats, default: enough repeats for some tens of
milliseconds) with a CUDA event between repeats, and the median region gives ms_per_step.  With CUDA graphs
(default) every warm-up and timed launch is a graph node, whatever K is.  `--config 3 --chain` times the
16 chained layers of config 3 as one graph (a step = the whole chain over the batch).

Prints ONE JSON line.  With --gpus N > 1 (under torchrun) every rank runs an
independent replica on its own GPU (the path has no exchange step); the value is the
sum over ranks divided by the slowest rank's time.
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

from paper_2110_14871_b200 import inputs as gi  # noqa: E402

METRIC = "GDWS layer images/sec"
UNIT = "images/s"
L2_BYTES = 126e6


# ------------------------------------------------------------------------------------------
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def layer_numbers(spec: gi.LayerSpec, G: int):
    """Algorithmic work of one step: Eq. 3 MACs and the compulsory HBM bytes
    (x once, y once, weights once; the intermediate channels never counted)."""
    e = 4 if spec.dtype == "f32" else 2
    px = spec.N * spec.Ho * spec.Wo
    macs = px * G * (spec.k * spec.k + spec.D)
    nbytes = spec.N * spec.H * spec.W * spec.C * e + px * spec.D * e + (G * spec.k * spec.k + spec.D * G) * e + 4 * spec.D
    return px, macs, nbytes


# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu captures
# summarised under profiles/ (key: config, layer, path, GDW stage).  An entry is removed when its kernel changes.
TRAFFIC_BYTES_PER_LAUNCH = {
    (1, 0, "fused", 2): 9180928,      # x + weights; y (8.39 MB) stays in L2 within the captured launch
    (2, 0, "fused", 1): 25794304,     # x + weights; y (25.7 MB) stays in L2
    (3, 0, "fused", 2): 93909504,     # x (67.1 MB) + the part of y that left L2
}


def layer_roofline_us(macs, nbytes, peaks, sustained=False):
    tf = peaks["bf16_tflops_sustained" if sustained else "bf16_tflops"]
    t_tensor = 2.0 * macs / (tf * 1e12) * 1e6
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9) * 1e6
    return max(t_tensor, t_hbm), t_tensor, t_hbm


def slowest_rank(value: float, device=None) -> float:
    """Max of `value` over all ranks of the default process group (the value itself when there is none).
    Replicas share nothing on the data path; this reduction of the measured time is the only exchange."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(units_per_rank: float, world: int, seconds_slowest: float) -> float:
    """Whole-job throughput of `world` independent replicas: all units over the slowest rank's time."""
    return world * units_per_rank / seconds_slowest


def percentile(v, q):
    v = sorted(v)
    return v[min(len(v) - 1, max(0, int(round(q * (len(v) - 1)))))]


def timed_regions(run_region, repeats):
    """Runs `run_region` `repeats` times back to back with a CUDA event between them; returns the
    milliseconds of each region (device time on the current stream)."""
    import torch
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    evs[0].record()
    for r in range(repeats):
        run_region()
        evs[r + 1].record()
    torch.cuda.synchronize()
    return [evs[r].elapsed_time(evs[r + 1]) for r in range(repeats)]


def choose_repeats(args, region_ms_estimate):
    """Repeats of the K-step region: given, or enough for about 60 ms of timed work (at least 5, at most 2000),
    never more than about 20 s in total."""
    if args.repeats > 0:
        return args.repeats
    r = int(np.ceil(60.0 / max(region_ms_estimate, 1e-3)))
    r = max(5, min(2000, r))
    return max(1, min(r, int(20000.0 / max(region_ms_estimate, 1e-3))))


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        self._period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _loop(self):
        nv = self._nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self._period)

    def __enter__(self):
        if self._nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()

    def summary(self):
        med = int(statistics.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------
def oracle_throughput(spec: gi.LayerSpec, target_s: float = 12.0):
    """Images/s of the CPU reference on a bounded sample of the workload (host cores): the first
    images of the batch, passed through the reference again and again until about `target_s`
    seconds of work have been timed."""
    from oracle import gdws_oracle as orc
    n = min(spec.N, 2)
    d = gi.make_layer(spec, N=n)
    run = lambda dd: orc.forward(dd.x, dd.g, dd.dw_w, dd.pw_w, dd.bias, stride=spec.stride, pad=spec.pad,
                                 relu=spec.relu, layout=spec.layout)
    t0 = time.perf_counter()
    run(d)
    probe = (time.perf_counter() - t0) / n
    n = int(max(1, min(spec.N, 0.25 * target_s / max(probe, 1e-6))))
    d = gi.make_layer(spec, N=n)
    run(d)                                   # warm-up of this size
    reps, t0 = 0, time.perf_counter()
    while True:
        run(d)
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= target_s or reps >= 10000:
            break
    return n * reps / dt, n, reps, dt, orc.num_threads()


def run_reference(args, spec):
    """--impl reference: the CPU reference as it stands, on the host cores, same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import gdws_oracle as orc
    d_full_g = gi.make_layer(spec, N=1).g
    G = int(d_full_g.sum())
    _, macs, _ = layer_numbers(spec, G)
    per_img = macs / spec.N
    # bounded sample: about 1.5 s of reference work per step
    probe_n = min(spec.N, 2)
    d = gi.make_layer(spec, N=probe_n)
    t0 = time.perf_counter()
    orc.forward(d.x, d.g, d.dw_w, d.pw_w, d.bias, stride=spec.stride, pad=spec.pad, relu=spec.relu, layout=spec.layout)
    probe = (time.perf_counter() - t0) / probe_n
    budget = min(1.5, 150.0 / max(1, args.steps + args.warmup))
    n = int(max(1, min(spec.N, budget / max(probe, 1e-6))))
    d = gi.make_layer(spec, N=n)
    run = lambda: orc.forward(d.x, d.g, d.dw_w, d.pw_w, d.bias, stride=spec.stride, pad=spec.pad, relu=spec.relu,
                              layout=spec.layout)
    for _ in range(args.warmup):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    sample = f"{n} of {spec.N} images per step ({per_img * n / 1e9:.3f} GMAC), {args.steps} steps"
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(spec, G) | {"note": "CPU reference (oracle/), fp64 direct loops"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def dense_conv_context(spec: gi.LayerSpec, data, x0, nsets: int, steps: int):
    """Context only, not part of the product path: the dense k x k convolution that the GDWS layer replaces
    (Eq. 1), run by the vendor library through torch (bf16, channels_last), with the dense weights rebuilt from
    the layer's factors (Property 1 and 2: W[d, c] = sum_j P[d, off_c + j] K[off_c + j]).  Same batch, same
    rotation of input buffers, CUDA events."""
    import torch
    import torch.nn.functional as F
    if spec.dtype != "bf16":
        return None
    k2 = spec.k * spec.k
    off = np.concatenate([[0], np.cumsum(data.g)]).astype(np.int64)
    Wd = np.zeros((spec.D, spec.C, k2), dtype=np.float32)
    Kf = data.dw_w.reshape(-1, k2).astype(np.float32)
    for c in range(spec.C):
        a, b = off[c], off[c + 1]
        if b > a:
            Wd[:, c, :] = data.pw_w[:, a:b].astype(np.float32) @ Kf[a:b]
    w = torch.from_numpy(Wd.reshape(spec.D, spec.C, spec.k, spec.k)).cuda().to(torch.bfloat16).contiguous(memory_format=torch.channels_last)
    b = torch.from_numpy(data.bias).cuda().to(torch.bfloat16)
    xs = [x0.permute(0, 3, 1, 2)]                       # NHWC storage seen as NCHW channels_last
    xs += [xs[0].clone(memory_format=torch.channels_last) for _ in range(min(nsets, 16) - 1)]
    run = lambda i: F.conv2d(xs[i % len(xs)], w, b, stride=spec.stride, padding=spec.pad)
    for i in range(5):
        run(i)
    torch.cuda.synchronize()
    n = max(10, min(steps, 200))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n):
        run(i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / n
    return {"what": "dense k x k conv of the same layer, vendor library via torch (bf16 channels_last, plain launches)",
            "ms_per_step": ms, "images_per_s": spec.N / (ms * 1e-3), "dense_macs": spec.N * spec.Ho * spec.Wo * spec.D * spec.C * k2}


PAPER_CONTEXT = ("paper (Table 1, App. A.1): whole networks at batch 1 on a Jetson Xavier NX (384-core Volta GPU), PyTorch 1.8, "
                 "frames/s baseline -> GDWS: ResNet-50 16 -> 37, WRN-28-4 17 -> 65, ResNet-18 28 -> 104, VGG-16 36 -> 129 (CIFAR-10)")


def workload_config(spec: gi.LayerSpec, G: int):
    return {"workload": f"{spec.name}: N={spec.N} C={spec.C} D={spec.D} {spec.H}x{spec.W} k={spec.k} "
                        f"stride={spec.stride} pad={spec.pad} g~{spec.g_dist} G={G} {spec.dtype} {spec.layout}",
            "global_batch": spec.N}


# ------------------------------------------------------------------------------------------
def run_ours(args, spec):
    import torch
    import torch.distributed as dist

    from paper_2110_14871_b200 import build as gbuild
    from paper_2110_14871_b200 import gdws

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        gbuild.build_library()
    if world > 1:
        dist.barrier()
    peaks = load_peaks()

    data = gi.make_layer(spec)
    G = data.G
    px, macs, nbytes = layer_numbers(spec, G)
    tdt = torch.float32 if spec.dtype == "f32" else torch.bfloat16
    code = gdws.F32 if spec.dtype == "f32" else gdws.BF16

    def dev(a):
        t = torch.from_numpy(np.ascontiguousarray(a))
        return (t.to(torch.bfloat16) if spec.dtype == "bf16" else t).cuda()

    x0, dw, pw = dev(data.x), dev(data.dw_w), dev(data.pw_w)
    bias = torch.from_numpy(data.bias).cuda()
    yshape = (spec.N, spec.D, spec.Ho, spec.Wo) if spec.layout == "NCHW" else (spec.N, spec.Ho, spec.Wo, spec.D)
    set_bytes = x0.numel() * x0.element_size() + int(np.prod(yshape)) * x0.element_size()
    nsets = max(2, int(np.ceil(3.2 * L2_BYTES / set_bytes))) if set_bytes < 2.5 * L2_BYTES else 1
    nsets = min(nsets, 64)
    xs = [x0] + [x0.clone() for _ in range(nsets - 1)]
    ys = [torch.empty(yshape, dtype=tdt, device="cuda") for _ in range(nsets)]

    plan = gdws.Plan(spec.C, spec.D, spec.k, spec.stride, spec.pad, data.g)
    plan.set_option(gdws.OPT_RELU, int(spec.relu))
    path = {"fused": gdws.PATH_FUSED, "unfused": gdws.PATH_UNFUSED, "auto": gdws.PATH_AUTO}[args.path]
    plan.set_option(gdws.OPT_PATH, path)
    plan.set_option(gdws.OPT_DW_MATH, args.dw_math)
    plan.set_option(gdws.OPT_A_LAYOUT, args.a_layout)
    if args.tile:
        plan.set_option(gdws.OPT_TILE, args.tile)
    if path == gdws.PATH_UNFUSED:
        ws = torch.empty(plan.workspace_bytes(code, spec.N, spec.H, spec.W) + 256, dtype=torch.uint8, device="cuda")
        plan.set_workspace(ws)
    f32 = spec.dtype == "f32"
    if not f32:
        plan.pack_weights(dw, pw, bias)
    wargs = dict(dw_w=dw, pw_w=pw, bias=bias) if f32 else {}
    stream = torch.cuda.current_stream()

    def step(i):
        plan.forward(xs[i % nsets], ys[i % nsets], spec.layout, stream=stream, **wargs)

    # one checked forward before timing: sampled parity against the CPU reference (rank 0)
    step(0)
    torch.cuda.synchronize()
    plan.status()
    l0 = plan.launch_count()
    step(0)
    launches_per_step = plan.launch_count() - l0

    # Launch mode.  With graphs, two graphs cover any K: one of `nsets` launches (one per buffer set) and one of
    # K mod nsets launches, so that every warm-up and timed launch is a graph node.
    graphs = None
    if not args.no_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(nsets):
                plan.forward(xs[i], ys[i], spec.layout, stream=side, **wargs)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()

        def capture(count):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(count):
                    plan.forward(xs[i % nsets], ys[i % nsets], spec.layout, stream=torch.cuda.current_stream(), **wargs)
            return g
        graphs = (capture(nsets), capture(args.steps % nsets) if args.steps % nsets else None)

    def run_region():
        if graphs is None:
            for i in range(args.steps):
                step(i)
        else:
            for _ in range(args.steps // nsets):
                graphs[0].replay()
            if graphs[1] is not None:
                graphs[1].replay()

    for _ in range(max(3, -(-args.warmup // max(1, args.steps)))):     # at least W warm-up steps, in whole regions
        run_region()
    torch.cuda.synchronize()
    probe = timed_regions(run_region, 3)
    repeats = choose_repeats(args, min(probe))
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local) as clk:
        region_ms = timed_regions(run_region, repeats)
    ms = statistics.median(region_ms)
    if world > 1:
        dist.barrier()
        ms = slowest_rank(ms, device="cuda")
    plan.status()
    sec_per_step = ms / 1e3 / args.steps
    value = aggregate_value(spec.N, world, sec_per_step)

    # end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    e2e = None
    if not f32 or True:
        xh = torch.from_numpy(np.ascontiguousarray(data.x))
        xh = (xh.to(torch.bfloat16) if spec.dtype == "bf16" else xh).pin_memory()
        yh = torch.empty(yshape, dtype=tdt).pin_memory()
        k_e2e = max(3, min(args.steps, 30))
        for _ in range(3):
            plan.forward_host(xh, yh, spec.layout, stream=stream, **wargs)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(k_e2e):
            plan.forward_host(xh, yh, spec.layout, stream=stream, **wargs)
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / k_e2e
        if world > 1:
            dt = slowest_rank(dt, device="cuda")
        e2e = {"value": aggregate_value(spec.N, world, dt), "unit": UNIT, "h2d_bytes_per_step": xh.numel() * xh.element_size(),
               "d2h_bytes_per_step": yh.numel() * yh.element_size(), "steps": k_e2e}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    t_roof, t_tensor, t_hbm = layer_roofline_us(macs, nbytes, peaks)
    t_roof_s, _, _ = layer_roofline_us(macs, nbytes, peaks, sustained=True)
    us = sec_per_step * 1e6
    # The default kernel runs the GDW stage on the fp32 FMA lanes.  Its bound there: 128 FMA lanes per SM at
    # the maximum SM clock.
    clocks = clk.summary()
    props = torch.cuda.get_device_properties(local)
    sm_mhz = float(clocks.get("sm_max_mhz") or 1965)
    derived_tflops = 2.0 * props.multi_processor_count * 128 * sm_mhz * 1e6 / 1e12
    fma_per_clk, fma_tmacs = gdws.measure_fma_rate(gdws.FMA_F32)       # measured now, on this device
    alu_tflops = 2.0 * fma_tmacs
    dw_macs = px * G * spec.k * spec.k
    t_alu = 2.0 * dw_macs / (alu_tflops * 1e12) * 1e6
    # Layer roofline: the slower of the Eq. 3 MACs at the tensor peak and the compulsory bytes at the copy bandwidth.
    # The ALU time of the GDW stage is reported beside it as a diagnostic (it binds the default kernel on the
    # 64-channel layers), not as part of the roofline: the GDW stage can also run on the tensor cores.
    bound = "tensor" if t_tensor >= t_hbm else "hbm"
    if bound == "tensor":
        achieved, peak, runit = 2.0 * macs / sec_per_step / 1e12, peaks["bf16_tflops"], "TFLOP/s"
        psrc = peaks["source"] + " burst"
    else:
        achieved, peak, runit = nbytes / sec_per_step / 1e9, peaks["hbm_gbs"], "GB/s"
        psrc = peaks["source"] + " copy"
    roof = {"bound": bound, "achieved": achieved, "peak": peak, "unit": runit, "frac": achieved / peak,
            "traffic": TRAFFIC_BYTES_PER_LAUNCH.get((args.config, args.layer, args.path, plan.gdw_stage())) if not f32 else None,
            "peak_source": psrc,
            "kernel": ("fused_tc_kernel" if plan.gdw_stage() == 2 else "fused_bf16_kernel") if (not f32 and path != gdws.PATH_UNFUSED) else "see config.path",
            "layer_roofline_us": t_roof, "t_tensor_us": t_tensor, "t_hbm_us": t_hbm,
            "frac_of_layer_roofline": t_roof / us, "frac_of_layer_roofline_sustained_peak": t_roof_s / us,
            "gdw_on_alus": {"t_alu_us": t_alu, "peak_tflops": alu_tflops,
                            "peak_source": "measured in this run: independent fp32 FMAs on all SMs (gdws_measure_fma_rate)",
                            "fma_per_clk_per_sm": fma_per_clk, "derived_peak_tflops": derived_tflops,
                            "frac_of_max_tensor_hbm_alu": max(t_roof, t_alu) / us}}

    cpu_v, cpu_n, cpu_reps, cpu_dt, cores = oracle_throughput(spec, target_s=args.cpu_seconds)
    cpu = {"value": cpu_v, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"the first {cpu_n} of {spec.N} images, {cpu_reps} passes, {cpu_dt:.1f} s of CPU reference work"}

    # parity of the timed configuration on sampled images
    parity = None
    if args.check:
        from oracle import gdws_oracle as orc
        torch.cuda.synchronize()
        sel = sorted(set([0, spec.N // 2, spec.N - 1]))
        yg = ys[0][sel].float().cpu().numpy().astype(np.float64)
        xsel = data.x[sel]
        ref, _ = orc.forward(xsel, data.g, data.dw_w, data.pw_w, data.bias, stride=spec.stride, pad=spec.pad,
                             relu=spec.relu, layout=spec.layout)
        parity = float(np.max(np.abs(yg - ref)) / np.max(np.abs(ref)))

    context = {"paper": PAPER_CONTEXT}
    if args.context:
        try:
            context["dense_conv"] = dense_conv_context(spec, data, x0, nsets, args.steps)
        except Exception as exc:      # context only: never fails the bench line
            context["dense_conv"] = {"unavailable": repr(exc)[:200]}

    cfg = workload_config(spec, G)
    cfg.update({"path": args.path, "gdw_stage": ("tensor cores" if plan.gdw_stage() == 2 else "ALUs") + (" (chosen by the library)" if args.dw_math == 0 else " (forced)"), "launch": "cuda graph replay (every warm-up and timed launch is a graph node)" if graphs is not None else "plain launches",
                "timing": {"repeats_of_the_k_step_region": repeats, "region_ms_median": ms, "region_ms_p10": percentile(region_ms, 0.1),
                           "region_ms_p90": percentile(region_ms, 0.9), "timed_ms_total": float(sum(region_ms))},
                "l2": f"rotating {nsets} input/output buffer sets ({nsets * set_bytes / 1e6:.0f} MB > 126 MB L2)"
                      if nsets > 1 else "one buffer set larger than L2",
                "tile": "TNxPHxPW=%dx%dx%d" % plan.tile(spec.N, spec.H, spec.W)[:3] if not f32 else None,
                "parallelism": "replicas" if world > 1 else "single GPU"})
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": sec_per_step * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": spec.dtype, "data": "synthetic", "config": cfg,
        "effective_tmacs": world * macs / sec_per_step / 1e12,
        "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches_per_step * args.steps * repeats,
        "clocks": clocks, "parity_max_rel_err": parity, "context": context,
    }
    print(json.dumps(out), flush=True)
    plan.destroy()
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------
def run_chain(args):
    """Config 3: the 16 chained 3x3 layers (ReLU between them), a step = the whole chain over the batch.
    One CUDA graph holds the 16 launches; y of layer l is x of layer l+1.  The metric is end-to-end images/s,
    the roofline the sum of the layers' rooflines."""
    import torch

    from paper_2110_14871_b200 import build as gbuild
    from paper_2110_14871_b200 import gdws

    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("--chain runs on one GPU")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(0)
    gbuild.build_library()
    peaks = load_peaks()
    layers = gi.config_layers(3)
    N = layers[0].N
    gen = torch.Generator(device="cuda").manual_seed(3000)
    acts = [torch.randn((N, layers[0].H, layers[0].W, layers[0].C), generator=gen, device="cuda").to(torch.bfloat16)]
    plans, macs_total, roof_total, per_layer = [], 0, 0.0, []
    for spec in layers:
        rng = np.random.Generator(np.random.PCG64(spec.seed))
        g = gi.make_g(rng, spec.C, spec.g_dist)
        G = int(g.sum())
        dw = torch.from_numpy(gi.round_to_bf16((rng.standard_normal((G, spec.k, spec.k)) / spec.k).astype(np.float32))).to(torch.bfloat16).cuda()
        pw = torch.from_numpy(gi.round_to_bf16((rng.standard_normal((spec.D, G)) / np.sqrt(G)).astype(np.float32))).to(torch.bfloat16).cuda()
        b = torch.from_numpy((rng.standard_normal(spec.D) * 0.1).astype(np.float32)).cuda()
        plan = gdws.Plan(spec.C, spec.D, spec.k, spec.stride, spec.pad, g)
        plan.set_option(gdws.OPT_RELU, int(spec.relu))
        plan.set_option(gdws.OPT_PATH, gdws.PATH_FUSED)
        plan.set_option(gdws.OPT_DW_MATH, args.dw_math)
        plan.pack_weights(dw, pw, b)
        plans.append(plan)
        acts.append(torch.empty((N, spec.Ho, spec.Wo, spec.D), dtype=torch.bfloat16, device="cuda"))
        _, macs, nbytes = layer_numbers(spec, G)
        t_roof, _, _ = layer_roofline_us(macs, nbytes, peaks)
        macs_total += macs
        roof_total += t_roof
        per_layer.append(t_roof)

    def chain(stream):
        for l, plan in enumerate(plans):
            plan.forward(acts[l], acts[l + 1], "NHWC", stream=stream)

    chain(torch.cuda.current_stream())
    torch.cuda.synchronize()
    for plan in plans:
        plan.status()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = None
    if not args.no_graph:
        with torch.cuda.stream(side):
            chain(side)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            chain(torch.cuda.current_stream())
    steps = args.steps if args.steps != 20000 else 20

    def run_region():
        for _ in range(steps):
            if graph is None:
                chain(torch.cuda.current_stream())
            else:
                graph.replay()

    for _ in range(3):
        run_region()
    torch.cuda.synchronize()
    probe = timed_regions(run_region, 2)
    repeats = choose_repeats(args, min(probe))
    with ClockSampler(0) as clk:
        region_ms = timed_regions(run_region, repeats)
    ms = statistics.median(region_ms)
    for plan in plans:
        plan.status()
    sec = ms / 1e3 / steps
    out = {
        "metric": "GDWS 16-layer chain end-to-end images/sec", "value": N / sec, "unit": UNIT, "n_gpus": 1, "steps": steps,
        "warmup": 3 * steps, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"c3 chain: N={N}, 16 layers 64@32x32 ... 512@4x4, k=3, g~U[1,9], ReLU between layers, bf16 NHWC",
                   "global_batch": N, "launch": "one cuda graph of the 16 launches" if graph is not None else "plain launches",
                   "gdw_stage": {1: "ALUs (forced)", 2: "tensor cores (forced)"}.get(args.dw_math, "chosen per layer by the library: " + "".join("T" if pl.gdw_stage() == 2 else "A" for pl in plans)),
                   "l2": "each layer reads what the previous one wrote (0.03-67 MB per tensor, 126 MB L2), as a chained network does",
                   "timing": {"repeats_of_the_k_step_region": repeats, "region_ms_p10": percentile(region_ms, 0.1),
                              "region_ms_p90": percentile(region_ms, 0.9)}},
        "effective_tmacs": macs_total / sec / 1e12,
        "roofline": {"bound": "sum of the layers' rooflines", "layer_roofline_us_sum": roof_total, "frac_of_summed_layer_rooflines": roof_total / (sec * 1e6),
                     "per_layer_roofline_us": per_layer, "peak_source": peaks["source"]},
        "gpu_launches": len(plans) * steps * repeats, "clocks": clk.summary(),
    }
    print(json.dumps(out), flush=True)
    for plan in plans:
        plan.destroy()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--layer", type=int, default=0)
    ap.add_argument("--path", default="fused", choices=["fused", "unfused", "auto"])
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-check", dest="check", action="store_false")
    ap.add_argument("--no-context", dest="context", action="store_false")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--dw-math", type=int, default=0)
    ap.add_argument("--a-layout", type=int, default=0)
    ap.add_argument("--tile", type=int, default=0)
    ap.add_argument("--repeats", type=int, default=0, help="repeats of the K-step timed region (0: choose)")
    ap.add_argument("--chain", action="store_true", help="config 3: the 16 chained layers as one step")
    args = ap.parse_args()
    if args.chain:
        if args.config != 3 or args.impl != "ours":
            raise SystemExit("--chain is the 16-layer chain of config 3 (our arm)")
        run_chain(args)
        return
    spec = gi.config_layers(args.config)[args.layer]
    if args.impl == "reference":
        if args.steps == 20000:
            args.steps, args.warmup = 20, 3
        run_reference(args, spec)
    else:
        run_ours(args, spec)


if __name__ == "__main__":
    main()
