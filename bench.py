#!/usr/bin/env python
"""Benchmark of the im2win hot path on B200.

A step is one pass of the whole hot path over one batch of the headline layer
(ResNet-style 3x3 layer, N=128 C=64 56x56 -> 64): im2win transform, filter
pack and convolution, once in fp32 (CUDA cores) and once in fp16-in /
fp32-accumulate (tensor cores).  The metric is convolution TFLOPS,
2*N*Co*Ho*Wo*C*Kh*Kw per precision, over the device time of the whole step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--report FILE]

prints one JSON line (rank 0).  `--report FILE` additionally times every layer
of the workload table kernel by kernel and writes one JSON object per layer.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2608_20725_b200 import replicas, workloads  # noqa: E402

METRIC = "conv TFLOPS (fp32 + fp16 passes of the layer, transform and filter pack included)"
UNIT = "TFLOP/s"
SM_COUNT = 148
FP32_LANES_PER_SM = 128
SM_MAX_GHZ = 1.965
# fp32 FFMA peak from unit counts and the maximum SM clock: 148 * 128 lanes * 2 flop * 1.965 GHz
FP32_PEAK_TFLOPS = SM_COUNT * FP32_LANES_PER_SM * 2 * SM_MAX_GHZ / 1e3
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            d = json.load(fh)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def layer_flops(layer, ho, wo):
    return 2.0 * layer.N * layer.Co * ho * wo * layer.C * layer.Kh * layer.Kw


# --------------------------------------------------------------------- clocks ----
class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU through NVML (read-only queries)
    from a background thread while the timed region runs."""

    REASONS = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
               "hw_thermal_slowdown": 0x40}

    def __init__(self, index: int, period_s: float = 0.002):
        self.index = index
        self.period = period_s
        self.samples = []
        self.stop_flag = threading.Event()
        self.thread = None
        self.handle = None
        self.nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if visible:
                ids = [v.strip() for v in visible.split(",") if v.strip()]
                if index < len(ids) and ids[index].isdigit():
                    phys = int(ids[index])
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.nvml = pynvml
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nvml = None

    def _sample(self):
        n = self.nvml
        try:
            mhz = float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM))
            reasons = int(n.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
            power = n.nvmlDeviceGetPowerUsage(self.handle) / 1000.0
            self.samples.append((mhz, reasons, power))
        except Exception:
            pass

    def _run(self):
        while not self.stop_flag.is_set():
            self._sample()
            time.sleep(self.period)

    def start(self):
        if self.nvml is None:
            return
        self._sample()
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

    def stop(self):
        if self.nvml is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self._sample()
        self.stop_flag.set()
        if self.thread is not None:
            self.thread.join(timeout=2)
        mhz = sorted(s[0] for s in self.samples)
        seen = 0
        for s in self.samples:
            seen |= s[1]
        reasons = sorted(k for k, bit in self.REASONS.items() if seen & bit)
        return {"sm_mhz": mhz[len(mhz) // 2] if mhz else None, "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(mhz), "power_w_max": max((s[2] for s in self.samples), default=None)}


# -------------------------------------------------------------- the GPU arm ----
class LayerRunner:
    """Device-resident buffers of one layer and the four calls of a step."""

    def __init__(self, layer, precisions=("f32", "f16"), sets=1):
        """`sets` > 1 keeps that many copies of every device buffer (inputs included), so that
        launches queued back to back can each work on memory the one before did not touch."""
        from paper_2608_20725_b200 import binding
        self.b = binding
        self.layer = layer
        self.dims = layer.dims()
        self.sets = sets
        x, f = workloads.make_inputs(layer)
        self.host = {}
        self.dev = {}
        self.dev_sets = {}
        for prec in precisions:
            tdt = torch.float32 if prec == "f32" else torch.float16
            xh, fh = x.to(tdt).contiguous(), f.to(tdt).contiguous()
            self.dev_sets[prec] = []
            for i in range(sets):
                window, scratch, y = binding.alloc_layer_buffers(self.dims, tdt)
                xd = xh.cuda() if i == 0 else self.dev_sets[prec][0]["x"].clone()
                self.dev_sets[prec].append(dict(x=xd, f=fh.cuda(), window=window, scratch=scratch, y=y))
            self.dev[prec] = self.dev_sets[prec][0]
            self.host[prec] = (xh, fh)
        code = binding.F32 if "f32" in precisions else binding.F16
        _, _, self.ho, self.wo = binding.im2win_workspace_size(self.dims, code)
        self.flops = layer_flops(layer, self.ho, self.wo)
        self.precisions = precisions
        self.nhwc = None

    def add_nhwc(self):
        """Buffers of the channel-innermost (NHWC) form of the fp16 path: same NCHW input and OIHW
        filter, NHWC window tensor, fp32 NCHW output."""
        b = self.b
        x, f = workloads.make_inputs(self.layer)
        x16, f16 = x.half().cuda(), f.half().cuda()
        cp = b.im2win_nhwc_workspace_size(self.dims)[4]
        self.nhwc_sets = []
        for i in range(self.sets):
            window, scratch, y = b.alloc_nhwc_buffers(self.dims)
            d = dict(x=x16 if i == 0 else x16.clone(), f=f16 if i == 0 else f16.clone(), window=window,
                     scratch=scratch, y=y, cp=cp, y16=torch.empty(y.shape, dtype=torch.float16, device="cuda"),
                     bias=torch.zeros(self.layer.Co, dtype=torch.float32, device="cuda"))
            d["epi16"] = b.make_epilogue(d["bias"], True, torch.float16, b.NCHW)
            d["x_nhwc"] = d["x"].permute(0, 2, 3, 1).contiguous()      # the same input, channel-innermost
            self.nhwc_sets.append(d)
        self.nhwc = self.nhwc_sets[0]

    def transform_nhwc(self, prec=None, i=0):
        d = self.nhwc_sets[i]
        self.b.im2win_transform_nhwc(d["x"], self.b.NCHW, d["window"], self.dims)

    def transform_nhwc_from_nhwc(self, prec=None, i=0):
        """The same window tensor from a channel-innermost input (what a chain of NHWC layers feeds)."""
        d = self.nhwc_sets[i]
        self.b.im2win_transform_nhwc(d["x_nhwc"], self.b.NHWC, d["window"], self.dims)

    def conv_nhwc(self, prec=None, i=0):
        d = self.nhwc_sets[i]
        self.b.im2win_conv_f16_nhwc(d["window"], d["f"], d["y"], d["scratch"], self.dims)

    def conv_nhwc_out16(self, prec=None, i=0):
        """The same convolution with the fused epilogue: bias, ReLU, binary16 NCHW output."""
        d = self.nhwc_sets[i]
        self.b.im2win_conv_f16_nhwc(d["window"], d["f"], d["y16"], d["scratch"], self.dims, d["epi16"])

    def conv_nhwc_packed(self, prec=None, i=0):
        d = self.nhwc_sets[i]
        self.b.im2win_conv_packed_nhwc(d["window"], d["y"], d["scratch"], self.dims)

    def transform(self, prec, i=0):
        d = self.dev_sets[prec][i]
        self.b.im2win_transform(d["x"], d["window"], self.dims)

    def conv(self, prec, i=0):
        d = self.dev_sets[prec][i]
        if prec == "f32":
            self.b.im2win_conv_f32(d["window"], d["f"], d["y"], d["scratch"], self.dims)
        else:
            self.b.im2win_conv_f16(d["window"], d["f"], d["y"], d["scratch"], self.dims)

    def conv_packed(self, prec, i=0):
        """The convolution alone, on the filter the last conv() call left packed in scratch."""
        d = self.dev_sets[prec][i]
        self.b.im2win_conv_packed(d["window"], d["y"], d["scratch"], self.dims)

    def step(self, events=None):
        """One pass of the hot path; with `events` (list) records an event before/after each call."""
        for prec in self.precisions:
            for name, fn in (("transform", self.transform), ("conv", self.conv)):
                if events is not None:
                    e0 = torch.cuda.Event(enable_timing=True)
                    e0.record()
                fn(prec)
                if events is not None:
                    e1 = torch.cuda.Event(enable_timing=True)
                    e1.record()
                    events.append((f"{name}_{prec}", e0, e1))

    def algorithmic_bytes(self, kernel):
        """Bytes each kernel must move once: input + window for a transform, window + output (+ filter) for a convolution."""
        l, es = self.layer, (4 if kernel.endswith("f32") else 2)
        x_el = l.N * l.C * l.H * l.W
        chans = self.nhwc["cp"] if kernel.endswith("nhwc") else l.C        # the NHWC form stores C rounded up to 8
        win_el = l.N * chans * self.ho * l.Kh * (l.W + 2 * l.pad)
        out_el = l.N * l.Co * self.ho * self.wo
        f_el = l.Co * l.C * l.Kh * l.Kw
        if kernel.startswith("transform"):
            return (x_el + win_el) * es
        if kernel.endswith("out16_nhwc"):
            return win_el * es + f_el * es + out_el * 2 + l.Co * 4
        return win_el * es + f_el * es + out_el * 4

    def memory_report(self):
        l = self.layer
        rep = {}
        for prec in self.precisions:
            es = 4 if prec == "f32" else 2
            win = l.N * l.C * self.ho * l.Kh * (l.W + 2 * l.pad) * es
            out = l.N * l.Co * self.ho * self.wo * 4
            rep[prec] = {"window_bytes": win, "output_bytes": out, "window_plus_output_bytes": win + out,
                         "scratch_bytes": self.dev[prec]["scratch"].numel(),
                         "im2col_bytes": l.N * l.C * l.Kh * l.Kw * self.ho * self.wo * es}
        if self.nhwc is not None:
            win = l.N * self.nhwc["cp"] * self.ho * l.Kh * (l.W + 2 * l.pad) * 2
            out = l.N * l.Co * self.ho * self.wo * 4
            rep["f16_nhwc"] = {"window_bytes": win, "output_bytes": out, "window_plus_output_bytes": win + out,
                               "scratch_bytes": self.nhwc["scratch"].numel(),
                               "im2col_bytes": l.N * l.C * l.Kh * l.Kw * self.ho * self.wo * 2}
        return rep


def kernel_rooflines(runner, avg_ms, peaks, peak_kind):
    """Roofline entry of every call of the step from its average device time."""
    out = {}
    for name, ms in avg_ms.items():
        sec = ms * 1e-3
        nbytes = runner.algorithmic_bytes(name)
        if name.startswith("transform"):
            a = nbytes / sec / 1e9
            out[name] = {"bound": "hbm", "achieved": a, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": a / peaks["hbm_gbs"], "peak_kind": peak_kind, "ms": ms}
        elif name == "conv_f32":
            a = runner.flops / sec / 1e12
            out[name] = {"bound": "alu", "achieved": a, "peak": FP32_PEAK_TFLOPS, "unit": "TFLOP/s",
                         "frac": a / FP32_PEAK_TFLOPS, "peak_kind": "148 SM x 128 lanes x 2 x 1.965 GHz", "ms": ms}
        else:
            tf = runner.flops / sec / 1e12
            # fp16 dense peak: measured bf16 GEMM peak (same tensor rate for fp16 and bf16)
            tensor_peak = peaks["bf16_tflops"]
            t_tensor = runner.flops / (tensor_peak * 1e12)
            t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
            if t_hbm > t_tensor:
                a = nbytes / sec / 1e9
                out[name] = {"bound": "hbm", "achieved": a, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                             "frac": a / peaks["hbm_gbs"], "peak_kind": peak_kind, "ms": ms, "tflops": tf}
            else:
                out[name] = {"bound": "tensor", "achieved": tf, "peak": tensor_peak, "unit": "TFLOP/s",
                             "frac": tf / tensor_peak, "peak_kind": peak_kind, "ms": ms, "tflops": tf}
            out[name]["frac_of_tensor_peak"] = tf / tensor_peak
    return out


def load_traffic():
    """Per-launch DRAM traffic of each kernel from the committed ncu summary, if present."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as fh:
            return json.load(fh)
    except Exception:
        return {}


def time_cpu_oracle(layer, target_seconds=12.0):
    """Times the oracle's im2win route (fp64, OpenMP) on a bounded slice of the batch."""
    import numpy as np
    import oracle
    x, f = workloads.make_inputs(layer)
    xn, fn = x.numpy(), f.numpy()
    dims = layer.dims()
    ho, wo = oracle.out_dims(dims)
    per_image = layer_flops(layer, ho, wo) / layer.N
    t0 = time.perf_counter()
    oracle.conv_im2win_range(xn, fn, dims, 0, 1)
    t1 = time.perf_counter() - t0
    n = int(max(1, min(layer.N, target_seconds / max(t1, 1e-6))))
    reps = 0
    t0 = time.perf_counter()
    while True:                                   # whole passes over the sample until ~target_seconds
        oracle.conv_im2win_range(xn, fn, dims, 0, n)
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= target_seconds or reps >= 200:
            break
    return {"value": per_image * n * reps / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"fp64 im2win route (transform + convolution) on {n} of {layer.N} images of {layer.name}, "
                      f"{reps} passes ({dt:.1f} s)"}


def run_gpu_arm(args):
    from paper_2608_20725_b200 import binding
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    layer = workloads.LAYERS[workloads.BENCH_LAYER]
    peaks, peak_kind = load_peaks()
    runner = LayerRunner(layer)
    torch.cuda.reset_peak_memory_stats()

    for _ in range(args.warmup):
        runner.step()
    for prec in runner.precisions:
        binding.im2win_check_status(runner.dev[prec]["scratch"])

    # ---- timed region: K steps, device time, max over ranks --------------------
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    events = []
    start = torch.cuda.Event(enable_timing=True)
    stop = torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(args.steps):
        runner.step(events)
    stop.record()
    barrier()
    clocks = sampler.stop()
    total_ms = start.elapsed_time(stop)
    for prec in runner.precisions:
        binding.im2win_check_status(runner.dev[prec]["scratch"])
    peak_alloc = torch.cuda.max_memory_allocated()

    per_call = {}
    for name, e0, e1 in events:
        per_call.setdefault(name, []).append(e0.elapsed_time(e1))
    avg_ms = {k: sum(v) / len(v) for k, v in per_call.items()}

    # ---- end to end: host buffers, copies inside the timed region ---------------
    e2e_sets = {}
    for prec in runner.precisions:
        xh, fh = runner.host[prec]
        code = binding.F32 if prec == "f32" else binding.F16
        nbytes = binding.im2win_layer_workspace_size(runner.dims, code)
        e2e_sets[prec] = dict(x=xh.pin_memory(), f=fh.pin_memory(),
                              y=torch.empty((layer.N, layer.Co, runner.ho, runner.wo), dtype=torch.float32).pin_memory(),
                              ws=torch.empty(nbytes, dtype=torch.uint8, device="cuda"))

    def e2e_step():
        for prec in runner.precisions:
            s = e2e_sets[prec]
            binding.im2win_layer_forward_host(s["x"], s["f"], s["y"], s["ws"], runner.dims)

    e2e_steps = max(1, min(args.steps, 5))
    e2e_step()
    barrier()
    es, ee = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    es.record()
    for _ in range(e2e_steps):
        e2e_step()
    ee.record()
    barrier()
    e2e_ms = es.elapsed_time(ee)
    h2d = sum(e2e_sets[p]["x"].numel() * e2e_sets[p]["x"].element_size()
              + e2e_sets[p]["f"].numel() * e2e_sets[p]["f"].element_size() for p in runner.precisions)
    d2h = sum(e2e_sets[p]["y"].numel() * 4 for p in runner.precisions)

    total_ms, e2e_ms = replicas.max_over_ranks([total_ms, e2e_ms], device="cuda")

    step_flops = runner.flops * len(runner.precisions)
    value = replicas.whole_job_rate(step_flops * args.steps, world, total_ms) / 1e12
    e2e_value = replicas.whole_job_rate(step_flops * e2e_steps, world, e2e_ms) / 1e12

    rooflines = kernel_rooflines(runner, avg_ms, peaks, peak_kind)
    traffic = load_traffic()
    dominant = max(avg_ms, key=avg_ms.get)
    roof = dict(rooflines[dominant])
    roof["kernel"] = dominant
    roof["traffic"] = traffic.get(f"{layer.name}:{dominant}")

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32+f16", "data": "synthetic",
        "config": {"workload": f"{layer.name}: N={layer.N} C={layer.C} H=W={layer.H} Co={layer.Co} "
                               f"K={layer.Kh}x{layer.Kw} stride={layer.stride} pad={layer.pad}, fp32 and fp16 passes",
                   "l2": "working set per pass (input+window+output >= 360 MB) exceeds the 126 MB L2",
                   "parallelism": f"batch replicas x{world}, no collective"},
        "tflops": {p: runner.flops / (avg_ms[f"conv_{p}"] * 1e-3) / 1e12 for p in runner.precisions},
        "tflops_with_transform": {p: runner.flops / ((avg_ms[f"conv_{p}"] + avg_ms[f"transform_{p}"]) * 1e-3) / 1e12
                                  for p in runner.precisions},
        "roofline": roof,
        "kernels": rooflines,
        "memory": dict(runner.memory_report(), torch_peak_allocated_bytes=peak_alloc),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
        "gpu_launches": 6 * args.steps,
        "clocks": clocks,
    }
    if rank == 0:
        if world == 1 and not args.no_per_layer:
            # every BASELINE config, call by call (the metric is "per layer"): 20 launches each
            del runner, e2e_sets
            torch.cuda.empty_cache()
            out["per_layer"] = per_layer_summary(layer_rows(peaks, peak_kind, iters=20, with_packed=False))
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = time_cpu_oracle(layer)
        print(json.dumps(out))
    if args.report and rank == 0:
        write_report(args.report, peaks, peak_kind,
                     names=args.report_layers.split(",") if args.report_layers else None)
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------------- per-layer report ----
def time_call(fn, iters, flush):
    """Average, best and median device time (ms) of fn over `iters` launches, each preceded by an
    L2 flush (the paper reports the best of 50 runs; the average is what the rooflines use)."""
    total = 0.0
    best = float("inf")
    samples = []
    for _ in range(2):                 # untimed: the call's own first-use costs stay out of the average
        fn()
    torch.cuda.synchronize()
    for _ in range(iters):
        flush.zero_()
        # keep the GPU busy (~0.3 ms) while the host queues the events and the call, so that the
        # bracket measures device time, not launch latency
        torch.cuda._sleep(600_000)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        e1.synchronize()
        ms = e0.elapsed_time(e1)
        total += ms
        best = min(best, ms)
        samples.append(ms)
    samples.sort()
    return total / iters, best, samples[len(samples) // 2]


def time_back_to_back(fn, sets, launches):
    """Device time per launch (ms) of `launches` calls fn(i) queued back to back between one pair of
    events, call j on buffer set j % sets.  The sets together exceed the L2 several times (or one
    call's own buffers do), so no call finds its inputs cached; unlike time_call the figure leaves out
    the fixed cost of an isolated launch (event bracket, idle-GPU start, nothing queued behind it)."""
    for i in range(sets):
        fn(i)
    torch.cuda.synchronize()
    torch.cuda._sleep(600_000)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for j in range(launches):
        fn(j % sets)
    e1.record()
    e1.synchronize()
    return e0.elapsed_time(e1) / launches


L2_BYTES = 126 << 20


def buffer_sets_for(layer):
    """Buffer sets for back-to-back timing: one when a single call already moves two L2 sizes, else
    enough (at most 12) that the sets a call does not touch hold three L2 sizes."""
    from paper_2608_20725_b200 import binding
    _, _, ho, wo = binding.im2win_workspace_size(layer.dims(), binding.F32 if "f32" in layer.precisions else binding.F16)
    x_el = layer.N * layer.C * layer.H * layer.W
    win_el = layer.N * layer.C * ho * layer.Kh * (layer.W + 2 * layer.pad)
    out_el = layer.N * layer.Co * ho * wo
    smallest = min((x_el + win_el) * 2, win_el * 2 + out_el * 2)     # fewest bytes a timed call touches (fp16 sizes)
    if smallest >= 2 * L2_BYTES:
        return 1
    return max(2, min(12, 1 + -(-3 * L2_BYTES // smallest)))


def layer_rows(peaks, peak_kind, names=None, iters=20, with_packed=True):
    """Times every call of the named layers (default: all BASELINE configs) one by one: transform and
    convolution (filter pack included) per precision, L2 flushed before each launch; then the same
    calls queued back to back over rotating buffer sets."""
    from paper_2608_20725_b200 import binding
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # larger than the 126 MB L2
    rows = []
    table = dict(workloads.LAYERS)
    table.update(workloads.TABLE1_LAYERS)
    for name in (names or list(workloads.LAYERS)):
        layer = table[name]
        print(f"[report] {name}", file=sys.stderr, flush=True)
        sets = buffer_sets_for(layer)
        runner = LayerRunner(layer, layer.precisions, sets=sets)
        for _ in range(3):
            runner.step()
        torch.cuda.synchronize()
        avg, best, median, b2b = {}, {}, {}, {}
        for prec in layer.precisions:
            for kind, fn in (("transform", runner.transform), ("conv", runner.conv)):
                key = f"{kind}_{prec}"
                avg[key], best[key], median[key] = time_call(lambda: fn(prec), iters, flush)
                b2b[key] = time_back_to_back(lambda i: fn(prec, i), sets, iters)
            for d in runner.dev_sets[prec]:
                binding.im2win_check_status(d["scratch"])
        if "f16" in layer.precisions:
            # the channel-innermost (NHWC) form of the fp16 path on the same layer
            runner.add_nhwc()
            for _ in range(3):
                runner.transform_nhwc()
                runner.conv_nhwc()
            # conv_packed_*: the convolution on a filter packed beforehand (static weights), i.e. without
            # the pack kernel that conv_f16_nhwc runs on every call
            for key, fn in (("transform_f16_nhwc", runner.transform_nhwc),
                            ("transform_from_nhwc_f16_nhwc", runner.transform_nhwc_from_nhwc), ("conv_f16_nhwc", runner.conv_nhwc),
                            ("conv_packed_f16_nhwc", runner.conv_nhwc_packed),
                            ("conv_f16_out16_nhwc", runner.conv_nhwc_out16)):
                avg[key], best[key], median[key] = time_call(fn, iters, flush)
                b2b[key] = time_back_to_back(lambda i: fn(None, i), sets, iters)
            for d in runner.nhwc_sets:
                binding.im2win_check_status(d["scratch"])
        row = {"layer": name, "dims": layer.dims(), "gflop": runner.flops / 1e9, "avg_ms": avg, "best_ms": best,
               "median_ms": median, "back_to_back_ms": b2b, "buffer_sets": sets,
               "kernels": kernel_rooflines(runner, avg, peaks, peak_kind),
               "kernels_back_to_back": kernel_rooflines(runner, b2b, peaks, peak_kind),
               "conv_kernel": dict({p: binding.im2win_conv_kernel_name(layer.dims(), binding.F32 if p == "f32" else binding.F16)
                                    for p in layer.precisions},
                                   **({"f16_nhwc": binding.im2win_nhwc_kernel_name(layer.dims()),
                                       "f16_out16_nhwc": binding.im2win_nhwc_kernel_name(layer.dims(), runner.nhwc["epi16"])}
                                      if runner.nhwc is not None else {})),
               "memory": runner.memory_report()}
        if with_packed:
            # the convolution kernel without the filter pack (static weights), for reference
            packed = {}
            for prec in layer.precisions:
                a, b_, m = time_call(lambda: runner.conv_packed(prec), iters, flush)
                packed[f"conv_{prec}"] = {"avg_ms": a, "best_ms": b_, "median_ms": m}
            if runner.nhwc is not None:
                a, b_, m = time_call(runner.conv_nhwc_packed, iters, flush)
                packed["conv_f16_nhwc"] = {"avg_ms": a, "best_ms": b_, "median_ms": m,
                                           "back_to_back_ms": time_back_to_back(lambda i: runner.conv_nhwc_packed(None, i), sets, iters)}
            row["conv_without_pack"] = packed
        rows.append(row)
        del runner
        torch.cuda.empty_cache()
    return rows


def write_report(path, peaks, peak_kind, names=None, iters=20):
    rows = layer_rows(peaks, peak_kind, names, iters)
    os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
    with open(path, "w") as fh:
        for row in rows:
            fh.write(json.dumps(row) + "\n")


def per_layer_summary(rows):
    """The per-layer part of the bench line: for every BASELINE config and each of its calls the
    device time, the bounding roofline and the fraction reached, plus the memory figures."""
    out = {}
    for row in rows:
        entry = {}
        for key, k in row["kernels"].items():
            e = {"ms": round(k["ms"], 5), "bound": k["bound"], "frac": round(k["frac"], 4),
                 "achieved": round(k["achieved"], 2), "unit": k["unit"]}
            kb = row["kernels_back_to_back"][key]
            # the same call queued back to back over `buffer_sets` rotating buffer sets (no isolated-launch cost)
            e["back_to_back"] = {"ms": round(kb["ms"], 5), "bound": kb["bound"], "frac": round(kb["frac"], 4)}
            if key.startswith("conv"):
                e["tflops"] = round(row["gflop"] / k["ms"], 2)      # GFLOP per ms = TFLOP/s
                e["kernel"] = row["conv_kernel"]["f16_out16_nhwc" if key == "conv_f16_out16_nhwc" else "f16_nhwc"] \
                    if key.endswith("nhwc") else row["conv_kernel"][key.split("_")[1]]
                if "f16" in key:
                    e["frac_of_tensor_peak"] = round(k["frac_of_tensor_peak"], 4)
            entry[key] = e
        entry["buffer_sets"] = row["buffer_sets"]
        entry["memory"] = {p: {"window_bytes": m["window_bytes"], "output_bytes": m["output_bytes"],
                               "im2col_bytes": m["im2col_bytes"]} for p, m in row["memory"].items()}
        out[row["layer"]] = entry
    return out


def run_kernel_loop(spec, launches=3):
    """`LAYER:KERNEL[:BATCH]` -- a few launches of one kernel of one layer (for profilers)."""
    parts = spec.split(":")
    table = dict(workloads.LAYERS)
    table.update(workloads.TABLE1_LAYERS)
    layer = table[parts[0]]
    if len(parts) > 2:
        layer = layer.with_batch(int(parts[2]))
    if parts[1].endswith("_nhwc"):
        # the channel-innermost form: transform_f16_nhwc | conv_f16_nhwc
        runner = LayerRunner(layer, ("f16",))
        runner.add_nhwc()
        runner.transform_nhwc()
        fn = runner.transform_nhwc if parts[1].startswith("transform") else runner.conv_nhwc
        for _ in range(launches):
            fn()
        runner.b.im2win_check_status(runner.nhwc["scratch"])
        print(f"kernel-loop {spec}: {launches} launches done")
        return
    kind, prec = parts[1].rsplit("_", 1)
    runner = LayerRunner(layer, (prec,))
    runner.transform(prec)
    fn = runner.transform if kind == "transform" else runner.conv
    for _ in range(launches):
        fn(prec)
    runner.b.im2win_check_status(runner.dev[prec]["scratch"]) if kind == "conv" else torch.cuda.synchronize()
    print(f"kernel-loop {spec}: {launches} launches done")


# ------------------------------------------------------ the reference arm ----
def run_reference_arm(args):
    """Times the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    layer = workloads.LAYERS[workloads.BENCH_LAYER]
    x, f = workloads.make_inputs(layer)
    _, x16 = oracle.round_to_f16(x.numpy())
    _, f16 = oracle.round_to_f16(f.numpy())
    sets = {"f32": (x.numpy(), f.numpy()), "f16": (x16, f16)}
    dims = layer.dims()
    ho, wo = oracle.out_dims(dims)
    n_img = 16                                  # images per precision per step: a bounded sample of the batch
    flops_step = 2 * n_img * layer_flops(layer, ho, wo) / layer.N

    def step(i):
        for prec in ("f32", "f16"):
            xs, fs = sets[prec]
            b = (i * n_img) % (layer.N - n_img + 1)
            oracle.conv_im2win_range(xs, fs, dims, b, b + n_img)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(args.warmup + i)
    dt = time.perf_counter() - t0
    value = flops_step * args.steps / dt / 1e12
    sample = (f"fp64 im2win route (transform + convolution) on {n_img} of {layer.N} images of {layer.name} "
              f"per precision per step")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{layer.name}: N={layer.N} C={layer.C} H=W={layer.H} Co={layer.Co} "
                               f"K={layer.Kh}x{layer.Kw} stride={layer.stride} pad={layer.pad}, fp32 and fp16 passes",
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--report", default=None, help="also write a per-layer, per-kernel report (JSON lines)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-layer", action="store_true", help="skip the per-layer timings of the default run")
    ap.add_argument("--kernel-loop", default=None, metavar="LAYER:KERNEL[:BATCH]",
                    help="run a few launches of one kernel (e.g. cfg2:conv_f32) and exit; for profilers")
    ap.add_argument("--report-layers", default=None, help="comma-separated layer names for --report")
    args = ap.parse_args()
    if args.kernel_loop:
        run_kernel_loop(args.kernel_loop)
        return
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference_arm(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand with --gpus N: become N ranks (one per GPU) under torchrun
        import socket
        import subprocess
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    run_gpu_arm(args)


if __name__ == "__main__":
    main()
