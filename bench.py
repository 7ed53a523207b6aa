#!/usr/bin/env python
"""Benchmark of the fused-chain hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C2] [--impl reference]

A step is one fc_run of the workload's whole chain (producer -> epilogue -> reduction) over one
batch of seeded synthetic input.  The headline workload is C2 (the memory-bound chain the metric is
quoted on); `--workload C1|C3|C4|C5` selects another.  Rank 0 prints ONE JSON line.  With N > 1
(launched by torch.distributed.run) every rank runs its own batch (the chains' rows / images are
independent problems: weak scaling, no data-path collective); the time is the max over ranks.

`value` times fc_run with inputs resident in HBM (CUDA events on the launch stream): the timed region
of exactly `--steps` steps is taken five times and the median is reported (`ms_per_step_repeats`,
`ms_per_step_best` beside it).  `e2e` times fc_run_host with pinned HOST buffers, copies inside the
timed region.  `roofline` relates the kernel's algorithmic bytes or FLOPs per launch to the measured
peak of this machine's B200s (`frac`) and to the nominal peak the targets are stated against
(`frac_nominal`: 8 TB/s, 2250 TFLOP/s dense bf16).  `cpu_baseline` is the CPU oracle, as it stands, on a
bounded sample of the same workload.  `--impl reference` times that oracle as the reference arm.

`per_config` (rank 0 of a one-GPU run; `--no-per-config` leaves it out) holds one entry for each of the
five benchmark configurations C1..C5, each timed by the same protocol: fc_run enqueued back to back on one
stream, the number of calls per timed region chosen so that the region lasts at least 20 ms, five such
regions, median and best; configurations whose tensors fit in L2 (C1, C4, C5) are timed with an
L2-evicting write before every call (one event pair per call) and, beside it, back to back (`warm`).
Every entry has its own roofline fractions, its own clock sample over its own timed loop, the host cost
of an fc_run call, the unfused eager sequence on the same tensors, and the oracle's verdict on a sample
of its outputs.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from dataclasses import replace

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from fc_inputs import workloads as wl  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_BYTES = 126 * 1024 * 1024


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                p = json.load(f)
            return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured (MEASURED_PEAKS.json)"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback (earlier measurement on this pool)"


NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}   # what the targets are stated against (context for `frac`)
TARGET_FRAC_NOMINAL = {"hbm": 0.80, "tensor": 0.60}          # memory-bound chain >= 80 % of HBM peak, GEMM / conv >= 60 % of bf16 peak


def load_traffic_table():
    """DRAM bytes per launch (read, write) of each profiled workload's dominant kernel, from the table in
    profiles/dram_traffic.md, which the ncu summaries beside it are the sources of: a re-capture updates that
    one file.  Rows: | workload | kernel | dram read bytes | dram write bytes | summary file |"""
    table = {}
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    try:
        with open(path) as f:
            for line in f:
                cells = [c.strip() for c in line.strip().strip("|").split("|")]
                if len(cells) >= 4 and cells[2].isdigit() and cells[3].isdigit():
                    table[cells[0]] = int(cells[2]) + int(cells[3])
    except OSError:
        pass
    return table


_TRAFFIC = None


def load_traffic(workload: str, full_size: bool):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu capture of this workload's
    kernel (captures are of the full config sizes; None for a resized run or an unprofiled workload)."""
    global _TRAFFIC
    if _TRAFFIC is None:
        _TRAFFIC = load_traffic_table()
    return _TRAFFIC.get(workload) if full_size else None


# ------------------------------------------------------------------------------ units per workload
def units(ch):
    """(metric name, unit, algorithmic units per step, roofline bound)."""
    if ch.producer == "elementwise" or wl.collapses(ch):
        return "fused_chain_throughput", "GB/s", wl.algorithmic_bytes(ch) / 1e9, "hbm"
    return "fused_chain_throughput", "TFLOP/s", ch.flops() / 1e12, "tensor" if ch.in_dtype in ("bf16", "f16", "f8e4m3", "mxf8e4m3") else "alu"


def dtype_of(ch):
    return ch.in_dtype


# ------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) in a background thread."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.samples = []
        self._stop = threading.Event()
        self._period = period_s
        self._thread = None
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)
                reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                self.samples.append((time.perf_counter(), int(mhz), int(reasons)))
            except Exception:
                pass
            time.sleep(self._period)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self, t0: float, t1: float, note: str):
        if self._nv is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML not available"}
        nv = self._nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        sel = [s for s in self.samples if t0 <= s[0] <= t1]
        if not sel:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "note": note}
        bits = 0
        for s in sel:
            bits |= s[2]
        reasons = sorted(n for b, n in names.items() if bits & b)
        return {"sm_mhz": statistics.median(s[1] for s in sel), "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(sel), "note": note}


# ------------------------------------------------------------------------------ eager context
def eager_fn(ch, t):
    """The unfused PyTorch eager sequence of the chain (context only; never a parity reference)."""
    import torch
    import torch.nn.functional as F
    name = ch.name
    if name == "gemm_f32_bias_relu":
        return lambda: torch.relu(F.linear(t[0], t[1], t[2]))
    if name == "ew_affine_gelu_add_lse":
        def f():
            y = F.gelu(t[0] * t[1] + t[2], approximate="tanh") + t[3]
            return y, torch.logsumexp(y.float(), 1)
        return f
    if name == "ew_scale_add_softmax":
        scale = [o for o in ch.ops if o[0] == "scale"][0][1]
        return lambda: torch.softmax(t[0] * scale + t[1], dim=1)
    if name == "gemm_bf16_bias_gelu_scale_clamp":
        return lambda: torch.clamp(F.gelu(F.linear(t[0], t[1], t[2]), approximate="tanh") * 0.5, -1.0, 1.0)
    if name == "gemm_bf16_bias_scale_lse":
        return lambda: torch.logsumexp((F.linear(t[0], t[1], t[2]) * 0.5).float(), dim=1)
    if name.startswith("linear_bf16_row_"):
        red = {"row_sum": lambda y: y.float().sum(1), "row_mean": lambda y: y.float().mean(1), "row_max": lambda y: y.float().amax(1)}[ch.reduce]
        if ch.ops == (("bias_n", 2),):
            return lambda: red(F.linear(t[0], t[1], t[2]))
        return None
    if name == "gemm_f8e4m3_bias_gelu_scale_clamp":
        one = torch.ones((), device=t[0].device, dtype=torch.float32)
        def f():
            y = torch._scaled_mm(t[0], t[1].t(), scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
            return torch.clamp(F.gelu(y * (1.0 / ch.K ** 0.5) + t[2], approximate="tanh") * 0.5, -1.0, 1.0)
        try:
            f()
        except Exception:
            return None
        return f
    if name == "mlp_bf16":
        def f():
            h = F.linear(t[0], t[1], t[2])
            for l in range(1, len(ch.widths)):
                h = F.linear(torch.relu(h), t[1 + 2 * l], t[2 + 2 * l])
            return h
        return f
    if name == "gemm_bf16_row_softmax":
        return lambda: torch.softmax(t[0] @ t[1].t(), dim=1)
    if name == "conv_bf16_bias_relu_maxpool":
        x = t[0].permute(0, 3, 1, 2)
        w = t[1].permute(0, 3, 1, 2)
        return lambda: F.max_pool2d(torch.relu(F.conv2d(x, w, t[2], padding=ch.pad, stride=ch.stride)), 2).float()
    if name == "conv_bf16_bias_relu_avgpool_nchw":   # contiguous channel-first storage, as torch keeps it by default
        return lambda: F.adaptive_avg_pool2d(torch.relu(F.conv2d(t[0], t[1], t[2], padding=ch.pad)), 1).float()
    if name == "conv_bf16_bias_relu_avgpool":
        x = t[0].permute(0, 3, 1, 2)            # NHWC storage viewed as NCHW = channels_last
        w = t[1].permute(0, 3, 1, 2)
        return lambda: F.adaptive_avg_pool2d(torch.relu(F.conv2d(x, w, t[2], padding=ch.pad)), 1).float()
    return None


def network_entry(fc, binding, flush, with_eager, batch=4096):
    """The LeNet-shaped network (conv -> ReLU -> max-pool twice, three linear layers) as three chains per step (the
    pooled outputs stored in bf16, the next layer's operand type), every stage reading the previous stage's output in
    place; the unfused eager network on the same tensors beside it."""
    import torch
    import torch.nn.functional as F
    stages = wl.lenet_shaped(batch)
    runs, tensors, prev = [], [], None
    for k, ch in enumerate(stages):
        ins = [fc.to_device(a) for a in wl.make_inputs(ch, k)]
        if prev is not None:
            ins[0] = prev.reshape(ch.input_recipe[0][2])
        outs = binding.output_tensors(ch, "cuda")
        spec = fc.make_spec(ch)
        binding.ensure_workspace(spec)
        runs.append((spec, ins, outs))
        tensors.append(ins)
        prev = outs[0]
    prepared = [fc.PreparedRun(sp, i, o) for sp, i, o in runs]   # after the last ensure_workspace: the workspace is final

    def step():
        for pr in prepared:
            pr.run()
    ms = time_loop(step, 20, 3, flush)
    flops = sum(ch.flops() for ch in stages)
    ent = {"ms": ms, "value": flops / (ms * 1e-3) / 1e12, "unit": "TFLOP/s", "bound": "tensor", "chains_per_step": len(stages),
           "workload": f"LeNet-shaped network, batch {batch}: conv5x5 8->64 + ReLU + pool, conv5x5 64->128 + ReLU + pool, 3200->120->88->10"}
    if with_eager:
        c1, c2, fcs = tensors[0], tensors[1], tensors[2]
        x = c1[0].permute(0, 3, 1, 2)
        w1, w2 = c1[1].permute(0, 3, 1, 2), c2[1].permute(0, 3, 1, 2)

        def eager():
            h = F.max_pool2d(torch.relu(F.conv2d(x, w1, c1[2])), 2)
            h = F.max_pool2d(torch.relu(F.conv2d(h, w2, c2[2])), 2)
            h = h.permute(0, 2, 3, 1).reshape(batch, -1)
            h = torch.relu(F.linear(h, fcs[1], fcs[2]))
            h = torch.relu(F.linear(h, fcs[3], fcs[4]))
            return F.linear(h, fcs[5], fcs[6])
        ent["eager_ms"] = time_loop(eager, 10, 3, flush)
    return ent


def time_loop(fn, steps, warmup, flush=None):
    """CUDA-event timing on the current stream.  Without `flush`: one event pair around `steps`
    back-to-back calls.  With `flush`: an L2-evicting write before every call, one pair per call."""
    import torch
    for _ in range(warmup):
        if flush is not None:
            flush()
        fn()
    torch.cuda.synchronize()
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps
    total = 0.0
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        flush()
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    for a, b in evs:
        total += a.elapsed_time(b)
    return total / steps


# ------------------------------------------------------------------------------ CPU oracle legs
def oracle_sample(ch, ins, target_s=15.0):
    """A bounded sample of the workload for the CPU oracle: leading rows (or images) sized so that the
    oracle runs for roughly `target_s` seconds.  Returns (sub-chain, sub-inputs, description)."""
    import oracle
    threads = oracle.num_threads()
    # rough oracle speed on these host cores: ~0.5 GFLOP/s/thread for the naive contraction,
    # ~15 M elements/s/thread for the transcendental elementwise chain
    if ch.producer == "elementwise":
        rows = int(min(ch.M, max(1, target_s * 15e6 * threads / ch.N)))
        sub = replace(ch, M=rows)
        sub_ins = [a[:rows] if a.ndim == 2 else a for a in ins]
        return sub, sub_ins, f"first {rows} of {ch.M} rows"
    if ch.producer == "gemm_nt":
        rows = int(min(ch.M, max(1, target_s * 0.5e9 * threads / (2.0 * ch.N * ch.K))))
        sub = replace(ch, M=rows)
        sub_ins = [ins[0][:rows]] + list(ins[1:])
        return sub, sub_ins, f"first {rows} of {ch.M} rows of A (all of B)"
    per_img = 2.0 * ch.OH * ch.OW * ch.Cout * ch.R * ch.S * ch.Cin
    n = int(min(ch.batch, max(1, target_s * 0.5e9 * threads / per_img)))
    sub = replace(ch, batch=n)
    return sub, [ins[0][:n]] + list(ins[1:]), f"first {n} of {ch.batch} images"


def sample_units(sub):
    _, _, u, _ = units(sub)
    return u


def cpu_baseline_leg(ch, ins, gpu_outputs=None, target_s=15.0):
    """Times the oracle on the sample and (when GPU outputs are given) compares them on the sample."""
    import oracle
    oracle.build()
    sub, sub_ins, desc = oracle_sample(ch, ins, target_s)
    t0 = time.perf_counter()
    ref = oracle.run_chain(sub, sub_ins)
    dt = time.perf_counter() - t0
    _, unit, _, _ = units(ch)
    out = {"value": sample_units(sub) / dt, "unit": unit, "cores": oracle.num_threads(), "kind": "oracle",
           "sample": desc, "seconds": round(dt, 3)}
    if gpu_outputs is not None:
        from tests import util
        names = [r for r, _, _ in wl.output_shapes(ch)]
        n = sub.batch if ch.is_conv else sub.M
        worst = {}
        for name, t in zip(names, gpu_outputs):
            got = util.to_f64(t[:n])
            r = ref[name]
            worst[name] = float(np.abs(got - r).max())
            if any(op[0] == "linear" for op in ch.ops):
                util.check_chained(t[:n], r, util.flip_allowance(oracle, sub, sub_ins), f"bench {ch.name}:{name}")
            else:
                util.check(t[:n], r, f"bench {ch.name}:{name}")
        out["parity_on_sample"] = {"ok": True, "max_abs_err": worst}
    return out


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    oracle.build()
    ch = wl.ALL[args.workload]()
    ins = wl.make_inputs(ch, 0)
    metric, unit, _, _ = units(ch)
    # each step is a bounded sample of the workload, sized so that the whole run ends within a few minutes
    sub, sub_ins, desc = oracle_sample(ch, ins, target_s=max(0.05, min(5.0, 120.0 / max(1, args.steps + 1))))
    for _ in range(min(args.warmup, 1)):
        oracle.run_chain(sub, sub_ins)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.run_chain(sub, sub_ins)
    dt = (time.perf_counter() - t0) / args.steps
    value = sample_units(sub) / dt
    line = {"impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{args.workload}: {ch.name}", "step": f"CPU oracle on a sample: {desc}"},
            "cpu_baseline": {"value": value, "unit": unit, "cores": oracle.num_threads(), "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------ timing protocol
MIN_REGION_MS = 20.0
REPEATS = 5


def roofline_of(ch, workload, units_per_step, bound, ms, peaks, peaks_src, full_size, long_region=False):
    """Roofline object of one launch: achieved units / s against the measured peak (`frac`) and against the nominal
    peak the targets are stated against (`frac_nominal`)."""
    frac_sustained = None
    if bound == "hbm":
        peak, peak_unit, nominal = peaks["hbm_gbs"], "GB/s", NOMINAL_PEAKS["hbm_gbs"]
        peak_note = f"HBM copy bandwidth, {peaks_src}"
    elif bound == "tensor":
        mult = 2.0 if ch.in_dtype in ("f8e4m3", "mxf8e4m3") else 1.0   # no fp8 measurement on this machine: the measured bf16 peak times the nominal fp8 : bf16 ratio
        peak = mult * (peaks["bf16_tflops_sustained"] if long_region else peaks["bf16_tflops"])
        peak_unit, nominal = "TFLOP/s", mult * NOMINAL_PEAKS["bf16_tflops"]
        peak_note = f"cuBLAS bf16 {'sustained' if long_region else 'burst'}, {peaks_src}" + (" x 2 (nominal fp8 : bf16 ratio)" if mult > 1 else "")
        frac_sustained = units_per_step / (ms * 1e-3) / (mult * peaks["bf16_tflops_sustained"])
    else:
        peak, peak_unit = 148 * 128 * 2 * 1.965e9 / 1e12, "TFLOP/s"
        nominal = peak
        peak_note = "fp32 FMA: 148 SMs x 128 lanes x 2 flop x 1.965 GHz (derived)"
    achieved = units_per_step / (ms * 1e-3)
    r = {"bound": bound, "achieved": achieved, "peak": peak, "unit": peak_unit, "frac": achieved / peak,
         "frac_measured": achieved / peak, "frac_nominal": achieved / nominal, "peak_nominal": nominal,
         "traffic": load_traffic(workload, full_size), "peak_source": peak_note,
         "algorithmic_units_per_launch": units_per_step, "kernel_ms": ms}
    if frac_sustained is not None:
        r["frac_of_sustained_peak"] = frac_sustained
    if bound in TARGET_FRAC_NOMINAL:
        r["target_frac_nominal"] = TARGET_FRAC_NOMINAL[bound]
        r["target_met"] = bool(r["frac_nominal"] >= TARGET_FRAC_NOMINAL[bound])
    return r


def timed_regions(step, flush, n, repeats, barrier=None, max_over_ranks=None):
    """`repeats` timed regions of `n` calls each, CUDA events on the current stream, a synchronize (and the ranks'
    barrier) on both sides of every region.  Without `flush`: one event pair around the n back-to-back calls.
    With `flush`: an L2-evicting write before every call and one event pair per call (the region's time is the
    sum).  Returns the per-call milliseconds of every region (max over ranks)."""
    import torch
    sync = barrier if barrier is not None else torch.cuda.synchronize
    out = []
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n if flush else 1)]
    for _ in range(repeats):
        sync()
        if flush is None:
            a, b = evs[0]
            a.record()
            for _ in range(n):
                step()
            b.record()
            sync()
            ms = a.elapsed_time(b)
        else:
            for a, b in evs:
                flush()
                a.record()
                step()
                b.record()
            sync()
            ms = sum(a.elapsed_time(b) for a, b in evs)
        if max_over_ranks is not None:
            ms = max_over_ranks(ms)
        out.append(ms / n)
    return out


def calls_for_region(step, flush, min_ms=MIN_REGION_MS):
    """Number of calls that make a timed region last at least `min_ms`, from a short trial."""
    import math
    trial = timed_regions(step, flush, 10, 1)[0]
    return max(10, int(math.ceil(min_ms / max(trial, 1e-4))))


def host_cost_us(step, kernel_ms, calls):
    """Host time of one fc_run call: the host clock around batches of un-synchronised calls (batches small enough
    that the launch queue never fills, the stream drained after each), divided by the number of calls."""
    import torch
    batch = 256
    total, done = 0.0, 0
    torch.cuda.synchronize()
    while done < calls:
        t0 = time.perf_counter()
        for _ in range(batch):
            step()
        total += time.perf_counter() - t0
        torch.cuda.synchronize()
        done += batch
    return total / done * 1e6, done


def host_floor_us(fc, calls=20000):
    """What a call costs before any work is done: a chain that validation rejects at once, through the same ctypes
    path (the rest of host_us_per_call is validation, planning and the CUDA launch calls themselves)."""
    import ctypes
    ch = wl.CONFIGS["C1"]()
    spec = fc.make_spec(ch)
    spec.version = 0                          # rejected before anything else is looked at
    fn, ref = fc.lib().fc_run, ctypes.byref(spec)
    t0 = time.perf_counter()
    for _ in range(calls):
        fn(ref, None, 0, None, 0, None)
    return (time.perf_counter() - t0) / calls * 1e6


def config_entry(fc, binding, key, ch, ins, sampler, flush_buf, peaks, peaks_src, with_eager, oracle_s):
    """One per_config entry: the timing protocol, roofline, clocks, host cost, eager context, oracle parity."""
    import torch
    metric, unit, units_per_step, bound = units(ch)
    dev_in = [fc.to_device(a) for a in ins]
    outs = binding.output_tensors(ch, "cuda")
    spec = fc.make_spec(ch)
    binding.ensure_workspace(spec)
    cold = wl.input_bytes(ch) <= L2_BYTES
    flush = (lambda: flush_buf.zero_()) if cold else None
    step = fc.PreparedRun(spec, dev_in, outs).run
    for _ in range(3):
        if flush:
            flush()
        step()
    torch.cuda.synchronize()
    n = calls_for_region(step, flush)
    t0 = time.perf_counter()
    reps = timed_regions(step, flush, n, REPEATS)
    t1 = time.perf_counter()
    fc.fc_get_async_status()
    ms, best = statistics.median(reps), min(reps)
    ent = {"workload": ch.name, "ms": ms, "ms_best": best, "ms_repeats": reps, "calls_per_region": n, "repeats": REPEATS,
           "region_ms": ms * n, "value": units_per_step / (ms * 1e-3), "value_best": units_per_step / (best * 1e-3), "unit": unit,
           "l2": "L2 flushed (252 MiB write) before every timed call, one event pair per call" if cold else "tensors larger than L2, calls back to back",
           "roofline": roofline_of(ch, key, units_per_step, bound, ms, peaks, peaks_src, True),
           "clocks": sampler.summary(t0, t1, "sampled during this config's timed regions")}
    if cold:
        nw = calls_for_region(step, None)
        warm = timed_regions(step, None, nw, REPEATS)
        ent["warm"] = {"ms": statistics.median(warm), "ms_best": min(warm), "calls_per_region": nw,
                       "note": "same calls back to back, tensors resident in L2"}
    us, calls = host_cost_us(step, ms, 10240 if ms < 0.05 else 2048)
    ent["host_us_per_call"] = us
    ent["host_calls"] = calls
    # re-poisoned outputs, one more call, checked against the oracle on a sample
    for t in outs:
        t.fill_(float("nan"))
    step()
    fc.fc_get_async_status()
    if with_eager:
        fn = eager_fn(ch, dev_in)
        if fn is not None:
            torch.backends.cuda.matmul.allow_tf32 = False
            torch.backends.cudnn.allow_tf32 = False
            for _ in range(3):
                if flush:
                    flush()
                fn()
            ne = calls_for_region(fn, flush)
            er = timed_regions(fn, flush, ne, 3)
            ent["eager_ms"] = statistics.median(er)
            ent["faster_than_eager"] = bool(ms < ent["eager_ms"])
    if oracle_s > 0:
        leg = cpu_baseline_leg(ch, ins, outs, target_s=oracle_s)
        ent["parity_on_sample"] = dict(leg["parity_on_sample"], sample=leg["sample"], oracle_seconds=leg["seconds"])
        ent["cpu_oracle"] = {"value": leg["value"], "unit": leg["unit"], "cores": leg["cores"]}
    r = ent["roofline"]
    ent["target_met"] = bool(r["target_met"] if "target_met" in r else ent.get("faster_than_eager", False))
    return ent


# ------------------------------------------------------------------------------ main arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="C2", choices=sorted(wl.ALL))
    ap.add_argument("--impl", default="fc", choices=["fc", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-eager", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="leave out the per_config entries of C1..C5 (profiler captures)")
    ap.add_argument("--single-region", action="store_true", help="time the --steps region once instead of five times (profiler captures)")
    ap.add_argument("--all-configs", action="store_true", help="also time the extra workloads F1.. and the network N1 (context)")
    ap.add_argument("--rows", type=int, default=0, help="override M (or the conv batch): a smaller case of the same kernel for profiler captures")
    args = ap.parse_args()
    if args.impl == "reference":
        return reference_arm(args)
    args.warmup = max(args.warmup, 3)

    import torch
    import paper_2602_14293_b200 as fc
    from paper_2602_14293_b200 import binding

    from paper_2602_14293_b200.ranks import Ranks
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    rk = Ranks("nccl")
    rank, world, local_rank = rk.rank, rk.world, rk.local_rank
    barrier, max_over_ranks = rk.barrier, rk.max_over_ranks

    peaks, peaks_src = load_peaks()
    ch = wl.ALL[args.workload]()
    if args.rows > 0:
        ch = wl.ALL[args.workload](batch=args.rows) if ch.is_conv else wl.ALL[args.workload](M=args.rows)
    metric, unit, units_per_step, bound = units(ch)
    ins = wl.make_inputs(ch, seed=rk.batch_seed(0))   # every rank draws its own batch
    dev_in = [fc.to_device(a) for a in ins]
    outs = binding.output_tensors(ch, "cuda")
    spec = fc.make_spec(ch)
    binding.ensure_workspace(spec)
    in_bytes = wl.input_bytes(ch)
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")
    flush = (lambda: flush_buf.zero_()) if in_bytes <= L2_BYTES else None

    prepared = fc.PreparedRun(spec, dev_in, outs)     # arguments marshalled once; a step is one fc_run C call
    step = prepared.run

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        if flush:
            flush()
        step()
    barrier()
    regions = 1 if args.single_region else REPEATS
    launches1 = fc.fc_launch_count()
    t_wall0 = time.perf_counter()
    reps = timed_regions(step, flush, args.steps, regions, barrier, max_over_ranks)   # each region: EXACTLY --steps steps
    t_wall1 = time.perf_counter()
    launches = (fc.fc_launch_count() - launches1) // regions
    fc.fc_get_async_status()
    ms_per_step = statistics.median(reps)
    value = rk.aggregate(units_per_step, ms_per_step)

    clocks = sampler.summary(t_wall0, t_wall1, "sampled during the timed regions")
    if clocks.get("samples", 0) < 3:
        # the timed regions were shorter than a few sampling periods: sample a longer loop of the same kernel
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < 0.4:
            for _ in range(20):
                step()
            torch.cuda.synchronize()
        clocks = sampler.summary(t0, time.perf_counter(), "timed regions too short to sample; taken over a 0.4 s loop of the same kernel right after them")

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed) ----
    host_in = [t.cpu().pin_memory() for t in dev_in]
    host_out = binding.output_tensors(ch, "cpu", pinned=True)
    staging = torch.empty(fc.fc_staging_size(spec, host_in, host_out), dtype=torch.uint8, device="cuda")
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(2):
        fc.fc_run_host(spec, host_in, host_out, staging)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        fc.fc_run_host(spec, host_in, host_out, staging)
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1) / e2e_steps)
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = sum(t.numel() * t.element_size() for t in host_out)
    e2e = {"value": rk.aggregate(units_per_step, e2e_ms), "unit": unit, "ms_per_step": e2e_ms, "steps": e2e_steps,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
    del host_in, host_out, staging

    # ---- roofline of the (single) kernel of this workload ----
    roofline = roofline_of(ch, args.workload, units_per_step, bound, ms_per_step, peaks, peaks_src, args.rows <= 0,
                           long_region=ms_per_step * args.steps > 1000.0)

    line = {"metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "ms_per_step_best": min(reps), "ms_per_step_repeats": reps, "timed_regions": regions,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": dtype_of(ch), "data": "synthetic",
            "config": {"workload": f"{args.workload}: {ch.name}", "shape": {k: getattr(ch, k) for k in ("M", "N", "K", "batch", "H", "W", "Cin", "Cout") if getattr(ch, k)},
                       "ops": [o[0] for o in ch.ops], "reduce": ch.reduce,
                       "l2": "inputs larger than L2, no flush" if flush is None else "L2 flushed (252 MiB write) before every timed step",
                       "timing": f"{regions} regions of exactly {args.steps} steps each, median reported",
                       "parallelism": f"independent batches per GPU x{world}"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline}

    if rank == 0 and not args.no_eager:
        fn = eager_fn(ch, dev_in)
        if fn is not None:
            torch.backends.cuda.matmul.allow_tf32 = False
            torch.backends.cudnn.allow_tf32 = False
            ems = time_loop(fn, max(5, min(args.steps, 50)), 3, flush)
            line["eager"] = {"ms_per_step": ems, "value": units_per_step / (ems * 1e-3), "unit": unit,
                             "note": "unfused PyTorch eager sequence on the same GPU and tensors (context)"}

    per = {}
    if rank == 0 and world == 1 and not args.no_per_config:
        # the five benchmark configurations, each by the same protocol (see the module docstring)
        for key in sorted(wl.CONFIGS):
            c2 = wl.CONFIGS[key]()
            i2 = ins if (key == args.workload and args.rows <= 0) else wl.make_inputs(c2, 0)
            per[key] = config_entry(fc, binding, key, c2, i2, sampler, flush_buf, peaks, peaks_src, not args.no_eager,
                                    0.0 if args.no_cpu_baseline else 3.0)
            del i2
            torch.cuda.empty_cache()
        line["host_floor_us_per_call"] = host_floor_us(fc)
        line["targets"] = {"statement": "memory-bound chain >= 80 % of nominal HBM peak (8 TB/s); GEMM / conv chains >= 60 % of nominal dense "
                                        "bf16 peak (2250 TFLOP/s); every config within the oracle's tolerances and faster than eager",
                           "met": {k: v["target_met"] for k, v in per.items()},
                           "faster_than_eager": {k: v.get("faster_than_eager") for k, v in per.items()},
                           "parity": {k: v.get("parity_on_sample", {}).get("ok") for k, v in per.items()}}

    if rank == 0 and args.all_configs:
        for key in sorted(wl.ALL):
            if key == args.workload or key in per:
                continue
            c2 = wl.ALL[key]()
            i2 = [fc.to_device(a) for a in wl.make_inputs(c2, 0)]
            o2 = binding.output_tensors(c2, "cuda")
            s2 = fc.make_spec(c2)
            binding.ensure_workspace(s2)
            fl = (lambda: flush_buf.zero_()) if wl.input_bytes(c2) <= L2_BYTES else None
            ms = time_loop(fc.PreparedRun(s2, i2, o2).run, 50, 5, fl)
            _, u2, n2, b2 = units(c2)
            ent = {"ms": ms, "value": n2 / (ms * 1e-3), "unit": u2, "bound": b2}
            if b2 == "tensor":
                ent["frac_of_burst_peak"] = ent["value"] / peaks["bf16_tflops"]
            elif "gemm_tc_mode7" in fc.fc_last_plan():
                # an fp32 GEMM that ran as three tf32 products per product on the tensor cores (tf32: half the bf16 rate)
                ent["bound"] = "tensor (3 x tf32 per fp32 product; operand split kernels included in the time)"
                ent["tensor_tflops_executed"] = 3.0 * ent["value"]
                ent["frac_of_burst_peak_tf32"] = 3.0 * ent["value"] / (0.5 * peaks["bf16_tflops"])
            f2 = eager_fn(c2, i2)
            if f2 is not None and not args.no_eager:
                ent["eager_ms"] = time_loop(f2, 20, 3, fl)
            per[key] = ent
            del i2, o2
        per["N1"] = network_entry(fc, binding, lambda: flush_buf.zero_(), not args.no_eager)
    if per:
        line["per_config"] = per

    sampler.stop()
    if rank == 0 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline_leg(ch, ins, outs)
    if rank == 0:
        print(json.dumps(line))
    rk.finish()
    return 0


if __name__ == "__main__":
    sys.exit(main())
