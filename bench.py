#!/usr/bin/env python
"""Benchmark of the recurrence-matmul hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

Workloads c1..c5 are the matrix-multiply recurrence.  With no --workload the largest configuration that fits one GPU
(c3) is the headline and the line carries a `configs` object with the same record for c1, c2, c4 and c5 (each timed over
at least a quarter of a second of back-to-back steps) and `sustained` sub-records (at least one second) for c2 and c3.
t1 and t2 are the block lower-triangular solve built on the recurrence; a1 and a2 are the FlashAttention-2 recurrence; p1..p3 the prefix-sum recurrence; h1 and h2 the tiled Cholesky recurrence.

One step = one evaluation of the whole recurrence (weight load, B injection, the
multiply-accumulate chain along k, export of C) for one workload.  Prints ONE JSON
line.  `value` is throughput with operands resident in HBM; `e2e` is the same metric
through the host-buffer entry point, host<->device copies inside the timed region.
With --gpus N > 1 (under torchrun) every rank runs an independent replica on its own
GPU ("replicas only": the path has no exchange step) and the values add up.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
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
sys.path.insert(0, ROOT)

from paper_2511_09987_b200 import inputs  # noqa: E402

# nominal dense tensor ratios relative to bf16 (2.25 PFLOP/s): int8 4.5 POPS, tf32 1.1 PFLOP/s
NOMINAL_RATIO = {"bf16": 1.0, "i8": 2.0, "tf32": 0.5}
# datasheet dense peaks (TFLOP/s or TOPS), reported beside the measured ones as `frac_nominal`
NOMINAL_PEAK = {"bf16": 2250.0, "i8": 4500.0, "tf32": 1100.0}
NOMINAL_HBM_GBS = 7700.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_BYTES = 126 * 1024 * 1024
# FP32 FMA roof: 148 SMs x 128 lanes x 2 flop x max SM clock
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def unit_of(w):
    return "TOPS" if w.dtype == "i8" else "TFLOPS"


def tensor_kind(w):
    return "tf32" if w.dtype == "f32" else w.dtype


def bound_of(w, family, peaks):
    """Which roof bounds the dominant kernel of this workload: the ridge is the measured tensor rate of the dtype
    (bf16 cuBLAS burst x the nominal ratio of the dtype) over the measured copy bandwidth."""
    if family == "simt":
        return "alu"
    ai = 2.0 * w.macs / w.algorithmic_bytes
    ridge = float(peaks["bf16_tflops"]) * NOMINAL_RATIO[tensor_kind(w)] * 1e12 / (float(peaks["hbm_gbs"]) * 1e9)
    return "tensor" if ai > ridge else "hbm"


def tensor_roofline(achieved, kind, peaks, peak_kind):
    """Fractions of one tensor-bound figure: against the measured burst peak (`frac`, the denominator never depends on
    how long the timed region was), the measured sustained peak and the datasheet dense peak of the dtype."""
    burst = float(peaks["bf16_tflops"]) * NOMINAL_RATIO[kind]
    sustained = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])) * NOMINAL_RATIO[kind]
    return {"peak": burst, "frac": achieved / burst, "frac_measured": achieved / burst,
            "frac_measured_sustained": achieved / sustained, "peak_sustained": sustained,
            "frac_nominal": achieved / NOMINAL_PEAK[kind], "peak_nominal": NOMINAL_PEAK[kind],
            "peak_source": "%s bf16 cuBLAS burst x nominal %s/bf16 ratio %.1f (of %s); frac_measured_sustained uses the "
                           "seconds-long cuBLAS loop, frac_nominal the datasheet dense peak" % (peak_kind, kind, NOMINAL_RATIO[kind], peak_kind)}


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period: float = 0.004):
        self.samples, self.reasons, self.max_mhz, self.period = [], set(), None, period
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if visible:
                try:
                    phys = int(visible.split(",")[index])
                except ValueError:
                    phys = index
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def cpu_oracle_rate(w, target_seconds=12.0, threads=None):
    """Time the oracle (collapsed walker, as it stands) on a bounded sample of workload `w`.

    The sample is a prefix of rows of C (problems, for a batched workload; repeats of the whole workload when it
    is tiny), grown until the walk takes about `target_seconds`."""
    import oracle
    threads = threads or os.cpu_count() or 1
    one = inputs.scaled(w, batch=1)
    if w.batch > 1:
        A, B = inputs.make_operands(inputs.scaled(w, batch=min(w.batch, 64)))
    else:
        A, B = inputs.make_operands(one)

    def walk(units):
        t0 = time.perf_counter()
        if w.batch > 1:
            for b in range(units):
                oracle.collapsed(one.dtype, A[b % len(A)], B[b % len(B)], b_col_major=one.b_col_major, threads=threads)
        elif units <= one.M:
            oracle.collapsed(one.dtype, A, B, b_col_major=one.b_col_major, rows=np.arange(units), threads=threads)
        else:
            for _ in range(units // one.M):
                oracle.collapsed(one.dtype, A, B, b_col_major=one.b_col_major, threads=threads)
        return time.perf_counter() - t0

    units = 1 if w.batch > 1 else min(one.M, 2 * threads)
    limit = w.batch if w.batch > 1 else (one.M if one.macs > 1e8 else one.M * 100000)
    while True:
        dt = walk(units)
        if dt >= 0.5 * target_seconds or units >= limit:
            break
        grow = min(8.0, max(2.0, 0.9 * target_seconds / max(dt, 1e-3)))
        units = int(min(limit, units * grow))
        if w.batch == 1 and units > one.M:
            units = (units // one.M) * one.M
    if w.batch > 1:
        ops, what = 2.0 * units * one.macs, "problems 0..%d" % (units - 1)
    elif units <= one.M:
        ops, what = 2.0 * units * one.N * one.K, "rows 0..%d" % (units - 1)
    else:
        ops, what = 2.0 * (units // one.M) * one.macs, "%d repeats of the whole workload" % (units // one.M)
    sample = "%s of %s (M=%d N=%d K=%d), collapsed walker, %d threads, %.1f s" % (what, w.name, one.M, one.N, one.K, threads, dt)
    return ops / dt / 1e12, threads, sample, dt


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = os.cpu_count() or 1
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    vals, sample = [], ""
    for s in range(args.warmup + args.steps):
        v, threads, sample, _ = cpu_oracle_rate(w, target_seconds=per_step, threads=threads)
        if s >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    ops = 2.0 * w.macs
    line = {
        "impl": "reference", "metric": "recurrence_matmul_throughput", "value": value, "unit": unit_of(w), "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ops / (value * 1e12) * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": {"f32": "f32", "bf16": "bf16", "i8": "i8"}[w.dtype],
        "data": "synthetic", "config": {"workload": describe(w), "note": "ms_per_step extrapolated from the sampled rate"},
        "cpu_baseline": {"value": value, "unit": unit_of(w), "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": unit_of(w), "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def describe(w):
    s = "%s: %s M=%d N=%d K=%d seed=%d" % (w.name, w.dtype, w.M, w.N, w.K, w.seed)
    if w.batch > 1:
        s += " batch=%d" % w.batch
    if w.b_col_major:
        s += " B column-major"
    if w.fixed_k_order:
        s += " fixed-k-order"
    return s


def cuda_setup():
    import torch
    from paper_2511_09987_b200.replicas import Replicas
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    reps = Replicas("nccl", torch.device("cuda", local))
    return torch, reps, local


def measure_matmul(w, steps, args, torch, reps, local, *, min_seconds=0.0, sustained_seconds=0.0, cpu_seconds=12.0,
                   with_cpu=True, with_e2e=True):
    """One record for the matrix-multiply recurrence on workload `w`.

    The timed region is `steps` back-to-back steps (one library call each); when `min_seconds` is given and `steps` is
    None, the number of steps is chosen from a short calibration so that the region lasts at least that long.  Clocks
    are sampled by NVML inside the region.  `sustained_seconds` adds a second, longer region of its own."""
    from paper_2511_09987_b200 import binding
    world = reps.world
    peaks, peak_kind = load_peaks()

    # ---- operands: generated once on the host, uploaded; several device copies rotate so that a set has left L2
    # ---- before it is used again
    A, B = inputs.make_operands(w)
    hA = torch.from_numpy(A)
    hB = torch.from_numpy(B)
    if w.dtype == "bf16":
        hA, hB = hA.view(torch.bfloat16), hB.view(torch.bfloat16)
    hA, hB = hA.pin_memory(), hB.pin_memory()
    out_dt = torch.int32 if w.dtype == "i8" else torch.float32
    cshape = (w.batch, w.M, w.N) if w.batch > 1 else (w.M, w.N)
    set_bytes = w.algorithmic_bytes
    nsets = int(min(8, max(2, -(-3 * L2_BYTES // set_bytes))))
    sets = [(hA.cuda(), hB.cuda(), torch.empty(cshape, dtype=out_dt, device="cuda")) for _ in range(nsets)]
    stream = torch.cuda.current_stream()
    ops_step = 2.0 * w.macs

    def step(i):
        dA, dB, dC = sets[i % nsets]
        if w.batch > 1:
            binding.recurrence_matmul_batched(dA, dB, dC, b_col_major=w.b_col_major, fixed_k_order=w.fixed_k_order)
        else:
            binding.recurrence_matmul(dA, dB, dC, b_col_major=w.b_col_major, fixed_k_order=w.fixed_k_order)

    family = binding.kernel_for(w.batch, w.M, w.N, w.K, w.dtype, sets[0][0].data_ptr(), sets[0][1].data_ptr(),
                                sets[0][2].data_ptr(), b_col_major=w.b_col_major, fixed_k_order=w.fixed_k_order)

    def barrier():
        reps.barrier()
        torch.cuda.synchronize()

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def region(n, replay=None):
        """n steps between two events on the launching stream, a barrier and a synchronize on both sides."""
        barrier()
        e0.record(stream)
        if replay is not None:
            for _ in range(n // replay[1]):
                replay[0].replay()
        else:
            for i in range(n):
                step(i)
        e1.record(stream)
        barrier()
        return e0.elapsed_time(e1)

    for i in range(max(3, args.warmup)):
        step(i)
    barrier()
    if steps is None:  # calibrate: as many steps as fill `min_seconds`
        est = region(20) / 20.0
        steps = int(max(20, min(200000, -(-min_seconds * 1e3 // max(est, 1e-4)))))
    # launch-bound workloads (a few microseconds per kernel): replay the steps from a CUDA graph so that the
    # device, not the Python launch path, is what is timed.  The graph holds `chunk` launches; K steps = K/chunk replays.
    graph, chunk, plain_call_us = None, 1, None
    if args.graph == "on" or (args.graph == "auto" and ops_step < 5e7):
        plain_call_us = region(min(steps, 2000)) / min(steps, 2000) * 1e3   # the same steps as plain library calls
        chunk = max(1, min(100, steps))
        while steps % chunk:
            chunk -= 1
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step(0)                                    # first call on this stream outside the capture
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for i in range(chunk):
                    step(i)
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = binding.cyc_launch_count()
    ms = region(steps, (graph, chunk) if graph is not None else None)
    launches = steps if graph is not None else binding.cyc_launch_count() - launches0
    if binding.last_device_status() != binding.CYC_OK:
        raise SystemExit("a device-side wait timed out during the benchmark: " + binding.cyc_last_cuda_error().decode())
    # keep the GPU loaded a little longer if the timed region was too short to catch a clock sample
    extra_note = None
    if len(sampler.samples) < 3:
        t_end = time.time() + 0.3
        i = 0
        while time.time() < t_end:
            step(i)
            i += 1
            if i % 64 == 0:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        extra_note = "timed region shorter than three sampling periods; clocks sampled under the same load right after it"
    clocks = sampler.stop()
    if extra_note:
        clocks["note"] = extra_note

    ms = reps.max_over_ranks(ms)
    ms_per_step = ms / steps
    value = world * ops_step / (ms_per_step * 1e-3) / 1e12

    # ---- a second, seconds-long region: what the kernel sustains under the power cap
    sustained = None
    if sustained_seconds > 0:
        n = int(max(steps, -(-sustained_seconds * 1e3 // ms_per_step)))
        s2 = ClockSampler(local)
        s2.start()
        ms2 = reps.max_over_ranks(region(n))
        c2 = s2.stop()
        v2 = ops_step / (ms2 / n * 1e-3) / 1e12
        sustained = {"value": world * v2, "unit": unit_of(w), "steps": n, "seconds": ms2 * 1e-3, "ms_per_step": ms2 / n, "clocks": c2}

    # ---- end to end through the host entry point (pinned buffers, copies inside the timed region)
    e2e = None
    if with_e2e:
        hC = torch.empty(cshape, dtype=out_dt).pin_memory()
        e2e_steps = max(3, min(steps, 20))
        for _ in range(2):
            binding.recurrence_matmul_host(hA, hB, hC, b_col_major=w.b_col_major, fixed_k_order=w.fixed_k_order)
        barrier()
        t0 = time.perf_counter()
        e0.record(stream)
        for _ in range(e2e_steps):
            binding.recurrence_matmul_host(hA, hB, hC, b_col_major=w.b_col_major, fixed_k_order=w.fixed_k_order)
        e1.record(stream)
        barrier()
        e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / e2e_steps
        e2e = {"value": world * ops_step / (reps.max_over_ranks(e2e_ms) * 1e-3) / 1e12, "unit": unit_of(w),
               "h2d_bytes_per_step": int(hA.numel() * hA.element_size() + hB.numel() * hB.element_size()),
               "d2h_bytes_per_step": int(hC.numel() * hC.element_size()), "steps": e2e_steps, "ms_per_step": e2e_ms}
        del hC
    else:
        e2e = {"value": None, "unit": unit_of(w), "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0, "steps": 0}
    del sets, graph
    torch.cuda.empty_cache()

    # ---- roofline of the dominant (only) kernel: one launch per step
    kernel_s = ms_per_step * 1e-3
    bound = bound_of(w, family, peaks)
    traffic = load_traffic(w, family)
    if bound == "hbm":
        achieved, runit = w.algorithmic_bytes / kernel_s / 1e9, "GB/s"
        peak = float(peaks["hbm_gbs"])
        fr = {"peak": peak, "frac": achieved / peak, "frac_measured": achieved / peak, "frac_nominal": achieved / NOMINAL_HBM_GBS,
              "peak_nominal": NOMINAL_HBM_GBS, "peak_source": "%s STREAM-style copy (of %s); frac_nominal against 7.7 TB/s" % (peak_kind, peak_kind)}
    elif bound == "tensor":
        achieved, runit = ops_step / kernel_s / 1e12, ("TOPS" if w.dtype == "i8" else "TFLOP/s")
        fr = tensor_roofline(achieved, tensor_kind(w), peaks, peak_kind)
        if sustained is not None:
            sustained["frac_measured_sustained"] = sustained["value"] / world / fr["peak_sustained"]
            sustained["frac_nominal"] = sustained["value"] / world / fr["peak_nominal"]
    else:
        achieved, runit = ops_step / kernel_s / 1e12, "TFLOP/s"
        fr = {"peak": FP32_ALU_TFLOPS, "frac": achieved / FP32_ALU_TFLOPS, "frac_nominal": achieved / FP32_ALU_TFLOPS,
              "peak_source": "FP32 FMA roof: 148 SMs x 128 lanes x 2 x 1.965 GHz (derived, not measured)"}
    roofline = {"bound": bound, "achieved": achieved, "unit": runit, "traffic": traffic, "kernel": family, "kernel_us": kernel_s * 1e6}
    roofline.update(fr)
    if clocks.get("sm_mhz"):
        roofline["kernel_us_x_sm_mhz"] = kernel_s * 1e6 * clocks["sm_mhz"]   # clock-independent duration: microseconds x MHz = cycles

    if with_cpu and reps.rank == 0 and world == 1:
        cpu_v, cores, sample, _ = cpu_oracle_rate(w, target_seconds=cpu_seconds)
    else:
        cpu_v, cores, sample = None, 0, "skipped"
    if nsets * set_bytes > 2 * L2_BYTES:
        l2_note = "inputs rotate over %d device copies (%.0f MB in total, larger than the 126 MB L2)" % (nsets, nsets * set_bytes / 1e6)
    else:
        l2_note = ("working set of %d rotating copies is %.1f MB, far below L2: this workload is launch/latency-bound, "
                   "no DRAM figure is claimed for it" % (nsets, nsets * set_bytes / 1e6))
    rec = {
        "value": value, "unit": unit_of(w), "steps": steps, "ms_per_step": ms_per_step, "seconds": ms * 1e-3, "dtype": w.dtype,
        "config": {"workload": describe(w), "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": l2_note, "kernel": family,
                   "launch": ("CUDA graph of %d launches, replayed %d times" % (chunk, steps // chunk)) if chunk > 1 or args.graph == "on"
                   else "one library call per step"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
        "cpu_baseline": {"value": cpu_v, "unit": unit_of(w), "cores": cores, "kind": "oracle", "sample": sample},
    }
    if plain_call_us is not None:
        rec["plain_call_us"] = plain_call_us   # the same step as an ordinary library call from Python, no graph
    if sustained is not None:
        rec["sustained"] = sustained
    return rec


def run_ours(args, w, with_configs):
    """The headline workload timed over exactly --steps steps; with `with_configs` (the default run) the other
    configurations of the matrix-multiply recurrence follow as sub-records, each over a region of at least 0.25 s."""
    torch, reps, local = cuda_setup()
    kernel_only = args.kernel_only
    base = w.name.split("@")[0].split("+")[0]
    sustained = 1.0 if (with_configs or args.sustained) and base in ("c2", "c3") else 0.0
    head = measure_matmul(w, args.steps, args, torch, reps, local, sustained_seconds=sustained,
                          with_cpu=not kernel_only, with_e2e=not kernel_only)
    line = {"metric": "recurrence_matmul_throughput", "value": head["value"], "unit": head["unit"], "n_gpus": reps.world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic"}
    for k in ("config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline", "sustained", "plain_call_us"):
        if k in head:
            line[k] = head[k]
    if with_configs and reps.world == 1:
        subs = {}
        for name in ("c1", "c2", "c4", "c5"):
            if name == base:
                continue
            cw = inputs.WORKLOADS[name]
            subs[name] = measure_matmul(cw, None, args, torch, reps, local, min_seconds=0.25,
                                        sustained_seconds=1.0 if name == "c2" else 0.0, cpu_seconds=5.0)
        line["configs"] = subs
    if reps.rank == 0:
        print(json.dumps(line))
    reps.close()


def run_trsm(args, w):
    """Block lower-triangular solve L X = B (workloads t1, t2): one step = one whole solve (every tile product of the
    triangular space and every diagonal solve)."""
    import torch
    from paper_2511_09987_b200 import binding
    from paper_2511_09987_b200.replicas import Replicas

    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    reps = Replicas("nccl", torch.device("cuda", local))
    world, rank = reps.world, reps.rank
    peaks, peak_kind = load_peaks()
    L, B = inputs.make_trsm_operands(w)
    hL, hB = torch.from_numpy(L).pin_memory(), torch.from_numpy(B).pin_memory()
    hX = torch.empty_like(hB).pin_memory()
    dL, dB = hL.cuda(), hB.cuda()
    dX = torch.empty_like(dB)
    stream = torch.cuda.current_stream()

    def barrier():
        reps.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        binding.block_trsm(dL, dB, dX, tile=w.tile)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = binding.cyc_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        binding.block_trsm(dL, dB, dX, tile=w.tile)
    e1.record(stream)
    barrier()
    launches = binding.cyc_launch_count() - launches0
    if binding.last_device_status() != binding.CYC_OK:
        raise SystemExit("a device-side wait timed out during the benchmark: " + binding.cyc_last_cuda_error().decode())
    clocks = sampler.stop()
    ms_per_step = reps.max_over_ranks(e0.elapsed_time(e1)) / args.steps
    value = world * w.flops / (ms_per_step * 1e-3) / 1e12

    # end to end: pinned host L and B up, solve, X down, every step
    e2e_steps = 0 if args.kernel_only else max(3, min(args.steps, 10))

    def e2e_step():
        dL.copy_(hL, non_blocking=True)
        dB.copy_(hB, non_blocking=True)
        binding.block_trsm(dL, dB, dX, tile=w.tile)
        hX.copy_(dX, non_blocking=True)

    for _ in range(0 if args.kernel_only else 2):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / max(1, e2e_steps)
    e2e_value = None if args.kernel_only else world * w.flops / (reps.max_over_ranks(e2e_ms) * 1e-3) / 1e12
    if rank != 0:
        reps.close()
        return
    step_s = ms_per_step * 1e-3
    roofline = {"bound": "tensor", "achieved": value / world, "unit": "TFLOP/s", "traffic": None,
                "note": "the whole step is rated (n(n+1)m flop, the three TF32 products of each fp32 product counted once): "
                        "%d launches per solve" % (launches // max(1, args.steps)),
                "kernel": "tcgen05_3xtf32 (tile products) + trsm_diag (diagonal tiles)", "kernel_us": step_s * 1e6}
    roofline.update(tensor_roofline(value / world, "tf32", peaks, peak_kind))
    if args.kernel_only:
        cpu_v, cores, sample = None, 0, "skipped (--kernel-only)"
    else:
        cpu_v, cores, sample = cpu_trsm_rate(w, L, B)
    line = {
        "metric": "block_trsm_throughput", "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": describe_trsm(w), "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": "L, B, X and the partial-sum planes (%.0f MB) exceed the 126 MB L2" % (
                       (w.n * w.n + 2 * w.n * w.m) * 4 / 1e6) if (w.n * w.n + 2 * w.n * w.m) * 4 > 2 * L2_BYTES
                   else "working set below L2: latency-bound, no DRAM figure claimed",
                   "launch": "one library call per step"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "TFLOPS", "h2d_bytes_per_step": int((hL.numel() + hB.numel()) * 4),
                "d2h_bytes_per_step": int(hX.numel() * 4), "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "cpu_baseline": {"value": cpu_v, "unit": "TFLOPS", "cores": cores, "kind": "oracle", "sample": sample},
    }
    print(json.dumps(line))
    reps.close()


def describe_trsm(w):
    return "%s: block lower-triangular solve f32 n=%d m=%d tile=%d seed=%d coupling=%s" % (w.name, w.n, w.m, w.tile, w.seed, w.coupling)


def cpu_trsm_rate(w, L, B, target_seconds=12.0, threads=None):
    """Time the triangular-solve oracle (collapsed form, as it stands) on a prefix of the right-hand-side columns."""
    from oracle import trsm as otrsm
    threads = threads or os.cpu_count() or 1
    cols = min(w.m, threads)
    while True:
        t0 = time.perf_counter()
        otrsm.block_trsm(L, np.ascontiguousarray(B[:, :cols]), w.tile, threads=threads)
        dt = time.perf_counter() - t0
        if dt >= 0.5 * target_seconds or cols >= w.m:
            break
        cols = int(min(w.m, cols * min(8.0, max(2.0, 0.9 * target_seconds / max(dt, 1e-3)))))
    rate = w.n * (w.n + 1) * cols / dt / 1e12
    return rate, threads, "columns 0..%d of %s (n=%d), collapsed form, %d threads, %.1f s" % (cols - 1, w.name, w.n, threads, dt)


def run_trsm_reference(args, w):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    L, B = inputs.make_trsm_operands(w)
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    vals, sample, threads = [], "", os.cpu_count() or 1
    for s in range(args.warmup + args.steps):
        v, threads, sample = cpu_trsm_rate(w, L, B, target_seconds=per_step)
        if s >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    print(json.dumps({
        "impl": "reference", "metric": "block_trsm_throughput", "value": value, "unit": "TFLOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": w.flops / (value * 1e12) * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": describe_trsm(w), "note": "ms_per_step extrapolated from the sampled rate"},
        "cpu_baseline": {"value": value, "unit": "TFLOPS", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}))


def describe_attention(w):
    return "%s: FlashAttention-2 recurrence bf16 batch=%d N=%d M=%d d=%d seed=%d qk_std=%g" % (w.name, w.batch, w.N, w.M, w.d, w.seed, w.qk_std)


def cpu_attention_rate(w, Q, K, V, target_seconds=12.0, threads=None):
    """Time the attention oracle (fp64 recurrence over key tiles of 128, as it stands) on a prefix of the query rows of
    problem 0, repeated over problem 0 when one whole problem is too short a sample."""
    from oracle import fa2 as ofa2
    threads = threads or os.cpu_count() or 1
    rows = min(w.N, threads)
    while True:
        reps_ = max(1, rows // w.N)
        t0 = time.perf_counter()
        for _ in range(reps_):
            ofa2.attention(Q[0][:min(rows, w.N)], K[0], V[0], 128, threads=threads)
        dt = time.perf_counter() - t0
        if dt >= 0.5 * target_seconds or rows >= 4096 * w.N:
            break
        rows = int(rows * min(8.0, max(2.0, 0.9 * target_seconds / max(dt, 1e-3))))
        if rows > w.N:
            rows = (rows // w.N) * w.N
    done = reps_ * min(rows, w.N)
    rate = 4.0 * done * w.M * w.d / dt / 1e12
    what = "query rows 0..%d" % (rows - 1) if rows <= w.N else "%d passes over all %d query rows" % (reps_, w.N)
    return rate, threads, "%s of problem 0 of %s (M=%d d=%d), fp64 recurrence, %d threads, %.1f s" % (what, w.name, w.M, w.d, threads, dt)


def run_attention_reference(args, w):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    Q, K, V = inputs.make_attention_operands(inputs.AttentionWorkload(w.name, 1, w.N, w.M, w.d, seed=w.seed, qk_std=w.qk_std))
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    vals, sample, threads = [], "", os.cpu_count() or 1
    for s in range(args.warmup + args.steps):
        v, threads, sample = cpu_attention_rate(w, Q, K, V, target_seconds=per_step)
        if s >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    print(json.dumps({
        "impl": "reference", "metric": "flash_attention_throughput", "value": value, "unit": "TFLOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": w.flops / (value * 1e12) * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": describe_attention(w), "note": "ms_per_step extrapolated from the sampled rate"},
        "cpu_baseline": {"value": value, "unit": "TFLOPS", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}))


def run_attention(args, w):
    """FlashAttention-2 recurrence (workloads a1, a2): one step = one launch over every (problem, query tile)."""
    import torch
    from paper_2511_09987_b200 import binding
    from paper_2511_09987_b200.replicas import Replicas

    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    reps = Replicas("nccl", torch.device("cuda", local))
    world, rank = reps.world, reps.rank
    peaks, peak_kind = load_peaks()
    Q, K, V = inputs.make_attention_operands(w)
    hQ, hK, hV = (torch.from_numpy(x).view(torch.bfloat16).pin_memory() for x in (Q, K, V))
    hO = torch.empty((w.batch, w.N, w.d), dtype=torch.float32).pin_memory()
    set_bytes = w.algorithmic_bytes
    nsets = int(min(8, max(2, -(-3 * L2_BYTES // set_bytes))))
    sets = [(hQ.cuda(), hK.cuda(), hV.cuda(), torch.empty((w.batch, w.N, w.d), dtype=torch.float32, device="cuda")) for _ in range(nsets)]
    stream = torch.cuda.current_stream()

    def step(i):
        dQ, dK, dV, dO = sets[i % nsets]
        binding.flash_attention(dQ, dK, dV, dO)

    def barrier():
        reps.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = binding.cyc_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    barrier()
    launches = binding.cyc_launch_count() - launches0
    if binding.last_device_status() != binding.CYC_OK:
        raise SystemExit("a device-side wait timed out during the benchmark: " + binding.cyc_last_cuda_error().decode())
    clocks = sampler.stop()
    total_ms = reps.max_over_ranks(e0.elapsed_time(e1))
    ms_per_step = total_ms / args.steps
    value = world * w.flops / (ms_per_step * 1e-3) / 1e12

    # end to end: pinned host Q, K, V up, one launch, O down, every step
    e2e_steps = 0 if args.kernel_only else max(3, min(args.steps, 10))
    dQ, dK, dV, dO = sets[0]

    def e2e_step():
        dQ.copy_(hQ, non_blocking=True)
        dK.copy_(hK, non_blocking=True)
        dV.copy_(hV, non_blocking=True)
        binding.flash_attention(dQ, dK, dV, dO)
        hO.copy_(dO, non_blocking=True)

    for _ in range(0 if args.kernel_only else 2):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / max(1, e2e_steps)
    e2e_value = None if args.kernel_only else world * w.flops / (reps.max_over_ranks(e2e_ms) * 1e-3) / 1e12
    if rank != 0:
        reps.close()
        return
    step_s = ms_per_step * 1e-3
    family = "fa2_d%d" % w.d
    roofline = {"bound": "tensor", "achieved": value / world, "unit": "TFLOP/s", "traffic": load_traffic(w, family),
                "note": "4 N M d flop per problem (both products, exponentials not counted)",
                "kernel": "fa2_kernel<%d>" % w.d, "kernel_us": step_s * 1e6}
    roofline.update(tensor_roofline(value / world, "bf16", peaks, peak_kind))
    if args.kernel_only:
        cpu_v, cores, sample = None, 0, "skipped (--kernel-only)"
    else:
        cpu_v, cores, sample = cpu_attention_rate(w, Q, K, V)
    if nsets * set_bytes > 2 * L2_BYTES:
        l2_note = "inputs rotate over %d device copies (%.0f MB in total, larger than the 126 MB L2)" % (nsets, nsets * set_bytes / 1e6)
    else:
        l2_note = "working set of %d rotating copies is %.1f MB, below L2: no DRAM figure is claimed" % (nsets, nsets * set_bytes / 1e6)
    line = {
        "metric": "flash_attention_throughput", "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": describe_attention(w), "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": l2_note, "launch": "one library call per step"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "TFLOPS", "h2d_bytes_per_step": int((hQ.numel() + hK.numel() + hV.numel()) * 2),
                "d2h_bytes_per_step": int(hO.numel() * 4), "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "cpu_baseline": {"value": cpu_v, "unit": "TFLOPS", "cores": cores, "kind": "oracle", "sample": sample},
    }
    print(json.dumps(line))
    reps.close()


def describe_scan(w):
    return "%s: prefix-sum recurrence %s rows=%d n=%d seed=%d" % (w.name, w.dtype, w.rows, w.n, w.seed)


def cpu_scan_rate(w, A, target_seconds=12.0):
    """Time the prefix-sum oracle (the literal walk, as it stands; one thread: the recurrence is a single dependency
    chain per row and the oracle does not split it) on a prefix of the elements, repeated when the workload is small."""
    from oracle import scan as oscan
    arith = "i32" if w.dtype == "i32" else "f64"
    flat = A.reshape(-1)
    count = min(flat.size, 1 << 20)
    while True:
        reps_ = max(1, count // flat.size)
        t0 = time.perf_counter()
        for _ in range(reps_):
            oscan.prefix_sum(flat[:min(count, flat.size)], arithmetic=arith)
        dt = time.perf_counter() - t0
        if dt >= 0.5 * target_seconds or count >= 64 * flat.size:
            break
        count = int(count * min(8.0, max(2.0, 0.9 * target_seconds / max(dt, 1e-3))))
        if count > flat.size:
            count = (count // flat.size) * flat.size
    done = reps_ * min(count, flat.size)
    what = "elements 0..%d as one sequence" % (count - 1) if count <= flat.size else "%d passes over all %d elements" % (reps_, flat.size)
    return done / dt / 1e9, 1, "%s of %s, literal walk (%s), 1 thread, %.1f s" % (what, w.name, arith, dt)


def run_scan_reference(args, w):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    A = inputs.make_scan_operand(w)
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    vals, sample = [], ""
    for s in range(args.warmup + args.steps):
        v, _, sample = cpu_scan_rate(w, A, target_seconds=per_step)
        if s >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    print(json.dumps({
        "impl": "reference", "metric": "prefix_sum_throughput", "value": value, "unit": "Gelem/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": w.elements / (value * 1e9) * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": describe_scan(w), "note": "ms_per_step extrapolated from the sampled rate"},
        "cpu_baseline": {"value": value, "unit": "Gelem/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "Gelem/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}))


def run_scan(args, w):
    """Prefix-sum recurrence (workloads p1, p2, p3): one step = one launch over every tile of every row."""
    import torch
    from paper_2511_09987_b200 import binding
    from paper_2511_09987_b200.replicas import Replicas

    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    reps = Replicas("nccl", torch.device("cuda", local))
    world, rank = reps.world, reps.rank
    peaks, peak_kind = load_peaks()
    A = inputs.make_scan_operand(w)
    hA = torch.from_numpy(A).pin_memory()
    hP = torch.empty_like(hA).pin_memory()
    set_bytes = w.algorithmic_bytes
    nsets = int(min(8, max(2, -(-3 * L2_BYTES // set_bytes))))
    sets = [(hA.cuda(), torch.empty(A.shape, dtype=hA.dtype, device="cuda")) for _ in range(nsets)]
    stream = torch.cuda.current_stream()

    def step(i):
        dA, dP = sets[i % nsets]
        binding.prefix_sum(dA, dP)

    def barrier():
        reps.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = binding.cyc_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    barrier()
    launches = binding.cyc_launch_count() - launches0
    if binding.last_device_status() != binding.CYC_OK:
        raise SystemExit("a device-side wait timed out during the benchmark: " + binding.cyc_last_cuda_error().decode())
    clocks = sampler.stop()
    ms_per_step = reps.max_over_ranks(e0.elapsed_time(e1)) / args.steps
    value = world * w.elements / (ms_per_step * 1e-3) / 1e9

    e2e_steps = 0 if args.kernel_only else max(3, min(args.steps, 10))
    dA, dP = sets[0]

    def e2e_step():
        dA.copy_(hA, non_blocking=True)
        binding.prefix_sum(dA, dP)
        hP.copy_(dP, non_blocking=True)

    for _ in range(0 if args.kernel_only else 2):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / max(1, e2e_steps)
    e2e_value = None if args.kernel_only else world * w.elements / (reps.max_over_ranks(e2e_ms) * 1e-3) / 1e9
    if rank != 0:
        reps.close()
        return
    step_s = ms_per_step * 1e-3
    achieved = w.algorithmic_bytes / step_s / 1e9
    peak = float(peaks["hbm_gbs"])
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": load_traffic(w, "scan"),
                "peak_source": "%s STREAM-style copy; 8 bytes per element (read once, written once); the step also holds a "
                               "memset of the tile descriptors (8 bytes per 16384 elements)" % peak_kind,
                "kernel": "scan_kernel<%s>" % ("float" if w.dtype == "f32" else "int"), "kernel_us": step_s * 1e6}
    if args.kernel_only:
        cpu_v, cores, sample = None, 0, "skipped (--kernel-only)"
    else:
        cpu_v, cores, sample = cpu_scan_rate(w, A)
    if nsets * set_bytes > 2 * L2_BYTES:
        l2_note = "inputs rotate over %d device copies (%.0f MB in total, larger than the 126 MB L2)" % (nsets, nsets * set_bytes / 1e6)
    else:
        l2_note = "working set of %d rotating copies is %.1f MB, below L2: no DRAM figure is claimed" % (nsets, nsets * set_bytes / 1e6)
    line = {
        "metric": "prefix_sum_throughput", "value": value, "unit": "Gelem/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": describe_scan(w), "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": l2_note, "launch": "one library call per step"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "Gelem/s", "h2d_bytes_per_step": int(hA.numel() * 4),
                "d2h_bytes_per_step": int(hP.numel() * 4), "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "cpu_baseline": {"value": cpu_v, "unit": "Gelem/s", "cores": cores, "kind": "oracle", "sample": sample},
    }
    print(json.dumps(line))
    reps.close()


def describe_chol(w):
    return "%s: tiled Cholesky f32 n=%d tile=%d seed=%d coupling=%s" % (w.name, w.n, w.tile, w.seed, w.coupling)


def cpu_chol_rate(w, A, target_seconds=12.0, threads=None):
    """Time the Cholesky oracle (tiled form, as it stands) on a leading principal block of A."""
    from oracle import chol as ochol
    threads = threads or os.cpu_count() or 1
    m = min(w.n, 512)
    while True:
        t0 = time.perf_counter()
        ochol.cholesky(np.ascontiguousarray(A[:m, :m]), w.tile, threads=threads)
        dt = time.perf_counter() - t0
        if dt >= 0.5 * target_seconds or m >= w.n:
            break
        m = int(min(w.n, m * min(2.0, max(1.26, (0.9 * target_seconds / max(dt, 1e-3)) ** (1.0 / 3.0)))))
    rate = (m ** 3 / 3.0) / dt / 1e12
    return rate, threads, "leading %d x %d block of %s, tiled form (tile %d), fp64, %d threads, %.1f s" % (m, m, w.name, w.tile, threads, dt)


def run_chol_reference(args, w):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    A = inputs.make_chol_operand(w)
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    vals, sample, threads = [], "", os.cpu_count() or 1
    for s in range(args.warmup + args.steps):
        v, threads, sample = cpu_chol_rate(w, A, target_seconds=per_step)
        if s >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    print(json.dumps({
        "impl": "reference", "metric": "cholesky_throughput", "value": value, "unit": "TFLOPS", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": w.flops / (value * 1e12) * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": describe_chol(w), "note": "ms_per_step extrapolated from the sampled rate"},
        "cpu_baseline": {"value": value, "unit": "TFLOPS", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}))


def run_chol(args, w):
    """Tiled Cholesky (workloads h1, h2): one step = one whole factorisation (every SYRK / GEMM launch, every diagonal
    tile, every panel solve)."""
    import torch
    from paper_2511_09987_b200 import binding
    from paper_2511_09987_b200.replicas import Replicas

    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    reps = Replicas("nccl", torch.device("cuda", local))
    world, rank = reps.world, reps.rank
    peaks, peak_kind = load_peaks()
    A = inputs.make_chol_operand(w)
    hA = torch.from_numpy(A).pin_memory()
    hL = torch.empty_like(hA).pin_memory()
    dA = hA.cuda()
    dL = torch.empty_like(dA)
    stream = torch.cuda.current_stream()

    def barrier():
        reps.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        binding.cholesky(dA, dL, tile=w.tile)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = binding.cyc_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        binding.cholesky(dA, dL, tile=w.tile)
    e1.record(stream)
    barrier()
    launches = binding.cyc_launch_count() - launches0
    if binding.last_device_status() != binding.CYC_OK:
        raise SystemExit("a device-side wait timed out during the benchmark: " + binding.cyc_last_cuda_error().decode())
    clocks = sampler.stop()
    total_ms = reps.max_over_ranks(e0.elapsed_time(e1))
    ms_per_step = total_ms / args.steps
    value = world * w.flops / (ms_per_step * 1e-3) / 1e12

    e2e_steps = 0 if args.kernel_only else max(3, min(args.steps, 10))

    def e2e_step():
        dA.copy_(hA, non_blocking=True)
        binding.cholesky(dA, dL, tile=w.tile)
        hL.copy_(dL, non_blocking=True)

    for _ in range(0 if args.kernel_only else 2):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / max(1, e2e_steps)
    e2e_value = None if args.kernel_only else world * w.flops / (reps.max_over_ranks(e2e_ms) * 1e-3) / 1e12
    if rank != 0:
        reps.close()
        return
    step_s = ms_per_step * 1e-3
    roofline = {"bound": "tensor", "achieved": value / world, "unit": "TFLOP/s", "traffic": None,
                "note": "the whole step is rated (n^3/3 flop, the three TF32 products of each fp32 product counted once): "
                        "%d launches per factorisation" % (launches // max(1, args.steps)),
                "kernel": "tcgen05_3xtf32 (SYRK/GEMM sums) + chol_diag (diagonal tiles) + trsm_diag (tiles below)", "kernel_us": step_s * 1e6}
    roofline.update(tensor_roofline(value / world, "tf32", peaks, peak_kind))
    if args.kernel_only:
        cpu_v, cores, sample = None, 0, "skipped (--kernel-only)"
    else:
        cpu_v, cores, sample = cpu_chol_rate(w, A)
    line = {
        "metric": "cholesky_throughput", "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": describe_chol(w), "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": "A and L (%.0f MB) exceed the 126 MB L2" % (2 * w.n * w.n * 4 / 1e6) if 2 * w.n * w.n * 4 > 2 * L2_BYTES
                   else "working set below L2: latency-bound, no DRAM figure claimed",
                   "launch": "one library call per step"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "TFLOPS", "h2d_bytes_per_step": int(hA.numel() * 4), "d2h_bytes_per_step": int(hL.numel() * 4),
                "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "cpu_baseline": {"value": cpu_v, "unit": "TFLOPS", "cores": cores, "kind": "oracle", "sample": sample},
    }
    print(json.dumps(line))
    reps.close()


# CUDA sources each kernel family is built from (host-side launch code is not part of a kernel's identity)
KERNEL_SOURCES = {
    "simt": ["simt_kernel.cuh"],
    "tcgen05": ["ptx.cuh", "umma_kernel.cuh"],
    "tcgen05_pair": ["ptx.cuh", "umma_kernel.cuh", "umma_pair_kernel.cuh"],
    "tcgen05_pair_tall": ["ptx.cuh", "umma_kernel.cuh", "umma_pair_kernel.cuh", "umma_pair_tall_kernel.cuh"],
    "tcgen05_pair_splitk": ["ptx.cuh", "umma_kernel.cuh", "umma_pair_kernel.cuh", "splitk_reduce_kernel.cuh"],
    "tcgen05_3xtf32": ["ptx.cuh", "umma_kernel.cuh", "umma_pair_kernel.cuh", "umma_pair_tf32x3_kernel.cuh"],
    "tcgen05_3xtf32_ws": ["ptx.cuh", "umma_kernel.cuh", "umma_ws_tf32x3_kernel.cuh"],
    "scan": ["scan_kernel.cuh"],
    "fa2_d64": ["ptx.cuh", "umma_kernel.cuh", "fa2_kernel.cuh"],
    "fa2_d128": ["ptx.cuh", "umma_kernel.cuh", "fa2_kernel.cuh"],
}


def kernel_source_digest(family):
    """sha256 over the CUDA sources of one kernel family: ties a stored DRAM-traffic figure to the kernel it was taken from."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2511_09987_b200", "csrc")
    for name in KERNEL_SOURCES.get(family, sorted(os.listdir(csrc))):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(name.encode())
            h.update(f.read())
    return h.hexdigest()[:16]


def load_traffic(w, family):
    """DRAM bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum) for this workload's kernel.

    Read from profiles/dram_traffic.txt, lines `workload bytes digest`; a figure whose digest does not match the
    current sources of the kernel is stale and reported as null."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    digest = kernel_source_digest(family)
    with open(path) as f:
        for line in f:
            parts = line.split()
            if len(parts) >= 3 and not line.startswith("#") and parts[0] == w.name and parts[2] == digest:
                return float(parts[1])
    return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=None, choices=sorted(inputs.WORKLOADS) + sorted(inputs.TRSM_WORKLOADS) + sorted(inputs.ATTENTION_WORKLOADS) + sorted(inputs.SCAN_WORKLOADS)
                    + sorted(inputs.CHOL_WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--shape", default=None, help="M,N,K[,batch] (c1..c5), n,m[,tile] (t1, t2) batch,N,M,d (a1, a2), rows,n (p1..p3) or n[,tile] (h1, h2): a smaller case of the workload's recipe (for profiling)")
    ap.add_argument("--strict", action="store_true", help="set the fixed-k-order flag (fp32: the per-element FMA chain kernel)")
    ap.add_argument("--graph", default="auto", choices=["auto", "on", "off"],
                    help="replay the timed steps from a CUDA graph (auto: only for launch-bound workloads)")
    ap.add_argument("--kernel-only", action="store_true", help="skip the end-to-end and CPU-baseline legs (for profiling)")
    ap.add_argument("--sustained", action="store_true", help="add a region of at least one second (c2, c3) to a single-workload run")
    args = ap.parse_args()
    # no --workload: the largest configuration that fits one GPU (c3) is the headline, and the other four
    # configurations of the matrix-multiply recurrence follow as sub-records of the same line
    with_configs = args.workload is None and args.impl == "ours" and not args.kernel_only and not args.shape
    if args.workload is None:
        args.workload = "c3"
    if args.workload in inputs.TRSM_WORKLOADS:
        w = inputs.TRSM_WORKLOADS[args.workload]
        if args.shape:  # n,m[,tile]: a smaller case of the same recipe (for profiling)
            dims = [int(x) for x in args.shape.split(",")]
            w = inputs.TrsmWorkload(w.name + "@" + args.shape, dims[0], dims[1], dims[2] if len(dims) > 2 else w.tile, seed=w.seed,
                                    coupling=w.coupling)
        if args.steps is None:
            args.steps = 3 if args.impl == "reference" else {"t1": 500, "t2": 50}[w.name.split("@")[0]]
        (run_trsm_reference if args.impl == "reference" else run_trsm)(args, w)
        return
    if args.workload in inputs.CHOL_WORKLOADS:
        w = inputs.CHOL_WORKLOADS[args.workload]
        if args.shape:
            dims = [int(x) for x in args.shape.split(",")]
            w = inputs.CholWorkload(w.name + "@" + args.shape, dims[0], dims[1] if len(dims) > 1 else w.tile, seed=w.seed, coupling=w.coupling)
        if args.steps is None:
            args.steps = 3 if args.impl == "reference" else {"h1": 200, "h2": 30}[w.name.split("@")[0]]
        (run_chol_reference if args.impl == "reference" else run_chol)(args, w)
        return
    if args.workload in inputs.SCAN_WORKLOADS:
        w = inputs.SCAN_WORKLOADS[args.workload]
        if args.shape:
            dims = [int(x) for x in args.shape.split(",")]
            w = inputs.ScanWorkload(w.name + "@" + args.shape, dims[0], dims[1], w.dtype, seed=w.seed)
        if args.steps is None:
            args.steps = 3 if args.impl == "reference" else {"p1": 2000, "p2": 200, "p3": 200}[w.name.split("@")[0]]
        (run_scan_reference if args.impl == "reference" else run_scan)(args, w)
        return
    if args.workload in inputs.ATTENTION_WORKLOADS:
        w = inputs.ATTENTION_WORKLOADS[args.workload]
        if args.shape:
            dims = [int(x) for x in args.shape.split(",")]
            w = inputs.AttentionWorkload(w.name + "@" + args.shape, dims[0], dims[1], dims[2], dims[3], seed=w.seed, qk_std=w.qk_std)
        if args.steps is None:
            args.steps = 3 if args.impl == "reference" else {"a1": 500, "a2": 50}[w.name.split("@")[0]]
        (run_attention_reference if args.impl == "reference" else run_attention)(args, w)
        return
    w = inputs.WORKLOADS[args.workload]
    if args.shape:
        dims = [int(x) for x in args.shape.split(",")]
        w = inputs.scaled(w, name=w.name + "@" + args.shape, M=dims[0], N=dims[1], K=dims[2], batch=dims[3] if len(dims) > 3 else w.batch)
    if args.strict:
        w = inputs.scaled(w, name=w.name + "+strict", fixed_k_order=True)
    if args.impl == "reference":
        if args.steps is None:
            args.steps = 3
        run_reference(args, w)
        return
    if args.steps is None:
        args.steps = {"c1": 20000, "c2": 4000, "c3": 400, "c4": 4000, "c5": 3000}[w.name.split("@")[0].split("+")[0]]
    run_ours(args, w, with_configs)


if __name__ == "__main__":
    main()
