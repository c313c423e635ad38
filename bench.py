#!/usr/bin/env python
"""Benchmark of the GEMM hot path on B200:  C = A * B^T at N = 8192.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--size N] [--e2e-steps E] [--no-cpu-baseline]

One step = one pass of the whole path over one batch of seeded synthetic
operands: an FP16 GEMM, an INT8 GEMM and an INT4 GEMM (nibble unpack pre-pass
+ INT8 tensor-core kernel) of size N^3, each bracketed by CUDA events on the
launching stream.  The headline `value` is the FP16 rate (TFLOP/s, 2 N^3 per
GEMM); the INT8 / INT4 rates (TOP/s) and every fraction-of-peak are in
`precisions`.  Operands stay resident in HBM for `value`; `e2e` repeats the
FP16 GEMM with pinned host buffers and both copies inside the timed region.

Prints ONE JSON line on rank 0.  Under torchrun each rank runs an independent
replica of the same workload (no data-path collective; weak scaling).

Other modes (1 GPU, one JSON line per measurement): --sweep (precision x size,
N = 512..8192), --ablation (tile / raster / L2 / INT4 route at --size, with the
kernel's cycle accounting), --few-rows (M = 1..128 against the HBM roofline;
--shape M,N,K for any other shape), --selector-check (the automatic tile and
split-K choice against forced ones), --capture (the launches the profiler summaries under
profiles/ were taken from).
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

SPEC_PEAK = {"fp16": 2250.0, "s8": 4500.0, "s4": 4500.0}   # vendor dense figures, T(FL)OP/s
UNIT = {"fp16": "TFLOP/s", "s8": "TOP/s", "s4": "TOP/s"}
KERNEL_LAUNCHES = {"fp16": 1, "s8": 1, "s4": 2}            # s4: unpack launch + GEMM
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic_fp16_gemm.txt")


def captured_traffic(size, lib_version):
    """DRAM bytes per launch of the FP16 GEMM kernel from the last profiler capture of this
    workload (key = value lines written beside the capture's summary), or None when no capture
    of this size exists or it was taken with another version of the library."""
    try:
        kv = {}
        with open(TRAFFIC_FILE) as f:
            for line in f:
                if "=" in line and not line.lstrip().startswith("#"):
                    k, v = line.split("=", 1)
                    kv[k.strip()] = v.strip()
        if int(kv["library_version"]) != lib_version:
            return None, "capture is of library version %s" % kv["library_version"]
        r, w = kv.get("n%d_dram_read_bytes" % size), kv.get("n%d_dram_write_bytes" % size)
        if r is None or w is None:
            return None, "no capture at this size"
        return int(r) + int(w), kv.get("capture", "")
    except (OSError, KeyError, ValueError):
        return None, "no capture on file"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"bf16_burst": float(d["bf16_tflops"]),
                "bf16_sustained": float(d["bf16_tflops_sustained"]),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    except Exception:
        return {"bf16_burst": 1590.0, "bf16_sustained": 1400.0, "hbm_gbs": 6650.0,
                "source": "fallback"}


class ClockSampler:
    """Samples SM clock, power and throttle reasons while a region runs (read-only NVML
    queries every ~5 ms in a thread; falls back to an nvidia-smi loop if NVML is missing)."""
    REASONS = ((0x4, "sw_power_cap"), (0x8, "hw_slowdown"), (0x20, "sw_thermal_slowdown"),
               (0x40, "hw_thermal_slowdown"), (0x80, "hw_power_brake_slowdown"))
    SMI_FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
                  "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
                  "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.sm, self.pw = [], []
        self.mask = 0
        self.sm_max = None
        self.stop_flag = threading.Event()
        self.thread = None
        self.proc = None
        self.nvml = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nvml = pynvml
            self.thread = threading.Thread(target=self._poll_nvml, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.SMI_FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read_smi, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _poll_nvml(self):
        n = self.nvml
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)))
                self.pw.append(n.nvmlDeviceGetPowerUsage(self.handle) / 1000.0)
                self.mask |= int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
            except Exception:
                pass
            time.sleep(0.005)

    def _read_smi(self):
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        bits = {"sw_power_cap": 0x4, "hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20,
                "hw_thermal_slowdown": 0x40}
        for line in self.proc.stdout:
            r = [x.strip() for x in line.split(",")]
            if len(r) < 7:
                continue
            try:
                self.sm.append(float(r[0]))
                self.sm_max = float(r[1])
                self.pw.append(float(r[2]))
            except ValueError:
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    self.mask |= bits[name]

    def stop(self):
        self.stop_flag.set()
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)
        if self.nvml is None and self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no NVML, no nvidia-smi"]}
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None,
                "sm_min_mhz": min(self.sm) if self.sm else None,
                "sm_max_mhz": self.sm_max,
                "power_w_max": max(self.pw) if self.pw else None,
                "power_w_mean": statistics.mean(self.pw) if self.pw else None,
                # second half of the samples: the regime the region settled in
                "sm_mhz_settled": statistics.median(self.sm[len(self.sm) // 2:]) if self.sm else None,
                "power_w_settled": statistics.median(self.pw[len(self.pw) // 2:]) if self.pw else None,
                "samples": len(self.sm),
                "source": "nvml" if self.nvml is not None else "nvidia-smi",
                "reasons": sorted(name for bit, name in self.REASONS if self.mask & bit)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except (ValueError, IndexError):
            return local
    return local


# --------------------------------------------------------------------- reference arm
def run_reference(args, rank):
    """Times the CPU oracle, as it stands, on a bounded sample of the same FP16
    workload (a block of rows of C, all columns), on this machine's host cores."""
    if rank != 0:
        return
    import numpy as np
    import oracle
    from paper_2608_10103_b200 import synth
    N = args.size
    A, B = synth.fp16_normal_clipped(N, N, N, seed=3)
    rows = np.arange(args.ref_rows, dtype=np.int32)
    ops = synth.gemm_ops(len(rows), N, N)
    for _ in range(args.warmup):
        oracle.gemm_fp16(A, B, rows=rows[:2])
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.gemm_fp16(A, B, rows=rows)
    dt = time.perf_counter() - t0
    value = ops * args.steps / dt / 1e12
    sample = "%d rows x %d cols of C per step (K=%d)" % (len(rows), N, N)
    line = {
        "impl": "reference", "metric": "fp16_gemm_tflops_n%d" % N, "value": value,
        "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "FP16 GEMM M=N=K=%d, N(0,1) clipped to [-4,4], seed 3" % N,
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oracle.threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- our arm
def cpu_baseline(N, A, B, target_seconds=12.0):
    """The oracle, as it stands, on a block of rows of the FP16 problem sized to
    take about `target_seconds` on this machine's cores."""
    import numpy as np
    import oracle
    from paper_2608_10103_b200 import synth

    def run(n):
        t0 = time.perf_counter()
        oracle.gemm_fp16(A, B, rows=np.arange(n, dtype=np.int32))
        return time.perf_counter() - t0

    th = oracle.threads()
    n_a, n_b = 2 * th, 6 * th
    t_a, t_b = run(n_a), run(n_b)
    per_row = max((t_b - t_a) / (n_b - n_a), 1e-7)
    fixed = max(t_a - n_a * per_row, 0.0)          # one-off operand decode
    nrows = int((target_seconds - fixed) / per_row) // th * th
    nrows = max(n_b, min(N, nrows))
    dt = run(nrows)
    return {"value": synth.gemm_ops(nrows, N, N) / dt / 1e12, "unit": "TFLOP/s",
            "cores": th, "kind": "oracle",
            "sample": "%d rows x %d cols of the FP16 C (K=%d), %.1f s" % (nrows, N, N, dt)}


def run_ours(args, rank, world):
    import numpy as np
    import torch
    from paper_2608_10103_b200 import binding, replicas, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the GEMM path has no CPU fallback")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    binding.lib()
    if args.override:
        binding.gemm_set_config_override(*[int(x) for x in args.override.split(",")])
    if args.l2_policy >= 0:
        binding.gemm_set_l2_policy(args.l2_policy)
    if args.family:
        binding.gemm_set_kernel_family(args.family)
    N = args.size
    ops = synth.gemm_ops(N, N, N)
    stream = torch.cuda.current_stream()

    # Operands: the named N = 8192 configurations (FP16: N(0,1) clipped, seed 3; INT8 / INT4:
    # the sweep's uniform draws).  Each rank draws its own replica (seed + rank).
    want = args.precisions.split(",")
    host = {"fp16": synth.fp16_normal_clipped(N, N, N, seed=replicas.replica_seed(3, rank))}
    if "s8" in want:
        host["s8"] = synth.s8_uniform(
            N, N, N, seed=replicas.replica_seed(synth.sweep_seed("s8", 8192), rank))
    if "s4" in want:
        host["s4"] = synth.s4_uniform(
            N, N, N, seed=replicas.replica_seed(synth.sweep_seed("s4", 8192), rank))
    dev = {p: (torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()) for p, (a, b) in host.items()}
    out = {p: torch.empty((N, N), dtype=torch.float32 if p == "fp16" else torch.int32,
                          device="cuda") for p in host}
    precs = tuple(x for x in ("fp16", "s8", "s4") if x in args.precisions.split(","))
    if "fp16" not in precs:
        raise SystemExit("bench.py: --precisions must include fp16 (the headline)")

    def step(events=None):
        for p in precs:
            if events is not None:
                events[p][0].record(stream)
            binding.gemm(p, dev[p][0], dev[p][1], out[p], stream)
            if events is not None:
                events[p][1].record(stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()                       # before the warm-up, so that short runs get samples too
    for _ in range(args.warmup):
        step()
    barrier()
    evs = [{p: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
            for p in precs} for _ in range(args.steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record(stream)
    for i in range(args.steps):
        step(evs[i])
    stop.record(stream)
    barrier()
    clocks = sampler.stop()
    total_ms = start.elapsed_time(stop)
    per_prec_ms = {p: sum(e[p][0].elapsed_time(e[p][1]) for e in evs) / args.steps for p in precs}
    best_ms = {p: min(e[p][0].elapsed_time(e[p][1]) for e in evs) for p in precs}
    if binding.gemm_last_device_status() != 0:
        raise SystemExit("bench.py: a kernel reported a barrier timeout")

    # max over ranks (device time)
    times = replicas.max_over_ranks([total_ms] + [per_prec_ms[p] for p in precs], dist, "cuda")
    total_ms = times[0]
    worst = dict(zip(precs, times[1:]))

    # ---- cycle-based view (independent of the power-capped clock): one traced launch per
    #      precision gives the SM cycles it took and the SM clock it ran at
    cycles = {}
    flop_per_clk = {"fp16": 8192, "s8": 16384, "s4": 16384}   # per SM, dense, from the probe below
    num_sms = torch.cuda.get_device_properties(local).multi_processor_count
    binding.gemm_trace_enable(1)
    for p in precs:
        binding.gemm(p, dev[p][0], dev[p][1], out[p], stream)
        tr = binding.gemm_trace_read(num_sms)
        cyc = max(t["cycles"] for t in tr)
        mhz = statistics.median(t["cycles"] / t["nanos"] * 1e3 for t in tr if t["nanos"])
        cycles[p] = {"sm_cycles": cyc, "sm_mhz_during_kernel": mhz,
                     "pipe_utilisation": ops / (num_sms * flop_per_clk[p]) / cyc}
    binding.gemm_trace_enable(0)

    # ---- the sustained regime: each precision alone, back to back for >= --sustain-seconds,
    #      with the clock and power NVML saw meanwhile (energy per GEMM = mean power x time)
    sustained = {}
    if args.sustain_seconds > 0:
        for p in precs:
            n = max(args.steps, int(args.sustain_seconds * 1e3 / max(per_prec_ms[p], 1e-3)) + 1)
            for attempt in range(3):      # back to back the launches run faster than when bracketed
                barrier()
                s2 = ClockSampler(physical_gpu_index(local))
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s2.start()
                e0.record(stream)
                for _ in range(n):
                    binding.gemm(p, dev[p][0], dev[p][1], out[p], stream)
                e1.record(stream)
                barrier()
                c2 = s2.stop()
                ms = replicas.max_over_ranks([e0.elapsed_time(e1) / n], dist, "cuda")[0]
                if ms * n * 1e-3 >= args.sustain_seconds:
                    break
                n = int(n * args.sustain_seconds / (ms * n * 1e-3) * 1.1) + 1
            sustained[p] = {"launches": n, "seconds": ms * n * 1e-3, "ms": ms,
                            "value": replicas.whole_job_rate(ops, world, ms), "unit": UNIT[p],
                            "sm_mhz_settled": c2.get("sm_mhz_settled"),
                            "power_w_settled": c2.get("power_w_settled"),
                            "joules_per_gemm": (c2["power_w_settled"] * ms * 1e-3
                                                if c2.get("power_w_settled") else None),
                            "clock_samples": c2.get("samples"), "reasons": c2.get("reasons")}
        if binding.gemm_last_device_status() != 0:
            raise SystemExit("bench.py: a kernel reported a barrier timeout")

    # ---- MMA-issue-only peak of this machine, per kind (same run, same power regime): rate by
    #      CUDA events, cycles per 128x256x(32 B) MMA and clock by the probe's own counters
    mma_peak, mma_detail = {}, {}
    for kind in (() if args.no_peak_probe else ("fp16", "s8")):
        binding.gemm_mma_peak_probe(kind, 2048)
        torch.cuda.synchronize()
        binding.gemm_trace_enable(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        pops = binding.gemm_mma_peak_probe(kind, 200000)
        e1.record(stream)
        torch.cuda.synchronize()
        tr = binding.gemm_trace_read(num_sms)
        binding.gemm_trace_enable(0)
        mma_peak[kind] = pops / (e0.elapsed_time(e1) * 1e-3) / 1e12
        mma_detail[kind] = {
            "cycles_per_mma": statistics.mean(t["cycles"] for t in tr) / 200000,
            "sm_mhz_during_probe": statistics.median(t["cycles"] / t["nanos"] * 1e3 for t in tr)}
    if mma_peak:
        mma_peak["s4"] = mma_peak["s8"]
        mma_detail["s4"] = mma_detail["s8"]

    # ---- end to end: FP16 GEMM through the host-buffer entry point (pinned A, B, C):
    #      H2D of the operands, the kernels and D2H of C are all inside the timed region
    e2e = None
    if args.e2e_steps > 0:
        hA = torch.from_numpy(host["fp16"][0]).pin_memory()
        hB = torch.from_numpy(host["fp16"][1]).pin_memory()
        hC = torch.empty((N, N), dtype=torch.float32).pin_memory()
        binding.gemm_host("fp16", hA, hB, hC, stream)      # first call allocates device buffers
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.e2e_steps):
            binding.gemm_host("fp16", hA, hB, hC, stream)
        e1.record(stream)
        barrier()
        e2e_ms = replicas.max_over_ranks([e0.elapsed_time(e1)], dist, "cuda")[0] / args.e2e_steps
        e2e = {"value": replicas.whole_job_rate(ops, world, e2e_ms), "unit": "TFLOP/s",
               "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": hA.numel() * 2 + hB.numel() * 2,
               "d2h_bytes_per_step": hC.numel() * 4,
               "what": "gemm_host(FP16): pinned host A, B -> device in 2048-row blocks, C blocks "
                       "multiplied as operands arrive and copied back while later blocks run"}
        e2e["sampled_check_max_abs"] = float(
            (hC[:4, :64] - out["fp16"][:4, :64].cpu()).abs().max())

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    precisions = {}
    for p in precs:
        rate = replicas.whole_job_rate(ops, world, worst[p])
        precisions[p] = {
            "value": rate, "unit": UNIT[p], "ms": worst[p], "best_ms_rank0": best_ms[p],
            "frac_of_spec_peak": rate / world / SPEC_PEAK[p], "spec_peak": SPEC_PEAK[p],
            "frac_of_mma_only_peak": rate / world / mma_peak[p] if mma_peak else None,
            "mma_only_peak": mma_peak.get(p), "mma_only_probe": mma_detail.get(p),
            "sm_cycles": cycles[p]["sm_cycles"], "pipe_utilisation": cycles[p]["pipe_utilisation"],
            "sm_mhz_during_kernel": cycles[p]["sm_mhz_during_kernel"],
            "config": binding.gemm_query_config(p, N, N, N),
        }
        if p in sustained:
            sus = dict(sustained[p])
            sus["frac_of_spec_peak"] = sus["value"] / world / SPEC_PEAK[p]
            precisions[p]["sustained"] = sus
    if "s4" in worst and "s8" in worst:
        precisions["s4"]["overhead_vs_s8"] = worst["s4"] / worst["s8"] - 1.0

    fp16_rate_1gpu = ops / (worst["fp16"] * 1e-3) / 1e12
    traffic, traffic_note = captured_traffic(N, binding.gemm_version())
    # Which measured peak applies: the burst figure for a timed region shorter than a second
    # (the clock has not settled under the power cap), the sustained one for longer regions.
    region_s = total_ms * 1e-3
    short = region_s < 1.0
    frac_burst = fp16_rate_1gpu / peaks["bf16_burst"]
    frac_sustained = None
    if "fp16" in sustained:
        frac_sustained = sustained["fp16"]["value"] / world / peaks["bf16_sustained"]
    elif not short:
        frac_sustained = fp16_rate_1gpu / peaks["bf16_sustained"]
    line = {
        "metric": "fp16_gemm_tflops_n%d" % N, "value": precisions["fp16"]["value"],
        "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {
            "workload": "FP16 GEMM M=N=K=%d, N(0,1) clipped to [-4,4], seed 3, FP32 accumulate and C; "
                        "one step runs the GEMMs of this size for: %s" % (N, ",".join(precs)),
            "l2": "operands + C of every GEMM exceed the 126 MB L2; no flush",
            "replicas": "one independent problem per GPU" if world > 1 else "single GPU",
        },
        "precisions": precisions,
        "roofline": {
            "bound": "tensor", "achieved": fp16_rate_1gpu,
            "peak": peaks["bf16_burst"] if short else peaks["bf16_sustained"],
            "unit": "TFLOP/s",
            "frac": frac_burst if short else fp16_rate_1gpu / peaks["bf16_sustained"],
            "frac_burst": frac_burst, "frac_sustained": frac_sustained,
            "peak_burst": peaks["bf16_burst"], "peak_sustained": peaks["bf16_sustained"],
            "peak_spec": SPEC_PEAK["fp16"], "frac_of_spec": fp16_rate_1gpu / SPEC_PEAK["fp16"],
            "timed_region_s": region_s,
            "traffic": traffic, "traffic_source": traffic_note,
            "algorithmic_bytes": 2 * N * N * 2 + 4 * N * N,
            "peak_source": "%s cuBLAS bf16 %s figure: the timed region lasted %.3f s (< 1 s: burst, "
                           "else sustained); frac_sustained is the separate >= %.0f s FP16-only "
                           "leg against the sustained figure"
                           % (peaks["source"], "burst" if short else "sustained", region_s,
                              args.sustain_seconds),
            "kernel": "FP16 GEMM kernel N=%d (%s), avg of %d launches"
                      % (N, precisions["fp16"]["config"].split(" kind")[0], args.steps),
        },
        "clocks": clocks,
        "e2e": e2e,
        # INT4: pre-pass + GEMM; or the fused kernel, alone or behind the kernel that makes the
        # int8 image of A, where the library picks that route
        "gpu_launches": args.steps * sum(
            (2 if "a=int8_image" in binding.gemm_query_config(p, N, N, N) else 1)
            if "fused_unpack" in binding.gemm_query_config(p, N, N, N) else KERNEL_LAUNCHES[p]
            for p in precs),
    }
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(N, host["fp16"][0], host["fp16"][1])
    if dist is not None:
        dist.destroy_process_group()
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """Precision x size sweep (the paper's Sec. III-B sizes): one JSON line per cell.
    Each cell: seeded operands resident in HBM; `reps` launches are captured once in a
    CUDA graph and the graph is replayed between two CUDA events, so the number is device
    time and not the host's cost of issuing a call (which exceeds the kernel at N <= 1024;
    it is reported separately as `host_us_per_call`).  Median of 5 replays; an L2 flush
    (256 MB write) precedes each, so the first launch starts cold and, at sizes whose
    operands fit in L2, later ones run warm: the batch mean and a cold single launch are
    both reported."""
    import numpy as np
    import torch
    from paper_2608_10103_b200 import binding, synth
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    peaks = measured_peaks()

    def timed(fn, reps, cold=False):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if cold:   # operand lines the kernels marked "evict last" would outlive the flush
            binding.gemm_debug_reset_l2()
        flush.fill_(1)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    def graph_of(call, reps):
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for _ in range(reps):
                    call(side)
        torch.cuda.current_stream().wait_stream(side)
        return g

    # the box's own CPU rate beside the GPU numbers: the oracle, as it stands, on the full
    # N = 1024 problem of each precision (a fraction of a second each)
    import oracle
    cpu_rate = {}
    for prec in synth.PRECISIONS:
        A, B = synth.make(prec, 1024, 1024, 1024, synth.sweep_seed(prec, 1024))
        t0 = time.perf_counter()
        if prec == "fp16":
            oracle.gemm_fp16(A, B)
        elif prec == "s8":
            oracle.gemm_s8_i64(A, B)
        else:
            oracle.gemm_s4_i64(A, B, 1024)
        cpu_rate[prec] = synth.gemm_ops(1024, 1024, 1024) / (time.perf_counter() - t0) / 1e9
    # MMA-issue-only rate of this machine, per kind, measured once before the sweep
    mma_peak = {}
    for kind in ("fp16", "s8"):
        binding.gemm_mma_peak_probe(kind, 2048)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        pops = binding.gemm_mma_peak_probe(kind, 200000)
        e1.record()
        torch.cuda.synchronize()
        mma_peak[kind] = pops / (e0.elapsed_time(e1) * 1e-3) / 1e12
    mma_peak["s4"] = mma_peak["s8"]

    for prec in synth.PRECISIONS:
        for N in synth.SWEEP_SIZES:
            A, B = synth.make(prec, N, N, N, synth.sweep_seed(prec, N))
            dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
            C = torch.empty((N, N), dtype=torch.float32 if prec == "fp16" else torch.int32,
                            device="cuda")
            call = lambda st: binding.gemm(prec, dA, dB, C, st)
            # device time first (the host-cost loops below are a second of full-power work at
            # N = 8192 and would push the timed replays into the power-capped regime), after a
            # pause, so that every cell starts from the same power state
            torch.cuda.synchronize()
            time.sleep(1.0)
            reps = max(5, min(100, int(20.0 / max(timed(lambda: call(stream), 5), 1e-3))))
            g_many, g_one = graph_of(call, reps), graph_of(call, 1)
            warm = float(np.median([timed(g_many.replay, 1) for _ in range(5)])) / reps
            cold = float(np.median([timed(g_one.replay, 1, cold=True) for _ in range(5)]))
            n_host = 200 if N <= 2048 else 50
            for _ in range(300 if N <= 2048 else 50):   # also lets the host core reach its working clock
                call(stream)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(n_host):
                call(stream)
            host_us = (time.perf_counter() - t0) / n_host * 1e6
            torch.cuda.synchronize()
            # the library's own share of that: the C entry point called with arguments that
            # are already marshalled (what a C or C++ caller pays, plus one ctypes dispatch)
            fn = getattr(binding.lib(), {"fp16": "gemm_fp16", "s8": "gemm_s8", "s4": "gemm_s4"}[prec])
            c_args = (N, N, N, dA.data_ptr(), dB.data_ptr(), C.data_ptr(), int(stream.cuda_stream))
            t0 = time.perf_counter()
            for _ in range(n_host):
                fn(*c_args)
            host_us_c = (time.perf_counter() - t0) / n_host * 1e6
            torch.cuda.synchronize()
            # ... and without that dispatch: the same calls looped and timed inside the library
            host_us_native = min(binding.gemm_debug_host_cost(prec, dA, dB, C, stream, n_host)
                                 for _ in range(3)) * 1e-3
            ops = synth.gemm_ops(N, N, N)
            rate = ops / (warm * 1e-3) / 1e12
            ref = peaks["bf16_burst"] * (1 if prec == "fp16" else 2)
            print(json.dumps({
                "sweep": True, "precision": prec, "N": N, "seed": synth.sweep_seed(prec, N),
                "ms": warm, "reps": reps, "ms_cold_single_launch": cold,
                "host_us_per_call": host_us, "host_us_c_abi": host_us_c,
                "host_us_in_library": host_us_native,
                "value": rate, "unit": UNIT[prec], "frac_of_spec_peak": rate / SPEC_PEAK[prec],
                "frac_of_cublas_bf16_burst_scaled": rate / ref,
                "frac_of_mma_only_peak": rate / mma_peak[prec], "mma_only_peak": mma_peak[prec],
                "cpu_oracle_gops_n1024": cpu_rate[prec], "cpu_cores": oracle.threads(),
                "config": binding.gemm_query_config(prec, N, N, N)}), flush=True)
    if binding.gemm_last_device_status() != 0:
        raise SystemExit("bench.py: a kernel reported a barrier timeout")


def run_few_rows(args):
    """Problems with few rows (the shapes of LLM decoding, which the paper lists as the use it
    has in mind but does not measure, Sec. VI): bound by the bytes of B, so the roofline is HBM.
    One JSON line per (shape, precision, route): CUDA-graph replay of 12 calls after an L2
    flush (256 MB write), median of 7, every launch of a call included (split-K's zeroing of C,
    the INT4 pre-pass).  The calls rotate through as many copies of B as it takes to exceed
    twice the L2 capacity, so every call reads its B from HBM.  `achieved` = algorithmic bytes
    (A, B as stored, C once) / time."""
    import numpy as np
    import torch
    from paper_2608_10103_b200 import binding, synth
    torch.cuda.set_device(0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    hbm = measured_peaks()["hbm_gbs"]
    shapes = [(1, 8192, 8192), (8, 8192, 8192), (16, 8192, 8192), (32, 8192, 8192), (64, 8192, 8192),
              (16, 4096, 16384),
              (8, 4096, 4096), (128, 16384, 4096), (16, 28672, 8192), (32, 28672, 8192)]
    if args.shape:
        shapes = [tuple(int(x) for x in args.shape.split(","))]
    # The tile kernels load their long operand with L2 priority "evict last", and lines so marked
    # outlive the flush between replays: whatever ran after them found part of a B copy in L2
    # (FP16, M = 1, N = K = 8192, few-rows kernel: 25.8 us before the first tile route, 23.9 us
    # after).  Hence the reset in front of every route below.
    probe = ("read-only probe: a kernel that reads B once and does nothing else", 0, 0, "probe")
    few = ("kernel for a few rows where it exists (up to 32)", 0, 0, "raw", 3)
    routes = {"fp16": [probe, ("selector default", 0, 0, "raw"), few,
                       ("FP16 output, selector default", 0, 0, "out16"),
                       ("tile kernels, operands exchanged", 0, 2, "raw"),
                       ("tile kernels, operands not exchanged", 0, 1, "raw")],
              "s8": [probe, ("selector default", 0, 0, "raw"), few,
                     ("dequantised to FP16, selector default", 0, 0, "out16"),
                     ("tile kernels, operands exchanged", 0, 2, "raw"),
                     ("tile kernels, operands not exchanged", 0, 1, "raw")],
              "s4": [probe, ("selector default", 0, 0, "raw"), few,
                     ("dequantised to FP16, selector default", 0, 0, "out16"),
                     ("tile kernels: expanded in the kernel, operands exchanged", 2, 2, "raw"),
                     ("tile kernels: expanded in the kernel, both operands packed on CTA-pair tiles", 5, 0, "raw"),
                     ("pre-pass + INT8 GEMM", 1, 1, "raw")]}
    for M, N, K in shapes:
        for prec in [q for q in synth.PRECISIONS if q in args.precisions.split(",")]:
            A, B = synth.make(prec, M, N, K, seed=M + N)
            dA = torch.from_numpy(A).cuda()
            copies = max(2, -(-(256 << 20) // B.nbytes))
            dBs = [torch.from_numpy(B).cuda() for _ in range(copies)]
            dB = dBs[0]
            C32 = torch.empty((M, N), dtype=torch.float32 if prec == "fp16" else torch.int32,
                              device="cuda")
            C16 = torch.empty((M, N), dtype=torch.float16, device="cuda")
            rs = torch.rand(M, device="cuda") + 0.5
            cs = torch.rand(N, device="cuda") + 0.5

            def call(mode, b, stream=None):
                if mode == "probe":
                    binding.gemm_debug_read_probe(b, stream=stream)
                elif mode == "raw":
                    binding.gemm(prec, dA, b, C32, stream=stream)
                elif prec == "fp16":
                    binding.gemm_fp16_f16out(dA, b, C16, stream=stream)
                elif prec == "s8":
                    binding.gemm_s8_dequant(dA, b, rs, cs, C16, torch.float16, stream=stream)
                else:
                    binding.gemm_s4_dequant(dA, b, rs, cs, C16, torch.float16, stream=stream)

            # the operands were just made on the host: bring the GPU out of idle before the first
            # route is timed
            t_warm = time.time()
            while time.time() - t_warm < 0.3:
                for _ in range(50):
                    call("raw", dB)
                torch.cuda.synchronize()
            for name, scheme, swap, mode, *rest in routes[prec]:
                algo_bytes = A.nbytes + B.nbytes + M * N * (4 if mode == "raw" else 2)
                if mode == "probe":
                    algo_bytes = B.nbytes
                # every route starts alike: the "evict last" lines the route before left in L2
                # go back to normal status, so that the flush removes them
                binding.gemm_debug_reset_l2()
                binding.gemm_set_s4_scheme(scheme)
                binding.gemm_set_swap_ab(swap)
                binding.gemm_set_kernel_family(rest[0] if rest else 0)
                for _ in range(3):
                    call(mode, dB)
                torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    with torch.cuda.graph(g, stream=side):
                        for i in range(12):
                            call(mode, dBs[i % copies], side)
                torch.cuda.current_stream().wait_stream(side)
                ts = []
                for _ in range(7):
                    flush.fill_(1)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    g.replay()
                    e1.record()
                    torch.cuda.synchronize()
                    ts.append(e0.elapsed_time(e1) / 12)
                us = float(np.median(ts)) * 1e3
                gbs = algo_bytes / us / 1e3
                print(json.dumps({
                    "few_rows": True, "M": M, "N": N, "K": K, "precision": prec, "route": name,
                    "us": us, "value": synth.gemm_ops(M, N, K) / us / 1e6, "unit": UNIT[prec],
                    "roofline": {"bound": "hbm", "achieved": gbs, "peak": hbm, "unit": "GB/s",
                                 "frac": gbs / hbm, "traffic": None},
                    "algorithmic_bytes": algo_bytes, "b_copies_rotated": copies,
                    "config": binding.gemm_query_config(prec, M, N, K) if mode == "raw" else None}),
                    flush=True)
    binding.gemm_set_s4_scheme(0)
    binding.gemm_set_swap_ab(0)
    binding.gemm_set_kernel_family(0)
    if binding.gemm_last_device_status() != 0:
        raise SystemExit("bench.py: a kernel reported a barrier timeout")


def run_selector_check(args):
    """The selector's automatic choice against forced tile shapes and split-K factors: one JSON
    line per (shape, precision) with the automatic time, the best forced time and configuration,
    and the regret = automatic / best - 1.  CUDA-graph replay of 20 calls, median of 3, operands
    seeded and resident (square and rectangular shapes between 256 and 4096; the few-row shapes
    have a mode of their own)."""
    import statistics
    import torch
    from paper_2608_10103_b200 import binding, synth
    torch.cuda.set_device(0)
    forced = [(256, 0, 2, 1), (128, 0, 2, 1), (64, 0, 2, 1), (256, 0, 1, 1), (128, 0, 1, 1),
              (64, 0, 1, 1), (32, 0, 1, 1), (256, 0, 2, 2), (128, 0, 2, 2), (256, 0, 1, 2),
              (128, 0, 1, 2), (64, 0, 1, 2), (256, 0, 2, 3), (128, 0, 1, 4), (64, 0, 1, 4), (32, 0, 1, 8)]
    shapes = [(n, n, n) for n in (512, 768, 1024, 1280, 1536, 1792, 2048, 2304, 2560, 2816, 3072,
                                  3584, 4096)]
    shapes += [(512, 8192, 4096), (1024, 4096, 8192), (2048, 8192, 2048), (4096, 1024, 4096),
               (2304, 2304, 8192), (2560, 2560, 1024), (1792, 3584, 4096), (3000, 3000, 1024),
               (640, 1280, 2560), (384, 768, 4096), (512, 512, 8192), (768, 3072, 768)]
    if args.shape:
        shapes = [tuple(int(x) for x in args.shape.split(","))]

    def timed(call, reps=20):
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for _ in range(reps):
                call()
        g.replay()
        torch.cuda.synchronize()
        out = []
        for _ in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1) * 1e3 / reps)
        return statistics.median(out)

    for M, N, K in shapes:
        for prec in [q for q in ("fp16", "s8") if q in args.precisions.split(",")]:
            A, B = synth.make(prec, M, N, K, seed=M + N + K)
            dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
            C = torch.empty((M, N), dtype=torch.float32 if prec == "fp16" else torch.int32, device="cuda")
            binding.gemm_set_config_override(0, 0, 0, 0)
            auto_us = timed(lambda: binding.gemm(prec, dA, dB, C))
            chosen = binding.gemm_query_config(prec, M, N, K)
            best_us, best_cfg = None, None
            for cfg in forced:
                binding.gemm_set_config_override(*cfg)
                try:
                    us = timed(lambda: binding.gemm(prec, dA, dB, C))
                except binding.GemmError:
                    continue
                if best_us is None or us < best_us:
                    best_us, best_cfg = us, cfg
            binding.gemm_set_config_override(0, 0, 0, 0)
            print(json.dumps({"selector_check": True, "M": M, "N": N, "K": K, "precision": prec,
                              "auto_us": auto_us, "chosen": chosen, "best_forced_us": best_us,
                              "best_forced": "BN=%d cta_group=%d split_k=%d" % (best_cfg[0], best_cfg[2], best_cfg[3]),
                              "regret": auto_us / best_us - 1.0}), flush=True)


def run_ablation(args):
    """One-variable-at-a-time ablation at N = args.size (the analogue of the paper's Run 4):
    tile shape, raster band height, L2 policy, and load-only / MMA-only runs, each with
    the per-role cycle accounting of the kernel.  One JSON line per variant."""
    import numpy as np
    import torch
    from paper_2608_10103_b200 import binding, synth
    torch.cuda.set_device(0)
    num_sms = torch.cuda.get_device_properties(0).multi_processor_count
    N = args.size
    ops = synth.gemm_ops(N, N, N)
    data = {"fp16": synth.fp16_normal_clipped(N, N, N, seed=3),
            "s8": synth.s8_uniform(N, N, N, seed=synth.sweep_seed("s8", 8192)),
            "s4": synth.s4_uniform(N, N, N, seed=synth.sweep_seed("s4", 8192))}
    # (name, (BN, band height, CTAs per tile), L2 policy, trace bits, INT4 route, kernel family,
    #  ring depth); family 1 = the 256 x 256 pair tile, 2 = the 512 x 256 tile, 0 = automatic
    def V(name, override=(0, 0, 0), policy=11, trace=1, scheme=0, family=1, stages=0):
        return (name, override, policy, trace, scheme, family, stages)
    variants = [V("baseline (automatic choice)", family=0),
                V("kernel: 256x256 tile per CTA pair, 2 accumulator buffers"),
                V("kernel: 512x256 tile per CTA pair, accumulators fill TMEM", family=2)]
    variants += [V("tile 128x%d, one CTA" % bn, (bn, 0, 1)) for bn in (256, 128, 64, 32)]
    variants += [V("tile 256x%d, CTA pair" % bn, (bn, 0, 2)) for bn in (256, 128, 64)]
    variants += [V("256x256 pair tile, ring depth %d" % st, (256, 0, 2), stages=st) for st in (3, 4, 5, 6)]
    variants += [V("band height %d" % g, (256, g, 2)) for g in (2, 4, 8, 16, 32)]
    variants += [V("512x256 tile, band height %d" % g, (0, g, 0), family=2) for g in (2, 4, 6, 8, 16)]
    variants += [V("L2: no hints, forward K only", policy=4),
                 V("L2: no hints, serpentine K", policy=0),
                 V("L2: keep A, stream B", policy=1),
                 V("L2: keep A and B", policy=2),
                 V("L2: default + 128-byte promotion", policy=27),
                 V("ablate: no MMAs (loads + barriers only)", trace=3),
                 V("ablate: no loads (MMAs + barriers only)", trace=5),
                 V("epilogue waits with nanosleep back-off", trace=9),
                 V("epilogue: direct register -> global stores", trace=33),
                 V("epilogue: 16x256b TMEM loads, sector-complete direct stores (no staging)", trace=65),
                 V("512x256 tile, ablate: no MMAs", trace=3, family=2),
                 V("512x256 tile, ablate: no loads", trace=5, family=2)]
    # INT4: how the nibbles reach the int8 tensor-core path (the traced launch is the GEMM; a
    # separate pre-pass launch is inside the timed loop but not in the cycle accounting)
    s4_variants = [V("INT4 route 0: pre-pass launch to int8 + INT8 GEMM", scheme=1, family=0),
                   V("INT4 route 0': pre-pass inside the INT8 GEMM kernel, ahead of its tiles", scheme=4, family=0),
                   V("INT4 route 1: nibbles expanded in shared memory inside the GEMM kernel", scheme=5),
                   V("INT4 route 1': B expanded inside the kernel, A as an int8 image made in front "
                     "(the automatic choice at this size)", scheme=0, family=0),
                   V("INT4 route 1, ablate: no MMAs", trace=3, scheme=5),
                   V("INT4 route 1, ablate: no operand loads", trace=5, scheme=5)]
    for prec in [q for q in ("fp16", "s8", "s4") if q in args.precisions.split(",")]:
        dA, dB = (torch.from_numpy(x).cuda() for x in data[prec])
        C = torch.empty((N, N), dtype=torch.float32 if prec == "fp16" else torch.int32,
                        device="cuda")
        flop_per_clk = 8192 if prec == "fp16" else 16384
        for v in (s4_variants if prec == "s4" else variants):
            name, override, policy, trace, scheme, family, stages = v
            binding.gemm_set_s4_scheme(scheme)
            binding.gemm_set_kernel_family(family)
            binding.gemm_set_stages_override(stages)
            binding.gemm_set_config_override(*override)
            binding.gemm_set_l2_policy(policy)
            binding.gemm_trace_enable(trace)
            cfg = binding.gemm_query_config(prec, N, N, N)
            for _ in range(3):
                binding.gemm(prec, dA, dB, C)
            torch.cuda.synchronize()
            time.sleep(1.5)        # let the power state settle: every variant starts alike
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                binding.gemm(prec, dA, dB, C)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            tr = binding.gemm_trace_read(num_sms)
            a = {k: np.array([t[k] for t in tr], dtype=np.float64) for k in binding.TRACE_FIELDS}
            lead = a["mma_issue"] > 0
            kb_total = a["tiles"].mean() * (N * (2 if prec == "fp16" else 1) // 128)
            unpack = {}
            if a["unpack_busy"].max() > 0:
                unpack = {"unpack_cycles_per_kblock": {
                    k: float(a[f].mean() / kb_total) for k, f in (
                        ("wait_packed_operands", "unpack_wait_packed"),
                        ("wait_free_int8_slot", "unpack_wait_slot"), ("expanding", "unpack_busy"))}}
            cyc = float(a["cycles"].max())
            print(json.dumps({
                "ablation": name, "precision": prec, "N": N, "config": cfg,
                "ms": ms, "value": ops / (ms * 1e-3) / 1e12, "unit": UNIT[prec],
                "sm_cycles": cyc, "pipe_utilisation": ops / (num_sms * flop_per_clk) / cyc,
                "sm_mhz_during_kernel": float(np.median(a["cycles"] / a["nanos"] * 1e3)),
                "cycles_per_kblock": {
                    "mma_wait_operands": float(a["mma_wait_operands"][lead].mean() / kb_total),
                    "mma_issue": float(a["mma_issue"][lead].mean() / kb_total),
                    "mma_commit": float(a["mma_commit"][lead].mean() / kb_total),
                    "mma_wait_accumulators": float((a["mma_wait_accumulator"][lead].mean() +
                                                    a["mma_wait_accumulator1"][lead].mean()) / kb_total),
                    "producer_wait": float(a["producer_wait"].mean() / kb_total),
                    "producer_issue": float(a["producer_issue"].mean() / kb_total)},
                "epilogue_busy_frac": float(a["epilogue_busy"].mean() / a["cycles"].mean()),
                "result_valid": trace in (1, 9, 33, 65), **unpack}), flush=True)
    binding.gemm_set_s4_scheme(0)
    binding.gemm_set_kernel_family(0)
    binding.gemm_set_stages_override(0)
    binding.gemm_set_config_override(0, 0, 0)
    binding.gemm_set_l2_policy(11)
    binding.gemm_trace_enable(0)
    if binding.gemm_last_device_status() != 0:
        raise SystemExit("bench.py: a kernel reported a barrier timeout")


def run_library_compare(args):
    """Measurement only (no library kernel is on the product path): this library against the
    vendor GEMM that PyTorch calls (cuBLAS / cuBLASLt) on the same box, same operand values,
    at --size: alternating loops of >= --sustain-seconds each, after a 2 s pause, with the SM
    clock and board power NVML saw in the second half of the loop and the energy per GEMM
    (settled power x time per GEMM).  On a power-capped part time per GEMM is energy per GEMM
    divided by the cap, so energy is the figure to compare.  A short leg (20 launches after the
    pause: the burst regime) follows for FP16.  One JSON line per leg."""
    import torch
    from paper_2608_10103_b200 import binding, synth
    torch.cuda.set_device(0)
    N = args.size
    A, B = synth.fp16_normal_clipped(N, N, N, seed=3)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    C32 = torch.empty((N, N), dtype=torch.float32, device="cuda")
    C16 = torch.empty((N, N), dtype=torch.float16, device="cuda")
    bA, bB = dA.to(torch.bfloat16), dB.to(torch.bfloat16)
    Cb = torch.empty((N, N), dtype=torch.bfloat16, device="cuda")
    A8, B8 = synth.s8_uniform(N, N, N, seed=19)
    dA8, dB8 = torch.from_numpy(A8).cuda(), torch.from_numpy(B8).cuda()
    Ci = torch.empty((N, N), dtype=torch.int32, device="cuda")
    ops = synth.gemm_ops(N, N, N)
    index = physical_gpu_index(0)

    def leg(name, impl, fn, seconds, unit):
        # L2 lines this library's kernels marked "evict last" would stay through the other
        # implementation's whole leg (ordinary traffic does not displace them)
        binding.gemm_debug_reset_l2()
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(5):
            fn()
        e1.record()
        torch.cuda.synchronize()
        n = 20 if seconds <= 0 else int(seconds * 1e3 / (e0.elapsed_time(e1) / 5) * 1.15) + 1
        time.sleep(2.0)
        sampler = ClockSampler(index)
        sampler.start()
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        clocks = sampler.stop()
        ms = e0.elapsed_time(e1) / n
        pw = clocks.get("power_w_settled")
        print(json.dumps({
            "library_compare": True, "leg": name, "impl": impl, "N": N, "launches": n,
            "seconds": ms * n * 1e-3, "ms": ms, "value": ops / (ms * 1e-3) / 1e12, "unit": unit,
            "sm_mhz_settled": clocks.get("sm_mhz_settled"), "power_w_settled": pw,
            "joule_per_gemm": pw * ms * 1e-3 if pw else None, "reasons": clocks.get("reasons")}),
            flush=True)

    S = args.sustain_seconds
    dBt, bBt, dB8t = dB.t(), bB.t(), dB8.t()
    legs = [
        ("fp16 in, fp32 out", "this library", lambda: binding.gemm_fp16(dA, dB, C32), "TFLOP/s"),
        ("fp16 in, fp16 out", "this library", lambda: binding.gemm_fp16_f16out(dA, dB, C16), "TFLOP/s"),
        ("fp16 in, fp16 out", "torch.matmul", lambda: torch.matmul(dA, dBt, out=C16), "TFLOP/s"),
        ("bf16 in, bf16 out (same values)", "torch.matmul", lambda: torch.matmul(bA, bBt, out=Cb), "TFLOP/s"),
        ("int8 in, int32 out", "this library", lambda: binding.gemm_s8(dA8, dB8, Ci), "TOP/s"),
        ("int8 in, int32 out", "torch._int_mm", lambda: torch._int_mm(dA8, dB8t, out=Ci), "TOP/s"),
    ]
    for rnd in range(2):  # twice round, so that a drift of the box shows
        for name, impl, fn, unit in legs:
            leg(name, impl, fn, S, unit)
    for name, impl, fn, unit in legs[:4]:
        leg(name + " (20 launches)", impl, fn, 0, unit)
    if binding.gemm_last_device_status() != 0:
        raise SystemExit("bench.py: a kernel reported a barrier timeout")


def run_capture(args):
    """Workload for profiler captures (the summaries under profiles/ name the full command): the
    FP16 GEMM at --size (seed 3) on both kernel families and a few raster band heights, two
    launches each, inside a cudaProfilerStart/Stop range, so that `ncu --profile-from-start off`
    sees exactly these launches.  Prints which configuration each pair of launches ran."""
    import torch
    from paper_2608_10103_b200 import binding, synth
    torch.cuda.set_device(0)
    N = args.size
    A, B = synth.fp16_normal_clipped(N, N, N, seed=3)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    C = torch.empty((N, N), dtype=torch.float32, device="cuda")
    cases = [("automatic", 0, 0), ("256x256 pair tile", 1, 0), ("512x256 tile, band 4", 2, 4),
             ("512x256 tile, band 5", 2, 5), ("512x256 tile, band 6", 2, 6), ("512x256 tile, band 8", 2, 8)]

    def setup(fam, g):
        binding.gemm_set_kernel_family(fam)
        binding.gemm_set_config_override(0, g, 0, 0)

    for _, fam, g in cases:
        setup(fam, g)
        binding.gemm_fp16(dA, dB, C)
    torch.cuda.synchronize()
    torch.cuda.profiler.start()
    for name, fam, g in cases:
        setup(fam, g)
        for _ in range(2):
            binding.gemm_fp16(dA, dB, C)
        print(json.dumps({"capture": name, "config": binding.gemm_query_config("fp16", N, N, N)}),
              flush=True)
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    setup(0, 0)
    if binding.gemm_last_device_status() != 0:
        raise SystemExit("bench.py: a kernel reported a barrier timeout")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--size", type=int, default=8192)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--sustain-seconds", type=float, default=2.0,
                    help="length of the per-precision back-to-back legs (0 = skip them)")
    ap.add_argument("--ref-rows", type=int, default=32)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-peak-probe", action="store_true")
    ap.add_argument("--few-rows", action="store_true",
                    help="few-row (LLM decoding) shapes, every precision and INT4 route, against the "
                         "HBM roofline (1 GPU)")
    ap.add_argument("--shape", default="", help="--few-rows: only this M,N,K")
    ap.add_argument("--ablation", action="store_true",
                    help="tile / raster / L2 / load-vs-MMA ablation with cycle accounting (1 GPU)")
    ap.add_argument("--selector-check", action="store_true",
                    help="automatic tile / split-K choice against forced ones, one JSON line per shape")
    ap.add_argument("--capture", action="store_true",
                    help="profiler workload: FP16 GEMM at --size, both kernel families and band "
                         "heights, inside a profiler range (1 GPU)")
    ap.add_argument("--library-compare", action="store_true",
                    help="measurement only: this library against torch.matmul / torch._int_mm "
                         "(the vendor GEMM) in alternating sustained loops with power and clock")
    ap.add_argument("--sweep", action="store_true",
                    help="precision x size sweep N=512..8192, one JSON line per cell (1 GPU)")
    ap.add_argument("--precisions", default="fp16,s8,s4")
    ap.add_argument("--l2-policy", type=int, default=-1, help="ablation: gemm_set_l2_policy")
    ap.add_argument("--family", type=int, default=0,
                    help="ablation: gemm_set_kernel_family (1 = 256x256 pair tile, 2 = 512x256)")
    ap.add_argument("--override", default="",
                    help="ablation: BN,GROUP_M,CTA_GROUP passed to gemm_set_config_override")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.capture:
        if rank == 0:
            run_capture(args)
    elif args.library_compare:
        if rank == 0:
            run_library_compare(args)
    elif args.selector_check:
        if rank == 0:
            run_selector_check(args)
    elif args.ablation:
        if rank == 0:
            run_ablation(args)
    elif args.few_rows:
        if rank == 0:
            run_few_rows(args)
    elif args.sweep:
        if rank == 0:
            run_sweep(args)
    elif args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world)


if __name__ == "__main__":
    main()
