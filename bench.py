#!/usr/bin/env python
"""Benchmark of the tensor-contraction hot path.

A step is one execution of the fp64 coupled-cluster ladder contraction
R[a,b,i,j] += sum_{c,d} V[a,b,c,d] T[c,d,i,j]  (a,b,c,d = 128; i,j = 32; 0.55 TFLOP per step)
through the C-ABI library.  `value` is GFLOP/s with the operands resident in HBM; `e2e` is the
same metric through btc_execute_host with pinned HOST buffers (copies inside the timed region).
The same line carries `peaks` (what this device's pipes and memory sustain, measured at the start
of the run with the library's micro-benchmarks) and `per_config`: every other workload timed in the
same process (small ones also as a replayed CUDA graph and over many buffer sets in one batched
call), each with its rate and roofline fraction.  `--workload NAME` times one workload alone.
`--impl reference` times the CPU oracle on a bounded sample of the headline workload instead.
Prints one JSON line.
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
sys.path.insert(0, ROOT)

WORKLOAD = "cfg2_f64_ccsd_ladder"
METRIC = "contraction GFLOP/s"
# Peaks from unit counts and clocks (148 SMs, 1.965 GHz): 64 FP64 FMA/clk/SM on the FP64 tensor
# (DMMA) pipe, 128 FP32 FMA/clk/SM on the FMA pipe.  Register-resident loops on this pool
# measured 37.1 TFLOP/s (DMMA) and 72.3 TFLOP/s (FFMA).
FP64_PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def measured_hbm_gbs():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except (OSError, KeyError, ValueError):
        return 6650.0, "fallback"


def measured_tf32_tflops():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"]) * 1.1 / 2.25, "measured"
    except (OSError, KeyError, ValueError):
        return 1590.0 * 1.1 / 2.25, "fallback"


PEAKS = {}    # filled by measure_peaks(): this device, this run


def measure_peaks(api, handle, torch):
    """The library's micro-benchmarks (btc_measure_peak): arithmetic pipes in TFLOP/s, memory in GB/s."""
    st = torch.cuda.current_stream().cuda_stream
    buf = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")      # 1 GiB: eight times the L2
    out = {}
    for name, which in (("fp64_fma_tflops", api.PEAK_FP64_FMA), ("fp64_mma_m16n8k16_tflops", api.PEAK_FP64_MMA_K16),
                        ("fp64_mma_m8n8k4_tflops", api.PEAK_FP64_MMA_K4), ("fp32_fma_tflops", api.PEAK_FP32_FMA),
                        ("tf32_mma_sync_tflops", api.PEAK_TF32_MMA_SYNC)):
        out[name] = api.measure_peak(handle, which, st, repeats=2) / 1e12
    for name, which in (("hbm_read_gbs", api.PEAK_HBM_READ), ("hbm_write_gbs", api.PEAK_HBM_WRITE), ("hbm_copy_gbs", api.PEAK_HBM_COPY)):
        out[name] = api.measure_peak(handle, which, st, buf.data_ptr(), buf.numel(), repeats=5) / 1e9
    del buf
    torch.cuda.empty_cache()
    out["how"] = ("btc_measure_peak: register-resident FMA / MMA loops (8 CTAs of 256 threads per SM, 4096 iterations); "
                  "one pass of 16-byte accesses over 1 GiB (copy: read + written bytes); CUDA events")
    PEAKS.update(out)
    return out


def roofline_for(w, kernel_ms, variant=-1, units=1):
    """Roofline entry of the dominant kernel for this workload (`units` buffer sets per launch): whichever
    of the arithmetic pipe the kernel runs on and HBM needs longer for the algorithmic work is the bound."""
    flops, nbytes = units * w.flops(), units * w.algorithmic_bytes()
    hbm, src = measured_hbm_gbs()
    t_hbm = nbytes / (hbm * 1e9)
    achieved = flops / (kernel_ms * 1e-3) / 1e12
    gbs = nbytes / (kernel_ms * 1e-3) / 1e9
    f32 = w.dtype in ("f32", "c32")
    umma = f32 and (10 <= variant <= 21 or variant == 23)
    if variant == 100:
        # at most four contracted indices: FMA pipe of the element type
        kernel, bound, executed = "stream_kernel", "alu", flops
        peak = FP32_PEAK_TFLOPS if f32 else FP64_PEAK_TFLOPS
        peak_measured = PEAKS.get("fp32_fma_tflops" if f32 else "fp64_fma_tflops")
        source = "FMA pipe of the element type (unit count); peak_measured = the register-resident FMA loop of this run"
    elif not f32:
        kernel, bound, executed = "tiled_f64_kernel", "tensor", flops
        peak, peak_measured = FP64_PEAK_TFLOPS, PEAKS.get("fp64_mma_m16n8k16_tflops")
        source = ("FP64 tensor (DMMA) pipe: 148 SMs x 64 FMA/clk x 2 x 1.965 GHz (unit count); peak_measured = the "
                  "register-resident m16n8k16 loop of this run")
    elif umma:
        # tcgen05 3xTF32: three TF32 MMAs per product; TF32 dense peak = measured bf16 burst peak x the
        # nominal TF32 : bf16 ratio (1.1 : 2.25)
        kernel, bound, executed = ("skinny_umma_kernel" if variant == 23 else "tiled_umma_tf32x3_kernel"), "tensor", 3 * flops
        peak, tsrc = measured_tf32_tflops()
        peak_measured = None
        source = f"TF32 dense = bf16 cuBLAS burst peak ({tsrc}) x 1.1/2.25; executed flops = 3 x useful (3xTF32)"
    else:
        kernel = "tiled_tf32x3_kernel" if (w.dtype == "c32" or 6 <= variant <= 9 or variant == 22) else "tiled_f32_kernel"
        bound, executed = "alu", flops
        peak, peak_measured = FP32_PEAK_TFLOPS, PEAKS.get("fp32_fma_tflops")
        source = ("FP32 FMA pipe: 148 SMs x 128 FMA/clk x 2 x 1.965 GHz (unit count); peak_measured = the "
                  "register-resident FFMA loop of this run")
    t_pipe = executed / (peak * 1e12)
    if t_hbm >= t_pipe:
        out = {"bound": "hbm", "achieved": gbs, "peak": hbm, "unit": "GB/s", "frac": gbs / hbm, "traffic": None,
               "peak_source": f"STREAM-style copy, {src}; HBM needs {t_hbm * 1e3:.4f} ms for the algorithmic bytes, "
                              f"the arithmetic pipe {t_pipe * 1e3:.4f} ms",
               "peak_measured": PEAKS.get("hbm_copy_gbs"), "useful_tflops": achieved}
    else:
        ach = executed / (kernel_ms * 1e-3) / 1e12
        out = {"bound": bound, "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak, "traffic": None,
               "peak_source": source, "peak_measured": peak_measured, "useful_tflops": achieved}
        if peak_measured:
            out["frac_of_measured"] = ach / peak_measured
        if bound == "alu":
            tf32_sync = PEAKS.get("tf32_mma_sync_tflops") or 277.0
            out["note"] = ("this kernel computes each product as three TF32 tensor-core MMAs (mma.sync m16n8k8, measured "
                           f"{tf32_sync:.0f} TFLOP/s in this run): it executes {3 * achieved:.1f} tensor TFLOP/s = "
                           f"{3 * achieved / tf32_sync:.2f} of that peak")
    # DRAM bytes of one launch from a one-pass ncu capture of this kernel on this workload
    # (dram__bytes_read.sum + dram__bytes_write.sum = 3.28 GB + 0.124 GB)
    if w.name == "cfg2_f64_ccsd_ladder" and variant == 2 and units == 1:
        out["traffic"] = 3.40e9
    out["kernel"], out["kernel_ms"] = kernel, kernel_ms
    return out


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", help="one workload name, or 'all': the headline workload plus per_config")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--results-from", default="", help="write RESULTS.md from a file holding a JSON line of the default run (no GPU needed)")
    ap.add_argument("--results-out", default=os.path.join(os.path.dirname(os.path.abspath(__file__)), "RESULTS.md"))
    ap.add_argument("--variant", type=int, default=-1, help="force a tile variant (tuning runs)")
    ap.add_argument("--batched", type=int, default=0,
                    help="one step = one btc_execute_batched call over this many distinct (A, B, D) buffer sets")
    return ap.parse_args()


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


class OracleSampler:
    """Times the CPU oracle (element-precision accumulators, as it stands) on randomly chosen
    elements of D of the workload."""

    def __init__(self, w):
        import numpy as np
        import oracle
        from paper_2601_07827_b200 import inputs
        self.oracle, self.w = oracle, w
        A, B, C, D = inputs.make_workload_tensors(w)
        self.keep = (A, B, C, D)
        h, m, n, _ = w.groups()
        self.total = h * m * n
        self.flops_per_elem = w.flops() / self.total
        self.rng = np.random.default_rng(12345)
        self.args = (A.numpy(), w.labelsA, B.numpy(), w.labelsB, C.numpy() if C is not None else None,
                     w.labelsD, D.numpy(), w.labelsD, w.alpha, w.beta)
        self.kw = dict(conjA=w.conjA, conjB=w.conjB, conjC=w.conjC, native_acc=True, with_scale=False)

    def run(self, count):
        """(GFLOP/s, seconds) for `count` random elements."""
        sample = self.rng.integers(0, self.total, size=count)
        t0 = time.perf_counter()
        self.oracle.contract(*self.args, want=sample, **self.kw)
        dt = time.perf_counter() - t0
        return count * self.flops_per_elem / dt / 1e9, dt

    def count_for(self, seconds):
        probe = int(min(self.total, 2048))
        _, dt = self.run(probe)
        return int(min(self.total, max(probe, probe * seconds / max(dt, 1e-6))))


def cpu_baseline(w, seconds=15.0):
    s = OracleSampler(w)
    count = s.count_for(seconds)
    g, dt = s.run(count)
    return {"value": g, "unit": "GFLOP/s", "cores": s.oracle.num_threads(), "kind": "oracle",
            "sample": f"{count} of {s.total} elements of D chosen at random ({dt:.1f} s)"}


def run_reference(args, w):
    """The oracle as it stands on the host cores; each step is a bounded sample of the workload."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    s = OracleSampler(w)
    per_step = max(1.0, min(10.0, 120.0 / max(1, args.steps + args.warmup)))
    count = s.count_for(per_step)
    vals, times = [], []
    for i in range(args.warmup + args.steps):
        g, dt = s.run(count)
        if i >= args.warmup:
            vals.append(g)
            times.append(dt)
    value = statistics.mean(vals)
    desc = f"{count} of {s.total} elements of D chosen at random per step"
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "groups_batch_M_N_K": list(w.groups()), "step": desc},
        "cpu_baseline": {"value": value, "unit": "GFLOP/s", "cores": s.oracle.num_threads(), "kind": "oracle",
                         "sample": desc},
        "e2e": {"value": value, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(out))


def max_over_ranks(ms: float, device="cpu") -> float:
    """Largest per-rank time; a no-op outside torch.distributed (single process)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms: float) -> float:
    """Independent replicas (weak scaling): all ranks' units over the slowest rank's time."""
    return world * units_per_rank / (ms * 1e-3)


def small_problem_latency(step, stream, torch):
    """For workloads with microseconds of work: median single-call latency, back-to-back plain
    launches, and replay of a CUDA graph holding 100 calls (all in microseconds per call)."""
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    with torch.cuda.stream(side):
        run = lambda: step(side)
        for _ in range(5):
            run()
        side.synchronize()
        single = []
        for _ in range(200):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(side); run(); b.record(side); side.synchronize()
            single.append(a.elapsed_time(b) * 1e3)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        for _ in range(1000):
            run()
        e1.record(side); side.synchronize()
        plain = e0.elapsed_time(e1)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for _ in range(100):
                run()
        g.replay(); side.synchronize()
        e0.record(side)
        for _ in range(10):
            g.replay()
        e1.record(side); side.synchronize()
        graph = e0.elapsed_time(e1)
    stream.wait_stream(side)
    return {"single_call_us_median": statistics.median(single), "back_to_back_us": plain,
            "graph_replay_us": graph, "calls": {"single": 200, "back_to_back": 1000, "graph": 1000}}


def ew_kernel_name(code):
    return {1: "elementwise_direct_kernel", 2: "elementwise_transposing_kernel", 3: "elementwise_vector_kernel"}.get(code, "?")


def measure_elementwise(args, w, torch, api, inputs, handle, sample_clocks=True):
    """One step = one C := alpha op(A) + beta op(B) over device-resident tensors; GB/s of algorithmic
    bytes against the measured HBM bandwidth."""
    A, B, C = inputs.make_elementwise_tensors(w, device="cuda")
    dt = api.dtype_code(C.dtype)
    tA = api.TensorInfo(handle, dt, A.extents, A.strides)
    tC = api.TensorInfo(handle, dt, C.extents, C.strides)
    tB = api.TensorInfo(handle, dt, B.extents, B.strides) if B is not None else None
    op = api.Elementwise(handle, tA, w.labelsA, tB, tC, w.labelsC, w.alpha, w.beta)
    stream = torch.cuda.current_stream()
    pB = B.data_ptr() if B is not None else 0

    def step():
        op.execute(stream.cuda_stream, A.data_ptr(), pB, C.data_ptr())
    for _ in range(max(1, args.warmup)):
        step()
    sampler = ClockSampler(0) if sample_clocks else None
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    ms = e0.elapsed_time(e1) / args.steps
    gbs = w.algorithmic_bytes() / (ms * 1e-3) / 1e9
    peak, src = measured_hbm_gbs()
    kernel = op.kernel_ran
    return {
        "metric": "elementwise GB/s", "value": gbs, "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "labels": [w.labelsA, w.labelsC], "kernel": kernel, "num_modes": list(op.num_modes),
                   "l2": "tensors exceed L2"},
        "clocks": clocks, "gpu_launches": args.steps,
        "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak, "traffic": None,
                     "peak_source": f"STREAM-style copy, {src}", "peak_measured": PEAKS.get("hbm_copy_gbs"),
                     "kernel": ew_kernel_name(kernel), "kernel_ms": ms}}


def run_elementwise(args, w):
    """`--workload ew...` alone."""
    import torch
    from paper_2601_07827_b200 import build, inputs
    build.build()
    from paper_2601_07827_b200 import api
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    print(json.dumps(measure_elementwise(args, w, torch, api, inputs, api.Handle())))


def measure_batched(args, w, n, torch, api, inputs, handle, sample_clocks=True):
    """N distinct buffer sets of the workload (more than L2 together for the small workloads), one
    pointer-array call per step: the device-side rate of a small contraction without the per-call
    launch latency."""
    A, B, C, D = inputs.make_workload_tensors(w, device="cuda")
    rep = lambda t: torch.stack([t.buffer] * n).contiguous()
    pA, pB, pD = rep(A), rep(B), rep(D)
    pC = rep(C) if (C is not None and not w.in_place) else None
    dt = api.dtype_code(D.dtype)
    tA = api.TensorInfo(handle, dt, A.extents, A.strides)
    tB = api.TensorInfo(handle, dt, B.extents, B.strides)
    tD = api.TensorInfo(handle, dt, D.extents, D.strides)
    op = api.Contraction(handle, tA, w.labelsA, tB, w.labelsB, tD if C is not None else None, w.labelsD, tD, w.labelsD,
                         w.alpha, w.beta, w.conjA, w.conjB, w.conjC)
    op.set_attr(api.ATTR_BATCH_HINT, n)
    if args.variant >= 0:
        op.set_attr(api.ATTR_VARIANT, args.variant)
    item = D.buffer.element_size()
    ptrs = lambda pool, t: [pool.data_ptr() + (i * t.buffer.numel() + t.origin) * item for i in range(n)]
    lA, lB, lD = ptrs(pA, A), ptrs(pB, B), ptrs(pD, D)
    lC = None if C is None else (lD if w.in_place else ptrs(pC, C))
    ws_bytes = op.batched_workspace_size(n)
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    step = lambda: op.execute_batched(stream.cuda_stream, lA, lB, lC, lD, workspace=ws.data_ptr(), workspace_bytes=ws_bytes)
    for _ in range(max(1, args.warmup)):
        step()
    sampler = ClockSampler(0) if sample_clocks else None
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    ms = e0.elapsed_time(e1) / args.steps
    total_bytes = n * w.algorithmic_bytes()
    roof = roofline_for(w, ms, op.variant, units=n)
    return {
        "metric": METRIC, "value": n * w.flops() / (ms * 1e-3) / 1e9, "unit": "GFLOP/s", "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "batched_entries": n, "us_per_entry": 1e3 * ms / n, "kernel": op.kernel,
                   "tile": list(op.tile), "variant": op.variant, "split_k": op.split_k,
                   "l2": "buffer sets exceed L2" if total_bytes > 126e6 else "buffer sets fit in L2"},
        "clocks": clocks, "gpu_launches": args.steps * (2 if op.split_k > 1 else 1),
        "roofline": roof}


def run_batched(args, w):
    """`--batched N` alone."""
    import torch
    from paper_2601_07827_b200 import build, inputs
    build.build()
    from paper_2601_07827_b200 import api
    torch.cuda.set_device(0)
    print(json.dumps(measure_batched(args, w, args.batched, torch, api, inputs, api.Handle())))


def measure_single(args, w, torch, api, inputs, handle, latency=False):
    """Device-side time of one execute of a contraction workload (operands resident in HBM)."""
    A, B, C, D = inputs.make_workload_tensors(w, device="cuda")
    dt = api.dtype_code(D.dtype)
    tA = api.TensorInfo(handle, dt, A.extents, A.strides)
    tB = api.TensorInfo(handle, dt, B.extents, B.strides)
    tD = api.TensorInfo(handle, dt, D.extents, D.strides)
    op = api.Contraction(handle, tA, w.labelsA, tB, w.labelsB, tD if C is not None else None, w.labelsD, tD, w.labelsD,
                         w.alpha, w.beta, w.conjA, w.conjB, w.conjC)
    ws_bytes = op.workspace_size()
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    pC = C.data_ptr() if C is not None else 0

    def step(status=False, on=None):
        return op.execute((on or stream).cuda_stream, A.data_ptr(), B.data_ptr(), pC, D.data_ptr(),
                          workspace=ws.data_ptr(), workspace_bytes=ws_bytes, want_status=status)
    st = step(status=True)
    for _ in range(max(1, args.warmup)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    out = {"workload": w.name, "mode": "single execute, back to back", "dtype": w.dtype, "ms": ms,
           "gflops": w.flops() / (ms * 1e-3) / 1e9, "gbs": w.algorithmic_bytes() / (ms * 1e-3) / 1e9,
           "kernel": st["kernel"], "variant": st["variant"], "tile": list(op.tile), "split_k": op.split_k,
           "launches": st["launches"], "groups_batch_M_N_K": list(w.groups()),
           "l2": "inputs exceed L2" if w.algorithmic_bytes() > 126e6 else "operands fit in L2 (L2-resident figure)",
           "roofline": roofline_for(w, ms, st["variant"])}
    if latency:
        lat = small_problem_latency(lambda s_: step(on=s_), stream, torch)
        out["latency"] = lat
        out["mode"] = "per call inside a replayed CUDA graph of 100 calls"
        out["ms"] = lat["graph_replay_us"] * 1e-3
        out["gflops"] = w.flops() / (out["ms"] * 1e-3) / 1e9
        out["gbs"] = w.algorithmic_bytes() / (out["ms"] * 1e-3) / 1e9
        out["roofline"] = roofline_for(w, out["ms"], st["variant"])
    return out


def per_config(args, torch, api, inputs, handle):
    """Every workload other than the headline one, timed in this process; small ones three ways."""
    W, E = inputs.workloads(), inputs.elementwise_workloads()
    sub = argparse.Namespace(**vars(args))
    sub.steps, sub.warmup, sub.variant = 20, 3, -1
    out = []

    def flat(d, mode):        # a full bench line reduced to a per_config entry
        c = d["config"]
        return {"workload": c["workload"], "mode": mode, "dtype": d["dtype"], "ms": d["ms_per_step"],
                "gflops": d["value"] if d["unit"] == "GFLOP/s" else None,
                "gbs": d["roofline"]["achieved"] if d["roofline"]["unit"] == "GB/s" else None,
                "kernel": c.get("kernel"), "variant": c.get("variant"), "tile": c.get("tile"), "split_k": c.get("split_k"),
                "l2": c.get("l2"), "roofline": d["roofline"]}
    plan = [("single", "cfg1_f64_small", True), ("batched", "cfg1_f64_small", 148),
            ("single", "cfg3_f32_batched_permuted", False), ("single", "cfg4_c64_conj", False), ("single", "cfg4c_c32_conj", False),
            ("single", "cfg5_f32_tensor_network", True), ("batched", "cfg5_f32_tensor_network", 64),
            ("single", "cfg5b_f32_tensor_network_rev", True), ("batched", "cfg5b_f32_tensor_network_rev", 64),
            ("single", "cfg6_f64_case4_isolated", False), ("single", "cfg6b_f64_case4_isolated_fast", False), ("single", "cfg7_f32_outer_product", False)] + [("ew", name, None) for name in E]
    for kind, name, arg in plan:
        try:
            if kind == "single":
                out.append(measure_single(sub, W[name], torch, api, inputs, handle, latency=bool(arg)))
            elif kind == "batched":
                out.append(flat(measure_batched(sub, W[name], arg, torch, api, inputs, handle, sample_clocks=False),
                                f"{arg} buffer sets in one batched call"))
            else:
                out.append(flat(measure_elementwise(sub, E[name], torch, api, inputs, handle, sample_clocks=False), "single execute"))
        except Exception as e:      # one failing workload must not lose the line
            out.append({"workload": name, "error": f"{type(e).__name__}: {e}"})
        torch.cuda.empty_cache()
    return out


def write_results(src, dst):
    """RESULTS.md from the JSON line of a default run: every figure in the table is a field of that line."""
    with open(src) as f:
        lines = [l for l in f.read().splitlines() if l.startswith("{")]
    d = json.loads(lines[-1])
    pk, roof, e2e, cpu = d.get("peaks", {}), d["roofline"], d["e2e"], d.get("cpu_baseline") or {}

    def frac(r):
        if not r or r.get("frac") is None:
            return "-"
        names = {"hbm": "HBM copy bandwidth", "tensor": "tensor-pipe peak", "alu": "FMA-pipe peak"}
        return f"{r['frac']:.2f} of {names.get(r['bound'], r['bound'])} ({r['peak']:.4g} {r['unit']})"

    out = []
    out.append("# RESULTS - one B200, CUDA events, operands resident in HBM")
    out.append("")
    out.append(f"Written by `python bench.py --results-from <file>` from the JSON line of one default run (`python bench.py`,")
    out.append(f"{d['steps']} timed steps after {d['warmup']} warm-up steps for the headline workload); nothing here is typed by hand.")
    out.append(f"SM clock while timing: {d['clocks'].get('sm_mhz')} MHz of {d['clocks'].get('sm_max_mhz')}, throttle reasons {d['clocks'].get('reasons')}"
               + (f"; other workloads {d['per_config_clocks'].get('sm_mhz')} MHz, reasons {d['per_config_clocks'].get('reasons')}." if d.get("per_config_clocks") else "."))
    out.append("")
    if pk:
        out.append("Peaks measured in the same run by the library's own micro-kernels (`btc_measure_peak`): "
                   f"FP64 FMA {pk['fp64_fma_tflops']:.1f}, FP64 MMA m16n8k16 {pk['fp64_mma_m16n8k16_tflops']:.1f}, m8n8k4 {pk['fp64_mma_m8n8k4_tflops']:.1f}, "
                   f"FP32 FMA {pk['fp32_fma_tflops']:.1f}, TF32 mma.sync {pk['tf32_mma_sync_tflops']:.0f} TFLOP/s; HBM read {pk['hbm_read_gbs']:.0f}, "
                   f"write {pk['hbm_write_gbs']:.0f}, copy {pk['hbm_copy_gbs']:.0f} GB/s.  The roofline fractions below use the driver-measured copy bandwidth "
                   "and the unit-count pipe peaks named in each row's `roofline.peak_source`.")
        out.append("")
    out.append("| workload | mode | time per call | rate | fraction of the bounding roofline | kernel | launches |")
    out.append("|---|---|---|---|---|---|---|")
    out.append(f"| {d['config']['workload']} (headline) | single execute, back to back | {d['ms_per_step']:.3f} ms | {d['value'] / 1e3:.2f} TFLOP/s | "
               f"{frac(roof)} | {roof.get('kernel')} | {d['gpu_launches'] // d['steps']} |")
    for v in d.get("per_config", []):
        r = v.get("roofline", {})
        ms = v["ms"]
        t = f"{ms:.3f} ms" if ms >= 0.1 else f"{ms * 1e3:.1f} us"
        rate = ", ".join(x for x in (f"{v['gflops'] / 1e3:.2f} TFLOP/s" if v.get("gflops") else "",
                                     f"{v['gbs']:.0f} GB/s" if v.get("gbs") else "") if x)
        out.append(f"| {v['workload']} | {v.get('mode', '')} | {t} | {rate} | {frac(r)} | {r.get('kernel')} | {v.get('launches', '')} |")
    out.append("")
    out.append(f"End to end through `btc_execute_host` (pinned host buffers, copies inside the timed region), headline workload: "
               f"{e2e['value'] / 1e3:.2f} TFLOP/s ({e2e['h2d_bytes_per_step'] / 1e9:.2f} GB in, {e2e['d2h_bytes_per_step'] / 1e9:.2f} GB out per step).")
    if cpu:
        out.append(f"CPU oracle on the same box ({cpu.get('cores')} threads; {cpu.get('sample')}): {cpu.get('value'):.2f} {cpu.get('unit')} - a baseline for context, not a target.")
    out.append("")
    out.append("Every workload passes element-wise parity against the CPU oracle at these sizes (`tests/test_gpu_fullsize.py`, sampled")
    out.append("elements for the large ones) within 1e-12 (64-bit parts) / 1e-5 (32-bit parts) of sum |a||b|.  What bounds each row: DESIGN.md section 7.")
    with open(dst, "w") as f:
        f.write("\n".join(out) + "\n")


def main():
    args = parse()
    if args.results_from:
        write_results(args.results_from, args.results_out)
        return
    from paper_2601_07827_b200 import inputs
    with_per_config = args.workload == "all"
    if with_per_config:
        args.workload = WORKLOAD
    if args.workload in inputs.elementwise_workloads():
        if args.impl == "reference":
            raise SystemExit("the reference arm times the contraction oracle only")
        run_elementwise(args, inputs.elementwise_workloads()[args.workload])
        return
    w = inputs.workloads()[args.workload]
    if args.batched > 0 and args.impl != "reference":
        run_batched(args, w)
        return
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2601_07827_b200 import build
    build.build()
    from paper_2601_07827_b200 import api

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the contraction kernels have no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    handle = api.Handle()
    peaks = measure_peaks(api, handle, torch) if rank == 0 else None
    # ---- operands: every rank holds its own replica of the workload (no exchange on this path)
    A, B, C, D = inputs.make_workload_tensors(w, device="cuda")
    dt = api.dtype_code(D.dtype)
    tA = api.TensorInfo(handle, dt, A.extents, A.strides)
    tB = api.TensorInfo(handle, dt, B.extents, B.strides)
    tD = api.TensorInfo(handle, dt, D.extents, D.strides)
    tC = tD if C is not None else None
    t0 = time.perf_counter()
    op = api.Contraction(handle, tA, w.labelsA, tB, w.labelsB, tC, w.labelsD, tD, w.labelsD, w.alpha, w.beta,
                         w.conjA, w.conjB, w.conjC)
    plan_ms = 1e3 * (time.perf_counter() - t0)
    if args.variant >= 0:
        op.set_attr(api.ATTR_VARIANT, args.variant)
    ws_bytes = op.workspace_size()
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    pC = C.data_ptr() if C is not None else 0

    def step(status=False, on=None):
        return op.execute((on or stream).cuda_stream, A.data_ptr(), B.data_ptr(), pC, D.data_ptr(),
                          workspace=ws.data_ptr(), workspace_bytes=ws_bytes, want_status=status)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    st = step(status=True)
    launches_per_step = st["launches"]
    for _ in range(max(0, args.warmup - 1)):
        step()
    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    ev[0].record(stream)
    for i in range(args.steps):
        step()
        ev[i + 1].record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = ev[0].elapsed_time(ev[-1])
    kernel_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    total_ms = max_over_ranks(total_ms, "cuda")
    ms_per_step = total_ms / args.steps
    flops = w.flops()
    l2_note = ("inputs exceed L2" if w.algorithmic_bytes() > 126e6 else
               "operands fit in L2 and stay there between steps (L2-resident figure)")
    value = whole_job_rate(flops, world, ms_per_step) / 1e9

    # ---- end to end: host buffers (pinned), copies inside the timed region
    hA = inputs.StridedTensor(A.buffer.cpu().pin_memory(), A.extents, A.strides, A.origin)
    hB = inputs.StridedTensor(B.buffer.cpu().pin_memory(), B.extents, B.strides, B.origin)
    hD = inputs.StridedTensor(D.buffer.cpu().pin_memory(), D.extents, D.strides, D.origin)
    hC_ptr = hD.data_ptr() if (C is not None and w.in_place) else (
        0 if C is None else inputs.StridedTensor(C.buffer.cpu().pin_memory(), C.extents, C.strides, C.origin).data_ptr())
    item = A.buffer.element_size()
    h2d = (A.buffer.numel() + B.buffer.numel() + D.buffer.numel()) * item
    if C is not None and not w.in_place:
        h2d += C.buffer.numel() * item
    d2h = D.buffer.numel() * item

    def e2e_step():
        op.execute_host(stream.cuda_stream, hA.data_ptr(), hB.data_ptr(), hC_ptr, hD.data_ptr())
    e2e_value = None
    if args.e2e_steps > 0:   # 0 only for profiler captures of the kernel
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.e2e_steps):
            e2e_step()
        e1.record(stream)
        barrier()
        e2e_ms = max(e0.elapsed_time(e1), 1e3 * (time.perf_counter() - t0)) / args.e2e_steps
        e2e_value = whole_job_rate(flops, world, max_over_ranks(e2e_ms, "cuda")) / 1e9

    if rank == 0:
        kernel_avg_ms = statistics.mean(kernel_ms)
        out = {
            "metric": METRIC, "value": value, "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": w.name, "groups_batch_M_N_K": list(w.groups()), "kernel": op.kernel,
                       "tile": list(op.tile), "variant": op.variant, "split_k": op.split_k, "grid": list(op.grid),
                       "l2": l2_note, "plan_ms": plan_ms,
                       "parallelism": "independent replicas" if world > 1 else "single GPU"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "GFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline_for(w, kernel_avg_ms, op.variant),
            "peaks": peaks,
        }
        if ms_per_step < 0.2 and world == 1:
            # microseconds of work per call: the per-step figure above includes the host's call
            # overhead, so the device-side figures are reported beside it
            lat = small_problem_latency(lambda s_: step(on=s_), stream, torch)
            out["latency"] = lat
            per_call_ms = lat["graph_replay_us"] * 1e-3
            out["roofline"] = roofline_for(w, per_call_ms, op.variant)
            out["roofline"]["timing"] = "per call inside a replayed CUDA graph of 100 calls"
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline(w)
        if with_per_config and world == 1:
            del A, B, C, D, hA, hB, hD, ws
            torch.cuda.empty_cache()
            sampler = ClockSampler(local)
            sampler.start()
            out["per_config"] = per_config(args, torch, api, inputs, handle)
            out["per_config_clocks"] = sampler.stop()
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
