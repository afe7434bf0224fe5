#!/usr/bin/env python
"""Benchmark of the butterfly-rotation + INT4 quantization hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = load the angles (two table-build kernels) + rotate and quantize every row of the
LLaMA-7B-shaped workload (32768 bf16 rows of n = 4096, INT4 codes + fp16 scales).  Prints
one JSON line (rank 0).  The other operations (backward on the 128 x 2048-token learning
batch, inverse, n = 8192 INT2, weight folding) are timed after the K steps and reported
in the same line under "others".
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

METRIC = "butterfly+INT4-quant rows/s at n=4096"
UNIT = "rows/s"
WORKLOAD = "act4096_int4"

# Algorithmic work per row (n = 4096, L = 12): bytes = bf16 row + packed INT4 codes + fp16 scale;
# FP32 issue slots = 2 MUL + 2 FMA per pair (paper's FLOP table: 3 n log2 n flops) + n for the scale.
BYTES_PER_ROW = 4096 * 2 + 4096 // 2 + 2
SLOTS_PER_ROW = 4 * (4096 // 2) * 12 + 4096
# what the kernel executes: two FMAs per pair in stages 0..10 (scaled rotations), 2 MUL + 2 FMA per pair in the last
# stage (which absorbs the element factors), one FMA per element for the scale: n L + 2 n slots
EXECUTED_SLOTS_PER_ROW = 2 * (4096 // 2) * 11 + 4 * (4096 // 2) + 4096
FP32_LANES_PER_SM = 128
# dram bytes (read + write) per row of the forward+quant kernel, from the committed ncu capture of the
# current kernel on this workload; set back to None whenever that kernel changes.
NCU_TRAFFIC_BYTES_PER_ROW = (268692736 + 50886656) / 32768  # dram read + write of one k_fwdq4096 launch (profiles/)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "sm_max_mhz": float(d.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [l for (t, l) in self.lines if t0 - 0.05 <= t <= t1 + 0.15] or [l for (_, l) in self.lines]
        for line in rows:
            f = [p.strip() for p in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def time_oracle(fn, min_seconds=0.0):
    t0 = time.perf_counter()
    fn()
    return time.perf_counter() - t0


def _omp_set_threads(n: int) -> bool:
    """Thread count of the OpenMP runtime the oracle library uses (the oracle itself is left as it stands)."""
    import ctypes

    try:
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
        return True
    except OSError:
        return False


def cpu_baseline(sample_rows=32768):
    """The fp64 oracle, as it stands, on the host cores: forward + INT4 quantize on the first `sample_rows` rows of
    the workload with all cores (the headline figure) and with one thread, plus two smaller slices of the other
    workloads: forward + backward on 2048 rows of the learning batch and forward + INT2 on 2048 rows of n = 8192."""
    import oracle
    from paper_2509_09679_b200 import synth

    wl = synth.WORKLOADS[WORKLOAD]
    theta = wl.theta().double().numpy()
    x = wl.x(n_rows=sample_rows).double().numpy()
    oracle.forward_quant(theta, x[:64], wl.bits)  # load the library, warm caches
    cores = oracle.num_threads()
    dt = time_oracle(lambda: oracle.forward_quant(theta, x, wl.bits))
    out = {"value": sample_rows / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"first {sample_rows} of {wl.n_rows} rows of {WORKLOAD} (fp64 C oracle, OpenMP over rows), {dt:.2f} s"}
    slices = {}
    one = 2048
    if _omp_set_threads(1):
        dt1 = time_oracle(lambda: oracle.forward_quant(theta, x[:one], wl.bits))
        slices["forward_int4_n4096_1thread"] = {"rows_per_s": one / dt1, "rows": one, "cores": 1, "seconds": dt1}
        _omp_set_threads(cores)
    wl3 = synth.WORKLOADS["learn4096"]
    th3, x3, g3 = wl3.theta().double().numpy(), wl3.x(n_rows=one).double().numpy(), wl3.g(n_rows=one).double().numpy()
    dt3 = time_oracle(lambda: (oracle.forward(th3, x3), oracle.backward(th3, x3, g3)))
    slices["forward_backward_n4096"] = {"rows_per_s": one / dt3, "rows": one, "cores": cores, "seconds": dt3}
    wl4 = synth.WORKLOADS["act8192_int2"]
    th4, x4 = wl4.theta().double().numpy(), wl4.x(n_rows=one).double().numpy()
    dt4 = time_oracle(lambda: oracle.forward_quant(th4, x4, 2))
    slices["forward_int2_n8192"] = {"rows_per_s": one / dt4, "rows": one, "cores": cores, "seconds": dt4}
    out["slices"] = slices
    return out


def run_reference(args):
    """--impl reference: the CPU oracle on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2509_09679_b200 import synth

    wl = synth.WORKLOADS[WORKLOAD]
    sample_rows = 2048
    theta = wl.theta().double().numpy()
    x = wl.x(n_rows=sample_rows).double().numpy()
    for _ in range(args.warmup):
        oracle.forward_quant(theta, x, wl.bits)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.forward_quant(theta, x, wl.bits)
    dt = (time.perf_counter() - t0) / args.steps
    value = sample_rows / dt
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "n": wl.n, "rows_per_step": sample_rows, "bits": wl.bits},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": f"{sample_rows} rows of {WORKLOAD} per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def event_time_ms(torch, fn, iters):
    """Average device time of fn() over `iters` back-to-back calls on the current stream."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="bfq", choices=["bfq", "reference"])
    ap.add_argument("--no-others", action="store_true", help="skip the secondary operations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--rows", type=int, default=0, help="override the row count (profiler captures of a small case)")
    ap.add_argument("--n", type=int, default=4096, choices=[4096, 8192], help="row length for --op backward / inverse")
    ap.add_argument("--op", default="forward_quant", choices=["forward_quant", "backward", "inverse", "int2_8192", "composite5120", "dequant_gemm", "fma_peak"],
                    help="backward / int2_8192: time only bfq_backward on the learning batch / bfq_forward_quant "
                         "(INT2) on the n = 8192 activations (for profiler captures; prints a short JSON line, "
                         "not the benchmark line)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "bfq" else args.warmup
    if args.impl == "reference":
        return run_reference(args)

    import torch
    from paper_2509_09679_b200 import Plan, lib, synth

    lib()  # fail loudly if the CUDA library is missing
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    from paper_2509_09679_b200.replicas import Replicas

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ranks = Replicas(dev)
    rank, world, dist = ranks.rank, ranks.world, ranks.dist
    barrier, max_over_ranks = ranks.barrier, ranks.max_over_ranks

    if args.op == "fma_peak":
        from paper_2509_09679_b200 import measure_mma_rates

        m = measure_mma_rates(dev)
        # one merged phase of four butterfly stages at n = 4096 = 256 distinct 16 x 16 blocks; 128 token rows per MMA;
        # two bf16 terms for the block and two for the data = 4 MMAs (M = 128, N = 16, K = 16) per block
        merged = {"cycles_per_mma_m128_k16": m,
                  "merged_phase_cycles_per_row_per_sm": 256 * 4 * m["n16"] / 128,
                  "note": "three such phases per row; the FP32 kernel takes about 1100 cycles per row per SM in all"}
        print(json.dumps({"op": "fma_peak", **fma_rates(torch, dev), "tensor_core_small_n": merged}))
        return
    if args.op == "backward":
        return run_backward_only(torch, args, synth, Plan, dev)
    if args.op == "inverse":
        return run_inverse_only(torch, args, synth, Plan, dev)
    if args.op == "dequant_gemm":
        return run_gemm_only(torch, args, synth, Plan, dev)
    if args.op == "int2_8192":
        return run_int2_8192_only(torch, args, synth, Plan, dev)
    if args.op == "composite5120":
        return run_composite_only(torch, args, synth, Plan, dev)
    wl = synth.WORKLOADS[WORKLOAD]
    if args.rows:
        import dataclasses

        wl = dataclasses.replace(wl, n_rows=args.rows)
    # replicas only: every rank runs the whole workload on its own GPU with its own seed
    theta = wl.theta(device=dev, seed=wl.seed)
    x = wl.x(device=dev, seed=ranks.seed(wl.seed))
    plan = Plan(wl.n, dev)
    codes = torch.empty((wl.n_rows, wl.n * wl.bits // 8), dtype=torch.uint8, device=dev)
    scales = torch.empty((wl.n_rows,), dtype=torch.float16, device=dev)

    def step():
        plan.set_angles(theta)
        plan.forward_quant(x, wl.bits, codes=codes, scales=scales)

    for _ in range(args.warmup):
        step()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    # the clock sampler needs a moment to start: spend it on further untimed steps, so that the timed region does not
    # begin on a GPU that has just idled for a quarter of a second
    t_ready = time.time() + 0.25
    while time.time() < t_ready:
        step()
        torch.cuda.synchronize()
    # The timed region: exactly `steps` steps between two events, nothing else on the stream.  (An event recorded between
    # the table build and the forward kernel keeps that kernel from being launched programmatically ahead of the build's
    # end: with a pair of events around every forward launch the step reads 5 % longer and the kernel 4 % longer than
    # they run without them, so the per-launch figures are taken in passes of their own below.)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    e0.record()
    for k in range(args.steps):
        plan.set_angles(theta)
        plan.forward_quant(x, wl.bits, codes=codes, scales=scales)
    e1.record()
    barrier()
    t_wall1 = time.time()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    ms_step = ms_total / args.steps
    # the dominant kernel (forward+quant): average launch duration over max(steps, 200) launches back to back between
    # two events on the launching stream, right after the timed region (same plan, same buffers, inputs larger than L2)
    k_launches = max(args.steps, 200)
    k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    k0.record()
    for k in range(k_launches):
        plan.forward_quant(x, wl.bits, codes=codes, scales=scales)
    k1.record()
    torch.cuda.synchronize()
    kernel_ms_avg = max_over_ranks(k0.elapsed_time(k1) / k_launches)
    # ... and, for the spread, a pair of events around each forward launch of 200 further steps (reads longer, see above)
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(200)]
    for k in range(200):
        plan.set_angles(theta)
        kev[k][0].record()
        plan.forward_quant(x, wl.bits, codes=codes, scales=scales)
        kev[k][1].record()
    torch.cuda.synchronize()
    kernel_ms = [a.elapsed_time(b) for a, b in kev]
    kernel_stats = {"launches": k_launches, "method": "back-to-back launches between two events, after the timed region",
                    "per_launch_event_pairs_inside_steps": {"launches": len(kernel_ms), "mean_ms": sum(kernel_ms) / len(kernel_ms),
                                                            "min_ms": min(kernel_ms), "median_ms": statistics.median(kernel_ms),
                                                            "max_ms": max(kernel_ms),
                                                            "note": "an event between the table build and the kernel blocks the kernel's programmatic early launch"}}
    status = plan.device_status()
    if status != 0:
        raise SystemExit(f"device status {status}")
    value = ranks.whole_job_rate(wl.n_rows, ms_step)

    # ---- end-to-end through the public API with host buffers --------------------------------------
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(torch, args, wl, plan, theta, x, codes, scales, barrier, max_over_ranks, world)

    # ---- secondary operations (single rank, after the headline) -------------------------------------
    others = {}
    if rank == 0 and not args.no_others:
        others = time_others(torch, synth, Plan, dev)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    finish(torch, args, wl, synth, x, dev, world, value, ms_step, kernel_ms_avg, kernel_stats, clocks, e2e, others, dist)


def fma_rates(torch, dev):
    """Measured FP32 FMA issue rates (register-only kernels of the library) as cycles per instruction per scheduler
    and as chip-wide Tslot/s at the maximum SM clock, beside the nominal one FMA per lane per cycle."""
    from paper_2509_09679_b200 import measure_fma_rates

    r = measure_fma_rates(dev)
    props = torch.cuda.get_device_properties(dev)
    clock = measured_peaks()["sm_max_mhz"] * 1e6
    sched = props.multi_processor_count * 4
    return {"cycles_per_instruction_per_scheduler": r,
            "tslots_per_s": {"packed_3reg": sched * 64 / r["packed_3reg"] * clock / 1e12,
                             "packed_2reg": sched * 64 / r["packed_2reg"] * clock / 1e12,
                             "scalar_3reg": sched * 32 / r["scalar_3reg"] * clock / 1e12,
                             "scalar_2reg": sched * 32 / r["scalar_2reg"] * clock / 1e12,
                             "nominal": sched * 32 * clock / 1e12},
            "note": "three distinct register operands per FMA is what a rotation with per-pair constants needs"}


def run_backward_only(torch, args, synth, Plan, dev):
    """bfq_backward alone on (a prefix of) the learning batch, or with --n 8192 on a prefix of the n = 8192 activations
    with standard-normal gradient rows: warm-up, then `steps` timed launches."""
    wl = synth.WORKLOADS["learn4096" if args.n == 4096 else "act8192_int2"]
    rows = args.rows or (wl.n_rows if args.n == 4096 else wl.n_rows // 4)
    plan = Plan(wl.n, dev)
    plan.set_angles(wl.theta(device=dev))
    x, g = wl.x(device=dev, n_rows=rows), wl.g(device=dev, n_rows=rows)
    dx = torch.empty_like(x)
    dth = torch.empty((wl.L, wl.n // 2), dtype=torch.float32, device=dev)
    for _ in range(args.warmup):
        plan.backward(x, g, dx=dx, dtheta=dth)
    ms = event_time_ms(torch, lambda: plan.backward(x, g, dx=dx, dtheta=dth), args.steps)
    print(json.dumps({"op": "backward", "workload": "learn4096" if args.n == 4096 else "act8192_int2",
                      "rows": rows, "ms": ms, "rows_per_s": rows / (ms * 1e-3), "status": plan.device_status()}))


def run_inverse_only(torch, args, synth, Plan, dev):
    """bfq_inverse alone on (a prefix of) the learning batch's gradient rows, or with --n 8192 on standard-normal rows of
    that length (the row count of the n = 8192 activations)."""
    wl = synth.WORKLOADS["learn4096" if args.n == 4096 else "act8192_int2"]
    rows = args.rows or wl.n_rows
    plan = Plan(wl.n, dev)
    plan.set_angles(wl.theta(device=dev))
    g = wl.g(device=dev, n_rows=rows)
    out = torch.empty_like(g)
    for _ in range(args.warmup):
        plan.inverse(g, out=out)
    ms = event_time_ms(torch, lambda: plan.inverse(g, out=out), args.steps)
    print(json.dumps({"op": "inverse", "workload": "learn4096" if args.n == 4096 else "act8192_int2", "rows": rows, "ms": ms,
                      "rows_per_s": rows / (ms * 1e-3), "status": plan.device_status()}))


def run_gemm_only(torch, args, synth, Plan, dev):
    """bfq_dequant_gemm alone: 4-bit activation codes x 4-bit weight codes, the forward product of the calibration step
    (tokens = --rows or 2048, a 4096 x 4096 layer)."""
    from paper_2509_09679_b200 import GemmOperand

    n, out, tokens = 4096, 4096, args.rows or 2048
    plan = Plan(n, dev)
    plan.set_angles(synth.angles(n, "normal", 7003, dev))
    W = synth.rows(out, n, "normal", 7001, scale=0.02, dtype=torch.bfloat16).to(dev)
    X = synth.rows(tokens, n, "student_t3", 7002, outliers=8, outlier_scale=50.0, dtype=torch.bfloat16).to(dev)
    wc, ws, _ = plan.fold_weights(W, 4)
    ac, asc = plan.forward_quant(X, 4)
    c = torch.empty((tokens, out), dtype=torch.float32, device=dev)
    fn = lambda: plan.dequant_gemm(GemmOperand(ac, asc, 4), GemmOperand(wc, ws, 4), out=c)
    for _ in range(args.warmup):
        fn()
    ms = event_time_ms(torch, fn, args.steps)
    print(json.dumps({"op": "dequant_gemm", "m": tokens, "n": out, "k": n, "ms": ms,
                      "tflops": 2.0 * tokens * out * n / (ms * 1e-3) / 1e12, "status": plan.device_status()}))


def run_int2_8192_only(torch, args, synth, Plan, dev):
    """bfq_forward_quant (INT2) alone on (a prefix of) the n = 8192 activations."""
    wl = synth.WORKLOADS["act8192_int2"]
    rows = args.rows or wl.n_rows
    plan = Plan(wl.n, dev)
    plan.set_angles(wl.theta(device=dev))
    x = wl.x(device=dev, n_rows=rows)
    codes = torch.empty((rows, wl.n // 4), dtype=torch.uint8, device=dev)
    scales = torch.empty((rows,), dtype=torch.float16, device=dev)
    for _ in range(args.warmup):
        plan.forward_quant(x, 2, codes=codes, scales=scales)
    ms = event_time_ms(torch, lambda: plan.forward_quant(x, 2, codes=codes, scales=scales), args.steps)
    print(json.dumps({"op": "int2_8192", "workload": "act8192_int2", "rows": rows, "ms": ms,
                      "rows_per_s": rows / (ms * 1e-3), "status": plan.device_status()}))


def composite_inputs(torch, synth, Plan, dev, rows=None):
    """The paper's composite example, d = 5120 = 40 x 128: plan (Q2 angles), Cayley factor Q1, bf16 token rows."""
    c = synth.COMPOSITE_5120
    rows = rows or c["n_rows"]
    plan = Plan(c["n2"], dev)
    plan.set_angles(synth.angles(c["n2"], "normal", c["seed"], dev))
    q1 = plan.cayley(synth.cayley_params(c["n1"], c["seed"], device=dev), c["n1"])
    x = synth.rows(rows, c["n1"] * c["n2"], c["dist"], c["seed"] + 1, outliers=c["outliers"],
                   outlier_scale=c["outlier_scale"], dtype=torch.bfloat16, device=dev)
    return plan, q1, x


def run_composite_only(torch, args, synth, Plan, dev):
    """bfq_composite_forward_quant (INT4) alone on (a prefix of) the d = 5120 token rows."""
    plan, q1, x = composite_inputs(torch, synth, Plan, dev, args.rows)
    rows = x.shape[0]
    codes = torch.empty((rows, 2560), dtype=torch.uint8, device=dev)
    scales = torch.empty((rows,), dtype=torch.float16, device=dev)
    for _ in range(args.warmup):
        plan.composite_forward_quant(q1, x, 4, codes=codes, scales=scales)
    ms = event_time_ms(torch, lambda: plan.composite_forward_quant(q1, x, 4, codes=codes, scales=scales), args.steps)
    print(json.dumps({"op": "composite5120", "workload": "composite 40x128 int4", "rows": rows, "ms": ms,
                      "rows_per_s": rows / (ms * 1e-3), "gbs": rows * (2 * 5120 + 2560 + 2) / (ms * 1e-3) / 1e9,
                      "status": plan.device_status()}))


def run_e2e(torch, args, wl, plan, theta, x, codes, scales, barrier, max_over_ranks, world):
    x_host = x.to("cpu").pin_memory()
    codes_host = torch.empty(codes.shape, dtype=codes.dtype).pin_memory()
    scales_host = torch.empty(scales.shape, dtype=scales.dtype).pin_memory()
    from paper_2509_09679_b200.host_pipeline import HostForwardQuant

    # rows from pinned host memory, codes + scales back to pinned host memory, every step; the copies of one chunk of
    # rows overlap the kernels of another (three streams)
    pipe = HostForwardQuant(plan, wl.n_rows, wl.bits, dtype=x.dtype, chunks=8)

    def e2e_step():
        pipe(x_host, codes_host, scales_host, before=lambda: plan.set_angles(theta))

    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        e2e_step()
    barrier()
    ms_e2e = max_over_ranks(event_time_ms(torch, e2e_step, e2e_steps))
    return {"value": world * wl.n_rows / (ms_e2e * 1e-3), "unit": UNIT, "ms_per_step": ms_e2e,
            "h2d_bytes_per_step": x_host.numel() * x_host.element_size(),
            "d2h_bytes_per_step": codes_host.numel() + scales_host.numel() * 2}


def finish(torch, args, wl, synth, x, dev, world, value, ms_step, kernel_ms_avg, kernel_stats, clocks, e2e, others, dist):
    peaks = measured_peaks()
    props = torch.cuda.get_device_properties(dev)
    alu_peak = props.multi_processor_count * FP32_LANES_PER_SM * peaks["sm_max_mhz"] * 1e6  # slots/s
    t_kernel = kernel_ms_avg * 1e-3
    slots_per_s = SLOTS_PER_ROW * wl.n_rows / t_kernel
    gbs = BYTES_PER_ROW * wl.n_rows / t_kernel / 1e9
    t_alu = SLOTS_PER_ROW * wl.n_rows / alu_peak
    t_hbm = BYTES_PER_ROW * wl.n_rows / (peaks["hbm_gbs"] * 1e9)
    bound = "alu" if t_alu >= t_hbm else "hbm"
    roofline = {
        "bound": bound,
        "achieved": slots_per_s / 1e12 if bound == "alu" else gbs,
        "peak": alu_peak / 1e12 if bound == "alu" else peaks["hbm_gbs"],
        "unit": "Tslot/s (FP32 issue slots: MUL or FMA per lane)" if bound == "alu" else "GB/s",
        "frac": max(t_alu, t_hbm) / t_kernel,
        "traffic": None if NCU_TRAFFIC_BYTES_PER_ROW is None else NCU_TRAFFIC_BYTES_PER_ROW * wl.n_rows,
        "kernel": "forward+quant", "kernel_ms": kernel_ms_avg, "kernel_ms_stats": kernel_stats,
        # the same launch against the bound of the formulation the kernel executes (n L + 2 n slots per row)
        "frac_executed_form": EXECUTED_SLOTS_PER_ROW * wl.n_rows / alu_peak / t_kernel,
        "executed_slots": EXECUTED_SLOTS_PER_ROW * wl.n_rows,
        "alu_measured": fma_rates(torch, dev),
        "algorithmic_bytes": BYTES_PER_ROW * wl.n_rows, "algorithmic_slots": SLOTS_PER_ROW * wl.n_rows,
        "hbm_achieved_gbs": gbs, "hbm_frac": gbs / peaks["hbm_gbs"], "hbm_peak_gbs": peaks["hbm_gbs"],
        "peaks": f"HBM {peaks['source']}; ALU = SMs x 128 lanes x {peaks['sm_max_mhz']:.0f} MHz",
    }
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "n": wl.n, "rows": wl.n_rows, "bits": wl.bits, "input": "bf16",
                   "l2": "inputs larger than L2 (268 MB per step)", "parallelism": "replicas only",
                   "x_checksum": f"{synth.checksum64(x[:256]):016x}"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": 3 * args.steps, "roofline": roofline,
        "gbs": gbs, "others": others,
    }
    if not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline()
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def time_others(torch, synth, Plan, dev):
    """Hadamard / unquantized variants of the headline, backward (learning batch), inverse, n = 8192 INT2 and
    weight folding: device-timed, inputs resident, 3 warm-up + a few timed launches each.  alu_frac uses the
    paper's FLOP table: 4 slots per pair for the butterfly, 1 (an add or a subtract per element) for Hadamard."""
    res = {}
    alu_peak = torch.cuda.get_device_properties(dev).multi_processor_count * FP32_LANES_PER_SM * 1.965e9

    def record(name, rows, n, L, slots_per_pair, bytes_per_row, fn, iters):
        for _ in range(3):
            fn()
        ms = event_time_ms(torch, fn, iters)
        slots = slots_per_pair * (n // 2) * L * rows
        res[name] = {"rows_per_s": rows / (ms * 1e-3), "ms": ms, "gbs": bytes_per_row * rows / (ms * 1e-3) / 1e9,
                     "alu_frac": slots / alu_peak / (ms * 1e-3), "rows": rows, "n": n}

    # the fixed Hadamard rotation and the unquantized (16-bit activation) outputs on the headline rows
    wl = synth.WORKLOADS[WORKLOAD]
    plan = Plan(wl.n, dev)
    plan.set_angles(wl.theta(device=dev))
    x = wl.x(device=dev)
    codes = torch.empty((wl.n_rows, wl.n // 2), dtype=torch.uint8, device=dev)
    scales = torch.empty((wl.n_rows,), dtype=torch.float16, device=dev)
    y = torch.empty_like(x)
    record("hadamard_int4_n4096", wl.n_rows, wl.n, wl.L, 1, BYTES_PER_ROW,
           lambda: plan.hadamard_quant(x, 4, codes=codes, scales=scales), 20)
    record("forward_int4_stats_n4096", wl.n_rows, wl.n, wl.L, 4, BYTES_PER_ROW + 8,
           lambda: plan.forward_quant_stats(x, 4), 10)
    record("forward_bf16_n4096", wl.n_rows, wl.n, wl.L, 4, 4 * wl.n, lambda: plan.forward(x, out=y), 20)
    codes2 = torch.empty((wl.n_rows, wl.n // 4), dtype=torch.uint8, device=dev)
    codes8 = torch.empty((wl.n_rows, wl.n), dtype=torch.uint8, device=dev)
    x32 = x.float()
    record("forward_int4_fp32_rows_n4096", wl.n_rows, wl.n, wl.L, 4, 4 * wl.n + wl.n // 2 + 2,
           lambda: plan.forward_quant(x32, 4, codes=codes, scales=scales), 20)
    del x32
    record("forward_int2_n4096", wl.n_rows, wl.n, wl.L, 4, 2 * wl.n + wl.n // 4 + 2,
           lambda: plan.forward_quant(x, 2, codes=codes2, scales=scales), 20)
    record("forward_int8_n4096", wl.n_rows, wl.n, wl.L, 4, 3 * wl.n + 2,
           lambda: plan.forward_quant(x, 8, codes=codes8, scales=scales), 20)
    del codes2, codes8
    record("hadamard_bf16_n4096", wl.n_rows, wl.n, wl.L, 1, 4 * wl.n, lambda: plan.hadamard(x, out=y), 20)
    del x, y, codes, scales, plan
    # angle-learning step: forward + backward on 128 x 2048 rows of n = 4096
    wl = synth.WORKLOADS["learn4096"]
    theta = wl.theta(device=dev)
    plan = Plan(wl.n, dev)
    plan.set_angles(theta)
    x = wl.x(device=dev)
    g = wl.g(device=dev)
    dx = torch.empty_like(x)
    dth = torch.empty((wl.L, wl.n // 2), dtype=torch.float32, device=dev)
    record("backward_n4096", wl.n_rows, wl.n, wl.L, 14, 3 * 2 * wl.n,
           lambda: plan.backward(x, g, dx=dx, dtheta=dth), 3)
    record("inverse_n4096", wl.n_rows, wl.n, wl.L, 4, 2 * 2 * wl.n, lambda: plan.inverse(g, out=dx), 3)
    # the same two on fp32 rows (a quarter of the batch)
    q = wl.n_rows // 4
    x32, g32 = x[:q].float(), g[:q].float()
    dx32 = torch.empty_like(x32)
    record("backward_fp32_rows_n4096", q, wl.n, wl.L, 14, 3 * 4 * wl.n,
           lambda: plan.backward(x32, g32, dx=dx32, dtheta=dth), 3)
    record("inverse_fp32_rows_n4096", q, wl.n, wl.L, 4, 2 * 4 * wl.n, lambda: plan.inverse(g32, out=dx32), 3)
    del x32, g32, dx32
    del x, g, dx
    torch.cuda.empty_cache()
    # n = 8192 INT2
    wl = synth.WORKLOADS["act8192_int2"]
    plan8 = Plan(wl.n, dev)
    plan8.set_angles(wl.theta(device=dev))
    x = wl.x(device=dev)
    codes = torch.empty((wl.n_rows, wl.n // 4), dtype=torch.uint8, device=dev)
    scales = torch.empty((wl.n_rows,), dtype=torch.float16, device=dev)
    record("forward_int2_n8192", wl.n_rows, wl.n, wl.L, 4, 2 * wl.n + wl.n // 4 + 2,
           lambda: plan8.forward_quant(x, 2, codes=codes, scales=scales), 5)
    codes4 = torch.empty((wl.n_rows, wl.n // 2), dtype=torch.uint8, device=dev)
    record("forward_int4_n8192", wl.n_rows, wl.n, wl.L, 4, 2 * wl.n + wl.n // 2 + 2,
           lambda: plan8.forward_quant(x, 4, codes=codes4, scales=scales), 5)
    del codes4
    x32 = x.float()
    record("forward_int2_fp32_rows_n8192", wl.n_rows, wl.n, wl.L, 4, 4 * wl.n + wl.n // 4 + 2,
           lambda: plan8.forward_quant(x32, 2, codes=codes, scales=scales), 5)
    del x32
    y8 = torch.empty_like(x)
    record("forward_bf16_n8192", wl.n_rows, wl.n, wl.L, 4, 4 * wl.n, lambda: plan8.forward(x, out=y8), 5)
    record("inverse_n8192", wl.n_rows, wl.n, wl.L, 4, 4 * wl.n, lambda: plan8.inverse(x, out=y8), 5)
    record("hadamard_int2_n8192", wl.n_rows, wl.n, wl.L, 1, 2 * wl.n + wl.n // 4 + 2,
           lambda: plan8.hadamard_quant(x, 2, codes=codes, scales=scales), 5)
    record("hadamard_bf16_n8192", wl.n_rows, wl.n, wl.L, 1, 4 * wl.n, lambda: plan8.hadamard(x, out=y8), 5)
    # backward at n = 8192 (forward cluster kernel for the last stage's sums + the n = 4096 backward kernel per half): a quarter of the rows
    rows8 = wl.n_rows // 4
    g8 = torch.randn((rows8, wl.n), device=dev, dtype=torch.float32).to(x.dtype)
    dx8 = torch.empty_like(g8)
    dth8 = torch.empty((wl.L, wl.n // 2), dtype=torch.float32, device=dev)
    record("backward_n8192", rows8, wl.n, wl.L, 14, 3 * 2 * wl.n,
           lambda: plan8.backward(x[:rows8], g8, dx=dx8, dtheta=dth8), 3)
    del x, y8, g8, dx8
    wl = synth.WORKLOADS["fold8192_int2"]
    W = wl.x(device=dev)
    record("fold_int2_n8192", wl.n_rows, wl.n, wl.L, 4, 2 * wl.n + wl.n // 4 + 2,
           lambda: plan8.fold_weights(W, 2), 5)
    record("fold_int2_with_rows_n8192", wl.n_rows, wl.n, wl.L, 4, 4 * wl.n + wl.n // 4 + 2,
           lambda: plan8.fold_weights(W, 2, want_rotated=True), 5)
    del W, plan8
    torch.cuda.empty_cache()
    # composite 40 x 128 (d = 5120): both factors on the tensor cores (default), or butterfly-128 on the CUDA cores
    planc, q1, x = composite_inputs(torch, synth, Plan, dev)
    rows = x.shape[0]
    codes = torch.empty((rows, 2560), dtype=torch.uint8, device=dev)
    scales = torch.empty((rows,), dtype=torch.float16, device=dev)
    y = torch.empty_like(x)
    legs = (("composite_int4_d5120", 2 * 5120 + 2560 + 2,
             lambda: planc.composite_forward_quant(q1, x, 4, codes=codes, scales=scales)),
            ("composite_bf16_d5120", 4 * 5120, lambda: planc.composite_forward(q1, x, out=y)))
    # default: both factors on the tensor cores; *_fp32_butterfly: Q2 as an fp32 butterfly on the CUDA cores
    for suffix, env in (("", None), ("_fp32_butterfly", "1")):
        if env is None:
            os.environ.pop("BFQ_COMPOSITE_FP32_BUTTERFLY", None)
        else:
            os.environ["BFQ_COMPOSITE_FP32_BUTTERFLY"] = env
        for name, nbytes, fn in legs:
            for _ in range(3):
                fn()
            ms = event_time_ms(torch, fn, 10)
            gbs = nbytes * rows / (ms * 1e-3) / 1e9
            res[name + suffix] = {"rows_per_s": rows / (ms * 1e-3), "ms": ms, "gbs": gbs,
                                  "hbm_frac": gbs / measured_peaks()["hbm_gbs"], "rows": rows, "n": 5120}
    os.environ.pop("BFQ_COMPOSITE_FP32_BUTTERFLY", None)
    del planc, q1, x, codes, scales, y
    torch.cuda.empty_cache()
    # layer-calibration step (reconstruction loss + angle gradient) on a 4096 x 4096 layer, 2048 tokens, 4-bit weights and
    # activations, and its dense products alone (bfq_dequant_gemm; TFLOP/s counts 2 m n k once, whatever the number of
    # bf16 terms an operand is split into)
    from paper_2509_09679_b200 import GemmOperand
    from paper_2509_09679_b200.calibrate import LayerCalibrator

    n, out, tokens = 4096, 4096, 2048
    W = synth.rows(out, n, "normal", 7001, scale=0.02, dtype=torch.bfloat16).to(dev)
    X = synth.rows(tokens, n, "student_t3", 7002, outliers=8, outlier_scale=50.0, dtype=torch.bfloat16).to(dev)
    cal = LayerCalibrator(W, 4, 4, theta=synth.angles(n, "normal", 7003, dev) * 0.1)
    for _ in range(2):
        cal.loss_and_grad(X)
    ms = event_time_ms(torch, lambda: cal.loss_and_grad(X), 5)
    res["calibration_step_n4096_w4a4"] = {"ms": ms, "tokens": tokens, "out": out, "n": n, "tokens_per_s": tokens / (ms * 1e-3)}
    p = cal.plan
    wc, ws, _ = p.fold_weights(W, 4)
    ac, asc = p.forward_quant(X, 4)
    e = torch.randn((tokens, out), device=dev)
    peak = None
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak = float(json.load(f)["bf16_tflops"])
    except (OSError, KeyError, ValueError):
        pass
    gemms = (("dequant_gemm_codes_x_codes", lambda: p.dequant_gemm(GemmOperand(ac, asc, 4), GemmOperand(wc, ws, 4)), tokens, out, n),
             ("dequant_gemm_f32_x_codesT", lambda: p.dequant_gemm(GemmOperand(e), GemmOperand(wc, ws, 4, transposed=True)), tokens, n, out),
             ("dequant_gemm_f32T_x_codesT", lambda: p.dequant_gemm(GemmOperand(e, transposed=True), GemmOperand(ac, asc, 4, transposed=True)), out, n, tokens))
    for name, fn, m_, n_, k_ in gemms:
        for _ in range(2):
            fn()
        ms = event_time_ms(torch, fn, 10)
        tf = 2.0 * m_ * n_ * k_ / (ms * 1e-3) / 1e12
        res[name] = {"ms": ms, "m": m_, "n": n_, "k": k_, "tflops": tf,
                     "tensor_frac": None if peak is None else tf / peak}
    if p.device_status() != 0:
        raise SystemExit("device status after the calibration legs")
    return res


if __name__ == "__main__":
    main()
