#!/usr/bin/env python
"""Benchmark of the Generalized PolyDot coded matrix product on B200.

One "step" is one pass of the whole coded path over one batch of synthetic input:
encode W, encode X, the P worker products (one batched kernel), seeded error injection,
error detection/location, interpolation decode.  Workload: the 8192 x 8192 x 512 coded
matrix-matrix product (W split 2 x 4, X split 4 x 2, threshold 19, P = 25 nodes, additive
errors on each node with probability 0.1).  Shares are evaluated in FP64; the worker products
run either as exact int8 digit-plane contractions on the tcgen05 tensor cores with FP64
recombination (--precision sliced, the default) or as FP64 mma (--precision fp64); worker
outputs, location and decoding are FP64 in both.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--precision sliced|sliced40|fp64]
                    [--workload matmul|matvec|mlp_layer|sae_layer|positions] [--no-secondary]

Prints one JSON line.  The default line (matmul workload) also carries a `secondary` object with one
short run each of the other workloads (FP64-mma products, matrix-vector, MLP layer, autoencoder layer,
per-position correction), so that one run observes every path.  `value` is useful TFLOP/s = 2 N1 N0 B / time (the product the caller
asked for); the coded path executes P/(m n d) = 1.5625 times those flops.  With --gpus N
(launched through torch.distributed.run) every rank runs an independent replica of the
workload; there is no data-path collective.  Started with --gpus N > 1 and no RANK in the
environment, the script re-executes itself under torch.distributed.run with N ranks.
"""

from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "coded matmul TFLOP/s (encode+workers+locate+decode)"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0        # dense, per GPU
NOMINAL_FP64_TFLOPS = 37.0          # FP64 tensor, per GPU of an 8-GPU HGX B200 board (296 / 8)
NOMINAL_INT8_TOPS = 4500.0          # dense int8, per GPU
FALLBACK_BF16_SUSTAINED = 1400.0
FALLBACK_HBM_GBS = 6650.0
CPU_SAMPLE_ROWS = 1024              # rows of W in the CPU sample (1/8 of the workload)
TRAFFIC_BYTES_PER_LAUNCH = None     # dram read+write bytes of the dominant kernel from ncu (see profiles/)
TRAFFIC_BYTES_PER_LAUNCH_SLICED = {6: 1541924000,   # gemm_i8_sliced_kernel<6>: dram read 1.345208 GB + write 0.196716 GB (profiles/)
                                   5: None}         # five planes: no counters taken
TENSOR_PIPE_PCT_NCU = {6: 79.3, 5: None}            # sm__pipe_tensor_cycles_active, % of elapsed (profiles/)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_sustained": float(p["bf16_tflops_sustained"]),
                "bf16_burst": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_sustained": FALLBACK_BF16_SUSTAINED, "bf16_burst": 1590.0,
            "source": "fallback"}


# --------------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("uuid,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid = uuid
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 9 or (self.uuid and self.uuid not in parts[0]):
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------------------------------
# CPU baseline / reference arm: the oracle as it stands, on a bounded sample of the workload
# --------------------------------------------------------------------------------------------------
def oracle_sample_step(cfg, W, X, seed, stages=None):
    """One pass of the oracle's coded path over the sample; returns seconds.  `stages` (a dict)
    collects the seconds of each stage."""
    from oracle import inject as oinj
    from oracle import product as op
    from oracle.code import GPCode, FWD
    from oracle.locate import DECODE_FAILURE, locate_subspace, tolerances_for
    code = GPCode(W.shape[0], cfg.N0, cfg.B, cfg.m, cfg.n, cfg.d, 1, cfg.P)
    marks = [("start", time.perf_counter())]

    def mark(name):
        marks.append((name, time.perf_counter()))
    Ws = op.encode_W(W, code); mark("encode_A")
    Xs = op.encode_X(X, code); mark("encode_B")
    Z = op.worker_products(Ws, Xs); mark("worker_products")
    oinj.inject_additive(Z, seed, float(np.sqrt(np.mean(Z * Z))), prob=cfg.inject_prob); mark("inject")
    r = locate_subspace(Z, code.points, code.Q_f, tolerances_for(np.float64)); mark("locate")
    if r.outcome != DECODE_FAILURE:
        op.decode(Z, code, FWD, use=~r.flagged)
    mark("decode")
    if stages is not None:
        for (_, t0), (name, t1) in zip(marks[:-1], marks[1:]):
            stages[name] = stages.get(name, 0.0) + (t1 - t0)
    return marks[-1][1] - marks[0][1]


def oracle_uncoded_seconds(W, X):
    """The uncoded FP64 product of the same sample (the oracle's reference value)."""
    from oracle import product as op
    t0 = time.perf_counter()
    op.ref_forward(W, X)
    return time.perf_counter() - t0


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 0) for i in threadpool_info()]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import workloads as wl
    W, X = wl.matmul_inputs(cfg)
    Ws = np.ascontiguousarray(W[:CPU_SAMPLE_ROWS])
    for i in range(args.warmup):
        oracle_sample_step(cfg, Ws, X, cfg.inject_seeds[i % len(cfg.inject_seeds)])
    total = 0.0
    stages = {}
    for i in range(args.steps):
        total += oracle_sample_step(cfg, Ws, X, cfg.inject_seeds[i % len(cfg.inject_seeds)], stages)
    uncoded = oracle_uncoded_seconds(Ws, X)
    flops = 2.0 * CPU_SAMPLE_ROWS * cfg.N0 * cfg.B
    value = flops * args.steps / total / 1e12
    sample = (f"each step = first {CPU_SAMPLE_ROWS} of {cfg.N1} rows of W (same N0, B, code and P), rate scaled by the "
              "sample's flops; numpy FP64 oracle")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": dict(workload_config(cfg), precision=args.precision, sampled_rows_of_W=CPU_SAMPLE_ROWS),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample,
                         "stage_seconds_per_step": {k: round(v / args.steps, 4) for k, v in stages.items()},
                         "uncoded_product_seconds": round(uncoded, 4)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def max_over_ranks(values_ms, world: int, device: str):
    """Every rank times its own replica on its device; the job's time is the slowest rank's."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values_ms, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_tflops(flops_per_step_per_rank: float, steps: int, world: int, ms: float) -> float:
    """Aggregate over all replicas: units all ranks processed / slowest rank's time."""
    return flops_per_step_per_rank * steps * world / (ms * 1e-3) / 1e12


def measure_fp64_matmul_peak(torch) -> float:
    """cuBLAS FP64 GEMM 8192^3, best of 10 (the recipe that produced the bf16 figure, for FP64)."""
    n = 8192
    a = torch.randn((n, n), dtype=torch.float64, device="cuda")
    b = torch.randn((n, n), dtype=torch.float64, device="cuda")
    c = torch.empty((n, n), dtype=torch.float64, device="cuda")
    for _ in range(2):
        torch.matmul(a, b, out=c)
    best = float("inf")
    for _ in range(10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        torch.matmul(a, b, out=c)
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    del a, b, c
    return 2.0 * n ** 3 / (best * 1e-3) / 1e12


def workload_config(cfg):
    return {"workload": cfg.name, "N1": cfg.N1, "N0": cfg.N0, "B": cfg.B, "split": [cfg.m, cfg.n, cfg.d],
            "threshold": cfg.m * cfg.n * cfg.d + cfg.n - 1, "nodes": cfg.P,
            "injection": f"additive, per-node probability {cfg.inject_prob}",
            "l2": "inputs larger than L2 (W 268 MB, shares 1.68 GB)", "parallelism": "replicas"}


def measure_int8_matmul_peak(torch):
    """int8 x int8 -> int32 GEMM 8192^3 through torch._int_mm (cuBLASLt), best of 10, CUDA events: the
    recipe of the bf16 figure, for the integer tensor path.  Returns (TOP/s, note) or (None, why)."""
    n = 8192
    try:
        a = torch.randint(-128, 127, (n, n), dtype=torch.int8, device="cuda")
        b = torch.randint(-128, 127, (n, n), dtype=torch.int8, device="cuda")
        for _ in range(2):
            torch._int_mm(a, b)
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch._int_mm(a, b)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        del a, b
        return 2.0 * n ** 3 / (best * 1e-3) / 1e12, "measured here: torch._int_mm int8 8192^3, best of 10"
    except Exception as exc:                                  # the call is private API: may be absent
        return None, f"torch._int_mm unavailable ({type(exc).__name__})"


# --------------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------------
def run_ours(args, cfg, precision, steps, repeats, full):
    """The headline workload.  full = True: the whole measurement (device-resident timing repeated
    `repeats` times, end-to-end timing, clocks, CPU baseline); False: one short device-resident run."""
    import torch
    import torch.distributed as dist
    import paper_1811_10751_b200 as g
    import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    peaks = load_peaks()

    W, X = wl.matmul_inputs(cfg)
    sliced = precision in ("sliced", "sliced40")
    planes = {"sliced": 6, "sliced40": 5}.get(precision, 0)
    plan = g.gpd_plan((cfg.N1, cfg.N0, cfg.B), (cfg.m, cfg.n, cfg.d, 1), cfg.P,
                      precision={"sliced": g.GPD_PREC_FP64_SLICED, "sliced40": g.GPD_PREC_FP64_SLICED40,
                                 "fp64": g.GPD_PREC_FP64}[precision])
    assert plan.query(g.GPD_Q_ELEMENT_SIZE) == 8
    g.gpd_plan_upload(plan)                  # the plan's tables: allocated and copied before anything is timed
    stream = torch.cuda.Stream()
    side = torch.cuda.Stream(priority=-1)
    fork, join = torch.cuda.Event(), torch.cuda.Event()
    Wh, Xh = torch.from_numpy(W).pin_memory(), torch.from_numpy(X).pin_memory()
    Sh = torch.empty((cfg.N1, cfg.B), dtype=torch.float32).pin_memory()
    Wd, Xd = Wh.cuda(), Xh.cuda()
    Wsh, Xsh = plan.empty(g.GPD_Q_W_SHARE_ELEMS), plan.empty(g.GPD_Q_X_SHARE_ELEMS)
    Z = plan.empty(g.GPD_Q_OUT_ELEMS_FWD)
    S = torch.empty((cfg.N1, cfg.B), dtype=torch.float32, device="cuda")
    ws, res = plan.workspace(), g.new_results(1)
    res_h = torch.empty(g.RESULT_BYTES, dtype=torch.uint8).pin_memory()
    scale = 1.0                         # replaced below by the RMS of the clean worker outputs
    seeds = cfg.inject_seeds
    exec_flops = 2.0 * cfg.P * (cfg.N1 // cfg.m) * (cfg.N0 // cfg.n) * (cfg.B // cfg.d)
    useful_flops = 2.0 * cfg.N1 * cfg.N0 * cfg.B
    # encode W, encode X, products, inject, syndrome, locate finish, decode matrix, decode stream;
    # the digit-plane encoder of X takes two kernels (scales, then digits), the one of W is fused
    KERNELS_PER_STEP = 9 if sliced else 8

    def step(i, gemm_events=None, stage_events=None, Wd=Wd, Xd=Xd):
        def mark(name):
            if stage_events is not None:
                e = torch.cuda.Event(enable_timing=True)
                e.record(stream)
                stage_events.append((name, e))
        mark("start")
        if stage_events is None:
            # the two encoders are independent: X~ (small, latency-bound kernels) is encoded on a second
            # stream beside W~; the stage breakdown pass runs them one after the other instead
            fork.record(stream)
            side.wait_event(fork)
            g.gpd_encode_B(plan, g.GPD_OPERAND_X_FWD, Xd, Xsh, stream=side)
            join.record(side)
            g.gpd_encode_A(plan, Wd, Wsh, stream=stream)
            stream.wait_event(join)
        else:
            g.gpd_encode_A(plan, Wd, Wsh, stream=stream); mark("encode_A")
            g.gpd_encode_B(plan, g.GPD_OPERAND_X_FWD, Xd, Xsh, stream=stream); mark("encode_B")
        if gemm_events is not None:
            e0 = torch.cuda.Event(enable_timing=True); e0.record(stream)
        g.gpd_worker_gemm(plan, g.GPD_FWD, Wsh, Xsh, Z, stream=stream)
        if gemm_events is not None:
            e1 = torch.cuda.Event(enable_timing=True); e1.record(stream)
            gemm_events.append((e0, e1))
        mark("worker_gemm")
        g.gpd_inject(plan, g.GPD_FWD, Z, seeds[i % len(seeds)], g.GPD_INJECT_ADDITIVE, prob=cfg.inject_prob,
                     scale=scale, stream=stream); mark("inject")
        g.gpd_locate_errors(plan, g.GPD_FWD, Z, res, ws, stream=stream); mark("locate")
        g.gpd_decode(plan, g.GPD_FWD, Z, S, ws, result=res, stream=stream); mark("decode")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    with torch.cuda.stream(stream):
        g.gpd_encode_A(plan, Wd, Wsh, stream=stream)
        g.gpd_encode_B(plan, g.GPD_OPERAND_X_FWD, Xd, Xsh, stream=stream)
        g.gpd_worker_gemm(plan, g.GPD_FWD, Wsh, Xsh, Z, stream=stream)
        scale = float(Z.pow(2).mean().sqrt())        # injection scale = RMS of the clean outputs (caller's job)
        for i in range(warmup):
            step(i)
    barrier()
    sampler = None
    if full:
        uuid = str(torch.cuda.get_device_properties(local).uuid)
        sampler = ClockSampler(uuid)
        sampler.start()
        time.sleep(0.3)

    # ---- device-resident timing: `repeats` timed regions of exactly `steps` steps each --------------
    gemm_events = []
    region_ms = []
    for _ in range(repeats):
        barrier()
        t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            t_start.record(stream)
            for i in range(steps):
                step(i, gemm_events)
            t_end.record(stream)
        barrier()
        region_ms.append(t_start.elapsed_time(t_end))
    gemm_ms = float(np.mean([a.elapsed_time(b) for a, b in gemm_events]))

    # ---- end to end: host buffers in, result out, every step ------------------------------------
    e2e_ms = 0.0
    if full:
        barrier()
        e_start, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        # Two device input buffers: the copy of step i+1's inputs (copy stream) overlaps step i's
        # kernels (compute stream).  The first copy is not overlapped and is inside the timed region.
        copy_stream = torch.cuda.Stream()
        in_bufs = [(Wd, Xd), (torch.empty_like(Wd), torch.empty_like(Xd))]
        ready = [torch.cuda.Event() for _ in range(2)]
        consumed = [torch.cuda.Event() for _ in range(2)]
        e_start.record(stream)
        copy_stream.wait_event(e_start)
        for i in range(steps):
            b = i % 2
            with torch.cuda.stream(copy_stream):
                if i >= 2:
                    copy_stream.wait_event(consumed[b])
                in_bufs[b][0].copy_(Wh, non_blocking=True)
                in_bufs[b][1].copy_(Xh, non_blocking=True)
                ready[b].record(copy_stream)
            with torch.cuda.stream(stream):
                stream.wait_event(ready[b])
                step(i, Wd=in_bufs[b][0], Xd=in_bufs[b][1])
                consumed[b].record(stream)
                Sh.copy_(S, non_blocking=True)
                res_h.copy_(res, non_blocking=True)
        e_end.record(stream)
        barrier()
        e2e_ms = e_start.elapsed_time(e_end)
    clocks = sampler.stop() if sampler else None

    # ---- per-stage breakdown (context; separate short pass) ---------------------------------------
    stage_ms = {}
    with torch.cuda.stream(stream):
        for i in range(3):
            ev = []
            step(i, stage_events=ev)
            torch.cuda.synchronize()
            for (n0, a), (n1, b) in zip(ev[:-1], ev[1:]):
                stage_ms.setdefault(n1, []).append(a.elapsed_time(b))
    stage_ms = {k: round(float(np.mean(v)), 4) for k, v in stage_ms.items()}

    # ---- check of the last step's result (not timed): sampled rows against a direct FP64 product ---
    r = g.read_results(res)[0]
    rows = torch.arange(0, cfg.N1, max(1, cfg.N1 // 64), device="cuda")
    ref = Wd[rows].double() @ Xd.double()
    rel = float((S[rows].double() - ref).norm() / ref.norm())
    check = {"outcome": int(r.outcome), "flagged": [p for p in range(cfg.P) if r.flagged[p]],
             "rel_err_sampled_rows": rel, "device_status": g.gpd_device_status()}

    # the job's time of a region is the slowest rank's; the line reports the median region
    reduced = max_over_ranks(region_ms + [e2e_ms, gemm_ms], world, "cuda")
    region_ms, e2e_ms, gemm_ms = reduced[:repeats], reduced[repeats], reduced[repeats + 1]
    ms = float(np.median(region_ms))
    value = whole_job_tflops(useful_flops, steps, world, ms)

    if sliced:
        # The dominant kernel multiplies int8 digit planes: 21 (15) plane pairs per FP64-class product.
        # Its peak: an int8 GEMM measured in this process by the recipe of the bf16 figure; if that call
        # is unavailable, the measured bf16 figure times the nominal int8 : bf16 ratio of the part (2).
        pairs = planes * (planes + 1) // 2
        int8_ops = pairs * exec_flops
        derived = peaks["bf16_burst"] * NOMINAL_INT8_TOPS / NOMINAL_BF16_TFLOPS
        int8_measured, int8_note = measure_int8_matmul_peak(torch)
        peak = int8_measured if int8_measured else derived
        achieved = int8_ops / (gemm_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": "gemm_i8_sliced_kernel (P worker products, int8 digit planes, tcgen05)",
                    "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": TRAFFIC_BYTES_PER_LAUNCH_SLICED[planes] if args.scale_down == 1 else None,
                    "peak_source": int8_note if int8_measured else
                    f"{int8_note}; of {peaks['source']}: bf16 burst {peaks['bf16_burst']} TFLOP/s x nominal int8:bf16 ratio 2",
                    "peak_from_bf16_ratio": derived, "frac_of_bf16_ratio_peak": achieved / derived,
                    "peak_nominal_int8": NOMINAL_INT8_TOPS, "frac_of_nominal": achieved / NOMINAL_INT8_TOPS,
                    "tensor_pipe_pct_of_elapsed_ncu": TENSOR_PIPE_PCT_NCU[planes] if args.scale_down == 1 else None,
                    "ops": f"int8 multiply-adds counted as 2 operations; {pairs} digit-plane pairs per product",
                    "ops_per_launch": int8_ops, "ms_per_launch": gemm_ms,
                    "fp64_equivalent_tflops": exec_flops / (gemm_ms * 1e-3) / 1e12}
        fp64_measured = measure_fp64_matmul_peak(torch)
        roofline["fp64_peak_measured_here"] = fp64_measured       # torch.matmul FP64 8192^3, best of 10 (cuBLAS)
        roofline["fp64_equivalent_over_fp64_peak"] = roofline["fp64_equivalent_tflops"] / fp64_measured
    else:
        # FP64 tensor peak: MEASURED_PEAKS.json has no FP64 figure, and scaling its power-capped bf16
        # number by the nominal ratio gives a value below what the FP64 path delivers (FP64 does not
        # reach the power cap).  So the denominator is measured here the same way the bf16 one was:
        # torch.matmul (cuBLAS) FP64 8192^3, best of 10, CUDA events.
        fp64_measured = measure_fp64_matmul_peak(torch)
        fp64_from_ratio = peaks["bf16_sustained"] * NOMINAL_FP64_TFLOPS / NOMINAL_BF16_TFLOPS
        achieved = exec_flops / (gemm_ms * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": "dgemm_mma_kernel (P worker products, FP64 tensor path)",
                    "achieved": achieved, "peak": fp64_measured, "unit": "TFLOP/s", "frac": achieved / fp64_measured,
                    "traffic": TRAFFIC_BYTES_PER_LAUNCH,
                    "peak_source": "measured here: torch.matmul FP64 8192^3, best of 10 (cuBLAS)",
                    "peak_nominal_fp64": NOMINAL_FP64_TFLOPS,
                    "peak_from_bf16_ratio": fp64_from_ratio,
                    "flops_per_launch": exec_flops, "ms_per_launch": gemm_ms}
    # Sum of the stage rooflines (the stages depend on each other, so their floors add): algorithmic
    # bytes at the measured copy bandwidth, the products at the tensor peak of the arithmetic they run in.
    hbm = peaks["hbm_gbs"] * 1e9
    Lpos = (cfg.N1 // cfg.m) * (cfg.B // cfg.d)
    e_s = float(planes) if sliced else 8.0               # bytes per stored share value
    t_stage = {
        "encode_A": (cfg.N1 * cfg.N0 * 4 + cfg.P * (cfg.N1 // cfg.m) * (cfg.N0 // cfg.n) * e_s) / hbm,
        "encode_B": (cfg.N0 * cfg.B * 4 + cfg.P * (cfg.N0 // cfg.n) * (cfg.B // cfg.d) * e_s) / hbm,
        "worker_gemm": max((roofline.get("ops_per_launch") or roofline.get("flops_per_launch")) / (roofline["peak"] * 1e12),
                           (cfg.P * ((cfg.N1 // cfg.m) + (cfg.B // cfg.d)) * (cfg.N0 // cfg.n) * e_s + cfg.P * Lpos * 8) / hbm),
        "inject": 2 * cfg.inject_prob * cfg.P * Lpos * 8 / hbm,
        "locate": cfg.P * Lpos * 8 / hbm,
        "decode": (cfg.P * Lpos * 8 + cfg.N1 * cfg.B * 4) / hbm,
    }
    path_roofline = {"stages_us": {k: round(v * 1e6, 1) for k, v in t_stage.items()},
                     "sum_ms": sum(t_stage.values()) * 1e3,
                     "frac": sum(t_stage.values()) * 1e3 / (ms / steps),
                     "note": "sum of stage floors / measured ms_per_step; bytes at the measured copy bandwidth, "
                             "products at the peak named in roofline.peak_source"}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": "f64 (products: int8 digit planes, exact int32 accumulation)" if sliced else "f64",
        "data": "synthetic", "config": dict(workload_config(cfg), precision=precision),
        "executed_tflops": value * exec_flops / useful_flops,
        "timed_regions": {"count": repeats, "steps_each": steps, "reported": "median",
                          "ms_per_step": [round(v / steps, 5) for v in region_ms],
                          "min": min(region_ms) / steps, "max": max(region_ms) / steps},
        "gpu_launches": KERNELS_PER_STEP * steps,
        "roofline": roofline, "path_roofline": path_roofline, "stage_ms": stage_ms, "check": check,
    }
    if full:
        line["e2e"] = {"value": whole_job_tflops(useful_flops, steps, world, e2e_ms), "unit": UNIT,
                       "h2d_bytes_per_step": int(W.nbytes + X.nbytes),
                       "d2h_bytes_per_step": int(cfg.N1 * cfg.B * 4 + g.RESULT_BYTES), "ms_per_step": e2e_ms / steps}
        line["clocks"] = clocks
    if full and rank == 0 and world == 1 and cfg.N1 >= CPU_SAMPLE_ROWS:
        Wsmp = np.ascontiguousarray(W[:CPU_SAMPLE_ROWS])
        oracle_sample_step(cfg, Wsmp, X, seeds[0])                         # warm-up
        reps = 3
        stages = {}
        secs = sum(oracle_sample_step(cfg, Wsmp, X, seeds[i % len(seeds)], stages) for i in range(reps))
        line["cpu_baseline"] = {
            "value": 2.0 * CPU_SAMPLE_ROWS * cfg.N0 * cfg.B * reps / secs / 1e12, "unit": UNIT,
            "cores": cpu_threads(), "kind": "oracle",
            "sample": f"first {CPU_SAMPLE_ROWS} of {cfg.N1} rows of W (same N0, B, code and P), {reps} passes, "
                      f"{secs:.1f} s; numpy FP64 oracle",
            "stage_seconds_per_pass": {k: round(v / reps, 4) for k, v in stages.items()},
            "uncoded_product_seconds": round(oracle_uncoded_seconds(Wsmp, X), 4)}
    del Wsh, Xsh, Z
    plan.destroy()
    return line


def run_matvec(args, steps):
    """Secondary workload: the coded matrix-vector product (W 4096 x 4096 split 4 x 2, one input vector,
    threshold 9, P = 13, two single-bit flips in two node outputs).  Step = encode x, the 13 node
    products (one batched matrix-vector kernel over the stored shares of W), injection, location,
    decode; W's shares stay resident (the initial encoding of W is timed on its own)."""
    import torch
    import paper_1811_10751_b200 as g
    import workloads as wl
    cfg = wl.CONFIG_2_MATVEC
    peaks = load_peaks()
    W, X = wl.matmul_inputs(cfg)
    plan = g.gpd_plan((cfg.N1, cfg.N0, cfg.B), (cfg.m, cfg.n, cfg.d, 1), cfg.P)
    g.gpd_plan_upload(plan)
    esize = plan.query(g.GPD_Q_ELEMENT_SIZE)
    Wd, Xd = torch.from_numpy(W).cuda(), torch.from_numpy(X).cuda()
    Wsh, Xsh = plan.empty(g.GPD_Q_W_SHARE_ELEMS), plan.empty(g.GPD_Q_X_SHARE_ELEMS)
    Z = plan.empty(g.GPD_Q_OUT_ELEMS_FWD)
    S = torch.empty((cfg.N1, cfg.B), dtype=torch.float32, device="cuda")
    ws, res = plan.workspace(), g.new_results(1)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")    # larger than L2: the shares (109 MB) would fit
    stream = torch.cuda.Stream()
    g.gpd_encode_A(plan, Wd, Wsh)
    g.gpd_encode_B(plan, g.GPD_OPERAND_X_FWD, Xd, Xsh)
    g.gpd_worker_gemm(plan, g.GPD_FWD, Wsh, Xsh, Z)
    scale = float(Z.pow(2).mean().sqrt())
    gemv_events, step_events, enc_events = [], [], []

    def step(i, timed):
        # L2 flush between iterations (not timed): 256 MB written, then read back, so that L2 is left full of
        # clean lines (dirty ones would be written back under the timed kernels' reads and halve their bandwidth)
        flush.zero_()
        flush.amax()
        a, b, c, d = (torch.cuda.Event(enable_timing=True) for _ in range(4))
        a.record(stream)
        g.gpd_encode_B(plan, g.GPD_OPERAND_X_FWD, Xd, Xsh, stream=stream)
        b.record(stream)
        g.gpd_worker_gemm(plan, g.GPD_FWD, Wsh, Xsh, Z, stream=stream)
        c.record(stream)
        g.gpd_inject(plan, g.GPD_FWD, Z, cfg.inject_seeds[i % len(cfg.inject_seeds)], g.GPD_INJECT_BITFLIP,
                     count=cfg.inject_count, scale=scale, stream=stream)
        g.gpd_locate_errors(plan, g.GPD_FWD, Z, res, ws, stream=stream)
        g.gpd_decode(plan, g.GPD_FWD, Z, S, ws, result=res, stream=stream)
        d.record(stream)
        if timed:
            gemv_events.append((b, c))
            step_events.append((a, d))

    with torch.cuda.stream(stream):
        for i in range(3):
            step(i, False)
        for i in range(steps):
            step(i, True)
        for i in range(3):                               # the one-time encoding of W, on its own
            flush.zero_()
            flush.amax()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            g.gpd_encode_A(plan, Wd, Wsh, stream=stream)
            b.record(stream)
            enc_events.append((a, b))
    torch.cuda.synchronize()
    ms = float(np.mean([a.elapsed_time(b) for a, b in step_events]))
    gemv_ms = float(np.mean([a.elapsed_time(b) for a, b in gemv_events]))
    enc_ms = float(np.mean([a.elapsed_time(b) for a, b in enc_events]))
    # The step is a chain of eight short launches: the same calls captured once into a CUDA graph and
    # replayed (what a caller with a fixed step would do; the library's calls only enqueue work on the
    # stream they are given).  Reported beside the eager figure, never instead of it.
    graph_ms = None
    try:
        if getattr(args, "no_graph", False):
            raise RuntimeError("graph replay switched off")
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            g.gpd_encode_B(plan, g.GPD_OPERAND_X_FWD, Xd, Xsh, stream=stream)
            g.gpd_worker_gemm(plan, g.GPD_FWD, Wsh, Xsh, Z, stream=stream)
            g.gpd_inject(plan, g.GPD_FWD, Z, cfg.inject_seeds[0], g.GPD_INJECT_BITFLIP,
                         count=cfg.inject_count, scale=scale, stream=stream)
            g.gpd_locate_errors(plan, g.GPD_FWD, Z, res, ws, stream=stream)
            g.gpd_decode(plan, g.GPD_FWD, Z, S, ws, result=res, stream=stream)
        graph_events = []
        with torch.cuda.stream(stream):
            for i in range(3 + steps):
                flush.zero_()
                flush.amax()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                graph.replay()
                b.record(stream)
                if i >= 3:
                    graph_events.append((a, b))
        torch.cuda.synchronize()
        graph_ms = float(np.mean([a.elapsed_time(b) for a, b in graph_events]))
    except Exception as exc:                             # capture not possible here: the eager figure stands alone
        graph_ms = None
        graph_note = f"capture failed: {type(exc).__name__}"
        try:
            torch.cuda.synchronize()
        except Exception:
            pass
    r = g.read_results(res)[0]
    ref = Wd.double() @ Xd.double()
    rel = float((S.double() - ref).norm() / ref.norm())
    share_bytes = float(plan.query(g.GPD_Q_W_SHARE_ELEMS)) * esize
    enc_bytes = W.nbytes + share_bytes
    useful = 2.0 * cfg.N1 * cfg.N0 * cfg.B
    line = {"metric": METRIC, "value": useful / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": steps,
            "ms_per_step": ms, "dtype": "f32 shares, FP64 accumulation", "data": "synthetic",
            "config": {"workload": cfg.name, "split": [cfg.m, cfg.n, cfg.d], "nodes": cfg.P,
                       "threshold": plan.query(g.GPD_Q_THRESHOLD_FWD), "injection": "2 single-bit flips in 2 node outputs",
                       "step": "encode x + 13 node products + inject + locate + decode; W's shares resident",
                       "l2": "256 MB written and read back between iterations (L2 flush, not timed)"},
            "gemv_ms": gemv_ms, "graph_replay_ms_per_step": graph_ms, "encode_W_once_ms": enc_ms,
            "encode_W_hbm_frac": enc_bytes / (enc_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "check": {"outcome": int(r.outcome), "n_flagged": int(r.n_flagged), "rel_err": rel},
            "roofline": {"bound": "hbm", "kernel": "gemv_kernel (13 node products, shares read once)",
                         "achieved": share_bytes / (gemv_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": share_bytes / (gemv_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                         "peak_source": f"of {peaks['source']} copy bandwidth; bytes = the stored shares of W "
                                        f"({share_bytes / 1e6:.0f} MB) read once"}}
    plan.destroy()
    return line


def measure_tf32_matmul_peak(torch) -> float:
    """cuBLAS TF32 GEMM 8192^3, best of 10 (same recipe as the bf16 figure)."""
    n = 8192
    a = torch.randn((n, n), device="cuda")
    b = torch.randn((n, n), device="cuda")
    c = torch.empty((n, n), device="cuda")
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    for _ in range(2):
        torch.matmul(a, b, out=c)
    best = float("inf")
    for _ in range(10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        torch.matmul(a, b, out=c)
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    torch.backends.cuda.matmul.allow_tf32 = old
    return 2.0 * n ** 3 / (best * 1e-3) / 1e12


def run_layer(args, kind, steps):
    """Secondary workloads (not the headline line): the coded training step of one layer,
    step = coded forward + coded backward + coded update through coded_layer_step.
      mlp_layer: hidden layer of the MLP, 4096 x 4096 weights, batch 256, split 2 x 2, P = 10; thresholds
                 5 / 6, so FP32 shares and tensor-core 3xTF32 products
      sae_layer: encoder of the sparse autoencoder, 8192 x 1024 weights, batch 1024, split 4 x 4, P = 36;
                 thresholds 19 / 28: FP64-class arithmetic, with every product on int8 digit planes
                 (training mode; --precision fp64: FP64 shares and FP64 mma products)"""
    import torch
    import paper_1811_10751_b200 as g
    import workloads as wl
    if kind == "mlp_layer":
        c = wl.CONFIG_4_MLP
        N1, N0, B, m, n, P, prob, seed = c.widths[1], c.widths[1], c.B, c.m, c.n, c.P, c.inject_prob, c.seed
        act, wname = g.GPD_ACT_RELU, "cfg4_mlp_hidden_layer_4096x4096_b256"
    else:
        c = wl.CONFIG_5_AUTOENCODER
        N1, N0, B, m, n, P, prob, seed = c.n_hidden, c.n_visible, c.B, c.m, c.n, c.P, c.inject_prob, c.seed
        act, wname = g.GPD_ACT_SIGMOID, "cfg5_autoencoder_encoder_8192x1024_b1024"
    gen = torch.Generator(device="cuda").manual_seed(seed)
    W = torch.randn((N1, N0), device="cuda", generator=gen) * (2.0 / N0) ** 0.5
    X = torch.randn((N0, B), device="cuda", generator=gen).clamp_(min=0)
    D = torch.randn((N1, B), device="cuda", generator=gen) / B
    DT = D.t().contiguous()
    # thresholds above 9 (the autoencoder): every product on int8 digit planes (training mode) unless
    # --precision fp64 asks for the FP64 mma path; thresholds up to 9 (the MLP): FP32 shares, 3xTF32
    sliced = kind == "sae_layer" and args.precision != "fp64"
    plan = g.gpd_plan((N1, N0, B), (m, n, 1, 1), P,
                      precision=g.GPD_PREC_FP64_SLICED_TRAIN if sliced else g.GPD_PREC_AUTO)
    g.gpd_plan_upload(plan)
    f32 = plan.query(g.GPD_Q_ELEMENT_SIZE) == 4
    Wsh = plan.empty(g.GPD_Q_W_SHARE_ELEMS)
    g.gpd_encode_A(plan, W, Wsh)
    ws, res = plan.workspace(step=True), g.new_results(3)
    S, Xn = torch.empty((N1, B), device="cuda"), torch.empty((N1, B), device="cuda")
    CT = torch.empty((B, N0), device="cuda")
    stream = torch.cuda.Stream()

    def step(i):
        g.coded_layer_step(plan, g.GPD_PHASE_FWD, Wsh, X=X, activation=act, inject_seed=1000 + 16 * i,
                           inject_prob=prob, S_out=S, Xnext_out=Xn, CT_out=CT, results=res, workspace=ws,
                           stream=stream)
        g.coded_layer_step(plan, g.GPD_PHASE_BWD | g.GPD_PHASE_UPD, Wsh, X=X, Delta=D, DeltaT=DT, eta=1e-4,
                           inject_seed=1000 + 16 * i, inject_prob=prob, S_out=S, Xnext_out=Xn, CT_out=CT,
                           results=res, workspace=ws, stream=stream)

    with torch.cuda.stream(stream):
        for i in range(max(args.warmup, 3)):
            step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for i in range(steps):
            step(i)
        e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    # the same step captured once into a CUDA graph and replayed (reported beside the eager figure)
    graph_ms = None
    try:
        if getattr(args, "no_graph", False):
            raise RuntimeError("graph replay switched off")
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step(0)
        with torch.cuda.stream(stream):
            for _ in range(3):
                graph.replay()
            e0.record(stream)
            for _ in range(steps):
                graph.replay()
            e1.record(stream)
        torch.cuda.synchronize()
        graph_ms = e0.elapsed_time(e1) / steps
    except Exception:                                    # capture not possible here: the eager figure stands alone
        graph_ms = None
        try:
            torch.cuda.synchronize()
        except Exception:
            pass
    # the three tensor-core launches on their own
    Xsh, Dsh = plan.empty(g.GPD_Q_X_SHARE_ELEMS), plan.empty(g.GPD_Q_DT_SHARE_ELEMS)
    Dh, Xh = plan.empty(g.GPD_Q_DHAT_ELEMS), plan.empty(g.GPD_Q_XHAT_ELEMS)
    Zf, Zb = plan.empty(g.GPD_Q_OUT_ELEMS_FWD), plan.empty(g.GPD_Q_OUT_ELEMS_BWD)
    g.gpd_encode_B(plan, g.GPD_OPERAND_X_FWD, X, Xsh)
    g.gpd_encode_B(plan, g.GPD_OPERAND_DELTAT_BWD, DT, Dsh)
    g.gpd_encode_B(plan, g.GPD_OPERAND_DELTA_UPD, D, Dh)
    g.gpd_encode_B(plan, g.GPD_OPERAND_X_UPD, X, Xh)
    kern = {}
    for name, fn in (("forward", lambda: g.gpd_worker_gemm(plan, g.GPD_FWD, Wsh, Xsh, Zf)),
                     ("backward", lambda: g.gpd_worker_gemm(plan, g.GPD_BWD, Wsh, Dsh, Zb)),
                     ("update", lambda: g.gpd_update_shares(plan, Wsh, Dh, Xh, 1e-6, 0.0))):
        for _ in range(3):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        kern[name] = a.elapsed_time(b) / steps
    status = g.gpd_device_status()
    outcomes = [int(r.outcome) for r in g.read_results(res)[:2]]
    extra = {}
    if f32:
        peak = measure_tf32_matmul_peak(torch) / 3.0
        kernel = "sgemm_3xtf32_kernel (forward products)"
        src = "measured here: torch.matmul TF32 8192^3 best of 10, divided by 3 (3xTF32)"
        dtype = "f32 (3xTF32 products, FP64 encode/locate/decode arithmetic)"
    elif sliced:
        peak, src = measure_int8_matmul_peak(torch)
        if not peak:
            peak = load_peaks()["bf16_burst"] * NOMINAL_INT8_TOPS / NOMINAL_BF16_TFLOPS
            src += "; bf16 burst x nominal int8:bf16 ratio 2"
        kernel = "gemm_i8_sliced_kernel (forward products, 21 digit-plane pairs)"
        dtype = "f64 (products: int8 digit planes, exact int32 accumulation; FP64 shares beside the planes)"
        fp64_peak = measure_fp64_matmul_peak(torch)
        extra = {"fp64_equivalent_tflops": {k: 2.0 * P * (N1 // m) * (N0 // n) * B / (v * 1e-3) / 1e12 for k, v in kern.items()},
                 "fp64_peak_measured_here": fp64_peak, "frac_of_nominal": None}
    else:
        peak = measure_fp64_matmul_peak(torch)
        kernel = "dgemm_mma_kernel (forward products)"
        src = "measured here: torch.matmul FP64 8192^3, best of 10 (cuBLAS)"
        dtype = "f64"
    flops = 2.0 * P * (N1 // m) * (N0 // n) * B               # flops of one product over all nodes
    if sliced:
        flops *= 21                                           # executed int8 operations: 21 plane pairs per product
        extra["frac_of_nominal"] = flops / (kern["forward"] * 1e-3) / 1e12 / NOMINAL_INT8_TOPS
    useful = 3 * 2.0 * N1 * N0 * B
    line = {"metric": METRIC, "value": useful / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": dtype, "data": "synthetic",
            "config": {"workload": wname, "split": [m, n, 1, 1], "nodes": P,
                       "thresholds": [plan.query(g.GPD_Q_THRESHOLD_FWD), plan.query(g.GPD_Q_THRESHOLD_BWD)],
                       "step": "coded forward + backward + update of one layer",
                       "l2": f"shares {plan.query(g.GPD_Q_W_SHARE_ELEMS) * plan.query(g.GPD_Q_ELEMENT_SIZE) / 1e6:.0f} MB > L2"},
            "graph_replay_ms_per_step": graph_ms, "kernel_ms": kern, "device_status": status, "last_outcomes_fwd_bwd": outcomes,
            "roofline": {"bound": "tensor", "kernel": kernel,
                         "achieved": flops / (kern["forward"] * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                         "frac": flops / (kern["forward"] * 1e-3) / 1e12 / peak, "traffic": None,
                         "peak_source": src, **extra}}
    plan.destroy()
    return line


def run_positions(args, steps):
    """Secondary workload (not the headline line): per-codeword correction under the adversarial
    model on the worker outputs of the 8192 x 8192 x 512 product (P = 25, threshold 19, up to 3 errors
    per position).  1 % of the 1.05 M output positions carry 1-3 errors at nodes that differ from
    position to position; step = gpd_correct_positions + gpd_decode from all nodes."""
    import torch
    import paper_1811_10751_b200 as g
    import workloads as wl
    cfg = wl.CONFIG_3_MATMUL
    W, X = wl.matmul_inputs(cfg)
    plan = g.gpd_plan((cfg.N1, cfg.N0, cfg.B), (cfg.m, cfg.n, cfg.d, 1), cfg.P, precision=g.GPD_PREC_FP64_SLICED)
    Wd, Xd = torch.from_numpy(W).cuda(), torch.from_numpy(X).cuda()
    Wsh, Xsh = plan.empty(g.GPD_Q_W_SHARE_ELEMS), plan.empty(g.GPD_Q_X_SHARE_ELEMS)
    Z0 = plan.empty(g.GPD_Q_OUT_ELEMS_FWD)
    g.gpd_encode_A(plan, Wd, Wsh)
    g.gpd_encode_B(plan, g.GPD_OPERAND_X_FWD, Xd, Xsh)
    g.gpd_worker_gemm(plan, g.GPD_FWD, Wsh, Xsh, Z0)
    del Wsh, Xsh
    P, L = cfg.P, Z0.numel() // cfg.P
    R = P - plan.query(g.GPD_Q_THRESHOLD_FWD)
    scale = float(Z0.pow(2).mean().sqrt())
    rng = np.random.default_rng(cfg.seed + 77)
    hit = rng.choice(L, size=L // 100, replace=False)
    sizes = rng.integers(1, R // 2 + 1, size=hit.size)
    pos = np.repeat(hit, sizes)
    node = np.concatenate([rng.choice(P, size=k, replace=False) for k in sizes])
    val = rng.choice([-1.0, 1.0], size=pos.size) * rng.uniform(0.25, 8.0, size=pos.size) * scale
    Zbad = Z0.clone()
    Zbad.view(P, L)[torch.from_numpy(node).cuda(), torch.from_numpy(pos).cuda()] += torch.from_numpy(val).cuda()
    Z = torch.empty_like(Zbad)
    S = torch.empty((cfg.N1, cfg.B), dtype=torch.float32, device="cuda")
    ws_pos = torch.empty(plan.query(g.GPD_Q_POSITION_WORKSPACE_BYTES), dtype=torch.uint8, device="cuda")
    res_pos = torch.zeros(g.POSITION_RESULT_BYTES, dtype=torch.uint8, device="cuda")
    ws = plan.workspace()
    stream = torch.cuda.Stream()
    fix_events = []

    def step(timed):
        Z.copy_(Zbad, non_blocking=True)                 # the correction works in place: fresh corrupted outputs
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        g.gpd_correct_positions(plan, g.GPD_FWD, Z, workspace=ws_pos, result=res_pos, stream=stream)
        b.record(stream)
        g.gpd_decode(plan, g.GPD_FWD, Z, S, ws, use_mask=[True] * P, stream=stream)
        if timed:
            fix_events.append((a, b))

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            step(False)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(steps):
            step(True)
        e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    fix_ms = float(np.mean([a.elapsed_time(b) for a, b in fix_events]))
    r = g.read_position_result(res_pos)
    rows = torch.arange(0, cfg.N1, cfg.N1 // 64, device="cuda")
    ref = Wd[rows].double() @ Xd.double()
    rel = float((S[rows].double() - ref).norm() / ref.norm())
    peaks = load_peaks()
    nbytes = float(P) * L * Z.element_size()             # every worker output read once
    line = {"metric": "per-position error correction, positions per second", "value": L / (fix_ms * 1e-3),
            "unit": "positions/s", "n_gpus": 1, "steps": steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": "cfg3_outputs_scattered_errors", "positions": L, "nodes": P, "parity": R,
                       "errors_per_position": f"1..{R // 2} on 1 % of the positions",
                       "step": "copy of the corrupted outputs + gpd_correct_positions + gpd_decode from all nodes"},
            "correct_positions_ms": fix_ms,
            "check": {"outcome": int(r.outcome), "n_active": int(r.n_active), "n_corrected": int(r.n_corrected),
                      "n_failed": int(r.n_failed), "n_entries": int(r.n_entries), "entries_injected": int(pos.size),
                      "rel_err_sampled_rows": rel},
            "roofline": {"bound": "hbm", "kernel": "position_scan_kernel + position_fix_kernel (one call)",
                         "achieved": nbytes / (fix_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": nbytes / (fix_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                         "peak_source": f"of {peaks['source']} copy bandwidth; bytes = P x L x 8 read once "
                                        "(the repaired entries written back are 0.01 % of that)"}}
    return line


def ensure_library():
    """Built artefacts are not tracked: on a clean checkout compile libgpd.so once (nvcc, sm_100a)."""
    if os.path.exists(os.path.join(ROOT, "paper_1811_10751_b200", "libgpd.so")):
        return
    import importlib.util
    spec = importlib.util.spec_from_file_location("_gpd_build", os.path.join(ROOT, "paper_1811_10751_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod.build(force=False)


def relaunch_under_torchrun(args):
    """--gpus N > 1 without a launcher: start N ranks of this script (one per GPU) and pass their
    exit code on.  The ranks are independent replicas; rank 0 prints the line."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def under_profiler() -> bool:
    """True when a CUDA profiler has injected itself into this process (ncu, nsys, compute-sanitizer)."""
    return any(k in os.environ for k in ("CUDA_INJECTION64_PATH", "NV_COMPUTE_PROFILER_PERFWORKS_DIR",
                                         "NVTX_INJECTION64_PATH", "NV_NSIGHT_INJECTION_PORT_BASE"))


def brief(line):
    """What the `secondary` object keeps of a secondary workload's line."""
    keep = ("value", "unit", "ms_per_step", "graph_replay_ms_per_step", "dtype", "kernel_ms", "gemv_ms", "encode_W_once_ms", "encode_W_hbm_frac",
            "correct_positions_ms", "check", "last_outcomes_fwd_bwd", "device_status", "stage_ms", "path_roofline")
    out = {"workload": line["config"]["workload"], "metric": line["metric"]}
    out.update({k: line[k] for k in keep if k in line})
    if "path_roofline" in out:
        out["path_roofline"] = {"sum_ms": out["path_roofline"]["sum_ms"], "frac": out["path_roofline"]["frac"]}
    rf = line["roofline"]
    out["roofline"] = {k: rf[k] for k in ("bound", "kernel", "achieved", "peak", "unit", "frac", "peak_source") if k in rf}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scale-down", type=int, default=1,
                    help="profiling aid: same code on matrices this many times smaller per side")
    ap.add_argument("--precision", default="sliced", choices=["sliced", "sliced40", "fp64"],
                    help="worker products of the matmul workload: six (default) or five int8 digit planes on tcgen05, "
                         "or FP64 mma")
    ap.add_argument("--workload", default="matmul", choices=["matmul", "matvec", "mlp_layer", "sae_layer", "positions"],
                    help="matmul: the headline 8192 x 8192 x 512 coded product; the others are secondary: matvec, the "
                         "4096 x 4096 coded matrix-vector product; mlp_layer / sae_layer, the coded training step of one "
                         "MLP layer (FP32 path) / of the autoencoder's encoder (FP64 path); positions, per-position "
                         "correction of the headline product's outputs")
    ap.add_argument("--repeats", type=int, default=5, help="timed regions of --steps steps each (the median is reported)")
    ap.add_argument("--no-secondary", action="store_true",
                    help="leave the short runs of the other workloads out of the default line")
    ap.add_argument("--no-graph", action="store_true",
                    help="leave the CUDA-graph replay figures out (set by itself under a profiler: ncu "
                         "ends a process that launches into a stream capture)")
    args = ap.parse_args()
    args.no_graph = args.no_graph or under_profiler()
    if args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(relaunch_under_torchrun(args))
    import workloads as wl
    cfg = wl.CONFIG_3_MATMUL
    if args.scale_down > 1:
        cfg = wl.scaled_down(cfg, args.scale_down)
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if local == 0:
        ensure_library()
    else:                                            # the other ranks of a node wait for rank 0's build
        lib_path = os.path.join(ROOT, "paper_1811_10751_b200", "libgpd.so")
        for _ in range(1200):
            if os.path.exists(lib_path):
                break
            time.sleep(0.5)
    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (the library has no CPU fallback)")
    torch.cuda.set_device(local)
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if args.workload == "matmul":
        line = run_ours(args, cfg, args.precision, args.steps, max(1, args.repeats), full=True)
        if world == 1 and args.scale_down == 1 and not args.no_secondary:
            # one short run each of the other paths, so that a single default run observes them all
            short = max(3, min(args.steps, 10))
            fp64_args = argparse.Namespace(**dict(vars(args), precision="fp64"))
            sec = {}
            for name, fn in (("matmul_fp64_mma", lambda: run_ours(args, cfg, "fp64", short, 1, full=False)),
                             ("matvec", lambda: run_matvec(args, short)),
                             ("mlp_layer", lambda: run_layer(args, "mlp_layer", short)),
                             ("sae_layer", lambda: run_layer(args, "sae_layer", short)),
                             ("sae_layer_fp64_mma", lambda: run_layer(fp64_args, "sae_layer", short)),
                             ("positions", lambda: run_positions(args, short))):
                try:
                    sec[name] = brief(fn())
                except Exception as exc:                     # a secondary run never takes the headline line down
                    sec[name] = {"error": f"{type(exc).__name__}: {exc}"}
                torch.cuda.empty_cache()
            line["secondary"] = sec
    elif args.workload == "matvec":
        line = run_matvec(args, args.steps)
    elif args.workload == "positions":
        line = run_positions(args, args.steps)
    else:
        line = run_layer(args, args.workload, args.steps)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
