#!/usr/bin/env python
"""Benchmark of the GETT contraction path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--dtype bf16]
    python bench.py --impl reference ...        # the CPU oracle on the host cores

One step = one gett_contract call (pack A/B tiles, macro-kernel, alpha/beta
update of C; plus the slice reduction when the plan splits K) over one seeded
synthetic input set.  The headline line is the 8192^3 GEMM control through the
tensor path; the same line carries, under "workloads", one row per workload / dtype /
split-K variant (time, TFLOP/s, GB/s, roofline fraction, plan, clocks, ratio to the
equal-sized GEMM, sampled parity against the CPU oracle) and, under "targets", which of the
seven workload/dtype pairs reach 0.70 of their roofline (`--no-workloads` leaves both out).
Prints exactly one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import (BF16_F32, DTYPE_NAMES, F32, Contraction, TensorSpec, make_inputs,  # noqa: E402
                       packed_strides, workload)

METRIC = "TFLOP/s per contraction"
UNIT = "TFLOP/s"
from workloads import F64  # noqa: E402

DTYPE_BY_NAME = {"f32": F32, "bf16": BF16_F32, "f64": F64}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"],
                "bf16_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# fp32 FMA peak: 148 SMs x 128 lanes x 2 flop at the sampled SM clock (no measured
# figure exists for it; the clock is the one seen during the timed region).
def _fp32_peak_tflops(sm_mhz: float) -> float:
    return 148 * 128 * 2 * sm_mhz * 1e6 / 1e12


def _fp64_peak_tflops(sm_mhz: float) -> float:
    """Double-precision FMA peak: 148 SMs x 64 lanes x 2 flops x clock."""
    return 148 * 64 * 2 * sm_mhz * 1e6 / 1e12


def fma_peak(ffma, dtype, sm_mhz: float) -> float:
    """Denominator of the ALU-bound fractions: the larger of the register-only FMA loop measured
    in this run and the unit counts at the given SM clock (MHz)."""
    derived = _fp64_peak_tflops(sm_mhz) if dtype == F64 else _fp32_peak_tflops(sm_mhz)
    measured = (ffma["fp64"] if dtype == F64 else ffma["tflops"]) if ffma else 0.0
    return max(measured, derived)


def measure_ffma_peak(torch, index: int):
    """fp32 FMA rate of a register-only loop (plain and two-wide packed FMAs), timed with CUDA
    events: the measured denominator of the strict-fp32 roofline fractions."""
    import ctypes
    path = os.path.join(ROOT, "paper_1607_00145_b200", "libgett_b200_bench.so")
    if not os.path.exists(path):
        return None
    lib = ctypes.CDLL(path)
    fn = lib.gett_bench_ffma_peak
    fn.restype = ctypes.c_longlong
    fn.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
    out = torch.zeros(8, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()
    sms = torch.cuda.get_device_properties(index).multi_processor_count
    res = {}
    with clock_sampler(index) as clk:
        for name, packed in (("plain", 0), ("packed", 1), ("fp64", 2)):
            best = 0.0
            for rep in range(6):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                fmas = fn(packed, 4096 if packed < 2 else 512, 2 * sms, out.data_ptr(), stream.cuda_stream)
                e1.record(stream)
                torch.cuda.synchronize()
                if fmas < 0:
                    return None
                if rep:  # the first launch is a warm-up
                    best = max(best, 2.0 * fmas / (e0.elapsed_time(e1) / 1e3) / 1e12)
            res[name] = best
        t0 = time.perf_counter()  # long enough for a few clock samples
        while time.perf_counter() - t0 < 0.3:
            fn(1, 4096, 2 * sms, out.data_ptr(), stream.cuda_stream)
            torch.cuda.synchronize()
    c = clk.summary()
    res["tflops"] = max(res["plain"], res["packed"])  # fp32; res["fp64"] is the double-precision rate
    res["sm_mhz"] = c["sm_mhz"]
    res["reasons"] = c["reasons"]
    res["derived_at_sampled_clock"] = _fp32_peak_tflops(c["sm_mhz"]) if c["sm_mhz"] else None
    res["how"] = "register-only FMA loop, 32 chains/thread, 2 x 1024 threads per SM, best of 5, CUDA events"
    return res


def run_copy_probe():
    """One launch per access pattern of the 16-byte asynchronous copy (see csrc/copy_probe_bench.cu);
    prints the time of each; meant to be run under a profiler that counts the L2 -> SM bytes."""
    import ctypes
    import torch
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_1607_00145_b200", "libgett_b200_bench.so"))
    fn = lib.gett_bench_copy_probe
    fn.restype = ctypes.c_longlong
    fn.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
    span = 384 << 20  # more than one launch touches, so that no region is read twice
    buf = torch.ones(span + 4096, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    rows = []
    for rep in range(2):
        for pattern in range(12):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            asked = fn(pattern, 64, 148 * 4, buf.data_ptr(), span, stream.cuda_stream)
            e1.record(stream)
            torch.cuda.synchronize()
            if rep:
                rows.append({"pattern": pattern, "ms": e0.elapsed_time(e1), "bytes_asked": int(asked)})
    print(json.dumps({"copy_probe": rows}))


class NvmlSampler:
    """SM clock and throttle reasons read through NVML (read-only) every few ms."""
    BITS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
            0x4: "sw_power_cap"}

    def __init__(self, index: int, period: float = 0.005):
        import pynvml
        self.nv = pynvml
        pynvml.nvmlInit()
        self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
        self.period, self.sm, self.reasons = period, [], set()
        self.max = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        self._stop = threading.Event()
        self._t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for bit, name in self.BITS.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=5)

    def summary(self):
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.max, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.sm)), "sm_max_mhz": self.max,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


def clock_sampler(index: int):
    try:
        return NvmlSampler(index)
    except Exception:
        return ClockSampler(index)


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed region runs (fallback)."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self._stop = index, [], threading.Event()
        self._t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.index}",
                                      f"--query-gpu={self.FIELDS}",
                                      "--format=csv,noheader,nounits"],
                                     capture_output=True, text=True, timeout=5).stdout.strip()
                if out:
                    self.rows.append([x.strip() for x in out.split(",")])
            except Exception:
                pass
            self._stop.wait(0.2)

    def __enter__(self):
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=10)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(np.max(mx)),
                "reasons": sorted(reasons), "samples": len(sm)}


def equal_gemm(con: Contraction) -> Contraction:
    """The plain GEMM with the same M, N, K (Sec. 7: the equal-sized GEMM line)."""
    M, N, K = con.mnk()
    return Contraction("equal-gemm", TensorSpec([0, 2], [M, K], [1, M]),
                       TensorSpec([2, 1], [K, N], [1, K]), TensorSpec([0, 1], [M, N], [1, M]))


def roofline_time_s(con, dtype, beta, peaks, fp32_peak):
    flops = con.flops()
    peak = peaks["bf16_burst"] if dtype not in (F32, F64) else fp32_peak  # (f64 rows pass their own FMA peak)
    t_c = flops / (peak * 1e12)
    t_m = con.compulsory_bytes(dtype, beta) / (peaks["hbm_gbs"] * 1e9)
    return max(t_c, t_m), ("hbm" if t_m >= t_c else ("tensor" if dtype not in (F32, F64) else "alu"))


# --------------------------------------------------------------------------- #
def run_reference(args):
    """The CPU oracle as it stands, on the host cores, on a bounded sample."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workload(args.workload)
    dtype = DTYPE_BY_NAME[args.dtype]
    con = w.contraction
    a, b, c = make_inputs(con, dtype, w.dist, w.seed, w.beta)
    cores = oracle.default_threads()
    M, N, K = con.mnk()
    rng = np.random.default_rng(0)
    npts = max(cores, int(args.ref_macs // max(K, 1)))
    pts = np.stack([rng.integers(0, e, npts) for e in con.C.extents], axis=1)

    def step():
        oracle.points(con, dtype, w.alpha, a, b, w.beta, c, pts, threads=cores)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    tflops = 2.0 * npts * K / dt / 1e12
    sample = f"{npts} random outputs of {con.C.numel} per step ({npts * K:.3g} multiply-adds)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": tflops, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": f"{w.key} {DTYPE_NAMES[dtype]} {M}x{N}x{K}", "sample": sample},
        "cpu_baseline": {"value": tflops, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": tflops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline(w, dtype, a, b, c, budget_macs):
    import oracle
    con = w.contraction
    cores = oracle.default_threads()
    K = con.mnk()[2]
    npts = max(cores, int(budget_macs // max(K, 1)))
    rng = np.random.default_rng(0)
    pts = np.stack([rng.integers(0, e, npts) for e in con.C.extents], axis=1)
    t0 = time.perf_counter()
    oracle.points(con, dtype, w.alpha, a, b, w.beta, c, pts, threads=cores)
    dt = time.perf_counter() - t0
    return {"value": 2.0 * npts * K / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{npts} random outputs of {con.C.numel} ({npts * K:.3g} multiply-adds, "
                      f"{dt:.1f} s)"}


def _to_dev(x, torch):
    if x.dtype == np.uint16:
        return torch.from_numpy(x.view(np.int16)).cuda()
    return torch.from_numpy(x).cuda()


SEARCH = 0  # --search k: every plan of the pool runs is made with opts.search = k


def time_contraction(torch, g, con, dtype, alpha, beta, dev, steps, warmup, opts=None):
    """Device-timed launches of one plan on resident inputs.  Returns seconds/launch."""
    opts = dict(opts or {})
    if SEARCH:
        opts["search"] = SEARCH
    plan = g.Plan(con, dtype, **opts)
    a, b, c = dev
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        plan(alpha, a, b, beta, c, stream)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with clock_sampler(torch.cuda.current_device()) as clk:
        e0.record(stream)
        for _ in range(steps):
            plan(alpha, a, b, beta, c, stream)
        e1.record(stream)
        torch.cuda.synchronize()
    status = plan.device_status()
    info = plan.info.as_dict()
    info["clocks"] = clk.summary()
    plan.close()
    if status != 0:
        raise RuntimeError(f"device status {status}")
    return e0.elapsed_time(e1) / 1e3 / steps, info


def max_over_ranks(seconds: float, world: int, device) -> float:
    """Timed-region length of the job: the slowest replica's (all-reduce MAX over ranks)."""
    if world <= 1:
        return seconds
    import torch
    import torch.distributed as dist
    t = torch.tensor([seconds], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replicas_value(flops_per_replica: float, world: int, sec_per_step: float) -> float:
    """Whole-job TFLOP/s of `world` independent replicas (no data-path collective)."""
    return world * flops_per_replica / sec_per_step / 1e12


def e2e_chunks(con, g, dtype, opts, nchunk: int = 8):
    """Plan for one of `nchunk` slabs along C's slowest mode, or None if the layout does not allow
    contiguous slabs: returns (operand index 0 = A / 1 = B, nchunk, slab extent, plan)."""
    from workloads import Contraction, TensorSpec, packed_strides
    C = con.C
    if not C.labels or C.strides != packed_strides(C.extents):
        return None
    lab, ext = C.labels[-1], C.extents[-1]
    if ext % nchunk:
        return None
    for which, T in ((0, con.A), (1, con.B)):
        if T.labels and T.labels[-1] == lab and T.strides == packed_strides(T.extents):
            def cut(t):
                e = list(t.extents)
                e[-1] = ext // nchunk
                return TensorSpec(list(t.labels), e, list(t.strides))
            sub = Contraction(con.name + " slab", cut(con.A) if which == 0 else con.A,
                              cut(con.B) if which == 1 else con.B, cut(C), dict(con.label_names))
            return which, nchunk, ext // nchunk, g.Plan(sub, dtype, **opts)
    return None


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_1607_00145_b200 as g

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = _peaks()
    scale = {kv.split("=")[0]: int(kv.split("=")[1]) for kv in args.scale.split(",") if kv}
    if args.workload.startswith("paper:"):  # one of the paper's 48 contractions (Table III extents), by its string
        from workloads.paper_benchmark import paper_pool
        w = [x for x in paper_pool("sp") if x.key == args.workload[6:]][0]
    else:
        w = workload(args.workload, scale or None)
    dtype = DTYPE_BY_NAME[args.dtype]
    con = w.contraction
    M, N, K = con.mnk()
    a, b, c = make_inputs(con, dtype, w.dist, w.seed, w.beta)
    dev = (_to_dev(a, torch), _to_dev(b, torch), _to_dev(c, torch))
    nbytes_in = a.nbytes + b.nbytes + (c.nbytes if w.beta != 0.0 else 0)
    l2_note = "inputs_larger_than_l2" if nbytes_in + c.nbytes > 2 * 126e6 else "l2_flush_between_steps"
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") \
        if l2_note == "l2_flush_between_steps" else None

    opts = {}
    if args.path:
        opts["path"] = args.path
    if args.split_k:
        opts["split_k"] = args.split_k
    if world > 1:  # the CTA-pair variant is for single-GPU processes only
        opts["flags"] = g.GETT_OPT_NO_PAIR
    plan = g.Plan(con, dtype, **opts)
    info = plan.info.as_dict()
    stream = torch.cuda.current_stream()
    launches_per_step = 1 + (1 if info["split_k"] > 1 else 0)

    def step():
        plan(w.alpha, dev[0], dev[1], w.beta, dev[2], stream)

    # the FMA-rate loops run first, on a GPU that the timed region has not yet pushed into its power cap
    ffma = measure_ffma_peak(torch, local) if rank == 0 else None
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(args.steps)]
    with clock_sampler(local) as clk:
        t_wall0 = time.perf_counter()
        for e0, e1 in evs:
            if flush is not None:
                flush.zero_()
            e0.record(stream)
            step()
            e1.record(stream)
        torch.cuda.synchronize()
        # keep the sampler alive long enough for at least a few samples
        while not args.kernel_only and time.perf_counter() - t_wall0 < 1.5:
            step()
            torch.cuda.synchronize()
    if plan.device_status() != 0:
        raise RuntimeError(f"kernel reported status {plan.device_status()}")
    per = np.array([e0.elapsed_time(e1) for e0, e1 in evs]) / 1e3   # seconds per launch
    total = float(per.sum())
    total = max_over_ranks(total, world, torch.device("cuda", local))
    if world > 1:
        dist.barrier()
    sec_per_step = total / args.steps
    flops = con.flops()
    value = replicas_value(flops, world, sec_per_step)
    clocks = clk.summary()
    sm_mhz = clocks["sm_mhz"] or 1965.0
    # strict-fp32 (fp64) denominator: the larger of the in-run FMA loop and the unit counts at the
    # sampled clock, so that a loop measured under a power cap cannot flatter the fractions
    fp32_peak = fma_peak(ffma, F64 if dtype == F64 else F32, sm_mhz)

    # ---- roofline of the contraction kernel ----
    avg = float(per.mean())
    t_roof, bound = roofline_time_s(con, dtype, w.beta, peaks, fp32_peak)
    if bound == "hbm":
        achieved = con.compulsory_bytes(dtype, w.beta) / avg / 1e9
        peak, runit = peaks["hbm_gbs"], "GB/s"
        peak_note = f"{peaks['source']} HBM copy bandwidth"
    elif bound == "tensor":
        achieved = flops / avg / 1e12
        sustained = total > 1.0
        peak = peaks["bf16_sustained"] if sustained else peaks["bf16_burst"]
        runit = "TFLOP/s"
        peak_note = f"{peaks['source']} cuBLAS bf16 {'sustained' if sustained else 'burst'}"
    else:
        achieved = flops / avg / 1e12
        peak, runit = fp32_peak, "TFLOP/s"
        peak_note = ("the larger of the register-only FMA loop measured in this run and the unit counts "
                     f"(148 SM x {64 if dtype == F64 else 128} lanes x 2) at the sampled {sm_mhz:.0f} MHz")
    # DRAM bytes of one launch: not measured by this run (it needs a profiler pass); the figure
    # is the one-pass ncu capture of this same workload that the named summary records
    traffic, traffic_source = None, None
    tpath = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tpath) and not scale:
        with open(tpath) as f:
            ent = json.load(f).get(f"{w.key}:{DTYPE_NAMES[dtype]}:{info['path']}")
        if isinstance(ent, dict):
            traffic, traffic_source = ent.get("bytes"), ent.get("source")
    roofline = {"bound": bound, "achieved": achieved, "peak": peak, "unit": runit,
                "frac": achieved / peak, "traffic": traffic, "traffic_source": traffic_source,
                "peak_note": peak_note,
                "kernel_ms_avg": avg * 1e3, "kernel_ms_min": float(per.min()) * 1e3,
                "roofline_time_ms": t_roof * 1e3}

    out = None
    if rank == 0 and args.kernel_only:
        out = {"metric": METRIC, "value": value, "unit": UNIT, "ms_per_step": sec_per_step * 1e3,
               "config": {"workload": f"{w.key} {DTYPE_NAMES[dtype]} {M}x{N}x{K}", "info": info},
               "roofline": roofline, "clocks": clocks}
        if ffma:
            out["ffma_peak"] = ffma
        if args.all:
            out["workloads"] = run_all(torch, g, peaks, ffma, args)
            out["targets"] = targets_summary(out["workloads"])
        if args.pool:
            out.update(run_pool(torch, g, peaks, args))
        if args.paper_pool:
            from workloads.paper_benchmark import fig11_sweep, paper_pool
            out.update(run_pool(torch, g, peaks, args, paper_pool("sp"), "paper_pool"))
            out.update(run_pool(torch, g, peaks, args, fig11_sweep(), "fig11"))
            # the paper's own figures for the same statistic (one Haswell core, MKL GEMM): context only
            if args.paper_pool_dp and ffma:  # Table IV: the same contractions with their double-precision extents
                out.update(run_pool(torch, g, peaks, args, paper_pool("dp"), "paper_pool_dp", dtypes=(F64,),
                                    fp_peak=fma_peak(ffma, F64, 1965.0)))
            out["paper_pool_context"] = {"gett_vs_equal_gemm_percent_sp": {"min": 72.4, "mean": 98.1, "max": 141.4},
                                         "source": "Sec. 7.2, Fig. 9"}
    elif rank == 0:
        # ---- end to end through the C ABI with host buffers ----
        pin = [torch.from_numpy(x.view(np.int16) if x.dtype == np.uint16 else x).pin_memory()
               for x in (a, b, c)]
        c_host = torch.empty(c.size, dtype=torch.float32).pin_memory()
        e2e_steps = max(1, min(args.steps, args.e2e_steps))

        def e2e_step():
            dev[0].copy_(pin[0], non_blocking=True)
            dev[1].copy_(pin[1], non_blocking=True)
            if w.beta != 0.0:
                dev[2].copy_(pin[2], non_blocking=True)
            plan(w.alpha, dev[0], dev[1], w.beta, dev[2], stream)
            c_host.copy_(dev[2], non_blocking=True)

        note = "single-GPU figure; plan reused, pinned host buffers"
        chunks = e2e_chunks(con, g, dtype, opts)
        if chunks is not None:
            # C's slowest mode is also the slowest mode of the operand that carries it: cut both
            # along it into slabs that are contiguous in memory and overlap the copies of one
            # slab (both directions) with the contraction of another, on three streams.
            which, nchunk, step_elems, sub_plan = chunks
            s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
            whole = 1 - which  # the operand that is not cut is copied first
            opd_step = dev[which].numel() // nchunk
            c_step = dev[2].numel() // nchunk
            ev_in = [torch.cuda.Event() for _ in range(nchunk)]
            ev_done = [torch.cuda.Event() for _ in range(nchunk)]

            def e2e_step():  # noqa: F811
                s_in.wait_stream(stream)
                with torch.cuda.stream(s_in):
                    dev[whole].copy_(pin[whole], non_blocking=True)
                    for i in range(nchunk):
                        o = slice(i * opd_step, (i + 1) * opd_step)
                        dev[which][o].copy_(pin[which][o], non_blocking=True)
                        if w.beta != 0.0:
                            cs = slice(i * c_step, (i + 1) * c_step)
                            dev[2][cs].copy_(pin[2][cs], non_blocking=True)
                        ev_in[i].record(s_in)
                for i in range(nchunk):
                    stream.wait_event(ev_in[i])
                    o = slice(i * opd_step, (i + 1) * opd_step)
                    cs = slice(i * c_step, (i + 1) * c_step)
                    ops = [dev[0], dev[1]]
                    ops[which] = dev[which][o]
                    sub_plan(w.alpha, ops[0], ops[1], w.beta, dev[2][cs], stream)
                    ev_done[i].record(stream)
                    s_out.wait_event(ev_done[i])
                    with torch.cuda.stream(s_out):
                        c_host[cs].copy_(dev[2][cs], non_blocking=True)
                stream.wait_stream(s_out)

            note = (f"single-GPU figure; pinned host buffers; {nchunk} slabs along C's slowest mode, "
                    "copies of one slab overlapped with the contraction of another")

        e2e_step()
        torch.cuda.synchronize()
        if chunks is not None:  # the pipelined step must give the same C as one call
            plan(w.alpha, dev[0], dev[1], w.beta, dev[2].copy_(pin[2]), stream)
            torch.cuda.synchronize()
            if not torch.equal(dev[2].cpu(), c_host):
                raise RuntimeError("pipelined end-to-end step disagrees with the single call")
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        s1.record(stream)
        torch.cuda.synchronize()
        e2e_s = s0.elapsed_time(s1) / 1e3 / e2e_steps
        e2e = {"value": flops / e2e_s / 1e12, "unit": UNIT, "h2d_bytes_per_step": int(nbytes_in),
               "d2h_bytes_per_step": int(c.nbytes), "steps": e2e_steps, "note": note}

        # ---- equal-sized GEMM through the same kernels (Sec. 7) ----
        extra = {}
        if not con.is_plain_gemm():
            eg = equal_gemm(con)
            ga, gb, gc = make_inputs(eg, dtype, w.dist, w.seed, w.beta)
            gdev = (_to_dev(ga, torch), _to_dev(gb, torch), _to_dev(gc, torch))
            t_eq, _ = time_contraction(torch, g, eg, dtype, w.alpha, w.beta, gdev,
                                       max(3, args.steps // 2), args.warmup)
            extra["equal_gemm"] = {"tflops": flops / t_eq / 1e12, "speedup_vs_equal_gemm": t_eq / avg}
            del gdev

        base = cpu_baseline(w, dtype, a, b, c, 8 * args.ref_macs)
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec_per_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": DTYPE_NAMES[dtype] + "-in/f32-acc"
            if dtype != F32 else "f32", "data": "synthetic",
            "config": {"workload": f"{w.key} {DTYPE_NAMES[dtype]} {M}x{N}x{K} alpha={w.alpha} "
                                   f"beta={w.beta}", "l2": l2_note, "replicas": world,
                       "path": info["path"], "tile": [info["tile_m"], info["tile_n"], info["tile_k"]],
                       "stages": info["stages"], "split_k": info["split_k"],
                       "loaders": [info["loader_a"], info["loader_b"]],
                       "epilogue": info["epilogue"], "grid": info["grid"]},
            "roofline": roofline, "cpu_baseline": base, "e2e": e2e,
            "gpu_launches": args.steps * launches_per_step, "clocks": clocks, **extra,
        }
        if ffma:
            out["ffma_peak"] = ffma
        if not args.no_workloads and world == 1:
            del dev
            out["workloads"] = run_all(torch, g, peaks, ffma, args)
            out["targets"] = targets_summary(out["workloads"])
    plan.close()
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def time_plan(torch, plan, alpha, beta, dev, steps, warmup, flush):
    """Per-launch device times (seconds, one CUDA-event pair per launch on the launching
    stream) of a plan on resident inputs, the L2 flushed between launches when `flush` is
    given; returns (times, clock summary)."""
    a, b, c = dev
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        plan(alpha, a, b, beta, c, stream)
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    with clock_sampler(torch.cuda.current_device()) as clk:
        t0 = time.perf_counter()
        for e0, e1 in evs:
            if flush is not None:
                flush.zero_()
            e0.record(stream)
            plan(alpha, a, b, beta, c, stream)
            e1.record(stream)
        torch.cuda.synchronize()
        while time.perf_counter() - t0 < 0.05:  # at least a few clock samples under load
            plan(alpha, a, b, beta, c, stream)
            torch.cuda.synchronize()
    if plan.device_status() != 0:
        raise RuntimeError(f"device status {plan.device_status()}")
    return np.array([e0.elapsed_time(e1) for e0, e1 in evs]) / 1e3, clk.summary()


def equal_gemm_seconds(torch, g, con, dtype, alpha, beta, steps, flush):
    """Median launch time of the plain GEMM with the same M, N, K through the same library
    (Sec. 7: the equal-sized GEMM line); its operands are seeded uniform[-1, 1) device draws."""
    eg = equal_gemm(con)
    gen = torch.Generator(device="cuda").manual_seed(1234)
    def draw(n, as16):
        x = torch.empty(n, dtype=torch.float32, device="cuda").uniform_(-1.0, 1.0, generator=gen)
        return x.to(torch.bfloat16).view(torch.int16) if as16 else x
    dev = (draw(eg.A.span, dtype != F32), draw(eg.B.span, dtype != F32), draw(eg.C.span, False))
    plan = g.Plan(eg, dtype)
    try:
        t, _ = time_plan(torch, plan, alpha, beta, dev, steps, 3, flush)
        info = plan.info.as_dict()
    finally:
        plan.close()
    return float(np.median(t)), info


TARGET_PAIRS = [("cfg2", "bf16"), ("cfg2", "f32"), ("cfg3", "f32"), ("cfg4", "bf16"), ("cfg4", "f32"),
                ("cfg5", "bf16"), ("cfg5", "f32")]


def run_all(torch, g, peaks, ffma, args, keys=None):
    """One row per workload / dtype / variant: launch time (median and min of per-launch CUDA
    events), TFLOP/s, GB/s, roofline fraction and bound, the plan, the SM clock and throttle
    reasons sampled during the row, the ratio to the equal-sized GEMM through the same library,
    and -- the row's CPU-baseline leg -- the oracle timed on a bounded sample of the row's
    outputs, whose values also give the row's acceptance ratio.  fp32 fractions use the FMA
    peak of this run (`fma_peak`: the measured loop or the unit counts at the row's clock, whichever is larger)."""
    import oracle
    rows = []
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for key in keys or ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "splitk", "splitk_vec"):
        w = workload(key)
        con = w.contraction
        M, N, K = con.mnk()
        for dtype in w.dtypes:
            a, b, c = make_inputs(con, dtype, w.dist, w.seed, w.beta)
            dev = (_to_dev(a, torch), _to_dev(b, torch), _to_dev(c, torch))
            small = a.nbytes + b.nbytes + c.nbytes * (2 if w.beta != 0.0 else 1) <= 2 * 126e6
            flush = flush_buf if small else None
            variants = [("auto", {})]
            if key == "cfg3":
                # K = 24 is one slab of the vector kernels; only the scalar path can slice it
                variants += [("scalar split_k=1", {"path": 1, "split_k": 1}),
                             ("scalar split_k=2", {"path": 1, "split_k": 2})]
            if key in ("splitk", "splitk_vec"):
                variants += [("split_k=1", {"split_k": 1}), ("split_k=4", {"split_k": 4}),
                             ("split_k=16", {"split_k": 16})]
            # sampled outputs for the parity / CPU-baseline leg (the same for every variant)
            rng = np.random.default_rng(7)
            npts = int(max(64, min(4096, args.row_macs // max(K, 1))))
            ext = np.array(con.C.extents, dtype=np.int64)
            pts = np.concatenate([np.zeros((1, len(ext)), np.int64), (ext - 1)[None, :],
                                  np.stack([rng.integers(0, e, npts) for e in ext], axis=1)], axis=0)
            off = (pts * np.array(con.C.strides, dtype=np.int64)).sum(axis=1)
            cores = oracle.default_threads()
            t0 = time.perf_counter()
            ref, absacc = oracle.points(con, dtype, w.alpha, a, b, w.beta, c, pts, threads=cores)
            t_cpu = time.perf_counter() - t0
            scale = abs(w.alpha) * absacc
            if w.beta != 0.0:
                scale = scale + abs(w.beta) * np.abs(c[off].astype(np.float64))
            off_dev = torch.from_numpy(off).cuda()
            for name, opts in variants:
                row = {"workload": key, "dtype": DTYPE_NAMES[dtype], "variant": name, "mnk": [M, N, K]}
                try:
                    plan = g.Plan(con, dtype, **opts)
                except Exception as e:  # an unsupported forced option is reported, not fatal
                    row["error"] = str(e)
                    rows.append(row)
                    continue
                try:
                    # parity on a fresh C (NaN where beta == 0: C must not be read)
                    if w.beta == 0.0:
                        dev[2].fill_(float("nan"))
                    else:
                        dev[2].copy_(torch.from_numpy(c))
                    plan(w.alpha, dev[0], dev[1], w.beta, dev[2], torch.cuda.current_stream())
                    torch.cuda.synchronize()
                    got = dev[2][off_dev].cpu().numpy().astype(np.float64)
                    parity = float(np.max(np.abs(got - ref)) / np.max(scale)) if np.all(np.isfinite(got)) \
                        else float("inf")
                    if w.beta != 0.0:
                        dev[2].copy_(torch.from_numpy(c))
                    steps = args.all_steps if M * N * K < 4e12 else max(3, args.all_steps // 2)
                    t, clocks = time_plan(torch, plan, w.alpha, w.beta, dev, steps, 3, flush)
                    info = plan.info.as_dict()
                finally:
                    plan.close()
                med, tmin = float(np.median(t)), float(t.min())
                fp32_peak = fma_peak(ffma, dtype, clocks["sm_mhz"] or 1965.0)  # at this row's own clock
                t_roof, bound = roofline_time_s(con, dtype, w.beta, peaks, fp32_peak)
                row.update({
                    "ms": med * 1e3, "ms_min": tmin * 1e3, "tflops": con.flops() / med / 1e12,
                    "gbs": con.compulsory_bytes(dtype, w.beta) / med / 1e9, "bound": bound,
                    "roofline_ms": t_roof * 1e3, "roofline_frac": t_roof / med,
                    "roofline_frac_best": t_roof / tmin,
                    "path": info["path"], "tile": [info["tile_m"], info["tile_n"], info["tile_k"]],
                    "stages": info["stages"], "loaders": [info["loader_a"], info["loader_b"]],
                    "epilogue": info["epilogue"], "split_k": info["split_k"], "grid": info["grid"],
                    "swapped": info["swapped"], "l2": "flushed" if small else "inputs_larger_than_l2",
                    "sm_mhz": clocks["sm_mhz"], "clock_reasons": clocks["reasons"],
                    "parity_ratio": parity, "parity_points": int(len(off)), "parity_ok": bool(parity <= 1e-5),
                    "cpu_baseline": {"value": 2.0 * len(off) * K / t_cpu / 1e12, "unit": UNIT, "cores": cores,
                                     "kind": "oracle", "sample": f"{len(off)} outputs, {t_cpu:.2f} s"},
                })
                if name == "auto" and not con.is_plain_gemm():
                    t_eq, ginfo = equal_gemm_seconds(torch, g, con, dtype, w.alpha, w.beta, steps, flush)
                    row["equal_gemm_ms"] = t_eq * 1e3
                    row["speedup_vs_equal_gemm"] = t_eq / med
                rows.append(row)
            del dev, off_dev
    return rows


def targets_summary(rows):
    """The seven workload/dtype pairs of the stated target: roofline fraction of the automatic
    plan and whether it reaches 0.70."""
    out = []
    for key, dt in TARGET_PAIRS:
        r = [x for x in rows if x.get("workload") == key and x.get("dtype") == dt and x.get("variant") == "auto"
             and "roofline_frac" in x]
        if r:
            out.append({"workload": key, "dtype": dt, "bound": r[0]["bound"], "roofline_frac": r[0]["roofline_frac"],
                        "met": bool(r[0]["roofline_frac"] >= 0.70), "parity_ok": r[0]["parity_ok"]})
    return {"threshold": 0.70, "pairs": out, "met": sum(1 for x in out if x["met"]), "of": len(out)}


def ttgt_seconds(torch, g, con, dtype, alpha, beta, dev, steps, flush):
    """Transpose-Transpose-GEMM-Transpose on the GPU (Sec. 4, Listing 5), the approach GETT is
    measured against: A and B are unfolded into packed matrices A'[M,K], B'[K,N] by explicit
    transpositions into auxiliary memory (torch's permuting copy), multiplied by the plain GEMM of
    this library, and the result C'[M,N] is folded back into C's layout.  Transpositions that are
    the identity are skipped (as the paper's TTGT candidates do).  Returns (seconds, seconds spent
    in the transpositions).  Every tensor must be packed."""
    im, in_, ik = con.index_sets()
    ext = con.extent_of()

    def view(t, x):       # the flat device array as a torch view with one dim per mode (first mode fastest)
        return x.view(tuple(reversed(t.extents))).permute(*reversed(range(len(t.extents))))

    def unfold(t, x, rows, cols):   # -> packed matrix [prod rows, prod cols], rows fastest
        v = view(t, x)
        order = [t.labels.index(l) for l in rows + cols]
        identity = order == list(range(len(order)))
        return v.permute(*order), identity

    a, b, c = dev
    el = torch.bfloat16 if dtype != F32 else torch.float32
    a_t, b_t = (a.view(torch.bfloat16), b.view(torch.bfloat16)) if dtype != F32 else (a, b)
    M, N, K = con.mnk()
    eg = equal_gemm(con)
    plan = g.Plan(eg, dtype)
    a_m = torch.empty(M * K, dtype=el, device="cuda")
    b_m = torch.empty(K * N, dtype=el, device="cuda")
    c_m = torch.empty(M * N, dtype=torch.float32, device="cuda")
    va, ida = unfold(con.A, a_t, im, ik)
    vb, idb = unfold(con.B, b_t, ik, in_)
    c_order = [con.C.labels.index(l) for l in im + in_]
    idc = c_order == list(range(len(c_order)))
    vc = view(con.C, c)
    shape_a = tuple(reversed([ext[l] for l in im + ik]))
    shape_b = tuple(reversed([ext[l] for l in ik + in_]))
    shape_c = tuple(reversed([ext[l] for l in im + in_]))
    stream = torch.cuda.current_stream()

    def to_packed(dst, v, shape):   # dst (first-mode-fastest packed) <- v
        dst.view(shape).copy_(v.permute(*reversed(range(v.dim()))))

    def step(timers=None):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)] if timers is not None else None
        if ev:
            ev[0].record(stream)
        if not ida:
            to_packed(a_m, va, shape_a)
        if not idb:
            to_packed(b_m, vb, shape_b)
        if not idc and beta != 0.0:   # C' <- C for the update
            to_packed(c_m, vc.permute(*c_order), shape_c)
        if ev:
            ev[1].record(stream)
        am = a_m if not ida else a_t
        bm = b_m if not idb else b_t
        cm = c_m if not idc else c
        plan(alpha, am.view(torch.int16) if dtype != F32 else am, bm.view(torch.int16) if dtype != F32 else bm,
             beta, cm, stream)
        if ev:
            ev[2].record(stream)
        if not idc:   # C <- C'
            inv = [c_order.index(i) for i in range(len(c_order))]
            vc.copy_(c_m.view(shape_c).permute(*reversed(range(len(shape_c)))).permute(*inv))
        if ev:
            ev[3].record(stream)
            timers.append(ev)

    for _ in range(2):
        step()
    torch.cuda.synchronize()
    timers = []
    for _ in range(steps):
        if flush is not None:
            flush.zero_()
        step(timers)
    torch.cuda.synchronize()
    plan.close()
    tot = np.array([e[0].elapsed_time(e[3]) for e in timers]) / 1e3
    tr = np.array([e[0].elapsed_time(e[1]) + e[2].elapsed_time(e[3]) for e in timers]) / 1e3
    return float(np.median(tot)), float(np.median(tr))


def run_pool(torch, g, peaks, args, items=None, label="pool", dtypes=None, fp_peak=None):
    """A pool of contractions -- the seeded synthetic pool (workloads.pool) or the paper's own 48
    shapes and its Fig. 11 sweep (workloads.paper_benchmark): per item and dtype the plan,
    TFLOP/s, roofline fraction and the ratio to the equal-sized GEMM through the same library
    (the paper's Sec. 7 statistic), plus the distribution of that ratio."""
    from workloads import pool
    rows = []
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for w in (items if items is not None else pool()):
        con = w.contraction
        for dtype in (dtypes or w.dtypes):
            a, b, c = make_inputs(con, dtype, w.dist, w.seed, w.beta, cache=True)
            dev = (_to_dev(a, torch), _to_dev(b, torch), _to_dev(c, torch))
            t, info = time_contraction(torch, g, con, dtype, w.alpha, w.beta, dev, args.all_steps, 3)
            flush.zero_()
            mhz = info["clocks"]["sm_mhz"] or 1965.0
            t_roof, bound = roofline_time_s(con, dtype, w.beta, peaks, fp_peak or _fp32_peak_tflops(mhz))
            eg = equal_gemm(con)
            ga, gb, gc = make_inputs(eg, dtype, w.dist, w.seed, w.beta)
            gdev = (_to_dev(ga, torch), _to_dev(gb, torch), _to_dev(gc, torch))
            t_eq, _ = time_contraction(torch, g, eg, dtype, w.alpha, w.beta, gdev, args.all_steps, 3)
            M, N, K = con.mnk()
            extra = {}
            if args.ttgt and dtype != F64:
                t_ttgt, t_tr = ttgt_seconds(torch, g, con, dtype, w.alpha, w.beta, dev, args.all_steps, None)
                extra = {"ttgt_ms": t_ttgt * 1e3, "ttgt_transpose_share": t_tr / t_ttgt,
                         "speedup_vs_ttgt": t_ttgt / t}
            rows.append({**extra, "item": w.key, "spec": con.name, "dtype": DTYPE_NAMES[dtype], "mnk": [M, N, K],
                         "ms": t * 1e3, "tflops": con.flops() / t / 1e12, "bound": bound,
                         "roofline_frac": t_roof / t, "path": info["path"],
                         "loaders": [info["loader_a"], info["loader_b"]], "epilogue": info["epilogue"],
                         "tile": [info["tile_m"], info["tile_n"], info["tile_k"]],
                         "split_k": info["split_k"], "speedup_vs_equal_gemm": t_eq / t,
                         "model_us": info["model_us"], "candidates": info["candidates"],
                         "model_rank": info["model_rank"], "timed": info["timed"]})
            del dev, gdev
    out = {label: rows}
    for name in sorted(DTYPE_BY_NAME):
        r = np.array([x["speedup_vs_equal_gemm"] for x in rows if x["dtype"] == name])
        f = np.array([x["roofline_frac"] for x in rows if x["dtype"] == name])
        if r.size:
            out[f"{label}_ratio_to_equal_gemm_{name}"] = {
                "min": float(r.min()), "mean": float(r.mean()), "median": float(np.median(r)),
                "max": float(r.max()), "n": int(r.size)}
            tt = np.array([x["speedup_vs_ttgt"] for x in rows if x["dtype"] == name and "speedup_vs_ttgt" in x])
            if tt.size:
                out[f"{label}_speedup_vs_ttgt_{name}"] = {"min": float(tt.min()), "mean": float(tt.mean()),
                                                          "median": float(np.median(tt)), "max": float(tt.max()),
                                                          "n": int(tt.size)}
            out[f"{label}_roofline_frac_{name}"] = {
                "min": float(f.min()), "median": float(np.median(f)), "max": float(f.max()),
                "at_least_0.7": int((f >= 0.7).sum()), "n": int(f.size)}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--dtype", default="bf16", choices=sorted(DTYPE_BY_NAME))
    ap.add_argument("--path", type=int, default=0, help="force a gett_path_t")
    ap.add_argument("--split-k", type=int, default=0)
    ap.add_argument("--scale", default="", help="override extents, e.g. m=4096,n=4096 (profiling)")
    ap.add_argument("--pool", action="store_true",
                    help="with --kernel-only: also time the seeded pool of synthetic contractions")
    ap.add_argument("--paper-pool", action="store_true",
                    help="with --kernel-only: the paper's 48 contractions (Table III extents) and its Fig. 11 sweep")
    ap.add_argument("--paper-pool-dp", action="store_true",
                    help="with --paper-pool: also the 48 contractions with their Table IV extents in double precision")
    ap.add_argument("--copy-probe", action="store_true",
                    help="run the access-pattern probe of the 16-byte asynchronous copy and exit")
    ap.add_argument("--ttgt", action="store_true",
                    help="pool runs: also time Transpose-Transpose-GEMM-Transpose (torch transpositions + this "
                         "library's plain GEMM) and report GETT's speedup over it")
    ap.add_argument("--search", type=int, default=0,
                    help="pool runs: make every plan with opts.search = k (model ranking, k best timed)")
    ap.add_argument("--kernel-only", action="store_true",
                    help="skip the end-to-end, equal-GEMM and CPU legs (profiling runs)")
    ap.add_argument("--all", action="store_true", help="with --kernel-only: also time every workload")
    ap.add_argument("--no-workloads", action="store_true",
                    help="leave the per-workload rows and the targets summary out of the line")
    ap.add_argument("--all-steps", type=int, default=10)
    ap.add_argument("--row-macs", type=float, default=1.0e8,
                    help="multiply-adds in the oracle's sample of each per-workload row")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--ref-macs", type=float, default=5.0e8,
                    help="multiply-adds in the oracle's bounded sample")
    args = ap.parse_args()
    global SEARCH
    SEARCH = args.search
    if args.copy_probe:
        run_copy_probe()
        return
    if args.dtype == "f64":
        args.kernel_only = True  # (the end-to-end and equal-GEMM legs are set up for fp32 outputs)
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
