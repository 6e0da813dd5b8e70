#!/usr/bin/env python
"""Benchmark of the sparse x dense contraction path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--headline-only]

Headline (the JSON line's `value`): the CSR SpMM workload (1,048,576^2 matrix, ~20M nnz with
Zipf(1.8) row lengths capped at 10,000, dense B of 1,048,576 x 64 fp64). One STEP is one pass of the
whole path over that workload: comet_pack (COO -> CSR: keys, radix sort, levels) followed by
comet_spmm (merge-path partition, gather kernel, carry fix-up). `value` = compulsory bytes of the
step / step time in GB/s, with the COO entries and B resident in HBM when the timed region starts.
The per-kernel figures the metric asks for (GB/s and GFLOP/s per contraction, fraction of the
8 TB/s nominal and of the measured copy roofline) are in `kernels`, one entry per workload and op,
all at full size.

With --gpus N > 1 (launched by torch.distributed.run) every rank runs an independent replica of
the same workload (the path is defined on one GPU and has no exchange step); `value` is the sum.

--impl reference times the CPU oracle (oracle/) on the host cores on a bounded row sample of the
same workload and prints the same JSON line with "impl": "reference".
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

NOMINAL_GBS = 8000.0
FALLBACK_GBS = 6650.0
D, CU, CN, S = 0, 1, 2, 3


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_GBS, "fallback"


# --------------------------------------------------------------------------------------------- byte / flop models
def bytes_pack(nnz, order, out_index_bytes):
    """Compulsory bytes of packing: read the COO entries once, write the packed arrays once."""
    return nnz * (4 * order + 8) + out_index_bytes + nnz * 8


def model(op, fmt, case, t):
    """(compulsory bytes, flops) of one contraction; index 4 B, value 8 B; every operand once."""
    n = case.nnz
    if op == "spmv":
        I, J = case.dims
        return n * 12 + (I + 1) * 4 + J * 8 + I * 8, 2 * n
    if op == "spmm":
        I, J = case.dims
        return n * 12 + (I + 1) * 4 + J * case.R * 8 + I * case.R * 8, 2 * n * case.R
    F = t.c.crd_len[1]
    Sn = t.c.crd_len[0]
    if op == "ttv":
        K = case.dims[2]
        return n * 12 + (F + 1) * 4 + K * 8 + F * 8, 2 * n          # leaf arrays, leaf pos, v, values out
    if op == "ttm":
        K = case.dims[2]
        return n * 12 + (F + 1) * 4 + K * case.R * 8 + F * case.R * 8, 2 * n * case.R
    if op == "mttkrp":
        I, J, K = case.dims
        dense = (J + K + I) * case.R * 8
        if fmt == "coo":
            return n * 20 + dense, 3 * n * case.R
        return n * 12 + F * 8 + Sn * 8 + dense, 2 * n * case.R + 2 * F * case.R
    raise ValueError(op)


def roofline_obj(nbytes, ms, peak, peak_kind, kernel, traffic=None, **extra):
    """The roofline object of one kernel group: algorithmic bytes per call / CUDA-event time of the call."""
    gbs = nbytes / ms / 1e6
    out = {"kernel": kernel, "bound": "hbm", "achieved": round(gbs, 1), "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
           "frac": round(gbs / peak, 4), "frac_of_8000": round(gbs / NOMINAL_GBS, 4), "us_per_call": round(ms * 1e3, 1),
           "algorithmic_bytes": int(nbytes), "traffic": traffic}
    out.update(extra)
    return out


SPMM_SOURCES = ("contract_vec.cu", "spmm_heavy.cu", "spmm_heavy.cuh", "walk.cuh", "common.cuh")
SPMM_PROFILE = os.path.join("profiles", "spmm_config2.md")


def source_digest(names):
    h = hashlib.sha256()
    for n in names:
        with open(os.path.join(ROOT, "paper_2102_05187_b200", "csrc", n), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def spmm_traffic_from_profile():
    """DRAM bytes per comet_spmm call on the full workload, from the ncu summary under profiles/. The summary
    records the digest of the kernel sources it was taken with; if the sources have changed since, the figure is
    dropped (null) instead of being carried over to code it was not measured on."""
    info = {"profile": SPMM_PROFILE, "source_digest": source_digest(SPMM_SOURCES)}
    try:
        text = open(os.path.join(ROOT, SPMM_PROFILE)).read()
        traffic = float(re.search(r"traffic_bytes_per_call:\s*([0-9.eE+]+)", text).group(1))
        digest = re.search(r"source_digest:\s*([0-9a-f]+)", text).group(1)
        commit = re.search(r"commit:\s*([0-9a-f]+)", text)
        info["profile_commit"] = commit.group(1) if commit else None
        info["profile_source_digest"] = digest
        if digest != info["source_digest"]:
            info["stale"] = "kernel sources changed since the capture"
            return None, info
        return traffic, info
    except Exception as e:                                  # no summary, or not in the expected form
        info["stale"] = f"no usable profile summary ({type(e).__name__})"
        return None, info


def index_bytes(t):
    return 4 * sum(t.c.pos_len[l] + t.c.crd_len[l] for l in range(t.c.order))


# --------------------------------------------------------------------------------------------- timing helpers
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(value, dist, device):
    """The job-wide time of a measurement: the slowest rank's (identity when not distributed)."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(step_bytes, ms_per_step, world):
    """Whole-job throughput in GB/s of `world` independent replicas that each move step_bytes per step."""
    return world * step_bytes / ms_per_step / 1e6


def cuda_time(fn, reps, warm):
    """Median and min device time (ms) of fn over `reps` runs after `warm` untimed ones (CUDA events on the
    current stream)."""
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    return statistics.median(ts), min(ts)


# --------------------------------------------------------------------------------------------- our arm
def flush_l2(buf):
    buf.add_(1)


def per_kernel(comet, handle, steps, warm, peak, peak_kind="measured", scale=1.0, only=None):
    """Every workload (at full size unless `scale`): pack time and contraction time per op and format. `only`:
    restrict to these config numbers (profiling runs)."""
    out = []
    l2buf = torch.zeros(192 << 20, dtype=torch.uint8, device="cuda")      # > 126 MB L2
    plans = [(1, "spmv", "csr", (0, 1), (D, CU)), (2, "spmm", "csr", (0, 1), (D, CU)),
             (3, "ttv", "csf", (0, 1, 2), (CU, CU, CU)), (4, "ttm", "csf", (0, 1, 2), (CU, CU, CU)),
             (5, "mttkrp", "coo", (0, 1, 2), (CN, S, S)), (5, "mttkrp", "csf", (0, 1, 2), (CU, CU, CU))]
    case = None
    for cfg, op, fmt, order, attr in plans:
        if only and cfg not in only:
            continue
        if case is None or case.name[:2] != f"C{cfg}":
            case = synth.make(cfg, scale=scale, device="cuda")
        coords, val = case.coords, case.val
        small = cfg in (1, 3)              # working set near or below L2: flush between repetitions

        def do_pack():
            t = comet.pack(coords, val, case.dims, order, attr, handle)
            return t
        pack_ms = []
        for it in range(warm + min(steps, 5)):
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            t = do_pack()
            b.record()
            torch.cuda.synchronize()
            if it >= warm:
                pack_ms.append(a.elapsed_time(b))
            if it < warm + min(steps, 5) - 1:
                t.free()
        T = t
        if op == "spmv":
            x = case.dense["x"]
            y = torch.empty(case.dims[0], dtype=torch.float64, device="cuda")
            fn = lambda: comet.spmv(T, x, y)
        elif op == "spmm":
            B = case.dense["B"]
            C = torch.empty((case.dims[0], case.R), dtype=torch.float64, device="cuda")
            fn = lambda: comet.spmm(T, B, C)
        elif op == "ttv":
            v = case.dense["v"]
            Y = comet.ttv_symbolic(T, 2)
            fn = lambda: comet.ttv(T, 2, v, Y)
        elif op == "ttm":
            U = case.dense["U"]
            Y = comet.ttm_symbolic(T, 2, case.R)
            fn = lambda: comet.ttm(T, 2, U, Y)
        else:
            Fd = [None, case.dense["B"], case.dense["C"]]
            A = torch.empty((case.dims[0], case.R), dtype=torch.float64, device="cuda")
            fn = lambda: comet.mttkrp(T, 0, Fd, A)
        if small:
            run = lambda: (flush_l2(l2buf), fn())
            # time only fn: bracket it with events inside
            for _ in range(warm):
                run()
            ts = []
            for _ in range(steps):
                flush_l2(l2buf)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                fn()
                b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            med, mn = statistics.median(ts), min(ts)
        else:
            med, mn = cuda_time(fn, steps, warm)
        nbytes, flops = model(op, fmt, case, T)
        pbytes = bytes_pack(case.nnz, len(case.dims), index_bytes(T))
        pmed = statistics.median(pack_ms)
        out.append({
            "workload": case.name, "op": op, "format": fmt, "nnz": case.nnz,
            "segments": int(T.c.crd_len[1]) if len(case.dims) == 3 else int(case.dims[0]),
            "us_median": round(med * 1e3, 2), "us_min": round(mn * 1e3, 2),
            "compulsory_bytes": nbytes, "GBps": round(nbytes / med / 1e6, 1),
            "frac_of_8000": round(nbytes / med / 1e6 / NOMINAL_GBS, 4),
            "frac_of_peak": round(nbytes / med / 1e6 / peak, 4),
            "GFLOPs": round(flops / med / 1e6, 1),
            "l2": "flushed between repetitions" if small else "inputs larger than L2",
            "pack_us_median": round(pmed * 1e3, 1), "pack_compulsory_bytes": pbytes,
            "pack_GBps": round(pbytes / pmed / 1e6, 1),
            "roofline": roofline_obj(nbytes, med, peak, peak_kind, f"comet_{op} ({fmt}) on {case.name}"),
            "pack_roofline": roofline_obj(pbytes, pmed, peak, peak_kind, f"comet_pack -> {fmt} on {case.name}"),
        })
        if op == "mttkrp":
            # the two other modes of the SAME packed tensor (atomic accumulation, nothing re-packed)
            for mode in (1, 2):
                Fm = [synth.random_dense((d, case.R), case.seed, 70 + m, device="cuda") for m, d in enumerate(case.dims)]
                Fm[mode] = None
                Am = torch.empty((case.dims[mode], case.R), dtype=torch.float64, device="cuda")
                med, mn = cuda_time(lambda: comet.mttkrp(T, mode, Fm, Am), steps, warm)
                out.append({
                    "workload": case.name, "op": f"mttkrp-mode{mode + 1}-of-root-packed", "format": fmt, "nnz": case.nnz,
                    "segments": int(T.c.crd_len[1]), "us_median": round(med * 1e3, 2), "us_min": round(mn * 1e3, 2),
                    "compulsory_bytes": nbytes, "GBps": round(nbytes / med / 1e6, 1),
                    "frac_of_8000": round(nbytes / med / 1e6 / NOMINAL_GBS, 4),
                    "frac_of_peak": round(nbytes / med / 1e6 / peak, 4), "GFLOPs": round(flops / med / 1e6, 1),
                    "l2": "inputs larger than L2", "accumulation": "atomic adds (order not fixed)",
                    "roofline": roofline_obj(nbytes, med, peak, peak_kind, f"comet_mttkrp mode {mode + 1} of the root-packed {fmt}"),
                })
                del Fm, Am
        del T
        torch.cuda.empty_cache()
    return out


def cpu_baseline_sample(case, frac_rows):
    """Rows [0, I*frac) of the SpMM workload as host arrays (a bounded sample for the CPU oracle)."""
    I = case.dims[0]
    rows = max(1, int(I * frac_rows))
    keep = case.coords[0] < rows
    ci = case.coords[0][keep].cpu().numpy()
    cj = case.coords[1][keep].cpu().numpy()
    v = case.val[keep].cpu().numpy()
    B = case.dense["B"].cpu().numpy()
    return (rows, case.dims[1]), [ci, cj], v, B


def timed_cpu_baseline(dims, coords, val, B, reps=3):
    """The oracle's SpMM loop with double accumulators (-O3 -march=native): one thread and all the threads this
    process may use; mean of `reps` runs each. Bytes = the compulsory bytes of the SpMM on the sample."""
    from oracle import timed_baseline
    n = len(val)
    nbytes = n * 12 + (dims[0] + 1) * 4 + B.size * 8 + dims[0] * B.shape[1] * 8
    threads = timed_baseline.host_threads()
    out = {"host_threads": threads, "reps": reps, "what": "SpMM only, COO loops with double accumulators, gcc -O3 -march=native"}
    for label, t in (("threads_1", 1), ("threads_all", threads)):
        timed_baseline.spmm(coords, val, dims, B, t)       # warm-up (page faults of the output)
        ts = []
        for _ in range(reps):
            t0 = time.perf_counter()
            timed_baseline.spmm(coords, val, dims, B, t)
            ts.append(time.perf_counter() - t0)
        mean = sum(ts) / len(ts)
        out[label] = {"threads": t, "seconds": round(mean, 4), "GBps": round(nbytes / mean / 1e9, 3),
                      "GFLOPs": round(2 * n * B.shape[1] / mean / 1e9, 2)}
    return out


def oracle_step(dims, coords, val, B):
    import oracle
    t0 = time.perf_counter()
    pk = oracle.pack(coords, val, dims, (0, 1), (D, CU))
    oracle.spmm(coords, val, dims, B)
    dt = time.perf_counter() - t0
    n = len(val)
    nbytes = bytes_pack(n, 2, 4 * (dims[0] + 2 + n)) + n * 12 + (dims[0] + 1) * 4 + B.size * 8 + dims[0] * B.shape[1] * 8
    del pk
    return dt, nbytes


def run_kernels_only(args):
    """--kernels-only: the per-workload table alone (optionally scaled down and restricted), for profiling runs."""
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    import paper_2102_05187_b200 as comet
    handle = comet.Handle()
    peak, peak_kind = measured_peak()
    only = [int(x) for x in args.configs.split(",")] if args.configs else None
    table = per_kernel(comet, handle, max(1, args.steps), max(1, args.warmup), peak, peak_kind, args.kernels_scale, only)
    print(json.dumps({"kernels": table, "scale": args.kernels_scale}))


def run_ours(args):
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl")
    import paper_2102_05187_b200 as comet
    handle = comet.Handle()
    peak, peak_kind = measured_peak()

    case = synth.make(2, scale=args.scale, device="cuda")
    I, J = case.dims
    R = case.R
    coords, val, B = case.coords, case.val, case.dense["B"]
    C = torch.empty((I, R), dtype=torch.float64, device="cuda")
    n = case.nnz

    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    spmm_ms, pack_ms = [], []

    def step(record=False):
        if record:
            ev[0].record()
        A = comet.pack(coords, val, case.dims, (0, 1), (D, CU), handle)
        if record:
            ev[1].record()
        comet.spmm(A, B, C)
        if record:
            ev[2].record()
        return A

    for _ in range(args.warmup):
        step().free()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = handle.kernel_launches()
    torch.cuda.synchronize()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for _ in range(args.steps):
        A = step(record=True)
        torch.cuda.synchronize()          # pack syncs anyway; this only makes the per-call events readable
        pack_ms.append(ev[0].elapsed_time(ev[1]))
        spmm_ms.append(ev[1].elapsed_time(ev[2]))
        A.free()
    t_end.record()
    torch.cuda.synchronize()
    launches = handle.kernel_launches() - launches0
    clocks = sampler.stop()
    total_ms = t_start.elapsed_time(t_end)
    total_ms = max_over_ranks(total_ms, dist, "cuda")
    if dist:
        dist.barrier()
    ms_per_step = total_ms / args.steps

    A = step()
    torch.cuda.synchronize()
    spmm_bytes, spmm_flops = model("spmm", "csr", case, A)
    pack_bytes = bytes_pack(n, 2, index_bytes(A))
    step_bytes = pack_bytes + spmm_bytes
    value = aggregate_value(step_bytes, ms_per_step, world)

    # end to end through the host-buffer call: pinned COO + B in, C out, every step
    h_coords = [c.cpu().pin_memory() for c in coords]
    h_val = val.cpu().pin_memory()
    h_B = B.cpu().pin_memory()
    h_C = torch.empty((I, R), dtype=torch.float64).pin_memory()
    for _ in range(2):
        comet.spmm_from_host(h_coords, h_val, case.dims, h_B, h_C, handle)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = max(1, min(args.steps, 5))
    e0.record()
    for _ in range(e2e_steps):
        comet.spmm_from_host(h_coords, h_val, case.dims, h_B, h_C, handle)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    e2e_ms = max_over_ranks(e2e_ms, dist, "cuda")
    h2d = n * 16 + B.numel() * 8
    d2h = C.numel() * 8
    A.free()

    spmm_med = statistics.median(spmm_ms)
    traffic, traffic_info = spmm_traffic_from_profile() if args.scale == 1.0 else (None, {"stale": "not the full workload"})
    roofline = roofline_obj(
        spmm_bytes, spmm_med, peak, peak_kind,
        "comet_spmm: seg_gather_kernel<32,1,2> with two CTA roles (long rows by column blocks of B | general tiles), "
        "3 analysis kernels, 1 two-role fix-up launch", traffic=traffic, traffic_source=traffic_info,
        note="gather-bound: the 64-column rows of B (537 MB, 4x the L2) are gathered nnz times; the long rows are "
             "processed by column blocks so that their gathers hit L2, the short rows still pull their rows from DRAM")

    result = {
        "metric": "effective HBM GB/s of the SpMM path (compulsory bytes / time); per-kernel GB/s and GFLOP/s in `kernels`",
        "value": round(value, 2), "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "configs[1] CSR SpMM: 1,048,576^2 fp64, Zipf(1.8) rows capped at 10,000, B 1,048,576x64"
                               if args.scale == 1.0 else f"configs[1] at scale {args.scale}",
                   "step": "comet_pack(COO->CSR) + comet_spmm", "nnz": n, "R": R, "seed": case.seed,
                   "l2": "inputs larger than L2", "replicas": world,
                   "step_compulsory_bytes": step_bytes},
        "pack_ms_median": round(statistics.median(pack_ms), 4), "spmm_ms_median": round(spmm_med, 4),
        "spmm_GBps": round(spmm_bytes / spmm_med / 1e6, 1), "spmm_GFLOPs": round(spmm_flops / spmm_med / 1e6, 1),
        "clocks": clocks,
        "e2e": {"value": round(aggregate_value(step_bytes, e2e_ms, world), 2), "unit": "GB/s", "ms_per_step": round(e2e_ms, 3),
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "roofline": roofline,
    }

    if rank == 0 and not args.headline_only and world == 1:
        result["kernels"] = per_kernel(comet, handle, max(3, min(args.steps, 25)), max(3, args.warmup), peak, peak_kind)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        dims_s, coords_s, val_s, B_s = cpu_baseline_sample(case, args.sample_rows)
        dt, nbytes = oracle_step(dims_s, coords_s, val_s, B_s)
        result["cpu_baseline"] = {"value": round(nbytes / dt / 1e9, 4), "unit": "GB/s", "cores": 1, "kind": "oracle",
                                  "seconds": round(dt, 2), "host_cores": len(os.sched_getaffinity(0)),
                                  "sample": f"rows 0..{dims_s[0] - 1} of the workload ({len(val_s)} nnz), "
                                            "oracle.pack + oracle.spmm (long double sums), one thread; the same sample "
                                            "as --impl reference",
                                  "timed_double": timed_cpu_baseline(dims_s, coords_s, val_s, B_s)}
    if rank == 0:
        print(json.dumps(result))
    if dist:
        dist.barrier()
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------- reference arm
def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    case = synth.make(2, scale=args.scale, device="cpu")
    dims_s, coords_s, val_s, B_s = cpu_baseline_sample(case, args.sample_rows)
    for _ in range(args.warmup):
        oracle_step(dims_s, coords_s, val_s, B_s)
    times = []
    nbytes = 0
    for _ in range(args.steps):
        dt, nbytes = oracle_step(dims_s, coords_s, val_s, B_s)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = nbytes / ms / 1e6
    sample = (f"rows 0..{dims_s[0] - 1} of the workload ({len(val_s)} nnz), oracle.pack + oracle.spmm per step, "
              "one thread")
    print(json.dumps({
        "impl": "reference",
        "metric": "effective HBM GB/s of the SpMM path (compulsory bytes / time); per-kernel GB/s and GFLOP/s in `kernels`",
        "value": round(value, 4), "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", 1)), "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms, 2), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "configs[1] CSR SpMM (bounded row sample for the CPU oracle)",
                   "step": "oracle.pack(COO->CSR) + oracle.spmm", "nnz": len(val_s), "R": case.R, "seed": case.seed},
        "cpu_baseline": {"value": round(value, 4), "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample,
                         "host_cores": len(os.sched_getaffinity(0))},
        "e2e": {"value": round(value, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scale", type=float, default=1.0, help="workload scale (1.0 is the only reported one)")
    ap.add_argument("--headline-only", action="store_true", help="skip the per-kernel table")
    ap.add_argument("--kernels-only", action="store_true", help="only the per-workload table (profiling runs)")
    ap.add_argument("--kernels-scale", type=float, default=1.0, help="workload scale of --kernels-only")
    ap.add_argument("--configs", default="", help="comma-separated config numbers for --kernels-only (default: all)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sample-rows", type=float, default=1.0 / 8,
                    help="fraction of the rows in the CPU sample (the cpu_baseline leg and --impl reference use the same one)")
    args = ap.parse_args()
    if args.kernels_only:
        run_kernels_only(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # plain `python bench.py --gpus N`: start the N replicas (one process per GPU) and hand over to them
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 2000), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    if "WORLD_SIZE" in os.environ and int(os.environ["WORLD_SIZE"]) != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} does not match the launcher's WORLD_SIZE={os.environ['WORLD_SIZE']}")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
