#!/usr/bin/env python
"""Benchmark: forward + all gradients of one synthetic workload through the C ABI.

One step = tad_forward + tad_backward (every gradient) on device-resident inputs.  Prints ONE
JSON line (rank 0).  With --gpus N > 1 (under torchrun) every rank runs an independent replica
of the same workload on its own GPU; there is no data-path collective.
`--impl reference` times the float64 CPU oracle on a bounded sample of the same workload.
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

METRIC = "fwd+bwd tensor elements/s"
UNIT = "elements/s"

# rows of the output the oracle sample covers, per workload (about 10-30 s of CPU work on 16 cores)
ORACLE_SAMPLE_ROWS = {"cfg1": 64, "cfg2": 2048, "cfg3": 4096, "cfg4": 96, "cfg5": 1}
# ... and per step of the reference arm, which repeats it steps + warmup times (a second or two each)
REFERENCE_STEP_ROWS = {"cfg1": 64, "cfg2": 256, "cfg3": 4096, "cfg4": 16, "cfg5": 1}


# how every workload keeps the timed iterations from running out of L2 (126 MB)
L2_NOTE = {
    "cfg1": "launch-latency case: 100 KB of tensors, resident in L2 (no roofline fraction is meaningful)",
    "cfg2": "inputs larger than L2 (df and c are 268 MB each)",
    "cfg3": "inputs larger than L2 per step (df, f, W and dW are 67 MB each: 268 MB cross HBM between two launches of a part)",
    "cfg4": "inputs larger than L2 (df and f are 537 MB each)",
    "cfg5": "inputs larger than L2 (x and dx are 269 MB, df and f 134 MB each)",
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": float(d["hbm_gbs"]), "sm_max_mhz": float(d.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.samples = []
        self.proc = None
        self.thread = None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 6:
                self.samples.append(parts)

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=5)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for p in self.samples:
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for name, v in zip(names, p[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def source_digest() -> str:
    """Digest of the kernel sources: ncu counters recorded for another digest are stale."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_1711_01348_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        with open(os.path.join(csrc, name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str, part: str):
    """DRAM bytes per launch of one part from the committed ncu capture, or None if absent or stale."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as fh:
        rec = json.load(fh)
    if rec.get("source_digest") != source_digest():
        return None
    return rec.get(workload, {}).get(part)


def elements_per_step(expr) -> int:
    n = 1
    for s in expr.out_shape:
        n *= s
    for shape in expr.arg_shapes:
        m = 1
        for s in shape:
            m *= s
        n += m
    return n


def oracle_sample(key, expr, args, df, nthreads, table=None):
    """Runs the oracle, as it stands, on the first rows of the output; returns (seconds, elements)."""
    from oracle.oracle import Oracle
    rows = min((table or ORACLE_SAMPLE_ROWS)[key], expr.out_shape[0])
    lo = [0] * len(expr.out_shape)
    hi = [rows] + list(expr.out_shape[1:])
    orc = Oracle(expr)
    t0 = time.perf_counter()
    orc.forward(args, lo, hi, nthreads=nthreads)
    orc.backward(args, df, lo, hi, nthreads=nthreads)
    dt = time.perf_counter() - t0
    frac = rows / expr.out_shape[0]
    return dt, elements_per_step(expr) * frac, f"output rows [0, {rows}) of {expr.out_shape[0]} ({frac:.4%} of one step), forward + all gradients"


def run_reference(opts):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle.oracle import build as build_oracle, max_threads
    from workloads import configs as W
    build_oracle()
    expr, args, df = W.workload(opts.config, full=True)
    cores = max_threads()
    times = []
    sample = ""
    elems = 0.0
    for i in range(opts.warmup + opts.steps):
        dt, elems, sample = oracle_sample(opts.config, expr, args, df, cores, REFERENCE_STEP_ROWS)
        if i >= opts.warmup:
            times.append(dt)
    total = sum(times)
    value = elems * len(times) / total
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": opts.gpus,
            "steps": opts.steps, "warmup": opts.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": W.FULL[opts.config]().name, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


CONTRACT_HBM_GBS = 8000.0      # the bandwidth the benchmark spec names for the roofline (nominal HBM3e)


def time_workload(key, opts, dev, distributed, replicas, rows=0, saved_forward=False, steps=None, warmup=None):
    """Builds one workload on the device, runs warm-up + timed steps with a CUDA event around every part.
    One step = tad_forward, then exactly what tad_backward does: staging kernels, then every gradient.
    Returns a dict with the per-part times and what the caller needs for the end-to-end run."""
    import torch
    from paper_1711_01348_b200 import Plan
    from workloads import configs as W
    steps = opts.steps if steps is None else steps
    warmup = opts.warmup if warmup is None else warmup
    if rows:
        expr = W.profile_case(key, rows)
        args, df = W.make_inputs(expr, W.DIST[key], seed=0)
    else:
        expr, args, df = W.workload(key, full=True)
    plan = Plan(expr, saved_forward=saved_forward)
    d_args = [a.to(dev) for a in args]
    d_df = df.to(dev)
    f = torch.empty(expr.out_shape, dtype=torch.float32, device=dev)
    dargs = [torch.empty(s, dtype=torch.float32, device=dev) for s in expr.arg_shapes]
    ws = torch.zeros(max(256, plan.workspace_bytes()), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    arg_ptrs = [a.data_ptr() for a in d_args]
    # a plan compiled with saved_forward reads the forward output of the same step in its backward kernels
    bwd_ptrs = arg_ptrs + ([f.data_ptr()] if saved_forward else [])
    darg_ptrs = [d.data_ptr() for d in dargs]
    n_args = len(d_args)
    n_stages = plan.num_stages()
    parts = ["forward"] + (["stage"] if n_stages else []) + [f"d{name}" for name in expr.arg_names]
    n_parts = len(parts)

    def step(events=None):
        e = 0
        if events is not None:
            events[e].record(); e += 1
        plan.forward(arg_ptrs, f.data_ptr(), stream, ws.data_ptr(), ws.numel())
        if n_stages:
            if events is not None:
                events[e].record(); e += 1
            plan.backward_stage(bwd_ptrs, d_df.data_ptr(), ws.data_ptr(), ws.numel(), stream)
        for p in range(n_args):
            if events is not None:
                events[e].record(); e += 1
            plan.backward_arg(bwd_ptrs, d_df.data_ptr(), p, darg_ptrs[p], ws.data_ptr(), ws.numel(), stream)
        if events is not None:
            events[e].record()

    for _ in range(warmup):
        step()
    replicas.barrier(distributed)
    all_events = [[torch.cuda.Event(enable_timing=True) for _ in range(n_parts + 1)] for _ in range(steps)]
    t_begin = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    replicas.barrier(distributed)
    t_begin.record()
    for k in range(steps):
        step(all_events[k])
    t_end.record()
    replicas.barrier(distributed)
    total_ms = replicas.max_over_ranks(t_begin.elapsed_time(t_end), distributed, dev)
    part_ms = [sum(ev[i].elapsed_time(ev[i + 1]) for ev in all_events) / steps for i in range(n_parts)]
    return {"expr": expr, "args": args, "df": df, "plan": plan, "parts": parts, "part_ms": part_ms,
            "ms_per_step": total_ms / steps, "n_stages": n_stages, "steps": steps}


def part_records(run, peaks, fp32_clock_tflops, fp32_measured_tflops):
    """Per part: time, algorithmic work (the expression as written, counted by the plan), the roof that binds
    it and the achieved fraction against three denominators: `frac` (measured HBM copy bandwidth / FP32 peak
    by the maximum SM clock), `frac_measured_fma` (ALU parts: against the measured multiply-add rate) and
    `frac_contract` (the benchmark spec's 8 TB/s and the same FP32 peak)."""
    expr, plan = run["expr"], run["plan"]
    first_access = {}
    for q, a in enumerate(expr.accesses):
        first_access.setdefault(a.arg, []).append(q)
    out, launches = [], 0
    for i, name in enumerate(run["parts"]):
        if name == "forward":
            qs = [-1]
        elif name == "stage":
            qs = [-2 - st for st in range(run["n_stages"])]
        else:
            qs = first_access.get(expr.arg_names.index(name[1:]), [])
        flops = sum(plan.kernel_stats(q).alg_flops for q in qs)
        byts = sum(plan.kernel_stats(q).alg_bytes for q in qs)
        launches += sum(plan.kernel_stats(q).n_launches for q in qs)
        ms = run["part_ms"][i]
        t_alu = flops / (fp32_clock_tflops * 1e12)
        t_hbm = byts / (peaks["hbm_gbs"] * 1e9)
        bound = "alu" if t_alu >= t_hbm else "hbm"
        rec = {"part": name, "ms": ms, "alg_gflop": flops / 1e9, "alg_gb": byts / 1e9, "bound": bound,
               "frac": max(t_alu, t_hbm) / (ms * 1e-3) if ms > 0 else None}
        if ms > 0:
            rec["frac_contract"] = max(t_alu, byts / (CONTRACT_HBM_GBS * 1e9)) / (ms * 1e-3)
            if bound == "alu" and fp32_measured_tflops:
                rec["frac_measured_fma"] = flops / (fp32_measured_tflops * 1e12) / (ms * 1e-3)
        out.append(rec)
    return out, launches


def run_ours(opts):
    import torch
    from paper_1711_01348_b200 import measure_fp32_rate
    from workloads import configs as W

    from paper_1711_01348_b200 import replicas
    rank, local_rank, world = replicas.rank_info()
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    distributed = replicas.init("nccl")
    stream = torch.cuda.current_stream().cuda_stream

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    run = time_workload(opts.config, opts, dev, distributed, replicas, rows=opts.rows, saved_forward=opts.saved_forward)
    clocks = sampler.stop() if rank == 0 else None
    expr, args, df, plan = run["expr"], run["args"], run["df"], run["plan"]
    ms_per_step = run["ms_per_step"]

    # end to end: pinned host buffers in, results back, through tad_step_host
    e2e = None
    try:
        if opts.no_e2e:
            raise RuntimeError("skipped (--no-e2e)")
        h_args = [a.pin_memory() for a in args]
        h_df = df.pin_memory()
        h_f = torch.empty(expr.out_shape, dtype=torch.float32).pin_memory()
        h_dargs = [torch.empty(s, dtype=torch.float32).pin_memory() for s in expr.arg_shapes]
        staging = torch.empty(plan.staging_bytes(), dtype=torch.uint8, device=dev)
        e2e_steps = max(1, min(opts.steps, 3))

        def host_step():
            plan.step_host([a.data_ptr() for a in h_args], h_df.data_ptr(), h_f.data_ptr(),
                           [d.data_ptr() for d in h_dargs], staging.data_ptr(), staging.numel(), stream)
        host_step()
        replicas.barrier(distributed)
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            host_step()
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0) / e2e_steps
        e2e_s = replicas.max_over_ranks(e2e_s, distributed, dev)
        h2d = sum(a.numel() * 4 for a in args) + df.numel() * 4
        d2h = h_f.numel() * 4 + sum(d.numel() * 4 for d in h_dargs)
        e2e = {"value": world * elements_per_step(expr) / e2e_s, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": 1e3 * e2e_s}
        del staging, h_args, h_df, h_f, h_dargs
    except RuntimeError as exc:                       # e.g. not enough pinned memory
        e2e = {"value": None, "unit": UNIT, "error": str(exc)[:200]}

    if rank == 0:
        peaks = load_peaks()
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        fp32_clock = 2 * 128 * sms * peaks["sm_max_mhz"] * 1e6 / 1e12
        try:
            fp32_measured = measure_fp32_rate(stream)
        except Exception:                              # noqa: BLE001 - the fraction against it is then left out
            fp32_measured = None
        per_part, launches = part_records(run, peaks, fp32_clock, fp32_measured)
        # the roofline object describes the slowest backward part (the target is on the backward kernels)
        backward = [i for i, p in enumerate(per_part) if p["part"] not in ("forward",)]
        dom = max(backward or range(len(per_part)), key=lambda i: per_part[i]["ms"])
        d = per_part[dom]
        if d["bound"] == "alu":
            achieved = d["alg_gflop"] / 1e3 / (d["ms"] * 1e-3)
            roof = {"bound": "alu", "achieved": achieved, "peak": fp32_clock, "unit": "TFLOP/s",
                    "frac": achieved / fp32_clock, "traffic": None,
                    "peak_source": f"2 x 128 lanes x {sms} SMs x {peaks['sm_max_mhz']:.0f} MHz ({peaks['source']} clock)",
                    "peak_measured_fma": fp32_measured,
                    "frac_measured_fma": achieved / fp32_measured if fp32_measured else None}
        else:
            achieved = d["alg_gb"] / (d["ms"] * 1e-3)
            roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
                    "frac_contract": achieved / CONTRACT_HBM_GBS}
        roof["kernel"] = d["part"]
        roof["traffic"] = recorded_traffic(expr.name, d["part"])
        # the other workloads: same timing, parts only (cfg1 is a launch-latency case: times, no fractions)
        others = {}
        if opts.all_workloads and not distributed and not opts.rows:
            run = None
            torch.cuda.empty_cache()
            for key in ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"]:
                if key == opts.config:
                    continue
                r = time_workload(key, opts, dev, distributed, replicas, steps=max(opts.steps, 20), warmup=max(opts.warmup, 3))
                recs, nl = part_records(r, peaks, fp32_clock, fp32_measured)
                if key == "cfg1":
                    recs = [{"part": p["part"], "us": 1e3 * p["ms"]} for p in recs]
                others[key] = {"workload": r["expr"].name, "ms_per_step": r["ms_per_step"], "steps": r["steps"],
                               "gpu_launches_per_step": nl, "l2": L2_NOTE[key], "parts": recs}
                del r
                torch.cuda.empty_cache()
        cpu = None
        if not distributed and not opts.no_cpu_baseline and not opts.rows:
            from oracle.oracle import build as build_oracle, max_threads
            build_oracle()
            cores = max_threads()
            dt, elems, sample = oracle_sample(opts.config, expr, args, df, cores)
            cpu = {"value": elems / dt, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                   "seconds": dt}
        line = {"metric": METRIC, "value": world * elements_per_step(expr) / (ms_per_step * 1e-3), "unit": UNIT,
                "n_gpus": world, "steps": opts.steps, "warmup": opts.warmup, "ms_per_step": ms_per_step,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic",
                "config": {"workload": expr.name, "out_shape": expr.out_shape, "arg_shapes": expr.arg_shapes,
                           "l2": L2_NOTE[opts.config],
                           "saved_forward": bool(opts.saved_forward),
                           "parallelism": "replicas" if world > 1 else "single"},
                "roofline": roof, "parts": per_part,
                "fp32_peak": {"by_clock_tflops": fp32_clock, "measured_fma_tflops": fp32_measured,
                              "contract_hbm_gbs": CONTRACT_HBM_GBS, "measured_hbm_gbs": peaks["hbm_gbs"]},
                "workloads": others, "cpu_baseline": cpu, "e2e": e2e,
                "gpu_launches": launches * opts.steps, "clocks": clocks}
        print(json.dumps(line), flush=True)
    replicas.finish(distributed)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--single", dest="all_workloads", action="store_false",
                    help="time only the workload of --config (the default run also times the parts of the other four)")
    ap.add_argument("--saved-forward", action="store_true",
                    help="compile the plan with saved_forward: the backward kernels read f of the same step")
    ap.add_argument("--rows", type=int, default=0,
                    help="profiler captures only: the workload with a smaller leading extent (not a bench number)")
    opts = ap.parse_args()
    if opts.impl == "reference":
        run_reference(opts)
    else:
        run_ours(opts)


if __name__ == "__main__":
    main()
