#!/usr/bin/env python
"""Benchmark of the streaming-rollout frame update.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--pattern streaming]
    python bench.py --impl reference ...        # the CPU oracle on the host cores, same metric

A step is one sr_rollout_run over the workload's T frame updates of the whole batch; the metric is
frame updates per second (a frame = all node states of the next frame for the whole batch).  The
headline workload is c5, the largest of the five configurations; at one GPU the other four are
measured as well and reported under "workloads" in the same line.  One JSON line is printed by rank 0.

With --gpus N and no WORLD_SIZE in the environment the script starts N copies of itself, one per GPU
(independent replicas: the frame update has no exchange step; NCCL carries only the timing barrier and
the maximum over ranks).  Under torchrun it takes RANK / LOCAL_RANK / WORLD_SIZE from the environment.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import data, graphs  # noqa: E402

METRIC = "streaming_rollout_frames_per_sec"
UNIT = "frames/s"
ALL_WORKLOADS = ("c1", "c2", "c3", "c4", "c5")
# The paper's own CIFAR10 networks (Sec. A): shallowest and deepest of DSR0..DSR6, at a batch the paper does not fix.
PAPER_NETS = {"dsr0": dict(batch=128, frames=16), "dsr6": dict(batch=128, frames=16)}

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of ONE launch of the dominant kernel, from the ncu
# captures summarised under profiles/.  Every entry names its capture and the first 12 hex digits of the SHA-256 of
# the kernel source it was taken from; the number is reported only while that source is unchanged, else null.
TRAFFIC = {
    # workload: (bytes per launch, kernel source file, sha256[:12] of that file at capture time, summary under profiles/)
    "c5": (615.7e6, "sr_tc.cu", "6985e1c55246", "profiles/sr_tc_group_kernel_counters.md"),
    "c3": (245.2e6, "sr_tc.cu", "6985e1c55246", "profiles/sr_tc_group_kernel_counters.md"),
    "c4": (165.1e6, "sr_tc.cu", "6985e1c55246", "profiles/sr_tc_group_kernel_counters.md"),
    "c2": (8.0e6, "sr_resident.cu", "89436108f1ff", "profiles/sr_resident_kernel_c2.md"),     # one launch = all 32 frames
    "c1": (1.30e6, "sr_dense.cu", "9f15eb3bde12", "profiles/sr_dense_kernel_c1.md"),           # one launch = all 16 frames
}


def source_digest(name: str) -> str:
    p = os.path.join(ROOT, "paper_1806_04965_b200", "csrc", name)
    return hashlib.sha256(open(p, "rb").read()).hexdigest()[:12]


def traffic_of(workload: str):
    t = TRAFFIC.get(workload)
    if not t:
        return None, "no capture of the current kernel"
    nbytes, src, digest, where = t
    if source_digest(src) != digest:
        return None, "%s changed since the capture in %s" % (src, where)
    return float(nbytes), where


# ----------------------------------------------------------------------------- algorithmic work of one frame update
def frame_flops(spec) -> float:
    return 2.0 * graphs.macs_per_sample(spec) * spec.batch


def conv_flops(spec) -> float:
    return 2.0 * spec.batch * sum(
        (16 if e.pool == 2 else e.k * e.k) * spec.nodes[e.src].c * spec.nodes[e.tgt].h * spec.nodes[e.tgt].w * spec.nodes[e.tgt].c
        for e in spec.edges if e.kind == graphs.CONV)


def frame_bytes(spec) -> float:
    """Every node state read once and every non-input state written once per frame, plus the float
    output and the weights once."""
    el = 2 if spec.dtype == "bf16" else 4
    size = lambda v: spec.batch * v.h * v.w * v.c * el
    has_in = {e.tgt for e in spec.edges}
    has_out = {e.src for e in spec.edges}
    total = 0
    for vi, v in enumerate(spec.nodes):
        if vi in has_out:
            total += size(v)
        if vi in has_in:
            total += size(v)
    out = max(vi for vi in range(len(spec.nodes)) if vi not in {e.src for e in spec.edges if e.src != e.tgt})
    total += spec.batch * spec.nodes[out].c * 4
    for ei, e in enumerate(spec.edges):
        total += int(np.prod(data.weight_shape(spec, ei))) * el
    return float(total)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (the timing rule for N > 1: a job is as slow
    as its slowest replica).  Without a process group the values come back unchanged."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_frames_per_s(world: int, frames_per_step: int, ms_per_step: float) -> float:
    """Replicas only: every rank rolls out its own batch of sequences, so the job's frame rate is the sum."""
    return world * frames_per_step / ms_per_step * 1e3


def build_spec(args, name=None):
    kw = {}
    if name is None or name == args.workload:
        if args.batch:
            kw["batch"] = args.batch
        if args.frames:
            kw["frames"] = args.frames
    n = name or args.workload
    if n in PAPER_NETS:
        kw = dict(PAPER_NETS[n], **kw)
    return graphs.build(n, **kw)


def replica_spec(args, rank: int, name=None):
    spec = build_spec(args, name)
    spec.seed += rank                                            # every rank rolls out its own sequences
    return spec


def config_of(spec, args, world: int) -> dict:
    """The workload description both arms print (identical keys and values for the same command line)."""
    return {"workload": spec.name, "pattern": args.pattern, "batch": spec.batch, "frames_per_step": spec.frames,
            "l2": "flushed before every timed step, after the reset (192 MiB write)",
            "parallelism": "replicas x%d" % world,
            "why_this_workload": "largest single-GPU configuration (the metric names none)" if spec.name == "c5" else "chosen on the command line"}


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_ms: int = 50):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS,
                                       "--format=csv,noheader,nounits", "-lms", str(period_ms)], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.p.terminate()
        self.p.wait()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                pw.append(float(r[2]))
                for n, v in zip(names, r[4:8]):
                    if v.strip().lower() == "active":
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "power_w_max": max(pw) if pw else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- the oracle on the host cores
def time_oracle(spec, pattern, budget_s=15.0):
    """Times the oracle as it stands on a bounded sample: whole sequences of a few batch samples."""
    from oracle import frame_update as fu
    X, W, Bi = data.make_inputs(spec), data.make_weights(spec), data.make_biases(spec)
    macs = graphs.macs_per_sample(spec)
    est_rate = 4e10                                           # multiply-adds per second, rough, to size the sample
    n_s = int(max(1, min(spec.batch, budget_s * est_rate / (macs * spec.frames))))
    T = spec.frames
    if macs * T / est_rate > budget_s:                       # one sequence is already too long: fewer frames
        T = int(max(1, budget_s * est_rate / macs))
    samples = list(range(n_s))
    fu.build()
    reps, dt = 0, 0.0
    while True:                                              # small workloads: repeat until a few seconds have passed
        t0 = time.perf_counter()
        fu.rollout_spec(spec, pattern, X, W, Bi, samples=samples, frames=T)
        dt += time.perf_counter() - t0
        reps += 1
        if dt >= min(5.0, budget_s) or reps >= 50:
            break
    dt /= reps
    sample_frames = n_s * T
    frames_per_s = sample_frames / dt / spec.batch            # whole-batch frame updates per second
    return {"value": frames_per_s, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
            "sample": "%d of %d sequences x %d of %d frames, %d run(s) of %.2f s (%.1f sample-frames/s), scaled to the full batch"
                      % (n_s, spec.batch, T, spec.frames, reps, dt, sample_frames / dt),
            "seconds": dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = build_spec(args)
    vals = []
    for _ in range(args.warmup):
        time_oracle(spec, args.pattern, budget_s=2.0)
    for _ in range(args.steps):
        vals.append(time_oracle(spec, args.pattern, budget_s=max(2.0, min(15.0, 60.0 / max(1, args.steps)))))
    v = float(np.mean([x["value"] for x in vals]))
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * spec.frames / v, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(spec, args, max(1, args.gpus)),
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": vals[-1]["cores"], "kind": "oracle",
                             "sample": vals[-1]["sample"]},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- the CUDA library
def time_pattern(torch, spec, pattern, W, Bi, dev_in, steps, warmup, graph_frames, engine, flush, resident=(1, 0, 0), tc_pair=0):
    from paper_1806_04965_b200 import Graph
    G = Graph(spec.nodes, spec.edges, spec.patterns[pattern], batch=spec.batch, dtype=spec.dtype, engine=engine,
              graph_frames=graph_frames, resident=bool(resident[0]), resident_cluster=resident[1], resident_warps=resident[2],
              tc_pair=tc_pair)
    G.set_weights(W, Bi)
    T = spec.frames
    out = torch.empty((T, spec.batch, spec.nodes[G.output_node].c), dtype=torch.float32, device="cuda")
    ins0, ins = [x[0] for x in dev_in], [x[1:] for x in dev_in]
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        G.reset(ins0)
        G.run(ins, out)
    torch.cuda.synchronize()
    times = []
    l0 = G.launch_count()
    for _ in range(steps):
        G.reset(ins0)
        if flush is not None:
            flush.add_(1)                                     # evicts L2 (the reset's writes included) before the timed step
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        G.run(ins, out)
        b.record(stream)
        b.synchronize()
        times.append(a.elapsed_time(b))
    G.sync_status()
    launches = G.launch_count() - l0
    ms = float(np.mean(times))
    return G, out, {"ms_per_step": ms, "frames_per_s": T / ms * 1e3, "us_per_frame": ms * 1e3 / T,
                    "ms_min": float(np.min(times)), "launches": launches, "groups_per_frame": G.info["n_groups"],
                    "tensor_core_nodes": G.info["n_tensor_core_nodes"], "direct_nodes": G.info["n_direct_nodes"],
                    "resident_cluster": G.info["resident_cluster"]}


def time_single_steps(torch, G, dev_in, n=60):
    """Host-visible latency of one sr_rollout_step: from the call to the moment the host sees the frame finished."""
    ins0 = [x[0] for x in dev_in]
    T1 = int(dev_in[0].shape[0])
    out = torch.empty((G.batch, G.nodes[G.output_node].c), dtype=torch.float32, device="cuda")
    G.reset(ins0)
    torch.cuda.synchronize()
    call, whole = [], []
    for i in range(n + 5):
        frame = [x[1 + i % (T1 - 1)] for x in dev_in]
        t0 = time.perf_counter()
        G.step(frame, out)
        t1 = time.perf_counter()
        torch.cuda.synchronize()
        t2 = time.perf_counter()
        if i >= 5:
            call.append(1e6 * (t1 - t0))
            whole.append(1e6 * (t2 - t0))
    G.sync_status()
    return {"step_latency_us": float(np.median(whole)), "step_call_us": float(np.median(call)),
            "what": "median of %d single sr_rollout_step calls, host clock: call until torch.cuda.synchronize returns "
                    "(step_call_us: until the call returns)" % n}


def kernel_timing(torch, G, dev_in, out, flush, runs, graph_frames):
    """Mean duration of the dominant kernel's launches, bracketed by the library with CUDA events on the launching stream."""
    ins0, ins = [x[0] for x in dev_in], [x[1:] for x in dev_in]
    resident = G.info["resident_cluster"] > 0
    if not resident:
        G.set_option(1, 0)                                    # plain launches: events cannot be recorded inside a CUDA graph
    G.set_option(5, 1)
    G.reset(ins0)
    G.run(ins, out)
    G.kernel_time()
    for _ in range(runs):
        G.reset(ins0)
        flush.add_(1)
        G.run(ins, out)
    k_ms, n = G.kernel_time()
    G.set_option(5, 0)
    if not resident:
        G.set_option(1, graph_frames)
    return (1e3 * k_ms / n if n else None), n


def measure_workload(torch, args, name, rank, local, dist, pk, flush, steps, warmup, main):
    """All patterns of one workload, the dominant kernel alone, single-step latency and (main workload) end to end."""
    spec = replica_spec(args, rank, name)
    X, W, Bi = data.make_inputs(spec), data.make_weights(spec), data.make_biases(spec)
    tdt = torch.bfloat16 if spec.dtype == "bf16" else torch.float32
    host_in = [torch.from_numpy(np.ascontiguousarray(X[v], dtype=np.float32)).to(tdt).contiguous().pin_memory()
               for v in spec.input_nodes()]
    dev_in = [h.cuda() for h in host_in]
    T = spec.frames

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    first = args.pattern if main else "streaming"
    pats = [first] + [p for p in spec.patterns if p != first and not args.only_main]
    results, main_G, main_out, clocks = {}, None, None, None
    for p in pats:
        barrier()
        sampler = ClockSampler(local) if p == first else None
        G, out, r = time_pattern(torch, spec, p, W, Bi, dev_in, steps, warmup, args.graph_frames, args.engine, flush,
                                 (args.resident, args.resident_cluster, args.resident_warps), args.tc_pair)
        barrier()
        if p == first:
            clocks = sampler.stop()
            main_G, main_out = G, out
        else:
            del G, out
        results[p] = r
    res = results[first]
    ms = max_over_ranks([res["ms_per_step"]], dist, "cuda")[0]
    us_frame = ms * 1e3 / T
    fl, by, cfl = frame_flops(spec), frame_bytes(spec), conv_flops(spec)
    tensor_bound = spec.dtype == "bf16" and fl / by > 1e3 * pk["bf16_tflops_sustained"] / pk["hbm_gbs"]
    resident = res["resident_cluster"] > 0
    kernel_us, kernel_n = None, 0
    if resident or res["tensor_core_nodes"] > 0:
        kernel_us, kernel_n = kernel_timing(torch, main_G, dev_in, main_out, flush, 5 if resident else 3, args.graph_frames)
    groups = res["groups_per_frame"]
    traffic, traffic_from = traffic_of(spec.name)
    mhz = clocks.get("sm_mhz") if clocks else None
    if resident:
        # One launch covers all T frames with the states on chip, so its own DRAM traffic is far below the algorithmic
        # bytes (every state read and written once per frame): the figure below is algorithmic bytes / time, the
        # classification this workload has on a per-frame launch path, not the bound of this kernel (which is the
        # shared-memory pipe; see profiles/).
        ach = by * T / (kernel_us * 1e-6) / 1e9
        dense = spec.dtype != "bf16"
        roof = {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
                "frac_is": "algorithmic bytes / time over measured copy bandwidth; the states never leave the SM, so HBM does not bound this kernel",
                "kernel": "%s, mean of %d event-timed launches (%.1f us each = %.2f us per frame, %d frames per launch, %s)"
                          % ("sr_dense_kernel" if dense else "sr_resident_kernel", kernel_n, kernel_us, kernel_us / T, T,
                             "one cluster of %d CTAs per 8 sequences" % res["resident_cluster"] if dense
                             else "%d CTAs per sequence" % res["resident_cluster"])}
        if dense:
            roof["alu"] = {"achieved_gflops": fl * T / (kernel_us * 1e-6) / 1e9,
                           "note": "fp32 FMA on CUDA cores; weights and states resident in the shared memory of a cluster; a frame "
                                   "is one round of work units (shared-memory loads, reduction over the lanes) and one "
                                   "cluster barrier: latency-bound"}
        else:
            roof["tensor"] = {"achieved_tflops": fl * T / (kernel_us * 1e-6) / 1e12,
                              "frac_of_burst_peak": fl * T / (kernel_us * 1e-6) / 1e12 / pk["bf16_tflops"],
                              "note": "mma.sync path; states and weights resident in shared memory"}
    elif tensor_bound:
        if kernel_us:
            ach = cfl / groups / (kernel_us * 1e-6) / 1e12     # average over the group launches of a frame
            what = "sr_tc_group_kernel, mean of %d event-timed launches (%.1f us each, %d per frame)" % (kernel_n, kernel_us, groups)
        else:
            ach = fl / (us_frame * 1e-6) / 1e12
            what = "all launches of one frame update"
        roof = {"bound": "tensor", "achieved": ach, "peak": pk["bf16_tflops"], "unit": "TFLOP/s", "frac": ach / pk["bf16_tflops"],
                "peak_is": "burst cuBLAS bf16 figure (kernels are event-timed one by one)",
                "frac_of_sustained_peak": ach / pk["bf16_tflops_sustained"], "kernel": what, "kernel_us": kernel_us,
                "kernel_us_x_sm_mhz": kernel_us * mhz if (kernel_us and mhz) else None,
                "whole_frame": {"achieved": fl / (us_frame * 1e-6) / 1e12, "frac": fl / (us_frame * 1e-6) / 1e12 / pk["bf16_tflops"]}}
    else:
        ach = by / (us_frame * 1e-6) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
                "kernel": "all launches of one frame update (%s)" %
                          ("tensor-core kernel %.1f us of %.1f us" % (kernel_us, us_frame) if kernel_us else "CUDA-core kernels")}
    roof["traffic"] = traffic
    roof["traffic_from"] = traffic_from
    roof["peak_source"] = pk["source"]
    roof["algorithmic_flops_per_frame"] = fl
    roof["algorithmic_bytes_per_frame"] = by
    w = {"batch": spec.batch, "frames_per_step": T, "dtype": "bf16" if spec.dtype == "bf16" else "f32",
         "ms_per_step": ms, "us_per_frame": us_frame, "frames_per_s": T / ms * 1e3,
         "sample_frames_per_s": spec.batch * T / ms * 1e3,
         "patterns": {p: {k: r[k] for k in ("frames_per_s", "us_per_frame", "groups_per_frame", "launches", "resident_cluster")}
                      for p, r in results.items()},
         "roofline": roof, "clocks": clocks, "gpu_launches": int(res["launches"]),
         "nodes": {"tensor_core": res["tensor_core_nodes"], "cuda_core": res["direct_nodes"]}}
    w.update(time_single_steps(torch, main_G, dev_in))
    if main:
        # end to end through the public call with host buffers: copy in, reset + run, copy the outputs back
        out_host = torch.empty(tuple(main_out.shape), dtype=torch.float32).pin_memory()
        stream = torch.cuda.current_stream()
        e2e_ms = []
        for i in range(warmup + steps):
            flush.add_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            d = [h.to("cuda", non_blocking=True) for h in host_in]
            main_G.reset([x[0] for x in d])
            main_G.run([x[1:] for x in d], main_out)
            out_host.copy_(main_out, non_blocking=True)
            b.record(stream)
            b.synchronize()
            if i >= warmup:
                e2e_ms.append(a.elapsed_time(b))
        main_G.sync_status()
        e2e = max_over_ranks([float(np.mean(e2e_ms))], dist, "cuda")[0]
        w["e2e_ms_per_step"] = e2e
        w["h2d_bytes_per_step"] = int(sum(h.numel() * h.element_size() for h in host_in))
        w["d2h_bytes_per_step"] = int(out_host.numel() * 4)
    del main_G, main_out, dev_in, host_in
    torch.cuda.empty_cache()
    return spec, w


def measure_window(torch, args, flush, steps, warmup, W=8):
    """c4 without its recurrent edges under the sequential rollout: T frames as chained windows of size 1
    (sr_rollout_run) against windows of W frames evaluated at once (sr_rollout_window)."""
    from paper_1806_04965_b200 import Graph
    spec = graphs.build("c4ff")
    X, Wt, Bi = data.make_inputs(spec), data.make_weights(spec), data.make_biases(spec)
    dev = [torch.from_numpy(np.ascontiguousarray(X[v], dtype=np.float32)).to(torch.bfloat16).cuda().contiguous() for v in spec.input_nodes()]
    G = Graph(spec.nodes, spec.edges, spec.patterns["sequential"], batch=spec.batch, dtype=spec.dtype, graph_frames=args.graph_frames)
    G.set_weights(Wt, Bi)
    G.bind_window(W)
    T = spec.frames // W * W
    out = torch.empty((T, spec.batch, spec.nodes[G.output_node].c), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()

    def chained():
        G.run([x[1:T + 1] for x in dev], out)

    def windows():
        for t in range(0, T, W):
            G.rollout_window([x[t + 1:t + 1 + W] for x in dev], out[t:t + W])

    res = {}
    for name, fn in (("w1", chained), ("w%d" % W, windows)):
        times = []
        for i in range(warmup + steps):
            G.reset([x[0] for x in dev])
            flush.add_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            b.synchronize()
            if i >= warmup:
                times.append(a.elapsed_time(b))
        G.sync_status()
        res[name] = float(np.mean(times)) * 1e3 / T
    return {"graph": "c4 without recurrent edges", "pattern": "sequential", "batch": spec.batch, "frames": T, "W": W,
            "levels_per_frame": G.info["n_groups"], "us_per_frame_w1": res["w1"], "us_per_frame_w%d" % W: res["w%d" % W],
            "what": "w1 = sr_rollout_run (chained windows of size 1, one launch group per level and frame); "
                    "w%d = sr_rollout_window (one launch group per level for %d frames at once)" % (W, W)}


def run_cuda(args):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    flush = torch.zeros(192 * 1024 * 1024 // 4, dtype=torch.int32, device="cuda")
    pk = peaks()
    spec, main = measure_workload(torch, args, args.workload, rank, local, dist, pk, flush, args.steps, args.warmup, True)
    T = spec.frames
    line = {"metric": METRIC, "value": whole_job_frames_per_s(world, T, main["ms_per_step"]), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": main["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": main["dtype"], "data": "synthetic",
            "config": dict(config_of(spec, args, world), engine=args.engine, graph_frames=args.graph_frames,
                           resident_cluster=main["patterns"][args.pattern]["resident_cluster"]),
            "us_per_frame": main["us_per_frame"], "sample_frames_per_s": world * main["sample_frames_per_s"],
            "patterns": main["patterns"],
            "step_latency_us": main["step_latency_us"], "step_call_us": main["step_call_us"],
            "e2e": {"value": whole_job_frames_per_s(world, T, main["e2e_ms_per_step"]), "unit": UNIT,
                    "h2d_bytes_per_step": main["h2d_bytes_per_step"], "d2h_bytes_per_step": main["d2h_bytes_per_step"]},
            "gpu_launches": main["gpu_launches"], "roofline": main["roofline"], "clocks": main["clocks"],
            "nodes": main["nodes"]}
    if world == 1 and not args.only_main:
        # the other configurations, fewer steps each; same measurement, reported beside the headline
        others = {}
        for name in [n for n in args.also.split(",") if n and n != args.workload]:
            torch.cuda.synchronize()
            time.sleep(3.0)          # let the clocks recover from the power-capped headline run before the next workload
            _, w = measure_workload(torch, args, name, rank, local, None, pk, flush, max(3, min(args.steps, 10)), max(3, args.warmup), False)
            others[name] = w
        main_copy = {k: v for k, v in main.items() if k not in ("e2e_ms_per_step", "h2d_bytes_per_step", "d2h_bytes_per_step")}
        others[spec.name] = main_copy
        line["workloads"] = {k: others[k] for k in sorted(others)}
        paper = {}
        for name in [n for n in args.paper_nets.split(",") if n]:
            torch.cuda.synchronize()
            time.sleep(1.0)
            _, w = measure_workload(torch, args, name, rank, local, None, pk, flush, max(3, min(args.steps, 5)), max(3, args.warmup), False)
            paper[name] = w
        if paper:
            line["paper_networks"] = paper
        if "c4" in line["workloads"]:
            line["workloads"]["c4"]["deep_window"] = measure_window(torch, args, flush, max(3, min(args.steps, 10)), 3)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            cb = time_oracle(spec, args.pattern)
            cb.pop("seconds")
            line["cpu_baseline"] = cb
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- one process per GPU
def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def spawn_ranks(n: int, argv) -> int:
    """Starts n copies of this script, one per GPU, with the rendezvous variables torchrun would set.
    Rank 0 inherits stdout (it prints the JSON line); every rank inherits stderr."""
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    rc = 0
    for p in procs:
        p.wait()
        rc = rc or p.returncode
    return rc


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c5", choices=list(graphs.BUILDERS))
    ap.add_argument("--paper-nets", default=",".join(PAPER_NETS), help="the paper's own networks reported beside the configs (one GPU)")
    ap.add_argument("--also", default=",".join(ALL_WORKLOADS), help="workloads reported beside the headline at one GPU")
    ap.add_argument("--pattern", default="streaming")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--frames", type=int, default=0)
    ap.add_argument("--engine", default="auto", choices=["auto", "direct"])
    ap.add_argument("--graph-frames", type=int, default=16, help="frames per CUDA graph inside sr_rollout_run (0 = plain launches)")
    ap.add_argument("--resident", type=int, default=1, help="1: sr_rollout_run may use the shared-memory-resident kernel; 0: per-frame launches")
    ap.add_argument("--resident-cluster", type=int, default=0)
    ap.add_argument("--resident-warps", type=int, default=0)
    ap.add_argument("--tc-pair", type=int, default=0, help="tensor-core work items: 0 = library decides, 1 = single tiles, 2 = pairs of tiles")
    ap.add_argument("--only-main", action="store_true", help="time only --workload and --pattern")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "cuda":
        args.warmup = 3                                       # the timing rule: at least three untimed steps
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
