#!/usr/bin/env python
"""Benchmark of the streaming-rollout frame update.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--pattern streaming]
    python bench.py --impl reference ...        # the CPU oracle on the host cores, same metric

A step is one sr_rollout_run over the workload's T frame updates of the whole batch; the metric is
frame updates per second (a frame = all node states of the next frame for the whole batch).  One
JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import data, graphs  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum of one tensor-core group launch from the ncu captures summarised under
# profiles/ (null where no capture of the current kernel exists)
TRAFFIC = {"c2": 5.78e6, "c3": 264.1e6, "c4": 157.5e6, "c5": 612.4e6}
# the same for one launch of the resident kernel (all T frames of the workload); null until captured for the current kernel
TRAFFIC_RESIDENT = {"c2": 8.00e6}

METRIC = "streaming_rollout_frames_per_sec"
UNIT = "frames/s"


# ----------------------------------------------------------------------------- algorithmic work of one frame update
def frame_flops(spec) -> float:
    return 2.0 * graphs.macs_per_sample(spec) * spec.batch


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


def replica_spec(args, rank: int):
    spec = build_spec(args)
    spec.seed += rank                                            # every rank rolls out its own sequences
    return spec


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS,
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        self.p.wait()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for n, v in zip(names, r[4:8]):
                    if v.strip().lower() == "active":
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def build_spec(args):
    kw = {}
    if args.batch:
        kw["batch"] = args.batch
    if args.frames:
        kw["frames"] = args.frames
    return graphs.build(args.workload, **kw)


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
            "config": {"workload": spec.name, "pattern": args.pattern, "batch": spec.batch, "frames": spec.frames},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": vals[-1]["cores"], "kind": "oracle",
                             "sample": vals[-1]["sample"]},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- the CUDA library
def time_pattern(torch, spec, pattern, W, Bi, dev_in, steps, warmup, graph_frames, engine, flush, resident=(1, 0, 0)):
    from paper_1806_04965_b200 import Graph
    G = Graph(spec.nodes, spec.edges, spec.patterns[pattern], batch=spec.batch, dtype=spec.dtype, engine=engine,
              graph_frames=graph_frames, resident=bool(resident[0]), resident_cluster=resident[1], resident_warps=resident[2])
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
        if flush is not None:
            flush.add_(1)                                     # evicts L2 between timed steps
        G.reset(ins0)
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
    spec = replica_spec(args, rank)
    X, W, Bi = data.make_inputs(spec), data.make_weights(spec), data.make_biases(spec)
    tdt = torch.bfloat16 if spec.dtype == "bf16" else torch.float32
    host_in = [torch.from_numpy(np.ascontiguousarray(X[v], dtype=np.float32)).to(tdt).contiguous().pin_memory()
               for v in spec.input_nodes()]
    dev_in = [h.cuda() for h in host_in]
    flush = torch.zeros(192 * 1024 * 1024 // 4, dtype=torch.int32, device="cuda")
    pk = peaks()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    results = {}
    pats = [args.pattern] + [p for p in spec.patterns if p != args.pattern and not args.only_main]
    sampler = None
    for p in pats:
        barrier()
        if p == args.pattern:
            sampler = ClockSampler(local)
        G, out, r = time_pattern(torch, spec, p, W, Bi, dev_in, args.steps, args.warmup, args.graph_frames, args.engine,
                                 flush, (args.resident, args.resident_cluster, args.resident_warps))
        barrier()
        if p == args.pattern:
            clocks = sampler.stop()
        results[p] = r
        if p == args.pattern:
            main_G, main_out = G, out
    main = results[args.pattern]
    T = spec.frames
    # end to end through the public call with host buffers: copy in, reset + run, copy the outputs back
    out_host = torch.empty(tuple(main_out.shape), dtype=torch.float32).pin_memory()
    stream = torch.cuda.current_stream()
    e2e_ms = []
    for i in range(args.warmup + args.steps):
        flush.add_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        d = [h.to("cuda", non_blocking=True) for h in host_in]
        main_G.reset([x[0] for x in d])
        main_G.run([x[1:] for x in d], main_out)
        out_host.copy_(main_out, non_blocking=True)
        b.record(stream)
        b.synchronize()
        if i >= args.warmup:
            e2e_ms.append(a.elapsed_time(b))
    e2e_ms_mean = float(np.mean(e2e_ms))
    # max over ranks
    ms, e2e = max_over_ranks([main["ms_per_step"], e2e_ms_mean], dist, "cuda")
    fl, by = frame_flops(spec), frame_bytes(spec)
    intensity = fl / by
    tensor_bound = spec.dtype == "bf16" and intensity > 1e3 * pk["bf16_tflops_sustained"] / pk["hbm_gbs"]
    us_frame = ms * 1e3 / T
    # the dominant kernel alone: every tensor-core group launch of a few plain (non-graph) runs is bracketed
    # with CUDA events on the launching stream by the library
    kernel_us, kernel_n = None, 0
    resident = main["resident_cluster"] > 0
    if resident:
        # the resident kernel: ONE launch per step walks all T frames; event-timed by the library
        main_G.set_option(5, 1)
        ins0, ins = [x[0] for x in dev_in], [x[1:] for x in dev_in]
        main_G.reset(ins0)
        main_G.run(ins, main_out)
        main_G.kernel_time()
        for _ in range(5):
            flush.add_(1)
            main_G.reset(ins0)
            main_G.run(ins, main_out)
        k_ms, kernel_n = main_G.kernel_time()
        main_G.set_option(5, 0)
        kernel_us = 1e3 * k_ms / max(1, kernel_n)
    elif main["tensor_core_nodes"] > 0:
        main_G.set_option(1, 0)
        main_G.set_option(5, 1)
        ins0, ins = [x[0] for x in dev_in], [x[1:] for x in dev_in]
        main_G.reset(ins0)
        main_G.run(ins, main_out)
        main_G.kernel_time()
        for _ in range(3):
            flush.add_(1)
            main_G.reset(ins0)
            main_G.run(ins, main_out)
        k_ms, kernel_n = main_G.kernel_time()
        main_G.set_option(5, 0)
        main_G.set_option(1, args.graph_frames)
        kernel_us = 1e3 * k_ms / max(1, kernel_n)
    groups = main["groups_per_frame"]
    conv_fl = 2.0 * spec.batch * sum(
        (16 if e.pool == 2 else e.k * e.k) * spec.nodes[e.src].c * spec.nodes[e.tgt].h * spec.nodes[e.tgt].w * spec.nodes[e.tgt].c
        for e in spec.edges if e.kind == graphs.CONV)
    if resident:
        # algorithmic bytes of the T frames one launch covers / its duration.  The states stay on chip, so the
        # kernel's own DRAM traffic is far below the algorithmic bytes (which assume every state is read and
        # written once per frame): the HBM roofline is the classification the workload has on a per-frame
        # launch path, not what limits this kernel.
        ach = by * T / (kernel_us * 1e-6) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
                "traffic": TRAFFIC_RESIDENT.get(spec.name),
                "kernel": "sr_resident_kernel, mean of %d event-timed launches (%.1f us each = %.2f us per frame, %d frames per launch, "
                          "%d CTAs per sequence)" % (kernel_n, kernel_us, kernel_us / T, T, main["resident_cluster"]),
                "tensor": {"achieved_tflops": fl * T / (kernel_us * 1e-6) / 1e12,
                           "note": "mma.sync path; states and weights resident in shared memory"}}
    elif tensor_bound:
        if kernel_us:
            ach = conv_fl / groups / (kernel_us * 1e-6) / 1e12     # average over the group launches of a frame
            what = "sr_tc_group_kernel, mean of %d event-timed launches (%.1f us each, %d per frame)" % (kernel_n, kernel_us, groups)
        else:
            ach = fl / (us_frame * 1e-6) / 1e12
            what = "all launches of one frame update"
        roof = {"bound": "tensor", "achieved": ach, "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac": ach / pk["bf16_tflops_sustained"], "traffic": TRAFFIC.get(spec.name),
                "frac_of_burst_peak": ach / pk["bf16_tflops"], "kernel": what,
                "whole_frame": {"achieved": fl / (us_frame * 1e-6) / 1e12,
                                "frac": fl / (us_frame * 1e-6) / 1e12 / pk["bf16_tflops_sustained"]}}
    else:
        ach = by / (us_frame * 1e-6) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
                "traffic": TRAFFIC.get(spec.name),
                "kernel": "all launches of one frame update (%s)" %
                          ("tensor-core kernel %.1f us of %.1f us" % (kernel_us, us_frame) if kernel_us else "CUDA-core kernels")}
    roof["peak_source"] = pk["source"]
    roof["algorithmic_flops_per_frame"] = fl
    roof["algorithmic_bytes_per_frame"] = by
    line = {"metric": METRIC, "value": whole_job_frames_per_s(world, T, ms), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if spec.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": spec.name, "pattern": args.pattern, "batch": spec.batch, "frames_per_step": T,
                       "l2": "flushed between timed steps (192 MiB write)", "engine": args.engine,
                       "graph_frames": args.graph_frames, "parallelism": "replicas x%d" % world,
                       "resident_cluster": main["resident_cluster"]},
            "us_per_frame": us_frame, "sample_frames_per_s": world * spec.batch * T / ms * 1e3,
            "patterns": {p: {k: r[k] for k in ("frames_per_s", "us_per_frame", "groups_per_frame", "launches", "resident_cluster")}
                         for p, r in results.items()},
            "e2e": {"value": whole_job_frames_per_s(world, T, e2e), "unit": UNIT,
                    "h2d_bytes_per_step": int(sum(h.numel() * h.element_size() for h in host_in)),
                    "d2h_bytes_per_step": int(out_host.numel() * 4)},
            "gpu_launches": int(main["launches"]), "roofline": roof, "clocks": clocks,
            "nodes": {"tensor_core": main["tensor_core_nodes"], "cuda_core": main["direct_nodes"]}}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            cb = time_oracle(spec, args.pattern)
            cb.pop("seconds")
            line["cpu_baseline"] = cb
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c2", choices=list(graphs.BUILDERS))
    ap.add_argument("--pattern", default="streaming")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--frames", type=int, default=0)
    ap.add_argument("--engine", default="auto", choices=["auto", "direct"])
    ap.add_argument("--graph-frames", type=int, default=16, help="frames per CUDA graph inside sr_rollout_run (0 = plain launches)")
    ap.add_argument("--resident", type=int, default=1, help="1: sr_rollout_run may use the shared-memory-resident kernel; 0: per-frame launches")
    ap.add_argument("--resident-cluster", type=int, default=0)
    ap.add_argument("--resident-warps", type=int, default=0)
    ap.add_argument("--only-main", action="store_true", help="time only --pattern, not the other rollout patterns")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
