"""Helpers shared by the GPU parity tests: run a workload through the C-ABI binding and the
oracle on the same seeded inputs and compare node states frame by frame."""
from __future__ import annotations

import numpy as np

from oracle import frame_update as fu
from workloads import data, rng

TOL = {"bf16": 2e-2, "fp32": 1e-4}       # max-abs-diff relative to the node's output scale


def to_device(spec, arr, device="cuda:0"):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32)).to(device)
    return t.to(torch.bfloat16).contiguous() if spec.dtype == "bf16" else t.contiguous()


def make_graph(spec, pattern, engine="auto", graph_frames=0, weights=None, biases=None, **options):
    from paper_1806_04965_b200 import Graph
    G = Graph(spec.nodes, spec.edges, spec.patterns[pattern], batch=spec.batch, dtype=spec.dtype, engine=engine,
              graph_frames=graph_frames, **options)
    G.set_weights(weights, biases)
    return G


def rel_err(got: np.ndarray, want: np.ndarray) -> float:
    scale = max(1e-6, float(np.abs(want).max()))
    return float(np.abs(got.astype(np.float64) - want).max()) / scale


def check_stepwise(spec, pattern, engine="auto", samples=None, zero_bias=False, tol=None, **options):
    """Step frame by frame; compare EVERY node state at EVERY frame with the oracle on `samples`."""
    import torch
    X, W, Bi = data.make_inputs(spec), data.make_weights(spec), data.make_biases(spec, zero=zero_bias)
    samples = list(range(spec.batch)) if samples is None else samples
    want = fu.rollout_spec(spec, pattern, X, W, Bi, samples=samples)
    G = make_graph(spec, pattern, engine, 0, W, Bi, **options)
    ins = G.input_nodes
    dev = {v: to_device(spec, X[v]) for v in ins}
    G.reset([dev[v][0] for v in ins])
    out = torch.empty(G.out_shape(), dtype=torch.float32, device="cuda:0")
    tol = TOL[spec.dtype] if tol is None else tol
    worst = 0.0
    for t in range(1, spec.frames + 1):
        G.step([dev[v][t] for v in ins], out)
        for v in range(len(spec.nodes)):
            got = G.get_state(v).float().cpu().numpy()[samples]
            e = rel_err(got, want[v][t])
            worst = max(worst, e)
            assert e <= tol, "node %s frame %d pattern %s: rel err %.3e > %.1e" % (spec.nodes[v].name, t, pattern, e, tol)
        e = rel_err(out.cpu().numpy()[samples].reshape(want[G.output_node][t].shape), want[G.output_node][t])
        assert e <= tol, ("output", t, e)
    G.sync_status()
    return worst


def check_run(spec, pattern, engine="auto", graph_frames=0, samples=None, frames=None, tol=None, expect_resident=None,
              **options):
    """One sr_rollout_run over all frames; compare the output sequence and the final states."""
    X, W, Bi = data.make_inputs(spec), data.make_weights(spec), data.make_biases(spec)
    T = spec.frames if frames is None else frames
    samples = list(range(spec.batch)) if samples is None else samples
    want = fu.rollout_spec(spec, pattern, X, W, Bi, samples=samples, frames=T)
    G = make_graph(spec, pattern, engine, graph_frames, W, Bi, **options)
    if expect_resident is not None:
        assert G.info["resident_cluster"] == expect_resident, G.info
    ins = G.input_nodes
    out = G.rollout([to_device(spec, X[v][:T + 1]) for v in ins])
    G.sync_status()
    tol = TOL[spec.dtype] if tol is None else tol
    o = G.output_node
    got = out.cpu().numpy()[:, samples]
    e = rel_err(got.reshape(want[o][1:].shape), want[o][1:])
    assert e <= tol, ("output sequence", pattern, e)
    worst = e
    for v in range(len(spec.nodes)):
        g = G.get_state(v).float().cpu().numpy()[samples]
        e = rel_err(g, want[v][T])
        worst = max(worst, e)
        assert e <= tol, "final state of %s, pattern %s: rel err %.3e" % (spec.nodes[v].name, pattern, e)
    assert G.frame() == T
    return worst
