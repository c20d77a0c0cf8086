"""ctypes binding of oracle/frame_update.c (test infrastructure only).

`rollout(spec-like arguments)` evaluates the explicit rollout window for T frame
updates in double precision and returns every node state at every frame.
The visiting order inside a frame comes from the theory half (tableau levels).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, List, Sequence

import numpy as np

from . import rollout_theory as rt

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "frame_update.c")
_LIB = os.path.join(_HERE, "libsr_oracle.so")
_lib = None


class _Node(ctypes.Structure):
    _fields_ = [("h", ctypes.c_int32), ("w", ctypes.c_int32), ("c", ctypes.c_int32), ("act", ctypes.c_int32)]


class _Edge(ctypes.Structure):
    _fields_ = [("src", ctypes.c_int32), ("tgt", ctypes.c_int32), ("kind", ctypes.c_int32),
                ("k", ctypes.c_int32), ("stride", ctypes.c_int32), ("pool", ctypes.c_int32)]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP across samples)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.sro_rollout.restype = ctypes.c_int
    return _lib


def rollout(nodes: Sequence, edges: Sequence, R: Sequence[int], batch: int, frames: int,
            inputs: Dict[int, np.ndarray], weights: List[np.ndarray], biases: List[np.ndarray],
            round_states_bf16: bool = False, initial_states: Dict[int, np.ndarray] | None = None) -> List[np.ndarray]:
    """nodes: objects with h, w, c, act; edges: objects with src, tgt, kind, k, stride, pool.
    inputs: {input node: [T+1][B][H][W][C]}.  Returns one float64 array [T+1][B][H][W][C] per node.
    initial_states: {non-input node: [B][H][W][C]} makes the window continue an earlier one (its last frame is this
    window's frame 0, paper Sec. 4); nodes left out start at zero."""
    lib = _load()
    n_nodes, n_edges = len(nodes), len(edges)
    pairs = [(e.src, e.tgt) for e in edges]
    if not rt.is_network(n_nodes, pairs):
        raise ValueError("not a network")
    if not rt.is_valid(n_nodes, pairs, R):
        raise ValueError("invalid rollout pattern")
    levels = rt.frame_levels(n_nodes, pairs, R)
    order = sorted([v for v in range(n_nodes) if levels[v] > 0], key=lambda v: (levels[v], v))
    c_nodes = (_Node * n_nodes)(*[_Node(n.h, n.w, n.c, n.act) for n in nodes])
    c_edges = (_Edge * n_edges)(*[_Edge(e.src, e.tgt, e.kind, e.k, e.stride, e.pool) for e in edges])
    c_R = (ctypes.c_uint8 * n_edges)(*[int(r) for r in R])
    c_order = (ctypes.c_int32 * len(order))(*order)
    states = []
    for vi, n in enumerate(nodes):
        if vi in inputs:
            a = np.ascontiguousarray(inputs[vi], dtype=np.float64)
            assert a.shape == (frames + 1, batch, n.h, n.w, n.c), (a.shape, vi)
        else:
            a = np.zeros((frames + 1, batch, n.h, n.w, n.c), dtype=np.float64)
            if initial_states is not None and vi in initial_states:
                a[0] = np.asarray(initial_states[vi], dtype=np.float64).reshape(a[0].shape)
        states.append(a)
    w64 = [np.ascontiguousarray(w, dtype=np.float64) for w in weights]
    b64 = [np.ascontiguousarray(b, dtype=np.float64) for b in biases]
    dp = ctypes.POINTER(ctypes.c_double)
    c_w = (dp * n_edges)(*[w.ctypes.data_as(dp) for w in w64])
    c_b = (dp * n_nodes)(*[b.ctypes.data_as(dp) for b in b64])
    c_s = (dp * n_nodes)(*[s.ctypes.data_as(dp) for s in states])
    rc = lib.sro_rollout(n_nodes, c_nodes, n_edges, c_edges, c_R, c_order, len(order), batch, frames,
                         c_w, c_b, c_s, int(round_states_bf16), int(initial_states is not None))
    if rc != 0:
        raise RuntimeError("sro_rollout failed: %d" % rc)
    return states


def rollout_spec(spec, pattern: str, inputs=None, weights=None, biases=None, samples=None, frames=None, **kw):
    """Convenience: run a workloads.GraphSpec, optionally on a subset of batch samples
    (sequences are independent, so a subset is exact) and fewer frames."""
    T = spec.frames if frames is None else frames
    if samples is not None:
        inputs = {k: v[:T + 1, samples] for k, v in inputs.items()}
        batch = len(samples)
    else:
        inputs = {k: v[:T + 1] for k, v in inputs.items()}
        batch = spec.batch
    return rollout(spec.nodes, spec.edges, spec.patterns[pattern], batch, T, inputs, weights, biases, **kw)
