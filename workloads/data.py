"""Seeded synthetic inputs, weights and biases for a GraphSpec.

Inputs have the structure of the paper's data (Sec. 4 "Datasets", Table A1): a
static image per sequence in a fixed value range plus a fresh Gaussian noise
sample on every frame.  Weights are random (trained weights are not needed to
time or check the frame update).  All arrays are float32; for bf16 graphs every
value is rounded to bfloat16 once, here, so that any consumer sees identical
operands.

Layouts: a state or frame is [B][H][W][C]; a conv weight [C_out][k][k][C_in]; a
dense weight [C_out][H][W][C_in] (the source flattened in H, W, C order); a
global-average dense weight [C_out][C_in].
"""
from __future__ import annotations

from typing import Dict, List

import numpy as np

from . import rng
from .graphs import CONV, DENSE, GAP_DENSE, GraphSpec


def _maybe_bf16(spec: GraphSpec, x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return rng.round_to_bf16(x) if spec.dtype == "bf16" else x


def edge_fan_in(spec: GraphSpec, ei: int) -> int:
    e = spec.edges[ei]
    s = spec.nodes[e.src]
    if e.kind == CONV:
        return e.k * e.k * s.c
    if e.kind == DENSE:
        return s.h * s.w * s.c
    return s.c


def weight_shape(spec: GraphSpec, ei: int):
    e = spec.edges[ei]
    s, t = spec.nodes[e.src], spec.nodes[e.tgt]
    if e.kind == CONV:
        return (t.c, e.k, e.k, s.c)
    if e.kind == DENSE:
        return (t.c, s.h, s.w, s.c)
    return (t.c, s.c)


def make_weights(spec: GraphSpec) -> List[np.ndarray]:
    """Normal weights with variance gain / fan_in, where fan_in of a target node is
    summed over all its incoming edges (the sum over incoming edges is one
    convolution over the concatenated sources, paper Sec. A), so that the
    pre-activation variance does not grow with the in-degree."""
    fan = [0] * len(spec.nodes)
    for ei, e in enumerate(spec.edges):
        fan[e.tgt] += edge_fan_in(spec, ei)
    out = []
    for ei, e in enumerate(spec.edges):
        shp = weight_shape(spec, ei)
        n = int(np.prod(shp))
        w = rng.normal(spec.seed, 100 + ei, n) * np.sqrt(spec.weight_gain / fan[e.tgt])
        out.append(_maybe_bf16(spec, w.reshape(shp)))
    return out


def make_biases(spec: GraphSpec, zero: bool = True) -> List[np.ndarray]:
    """Channel-wise biases (float32 in every mode).  The benchmark configs use 0;
    tests ask for non-zero values so that a dropped bias is seen."""
    out = []
    for vi, v in enumerate(spec.nodes):
        if zero:
            out.append(np.zeros(v.c, dtype=np.float32))
        else:
            out.append((0.1 * rng.normal(spec.seed, 500 + vi, v.c)).astype(np.float32))
    return out


def _blobs(seed: int, stream: int, b: int, h: int, w: int) -> np.ndarray:
    """Smooth images in [0, 1): three Gaussian bumps per image."""
    p = rng.uniform(seed, stream, b * 3 * 4).reshape(b, 3, 4)
    yy, xx = np.meshgrid(np.arange(h), np.arange(w), indexing="ij")
    img = np.zeros((b, h, w))
    for j in range(3):
        cy, cx = p[:, j, 0] * h, p[:, j, 1] * w
        amp, sig = p[:, j, 2], 2.0 + 4.0 * p[:, j, 3]
        d2 = (yy[None] - cy[:, None, None]) ** 2 + (xx[None] - cx[:, None, None]) ** 2
        img += amp[:, None, None] * np.exp(-d2 / (2.0 * sig[:, None, None] ** 2))
    return np.minimum(img, 1.0 - 2.0 ** -10)


def make_inputs(spec: GraphSpec) -> Dict[int, np.ndarray]:
    """Frames 0..T for every input node: {node index: [T+1][B][H][W][C] float32}."""
    out = {}
    t1, b = spec.frames + 1, spec.batch
    for vi in spec.input_nodes():
        v = spec.nodes[vi]
        shp = (t1, b, v.h, v.w, v.c)
        per = v.h * v.w * v.c
        fam = spec.name[:2]
        if fam == "c1":
            base = rng.uniform(spec.seed, 10 + vi, b * per).reshape(1, b, v.h, v.w, v.c)
            x = base + 0.1 * rng.normal(spec.seed, 20 + vi, t1 * b * per).reshape(shp)
        elif fam == "c2":
            base = _blobs(spec.seed, 10 + vi, b, v.h, v.w)[None, :, :, :, None]
            x = base + 0.3 * rng.normal(spec.seed, 20 + vi, t1 * b * per).reshape(shp)
            occ = rng.uniform(spec.seed, 30 + vi, t1 * b).reshape(t1, b) < 0.25
            blk = min(8, v.h, v.w)
            oy = rng.integers(spec.seed, 31 + vi, t1 * b, v.h - blk + 1).reshape(t1, b)
            ox = rng.integers(spec.seed, 32 + vi, t1 * b, v.w - blk + 1).reshape(t1, b)
            for t, s in zip(*np.nonzero(occ)):
                x[t, s, oy[t, s]:oy[t, s] + blk, ox[t, s]:ox[t, s] + blk, :] = 0.0
        elif fam == "c3":
            base = rng.normal(spec.seed, 10 + vi, b * per).reshape(1, b, v.h, v.w, v.c)
            x = base + 0.5 * rng.normal(spec.seed, 20 + vi, t1 * b * per).reshape(shp)
        elif fam == "c4":
            base = rng.uniform(spec.seed, 10 + vi, b * per).reshape(1, b, v.h, v.w, v.c)
            ramp = (0.5 + 0.5 * np.arange(t1) / max(1, spec.frames)).reshape(t1, 1, 1, 1, 1)
            x = base * ramp + 0.2 * rng.normal(spec.seed, 20 + vi, t1 * b * per).reshape(shp)
        else:
            x = rng.normal(spec.seed, 20 + vi, t1 * b * per).reshape(shp)
        out[vi] = _maybe_bf16(spec, x)
    return out
