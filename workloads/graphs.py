"""Network graphs and rollout patterns of the synthetic workloads.

A network is a directed graph of nodes (layers) and edges (transformations); a
rollout pattern R maps every edge to 1 (the edge bridges one frame) or 0 (the
edge stays inside a frame) (paper Sec. 3, Definitions "network" and "rollout
pattern and window").  This module only describes graphs; it computes nothing
of the method.

Shapes follow the paper's experiments (Sec. A "Details about networks, data,
and training"): 28x28x1 and 32x32x3 image sequences, 3x3 convolutions whose
stride is input size / output size, dense heads with 10 or 43 classes.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List

from . import rng

CONV, DENSE, GAP_DENSE = 0, 1, 2
IDENTITY, RELU = 0, 1


@dataclass(frozen=True)
class Node:
    name: str
    h: int
    w: int
    c: int
    act: int = RELU


@dataclass(frozen=True)
class Edge:
    src: int
    tgt: int
    kind: int = CONV
    k: int = 3
    stride: int = 1
    pool: int = 0          # 2: the 3x3 stride-1 conv is followed by a 2x2 stride-2 average


@dataclass
class GraphSpec:
    name: str
    nodes: List[Node]
    edges: List[Edge]
    batch: int
    frames: int                       # T frame updates; T+1 input frames 0..T are generated
    dtype: str                        # "fp32" or "bf16"
    seed: int
    weight_gain: float = 2.0          # variance numerator: 2 (He) or 1
    patterns: Dict[str, List[int]] = field(default_factory=dict)

    def input_nodes(self) -> List[int]:
        has_in = {e.tgt for e in self.edges}
        return [i for i in range(len(self.nodes)) if i not in has_in]

    def index(self, name: str) -> int:
        return [n.name for n in self.nodes].index(name)


def streaming_pattern(spec: GraphSpec) -> List[int]:
    return [1] * len(spec.edges)


def sequential_pattern(spec: GraphSpec) -> List[int]:
    """R(e)=1 only for self-loops and edges that point back in node order.

    When every other edge goes forward in node order the within-frame edges
    cannot close a cycle, and no further edge can be set to 0, so this is a
    most-sequential pattern (unique when the net has no cycle longer than 1).
    """
    return [1 if e.src >= e.tgt else 0 for e in spec.edges]


def _edge_out_size(n_in: int, k: int, stride: int) -> int:
    pad = (k - 1) // 2
    return (n_in + 2 * pad - k) // stride + 1


def check_shapes(spec: GraphSpec) -> None:
    """Every edge must map its source shape to its target shape."""
    for e in spec.edges:
        s, t = spec.nodes[e.src], spec.nodes[e.tgt]
        if e.kind == CONV:
            oh, ow = _edge_out_size(s.h, e.k, e.stride), _edge_out_size(s.w, e.k, e.stride)
            if e.pool == 2:
                oh, ow = oh // 2, ow // 2
            assert (oh, ow) == (t.h, t.w), (spec.name, e, (oh, ow), (t.h, t.w))
        else:
            assert (t.h, t.w) == (1, 1), (spec.name, e)


def macs_per_sample(spec: GraphSpec) -> int:
    """Multiply-adds of one frame update of one sample (true K, true output counts;
    a pooled edge is counted as the 4x4 stride-2 convolution it equals)."""
    total = 0
    for e in spec.edges:
        s, t = spec.nodes[e.src], spec.nodes[e.tgt]
        if e.kind == CONV:
            k2 = 16 if e.pool == 2 else e.k * e.k
            total += t.h * t.w * t.c * k2 * s.c
        elif e.kind == DENSE:
            total += t.c * s.h * s.w * s.c
        else:
            total += t.c * s.c
    return total


# ----------------------------------------------------------------------------- tiny nets for the theory pins
def worked_example() -> GraphSpec:
    """Three scalar nodes x -> h -> y with a skip x -> y and a self-loop on h."""
    nodes = [Node("x", 1, 1, 1, IDENTITY), Node("h", 1, 1, 1, RELU), Node("y", 1, 1, 1, RELU)]
    edges = [Edge(0, 1, DENSE), Edge(1, 1, DENSE), Edge(1, 2, DENSE), Edge(0, 2, DENSE)]
    g = GraphSpec("worked_example", nodes, edges, batch=1, frames=4, dtype="fp32", seed=0)
    g.patterns = {"streaming": [1, 1, 1, 1], "sequential": [0, 1, 0, 0], "hybrid": [0, 1, 1, 0]}
    return g


def mnist_net(kind: str = "SR", batch: int = 4, frames: int = 6) -> GraphSpec:
    """The paper's MNIST nets FF / S / SR (Sec. A, paragraph MNIST): I 28x28x1,
    H1 7x7x16 (conv receptive field 7, stride 4), H2 128, O 10; S adds the skip
    H1->O, SR adds the self-recurrence H1->H1 (3x3, stride 1)."""
    nodes = [Node("I", 28, 28, 1, IDENTITY), Node("H1", 7, 7, 16), Node("H2", 1, 1, 128), Node("O", 1, 1, 10, IDENTITY)]
    edges = [Edge(0, 1, CONV, 7, 4), Edge(1, 2, DENSE), Edge(2, 3, DENSE)]
    if kind in ("S", "SR"):
        edges.append(Edge(1, 3, DENSE))
    if kind == "SR":
        edges.append(Edge(1, 1, CONV, 3, 1))
    g = GraphSpec("mnist_" + kind, nodes, edges, batch=batch, frames=frames, dtype="fp32", seed=77)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g)}
    return g


def chain_with_shortcut(longest: int, shortest: int = 4) -> GraphSpec:
    """A scalar chain of `longest` edges from input to output plus one skip that
    makes the shortest input-output path `shortest` edges long, and a self-loop on
    the first hidden node: the path structure the paper states for its CIFAR10
    nets (Sec. 4: shortest path 4, longest path growing with depth)."""
    n = longest + 1
    nodes = [Node("v%d" % i, 1, 1, 1, RELU if 0 < i < n - 1 else IDENTITY) for i in range(n)]
    edges = [Edge(i, i + 1, DENSE) for i in range(longest)]
    if longest > shortest:
        # skip from node (shortest-1) straight to the output node
        edges.append(Edge(shortest - 1, n - 1, DENSE))
    edges.append(Edge(1, 1, DENSE))
    g = GraphSpec("chain%d" % longest, nodes, edges, batch=1, frames=2 * n, dtype="fp32", seed=5)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g)}
    return g


def three_cycle_net() -> GraphSpec:
    """Input feeding a minimal cycle of length 3 (cf. the second network of the
    paper's Fig. 2, which has three most-sequential rollout patterns)."""
    nodes = [Node("i", 1, 1, 1, IDENTITY), Node("a", 1, 1, 1), Node("b", 1, 1, 1), Node("c", 1, 1, 1)]
    edges = [Edge(0, 1, DENSE), Edge(1, 2, DENSE), Edge(2, 3, DENSE), Edge(3, 1, DENSE)]
    return GraphSpec("three_cycle", nodes, edges, batch=1, frames=4, dtype="fp32", seed=6)


def ff_chain(depth: int, width: int = 8, batch: int = 2, frames: int | None = None) -> GraphSpec:
    """Skip-free feed-forward chain of `depth` dense edges."""
    nodes = [Node("v0", 1, 1, width, IDENTITY)] + [Node("v%d" % i, 1, 1, width) for i in range(1, depth + 1)]
    edges = [Edge(i, i + 1, DENSE) for i in range(depth)]
    g = GraphSpec("ff%d" % depth, nodes, edges, batch=batch, frames=frames or 2 * depth + 2, dtype="fp32", seed=9)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g)}
    return g


# ----------------------------------------------------------------------------- the five benchmark configs
def c1_mlp(batch: int = 8, frames: int = 16) -> GraphSpec:
    nodes = [Node("input", 1, 1, 784, IDENTITY), Node("h1", 1, 1, 128), Node("h2", 1, 1, 128),
             Node("out", 1, 1, 10, IDENTITY)]
    edges = [Edge(0, 1, DENSE), Edge(1, 2, DENSE), Edge(2, 3, DENSE), Edge(0, 3, DENSE), Edge(2, 2, DENSE)]
    g = GraphSpec("c1", nodes, edges, batch, frames, "fp32", seed=1001, weight_gain=1.0)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g)}
    return g


def c2_small_cnn(batch: int = 64, frames: int = 32, dtype: str = "bf16") -> GraphSpec:
    nodes = [Node("input", 28, 28, 1, IDENTITY), Node("c1", 28, 28, 32), Node("c2", 14, 14, 32),
             Node("c3", 7, 7, 64), Node("fc", 1, 1, 10, IDENTITY)]
    edges = [Edge(0, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 2), Edge(2, 2, CONV, 3, 1),
             Edge(1, 3, CONV, 3, 4),          # 28 -> 7 needs stride = input size / output size = 4
             Edge(2, 3, CONV, 3, 2), Edge(3, 4, DENSE)]
    g = GraphSpec("c2", nodes, edges, batch, frames, dtype, seed=1002)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g)}
    return g


def c3_six_node(batch: int = 256, frames: int = 20, size: int = 32, dtype: str = "bf16") -> GraphSpec:
    s = size
    nodes = [Node("in", s, s, 3, IDENTITY), Node("n1", s, s, 64), Node("n2", s, s, 64),
             Node("n3", s // 2, s // 2, 128), Node("n4", s // 2, s // 2, 128), Node("n5", s // 4, s // 4, 256),
             Node("out", 1, 1, 10, IDENTITY)]
    edges = [Edge(0, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 1), Edge(2, 3, CONV, 3, 2), Edge(3, 4, CONV, 3, 1),
             Edge(4, 5, CONV, 3, 2)]
    edges += [Edge(i, i, CONV, 3, 1) for i in range(1, 6)]                      # self-recurrence on n1..n5
    edges += [Edge(0, 2, CONV, 1, 1), Edge(1, 3, CONV, 1, 2), Edge(2, 4, CONV, 1, 2), Edge(3, 5, CONV, 1, 2)]
    edges += [Edge(5, 6, GAP_DENSE)]
    g = GraphSpec("c3", nodes, edges, batch, frames, dtype, seed=1003)
    # hybrid: a two-stage pipeline; within-frame edges inside {n1,n2,n3} and inside {n4,n5,out},
    # input edges within-frame, everything that crosses the halves or recurs bridges a frame
    first, second = {1, 2, 3}, {4, 5, 6}
    hyb = []
    for e in edges:
        if e.src == e.tgt:
            hyb.append(1)
        elif e.src == 0:
            hyb.append(0)
        elif (e.src in first and e.tgt in first) or (e.src in second and e.tgt in second):
            hyb.append(0)
        else:
            hyb.append(1)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g), "hybrid": hyb}
    return g


def c4_ten_node(batch: int = 128, frames: int = 64, size: int = 32, dtype: str = "bf16", recurrence: bool = True) -> GraphSpec:
    s = size
    chans = [64, 64, 128, 128, 128, 128, 256, 256, 256, 256]
    sizes = [s, s, s // 2, s // 2, s // 2, s // 2, s // 4, s // 4, s // 4, s // 4]
    nodes = [Node("in", s, s, 3, IDENTITY)] + [Node("n%d" % (i + 1), sizes[i], sizes[i], chans[i]) for i in range(10)]
    nodes.append(Node("out", 1, 1, 43, IDENTITY))
    edges = []
    for i in range(10):                       # chain in -> n1 -> ... -> n10; n2->n3 and n6->n7 are pooling edges
        pooled = (i + 1) in (3, 7)
        edges.append(Edge(i, i + 1, CONV, 3, 1, 2 if pooled else 0))
    if recurrence:
        edges += [Edge(i, i, CONV, 3, 1) for i in (2, 4, 6, 8)]
    edges += [Edge(2, 4, CONV, 3, 2), Edge(6, 8, CONV, 3, 2), Edge(2, 8, CONV, 3, 4)]
    edges += [Edge(10, 11, GAP_DENSE)]
    g = GraphSpec("c4" if recurrence else "c4ff", nodes, edges, batch, frames, dtype, seed=1004)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g)}
    return g


def c5_stress(batch: int = 32, frames: int = 128, size: int = 64, dtype: str = "bf16", seed: int = 1005) -> GraphSpec:
    n_conv = 16
    sizes = [size >> (i // 4) for i in range(n_conv)]
    nodes = [Node("in", size, size, 3, IDENTITY)] + [Node("n%d" % (i + 1), sizes[i], sizes[i], 128) for i in range(n_conv)]
    nodes.append(Node("out", 1, 1, 10, IDENTITY))
    edges = [Edge(0, 1, CONV, 3, 1)]
    for i in range(1, n_conv):
        edges.append(Edge(i, i + 1, CONV, 3, nodes[i].h // nodes[i + 1].h))
    # skip edges n_i -> n_j, j >= i+2, each with probability 0.3
    pairs = [(i, j) for i in range(1, n_conv + 1) for j in range(i + 2, n_conv + 1)]
    u = rng.uniform(seed, 900, len(pairs))
    for (i, j), p in zip(pairs, u):
        if p < 0.3:
            edges.append(Edge(i, j, CONV, 3, nodes[i].h // nodes[j].h))
    # six recurrent edges: self-loops and back-edges spanning up to 3 nodes, same spatial size only
    cands = [(j, i) for i in range(1, n_conv + 1) for j in range(i, min(i + 3, n_conv) + 1) if nodes[i].h == nodes[j].h]
    order = rng.bits64(seed, 901, len(cands)).argsort(kind="stable")
    for idx in sorted(order[:6].tolist()):
        j, i = cands[idx]
        edges.append(Edge(j, i, CONV, 3, 1))
    edges.append(Edge(n_conv, n_conv + 1, GAP_DENSE))
    g = GraphSpec("c5", nodes, edges, batch, frames, dtype, seed=seed)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g)}
    # three random hybrids: Bernoulli(1/2) on forward edges, recurrent edges always bridge a frame
    seq = g.patterns["sequential"]
    found, s = [], 0
    while len(found) < 3:
        bits = rng.uniform(seed, 910 + s, len(edges)) < 0.5
        pat = [1 if seq[i] == 1 else int(bits[i]) for i in range(len(edges))]
        s += 1
        if pat in found or pat == seq or pat == g.patterns["streaming"]:
            continue
        found.append(pat)
    for i, pat in enumerate(found):
        g.patterns["hybrid%d" % i] = pat
    return g


def mini_cnn(batch: int = 3, frames: int = 5, dtype: str = "bf16") -> GraphSpec:
    """A small image network with every kind of edge the frame update knows: a few-channel first layer,
    a pooling edge, recurrence, 1x1 skips with stride (one straight from the input), a hidden dense
    node, and an output that sums a dense and a global-average dense edge."""
    nodes = [Node("in", 16, 16, 3, IDENTITY), Node("n1", 16, 16, 32), Node("n2", 8, 8, 32), Node("n3", 4, 4, 64),
             Node("d", 1, 1, 16), Node("out", 1, 1, 10, IDENTITY)]
    edges = [Edge(0, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 1, 2), Edge(2, 2, CONV, 3, 1), Edge(2, 3, CONV, 3, 2),
             Edge(1, 3, CONV, 1, 4), Edge(0, 3, CONV, 1, 4), Edge(3, 4, DENSE), Edge(4, 5, DENSE), Edge(3, 5, GAP_DENSE),
             Edge(1, 1, CONV, 3, 1)]
    g = GraphSpec("mini", nodes, edges, batch, frames, dtype, seed=1010)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g),
                  "hybrid": [0, 1, 1, 0, 1, 0, 0, 1, 0, 1],
                  # the input feeds one node inside the frame and another across frames
                  "mixed_input": [1, 1, 1, 0, 1, 0, 0, 1, 0, 1]}
    return g


def dsr(k: int, batch: int = 4, frames: int = 6, dtype: str = "bf16", classes: int = 10, h1_recurrence: bool = True) -> GraphSpec:
    """The paper's CIFAR10 networks DSR0 .. DSR6 (Sec. A, paragraph CIFAR10): I 32x32x3; block 1 = H1, H11, H12, H13 at
    32x32x32; block 2 = H2, H21, H22, H23 at 16x16x64; HD 4x4x512; O 10.  DSR0 is I - H1 - H2 - HD - O with a
    self-recurrent H1; DSRk adds the first k of H11, H21, H12, H22, H13, H23.  Inside a block every earlier layer
    feeds every later one, and every layer of a block feeds the head of the next (H2, HD): 3x3 convolutions whose stride
    is input size / output size; I - H1 has receptive field 5.  The shortest input-output path has 4 edges, the longest
    4 + k.  DSR4 with 43 classes and without the H1 recurrence is the paper's GTSRB network."""
    assert 0 <= k <= 6
    added = ["H11", "H21", "H12", "H22", "H13", "H23"][:k]
    block1 = ["H1"] + [n for n in ("H11", "H12", "H13") if n in added]
    block2 = ["H2"] + [n for n in ("H21", "H22", "H23") if n in added]
    names = ["I"] + block1 + block2 + ["HD", "O"]
    nodes = [Node("I", 32, 32, 3, IDENTITY)] + [Node(n, 32, 32, 32) for n in block1] + [Node(n, 16, 16, 64) for n in block2]
    nodes += [Node("HD", 4, 4, 512), Node("O", 1, 1, classes, IDENTITY)]
    ix = {n: i for i, n in enumerate(names)}
    edges = [Edge(ix["I"], ix["H1"], CONV, 5, 1)]
    for blk, head, stride in ((block1, "H2", 2), (block2, "HD", 4)):
        for i, a in enumerate(blk):
            for b in blk[i + 1:]:
                edges.append(Edge(ix[a], ix[b], CONV, 3, 1))
            edges.append(Edge(ix[a], ix[head], CONV, 3, stride))
    edges.append(Edge(ix["HD"], ix["O"], DENSE))
    if h1_recurrence:
        edges.append(Edge(ix["H1"], ix["H1"], CONV, 3, 1))
    g = GraphSpec("dsr%d" % k, nodes, edges, batch, frames, dtype, seed=1020 + k)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g)}
    return g


def conv_sink(batch: int = 3, frames: int = 4, dtype: str = "bf16") -> GraphSpec:
    """A network whose output node is an image: in -> n1 (3x3) -> n2 (3x3, stride 2), recurrence on n1."""
    nodes = [Node("in", 8, 8, 3, IDENTITY), Node("n1", 8, 8, 16), Node("n2", 4, 4, 8, IDENTITY)]
    edges = [Edge(0, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 2), Edge(1, 1, CONV, 3, 1)]
    g = GraphSpec("sink", nodes, edges, batch, frames, dtype, seed=1011)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g)}
    return g


BUILDERS = {"mini": mini_cnn, "sink": conv_sink, "dsr0": lambda **kw: dsr(0, **kw), "dsr2": lambda **kw: dsr(2, **kw),
            "dsr4": lambda **kw: dsr(4, **kw), "dsr6": lambda **kw: dsr(6, **kw), "c1": c1_mlp, "c2": c2_small_cnn, "c3": c3_six_node, "c4": c4_ten_node, "c5": c5_stress,
            "c4ff": lambda **kw: c4_ten_node(recurrence=False, **kw)}


def with_copy_nodes(spec: GraphSpec, delays: List[int]):
    """Edges that bridge more than one frame, R(e) = d > 1, written with copy-nodes (paper Sec. 6: longer forward
    connections are covered by the theory through copy-nodes): edge e = (u, v) becomes the chain
    u -> c_1 -> ... -> c_{d-1} -> v, every link bridging one frame; a copy-node has the shape of u, the identity as its
    activation, no bias, and its one incoming edge is a 1x1 convolution whose weight is the identity matrix.
    Returns the expanded GraphSpec (pattern "p" with values in {0, 1}; edge i of spec is still edge i) and, per added
    edge, the channel count of its identity weight."""
    nodes, edges, R = list(spec.nodes), list(spec.edges), [min(int(d), 1) for d in delays]
    identity_channels = []
    for ei, d in enumerate(delays):
        e = spec.edges[ei]
        src = e.src
        for j in range(int(d) - 1):
            u = spec.nodes[e.src]
            nodes.append(Node("copy%d_%d" % (ei, j + 1), u.h, u.w, u.c, IDENTITY))
            edges.append(Edge(src, len(nodes) - 1, CONV, 1, 1))
            R.append(1)
            identity_channels.append(u.c)
            src = len(nodes) - 1
        edges[ei] = Edge(src, e.tgt, e.kind, e.k, e.stride, e.pool)
    g = GraphSpec(spec.name + "_copy", nodes, edges, spec.batch, spec.frames, spec.dtype, spec.seed, spec.weight_gain)
    g.patterns = {"p": R}
    return g, identity_channels


def build(name: str, **overrides) -> GraphSpec:
    g = BUILDERS[name](**overrides)
    check_shapes(g)
    return g
