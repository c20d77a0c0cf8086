"""GPU parity of the resident kernel (one thread-block cluster per sequence, all frames of a run in one
launch, states in shared memory) against the oracle: every edge kind, every cluster size, streaming,
sequential and hybrid patterns, runs split in two and runs continued by single steps of the launch path."""
import numpy as np
import pytest

from oracle import frame_update as fu
from tests import parity
from workloads import data, graphs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cluster", [1, 2, 4])
def test_mini_cnn_every_pattern(cluster):
    g = graphs.build("mini", batch=3, frames=5)
    for p in g.patterns:
        parity.check_run(g, p, expect_resident=cluster, resident_cluster=cluster)


@pytest.mark.parametrize("split", [1, 2])
def test_both_tile_widths(split):
    """16-channel work units for every convolutional node / for the nodes the cost rule picks (default: 32-channel units)."""
    for g in (graphs.build("mini", batch=3, frames=4), graphs.build("c2", batch=2, frames=4)):
        for p in g.patterns:
            parity.check_run(g, p, expect_resident=2, resident_cluster=2, resident_split=split)


@pytest.mark.parametrize("cin,cout,k,stride,pool,size,cluster", [
    (32, 32, 3, 1, 0, 12, 2), (64, 64, 3, 1, 0, 8, 1), (64, 32, 3, 2, 0, 16, 2), (128, 32, 3, 1, 0, 8, 2), (64, 96, 1, 2, 0, 8, 1),
    (32, 64, 5, 1, 0, 10, 2), (32, 32, 7, 4, 0, 28, 2), (64, 32, 3, 1, 2, 16, 4), (96, 32, 3, 1, 0, 9, 1), (32, 64, 1, 1, 0, 6, 2),
])
def test_single_conv_edge(cin, cout, k, stride, pool, size, cluster):
    """Source channel counts (k-step loops of every shape), filter sizes, strides, a pooled edge, odd image sizes."""
    from workloads.graphs import CONV, GAP_DENSE, IDENTITY, Edge, GraphSpec, Node, check_shapes
    out = size // stride // (2 if pool else 1)
    nodes = [Node("in", size, size, 2, IDENTITY), Node("a", size, size, cin), Node("n", out, out, cout), Node("o", 1, 1, 6, IDENTITY)]
    edges = [Edge(0, 1, CONV, 3, 1), Edge(1, 2, CONV, k, stride, pool), Edge(2, 2, CONV, 3, 1), Edge(2, 3, GAP_DENSE)]
    for R in ([1, 1, 1, 1], [0, 0, 1, 0]):
        g = GraphSpec("edge", nodes, edges, batch=2, frames=3, dtype="bf16", seed=99)
        g.patterns = {"p": R}
        check_shapes(g)
        parity.check_run(g, "p", expect_resident=cluster, resident_cluster=cluster)


@pytest.mark.parametrize("cluster,warps", [(2, 16), (2, 8), (2, 5), (4, 12), (2, 24), (2, 32), (4, 29)])
def test_c2_reduced(cluster, warps):
    g = graphs.build("c2", batch=3, frames=6)
    for p in g.patterns:
        parity.check_run(g, p, expect_resident=cluster, resident_cluster=cluster, resident_warps=warps)


@pytest.mark.parametrize("batch,frames", [(1, 1), (1, 2), (2, 3), (5, 7)])
def test_short_runs_and_small_batches(batch, frames):
    """One- and two-frame runs (the input look-ahead is longer than the run), a single sequence, an odd batch."""
    g = graphs.build("mini", batch=batch, frames=frames)
    for p in g.patterns:
        parity.check_run(g, p, expect_resident=2, resident_cluster=2)
    g = graphs.build("c2", batch=batch, frames=frames)
    parity.check_run(g, "streaming", expect_resident=2, resident_cluster=2)


def test_empty_run_is_a_no_op():
    import torch
    g = graphs.build("mini", batch=2, frames=2)
    X, W, Bi = data.make_inputs(g), data.make_weights(g), data.make_biases(g, zero=False)
    G = parity.make_graph(g, "streaming", "auto", 0, W, Bi)
    x = parity.to_device(g, X[0])
    G.reset([x[0]])
    before = [G.get_state(v).clone() for v in range(len(g.nodes))]
    G.run([x[1:1]])
    G.sync_status()
    assert G.frame() == 0
    for v in range(len(g.nodes)):
        assert torch.equal(G.get_state(v), before[v])


def random_small_network(seed):
    """A seeded random image network of the kind the resident kernel takes: 2-4 convolutional nodes of 32 or 64
    channels on shrinking images, a chain plus random skips (1x1 or 3x3, stride = size ratio) and self-loops, a
    dense or mean-dense head, and a random valid rollout pattern (forward edges drawn, recurrent edges bridge)."""
    from workloads.graphs import CONV, DENSE, GAP_DENSE, IDENTITY, Edge, GraphSpec, Node, check_shapes
    r = np.random.default_rng(seed)
    size = int(r.choice([8, 12, 16, 20]))
    nodes = [Node("in", size, size, int(r.choice([1, 2, 3])), IDENTITY)]
    sizes = [size]
    for i in range(int(r.integers(2, 5))):
        s = sizes[-1] // 2 if (sizes[-1] % 2 == 0 and sizes[-1] >= 8 and r.random() < 0.5) else sizes[-1]
        sizes.append(s)
        nodes.append(Node("n%d" % (i + 1), s, s, int(r.choice([32, 64]))))
    n_conv = len(nodes) - 1
    nodes.append(Node("out", 1, 1, int(r.integers(3, 13)), IDENTITY))
    edges = [Edge(i, i + 1, CONV, 3, sizes[i] // sizes[i + 1]) for i in range(n_conv)]
    for i in range(n_conv + 1):
        for j in range(i + 2, n_conv + 1):
            if r.random() < 0.4 and sizes[i] % sizes[j] == 0:
                edges.append(Edge(i, j, CONV, int(r.choice([1, 3])), sizes[i] // sizes[j]))
    for i in range(1, n_conv + 1):
        if r.random() < 0.4:
            edges.append(Edge(i, i, CONV, 3, 1))
    edges.append(Edge(n_conv, n_conv + 1, DENSE if r.random() < 0.5 else GAP_DENSE))
    g = GraphSpec("rand%d" % seed, nodes, edges, batch=int(r.integers(1, 4)), frames=int(r.integers(2, 6)), dtype="bf16", seed=2000 + seed)
    g.patterns = {"streaming": [1] * len(edges),
                  "random": [1 if e.src >= e.tgt else int(r.random() < 0.5) for e in edges]}
    check_shapes(g)
    return g, int(r.choice([1, 2, 4]))


@pytest.mark.parametrize("seed", range(12))
def test_random_small_networks(seed):
    g, cluster = random_small_network(seed)
    if min(v.h for v in g.nodes[:-1]) < cluster:
        cluster = 1
    for p in g.patterns:
        parity.check_run(g, p, resident_cluster=cluster)


def test_default_choice_and_opt_out():
    from paper_1806_04965_b200 import Graph
    g = graphs.build("c2", batch=4, frames=2)
    assert Graph(g.nodes, g.edges, g.patterns["streaming"], batch=4).info["resident_cluster"] == 4
    assert Graph(g.nodes, g.edges, g.patterns["streaming"], batch=64).info["resident_cluster"] == 2
    # states and weights of one sequence exceed one CTA's shared memory: two CTAs per sequence, in waves
    assert Graph(g.nodes, g.edges, g.patterns["streaming"], batch=100).info["resident_cluster"] == 2
    assert Graph(g.nodes, g.edges, g.patterns["streaming"], batch=4, resident_cluster=1).info["resident_cluster"] == 0
    assert Graph(g.nodes, g.edges, g.patterns["streaming"], batch=4, resident=False).info["resident_cluster"] == 0
    assert Graph(g.nodes, g.edges, g.patterns["streaming"], batch=4, engine="direct").info["resident_cluster"] == 0
    assert Graph(g.nodes, g.edges, g.patterns["streaming"], batch=4, dtype="fp32").info["resident_cluster"] == 0
    big = graphs.build("c3", batch=2, frames=2)        # megabytes of weights: stays on the launch path
    assert Graph(big.nodes, big.edges, big.patterns["streaming"], batch=2).info["resident_cluster"] == 0


@pytest.mark.parametrize("pattern", ["streaming", "sequential"])
def test_split_runs_and_steps_continue_each_other(pattern):
    """run(3) -> step, step -> run(4): the resident kernel picks the states up from, and hands them back to,
    the buffers the launch path uses; every output and the final states match the oracle."""
    import torch
    g = graphs.build("mini", batch=4, frames=9)
    X, W, Bi = data.make_inputs(g), data.make_weights(g), data.make_biases(g, zero=False)
    want = fu.rollout_spec(g, pattern, X, W, Bi)
    G = parity.make_graph(g, pattern, "auto", 0, W, Bi, resident_cluster=2)
    assert G.info["resident_cluster"] == 2
    x = parity.to_device(g, X[0])
    o = G.output_node
    out = torch.zeros((9, g.batch, 10), dtype=torch.float32, device="cuda:0")
    G.reset([x[0]])
    G.run([x[1:4]], out[0:3])
    G.step([x[4]], out[3])
    G.step([x[5]], out[4])
    G.run([x[6:10]], out[5:9])
    G.sync_status()
    assert G.frame() == 9
    assert parity.rel_err(out.cpu().numpy().reshape(want[o][1:].shape), want[o][1:]) <= parity.TOL["bf16"]
    for v in range(len(g.nodes)):
        assert parity.rel_err(G.get_state(v).float().cpu().numpy(), want[v][9]) <= parity.TOL["bf16"], g.nodes[v].name


def test_resident_and_launch_path_agree_at_full_size():
    g = graphs.build("c2")
    X, W, Bi = data.make_inputs(g), data.make_weights(g), data.make_biases(g)
    outs = []
    for resident in (True, False):
        G = parity.make_graph(g, "streaming", "auto", 16, W, Bi, resident=resident)
        assert (G.info["resident_cluster"] > 0) == resident
        outs.append(G.rollout([parity.to_device(g, X[0])]).cpu().numpy())
        G.sync_status()
    assert np.abs(outs[1]).max() > 0
    assert parity.rel_err(outs[0], outs[1].astype(np.float64)) <= parity.TOL["bf16"]
