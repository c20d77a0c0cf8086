"""GPU parity of the dense resident engine (small all-dense fp32 networks: weights and states in the shared memory of
one thread-block cluster, all frames of a run in one launch) against the oracle, and its hand-over to the per-frame
launch path: states left in global memory, frame counter, resumed runs."""
import numpy as np
import pytest

from tests import parity
from workloads import data, graphs
from workloads.graphs import DENSE, GAP_DENSE, IDENTITY, RELU, Edge, GraphSpec, Node, sequential_pattern, streaming_pattern

pytestmark = pytest.mark.gpu

# CTAs per cluster: sixteen when a frame is one tableau level (streaming), eight otherwise
CLUSTER = {"streaming": 16, "sequential": 8, "hybrid": 8}


def mlp(batch, frames, sizes=(36, 20, 10, 7), seed=31):
    """input -> h1 -> h2 -> out with a skip input -> out, a self-loop on h2 and a back-edge h2 -> h1."""
    nodes = [Node("in", 1, 1, sizes[0], IDENTITY), Node("h1", 1, 1, sizes[1], RELU), Node("h2", 1, 1, sizes[2], RELU),
             Node("out", 1, 1, sizes[3], IDENTITY)]
    edges = [Edge(0, 1, DENSE), Edge(1, 2, DENSE), Edge(2, 3, DENSE), Edge(0, 3, GAP_DENSE), Edge(2, 2, DENSE), Edge(2, 1, DENSE)]
    g = GraphSpec("mlp", nodes, edges, batch=batch, frames=frames, dtype="fp32", seed=seed, weight_gain=1.0)
    g.patterns = {"streaming": streaming_pattern(g), "sequential": sequential_pattern(g), "hybrid": [0, 1, 0, 1, 1, 1]}
    return g


@pytest.mark.parametrize("pattern", ["streaming", "sequential"])
def test_c1_runs_on_the_dense_resident_engine(pattern):
    g = graphs.build("c1")
    cluster = CLUSTER[pattern]
    parity.check_run(g, pattern, expect_resident=cluster)
    parity.check_run(g, pattern, frames=1, expect_resident=cluster)
    parity.check_run(g, pattern, resident=False, expect_resident=0)


@pytest.mark.parametrize("batch", [1, 8, 11, 40])
def test_odd_sizes_and_batches(batch):
    # channel counts that are no multiple of four (padded columns), more sequences than one cluster holds, a ragged last cluster
    g = mlp(batch, 7)
    for p in g.patterns:
        parity.check_run(g, p, expect_resident=CLUSTER[p])


def test_runs_and_steps_continue_each_other():
    import torch
    from oracle import frame_update as fu
    g = mlp(5, 12)
    X, W, Bi = data.make_inputs(g), data.make_weights(g), data.make_biases(g, zero=False)
    want = fu.rollout_spec(g, "streaming", X, W, Bi)
    G = parity.make_graph(g, "streaming", "auto", 0, W, Bi)
    assert G.info["resident_cluster"] == CLUSTER["streaming"]
    x = parity.to_device(g, X[0])
    G.reset([x[0]])
    out = torch.empty((4, 5, 7), dtype=torch.float32, device="cuda:0")
    G.run([x[1:5]], out)                              # resident: frames 1..4
    assert G.frame() == 4
    for t in (5, 6):                                   # launch path continues from the states the kernel left
        G.step([x[t]])
    G.run([x[7:11]], out)                              # resident again: frames 7..10
    G.step([x[11]])
    G.run([x[12:13]], out[:1])
    G.sync_status()
    assert G.frame() == 12
    o = G.output_node
    assert parity.rel_err(out[:1].cpu().numpy().reshape(want[o][12:13].shape), want[o][12:13]) <= 1e-4
    for v in range(len(g.nodes)):
        assert parity.rel_err(G.get_state(v).cpu().numpy(), want[v][12]) <= 1e-4, g.nodes[v].name


def test_results_are_reproducible_bit_for_bit():
    g = graphs.build("c1")
    X, W, Bi = data.make_inputs(g), data.make_weights(g), data.make_biases(g)
    outs = []
    for _ in range(2):
        G = parity.make_graph(g, "streaming", "auto", 0, W, Bi)
        outs.append(G.rollout([parity.to_device(g, X[0])]).cpu().numpy())
    assert np.array_equal(outs[0], outs[1])
