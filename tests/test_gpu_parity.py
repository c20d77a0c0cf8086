"""GPU parity: the CUDA library, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Tolerances: max-abs-diff relative to each node's output scale, 2e-2 for bfloat16
states, 1e-4 for fp32; the dyadic worked example must match exactly."""
import numpy as np
import pytest

from tests import parity
from workloads import data, graphs

pytestmark = pytest.mark.gpu


def test_worked_example_exact():
    import torch
    from paper_1806_04965_b200 import Graph
    g = graphs.worked_example()
    x = torch.tensor([1, 2, 0, 3, 1], dtype=torch.float32, device="cuda:0").reshape(5, 1, 1, 1, 1)
    w = [np.array(v, dtype=np.float32).reshape(1, 1, 1, 1) for v in (1, 0.5, 2, -1)]
    b = [np.zeros(1, np.float32), np.array([-0.5], np.float32), np.array([0.25], np.float32)]
    want = {"streaming": [(0.5, 0), (1.75, 0), (0.375, 3.75), (2.6875, 0)],
            "sequential": [(1.5, 1.25), (0.25, 0.75), (2.625, 2.5), (1.8125, 2.875)],
            "hybrid": [(1.5, 0), (0.25, 3.25), (2.625, 0), (1.8125, 4.5)]}
    for dtype in ("fp32", "bf16"):
        for p, R in g.patterns.items():
            G = Graph(g.nodes, g.edges, R, batch=1, dtype=dtype)
            G.set_weights(w, b)
            xs = x if dtype == "fp32" else x.to(torch.bfloat16)
            G.reset([xs[0]])
            got = []
            for t in range(1, 5):
                G.step([xs[t]])
                got.append((float(G.get_state(1).float().item()), float(G.get_state(2).float().item())))
            assert got == [(float(a), float(c)) for (a, c) in want[p]], (dtype, p, got)


@pytest.mark.parametrize("pattern", ["streaming", "sequential"])
def test_c1_mlp_full_size(pattern):
    parity.check_stepwise(graphs.build("c1"), pattern)
    parity.check_run(graphs.build("c1"), pattern)
    parity.check_run(graphs.build("c1"), pattern, graph_frames=4)


@pytest.mark.parametrize("kind", ["FF", "S", "SR"])
def test_paper_mnist_networks_fp32(kind):
    g = graphs.mnist_net(kind, batch=3, frames=5)
    for p in g.patterns:
        parity.check_stepwise(g, p, zero_bias=False)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("name,kw", [
    ("c2", dict(batch=3, frames=6)),
    ("c3", dict(batch=2, frames=4, size=16)),
    ("c4", dict(batch=2, frames=4, size=16)),
    ("c5", dict(batch=2, frames=4, size=16)),
])
def test_configs_reduced_direct_engine(name, kw, dtype):
    g = graphs.build(name, dtype=dtype, **kw)
    for p in g.patterns:
        parity.check_stepwise(g, p, engine="direct", zero_bias=False)


def test_run_equals_steps_and_resume():
    import torch
    g = graphs.build("c2", batch=4, frames=8, dtype="fp32")
    X, W, Bi = data.make_inputs(g), data.make_weights(g), data.make_biases(g, zero=False)
    A = parity.make_graph(g, "streaming", "direct", 0, W, Bi)
    Bg = parity.make_graph(g, "streaming", "direct", 3, W, Bi)
    x = parity.to_device(g, X[0])
    oa = A.rollout([x])
    ob = Bg.rollout([x])                     # CUDA graphs of 3 frames + 2 plain frames
    assert torch.equal(oa, ob)
    # resume: run 4 frames, move every state into a fresh graph, run the other 4
    C = parity.make_graph(g, "streaming", "direct", 0, W, Bi)
    C.reset([x[0]])
    C.run([x[1:5]])
    D = parity.make_graph(g, "streaming", "direct", 0, W, Bi)
    D.reset([x[4]])
    for v in range(len(g.nodes)):
        D.set_state(v, C.get_state(v))
    od = torch.empty((4, g.batch, 10), dtype=torch.float32, device="cuda:0")
    D.run([x[5:9]], od)
    assert torch.equal(od, oa[4:])
    assert A.launch_count() > 0


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_spatial_output_node_fills_a_full_frame(dtype):
    # the output node is an image: `out` holds [B][H][W][C] floats per frame, and consecutive frames of a run do not overlap
    import torch
    g = graphs.build("sink", dtype=dtype)
    for p in g.patterns:
        parity.check_stepwise(g, p, zero_bias=False)
        parity.check_run(g, p)
    from paper_1806_04965_b200 import Graph
    G = Graph(g.nodes, g.edges, g.patterns["streaming"], batch=g.batch, dtype=dtype)
    assert G.out_shape() == (g.batch, 4, 4, 8)
    G.set_weights(data.make_weights(g), data.make_biases(g, zero=False))
    X = data.make_inputs(g)
    # guard words behind the output buffer stay untouched
    buf = torch.full((g.frames * g.batch * 4 * 4 * 8 + 64,), 7.0, dtype=torch.float32, device="cuda:0")
    out = buf[:g.frames * g.batch * 4 * 4 * 8].view(g.frames, g.batch, 4, 4, 8)
    x = parity.to_device(g, X[0])
    G.reset([x[0]])
    G.run([x[1:]], out)
    G.sync_status()
    assert bool((buf[-64:] == 7.0).all())
    assert float(out.abs().max()) > 0


def test_expired_device_wait_is_reported_and_cleared_by_reset():
    # host-side hook only: with a wait limit of zero every tensor-core launch reports the expiry at its entry and
    # returns before it touches a barrier, a copy or an MMA; nothing on the GPU actually waits
    from paper_1806_04965_b200 import SrError
    g = graphs.build("c3", batch=2, frames=3, size=16)
    X, W, Bi = data.make_inputs(g), data.make_weights(g), data.make_biases(g)
    G = parity.make_graph(g, "streaming", "auto", 0, W, Bi, wait_limit_ms=0)
    assert G.info["n_tensor_core_nodes"] > 0 and G.info["resident_cluster"] == 0
    x = parity.to_device(g, X[0])
    G.rollout([x])
    for _ in range(2):                                  # the error stays recorded until the rollout starts over
        with pytest.raises(SrError) as e:
            G.sync_status()
        assert e.value.status == "SR_ERR_TIMEOUT"
    G.set_option(10, 1000)
    want = fu_rollout(g, X, W, Bi)
    out = G.rollout([x])                                # reset clears the error word
    G.sync_status()
    o = G.output_node
    assert parity.rel_err(out.cpu().numpy().reshape(want[o][1:].shape), want[o][1:]) <= parity.TOL["bf16"]
    parity.check_run(g, "streaming")                    # and a fresh graph is unaffected


def fu_rollout(g, X, W, Bi):
    from oracle import frame_update as fu
    return fu.rollout_spec(g, "streaming", X, W, Bi)


@pytest.mark.parametrize("name,kw,W", [("c4ff", dict(batch=3, frames=9, size=16), 4), ("dsr2", dict(batch=2, frames=7, h1_recurrence=False), 3),
                                        ("mini_ff", dict(), 5)])
def test_deep_window_equals_chained_windows(name, kw, W):
    # a network without recurrence under the sequential rollout: the W frames of a window do not depend on each other and
    # are evaluated at once (one launch group per level over W * B samples); results equal W single steps, the graph
    # stands at frame t + W afterwards and can be stepped on (two windows, then single steps to the end)
    import torch
    from workloads.graphs import CONV, GAP_DENSE, IDENTITY, Edge, GraphSpec, Node, sequential_pattern, streaming_pattern
    if name == "mini_ff":
        # a streaming input edge (reads the previous input frame) beside within-frame edges
        nodes = [Node("in", 16, 16, 3, IDENTITY), Node("a", 16, 16, 32), Node("b", 8, 8, 64), Node("o", 1, 1, 5, IDENTITY)]
        edges = [Edge(0, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 2), Edge(0, 2, CONV, 1, 2), Edge(2, 3, GAP_DENSE)]
        g = GraphSpec("mini_ff", nodes, edges, batch=3, frames=12, dtype="bf16", seed=77)
        g.patterns = {"sequential": [0, 0, 1, 0]}
    elif name == "dsr2":
        g = graphs.dsr(2, **kw)
    else:
        g = graphs.build(name, **kw)
    from oracle import frame_update as fu
    X, Wt, Bi = data.make_inputs(g), data.make_weights(g), data.make_biases(g, zero=False)
    want = fu.rollout_spec(g, "sequential", X, Wt, Bi)
    G = parity.make_graph(g, "sequential", "auto", 0, Wt, Bi)
    G.bind_window(W)
    x = {v: parity.to_device(g, X[v]) for v in G.input_nodes}
    G.reset([x[v][0] for v in G.input_nodes])
    o, tol = G.output_node, parity.TOL[g.dtype]
    t = 0
    for _ in range(2):
        out = torch.empty((W,) + G.out_shape(), dtype=torch.float32, device="cuda:0")
        G.rollout_window([x[v][t + 1:t + 1 + W] for v in G.input_nodes], out)
        assert G.frame() == t + W
        assert parity.rel_err(out.cpu().numpy().reshape(want[o][t + 1:t + 1 + W].shape), want[o][t + 1:t + 1 + W]) <= tol
        t += W
        for v in range(len(g.nodes)):
            assert parity.rel_err(G.get_state(v).float().cpu().numpy(), want[v][t]) <= tol, (g.nodes[v].name, t)
    while t < g.frames:
        G.step([x[v][t + 1] for v in G.input_nodes])
        t += 1
        for v in range(len(g.nodes)):
            assert parity.rel_err(G.get_state(v).float().cpu().numpy(), want[v][t]) <= tol, (g.nodes[v].name, t)
    G.sync_status()


def test_deep_window_refuses_patterns_with_recurrence():
    from paper_1806_04965_b200 import SrError
    g = graphs.build("c2", batch=2, frames=3)
    G = parity.make_graph(g, "streaming", "auto", 0, data.make_weights(g), data.make_biases(g))
    with pytest.raises(SrError) as e:
        G.bind_window(4)
    assert e.value.status == "SR_ERR_UNSUPPORTED"


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_edges_that_bridge_several_frames_run_as_chains_of_copy_nodes(dtype):
    # Sec. 6: R(e) > 1 is covered through copy-nodes.  The library takes patterns with values in {0, 1}; the expanded
    # graph (identity 1x1 copies, one frame per link) must reproduce the oracle's direct evaluation of the delays, on the
    # tensor cores (64-channel nodes, bf16) as on the CUDA cores (fp32).
    from oracle import frame_update as fu
    from workloads.graphs import CONV, GAP_DENSE, IDENTITY, Edge, GraphSpec, Node
    g = GraphSpec("delays", [Node("in", 16, 16, 3, IDENTITY), Node("a", 16, 16, 64), Node("b", 8, 8, 64), Node("o", 1, 1, 5, IDENTITY)],
                  [Edge(0, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 2), Edge(2, 2, CONV, 3, 1), Edge(1, 1, CONV, 3, 1), Edge(0, 2, CONV, 1, 2),
                   Edge(2, 3, GAP_DENSE)], batch=3, frames=7, dtype=dtype, seed=77)
    delays = [1, 1, 2, 3, 2, 1]                        # b's recurrence bridges 2 frames, a's 3, the skip from the input 2
    g.patterns["delayed"] = delays
    X, W, Bi = data.make_inputs(g), data.make_weights(g), data.make_biases(g, zero=False)
    want = fu.rollout_spec(g, "delayed", X, W, Bi)
    ex, ident = graphs.with_copy_nodes(g, delays)
    assert len(ex.nodes) == len(g.nodes) + 4
    W_ex = list(W) + [np.eye(c, dtype=np.float32).reshape(c, 1, 1, c) for c in ident]
    B_ex = list(Bi) + [np.zeros(n.c, dtype=np.float32) for n in ex.nodes[len(g.nodes):]]
    G = parity.make_graph(ex, "p", "auto", 0, W_ex, B_ex)
    if dtype == "bf16":
        assert G.info["n_tensor_core_nodes"] >= 2, G.info
    out = G.rollout([parity.to_device(ex, X[0])])
    G.sync_status()
    o = G.output_node
    assert o == 3
    tol = parity.TOL[dtype]
    assert parity.rel_err(out.cpu().numpy().reshape(want[o][1:].shape), want[o][1:]) <= tol
    for v in range(len(g.nodes)):
        assert parity.rel_err(G.get_state(v).float().cpu().numpy(), want[v][g.frames]) <= tol, g.nodes[v].name
