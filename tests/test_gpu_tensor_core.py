"""GPU parity of the tcgen05 implicit-GEMM engine against the oracle: single edges of every kind the
engine lowers (taps, strides, channel-block widths, staged few-channel inputs, pooled edges, several
incoming edges), ragged tiles, and the reduced benchmark graphs with the engine chosen automatically."""
import pytest

from tests import parity
from workloads.graphs import CONV, GAP_DENSE, IDENTITY, RELU, Edge, GraphSpec, Node, check_shapes, build

pytestmark = pytest.mark.gpu


def tiny(name, nodes, edges, batch=3, frames=3, R=None):
    g = GraphSpec(name, nodes, edges, batch=batch, frames=frames, dtype="bf16", seed=4321)
    g.patterns = {"p": R or [1] * len(edges)}
    check_shapes(g)
    return g


def run(g):
    # single tiles (work items from the shared list, then from per-CTA lists), then pairs of tiles that share every
    # weight box
    from paper_1806_04965_b200 import Graph
    G = Graph(g.nodes, g.edges, g.patterns["p"], batch=g.batch, dtype="bf16")
    assert G.info["n_tensor_core_nodes"] >= 1, G.info
    parity.check_stepwise(g, "p", zero_bias=False, tc_pair=1)
    parity.check_stepwise(g, "p", zero_bias=False, tc_lists=1)      # a work list per CTA instead of the shared list
    return parity.check_stepwise(g, "p", zero_bias=False, tc_pair=2)


@pytest.mark.parametrize("cin,cout,k,stride,size", [
    (64, 64, 3, 1, 16), (64, 128, 3, 2, 16), (128, 256, 3, 4, 16), (64, 64, 1, 1, 16), (64, 128, 1, 2, 16),
    (32, 64, 3, 1, 16), (16, 32, 3, 1, 16), (48, 64, 3, 1, 8), (128, 128, 3, 8, 32), (64, 32, 3, 1, 28),
    (32, 64, 3, 2, 14), (32, 64, 3, 4, 28), (256, 256, 3, 1, 8), (64, 96, 3, 1, 7),
])
def test_single_conv_edge(cin, cout, k, stride, size):
    out = size // stride
    for R in ([0], [1]):
        g = tiny("edge", [Node("in", size, size, cin, IDENTITY), Node("n", out, out, cout, RELU), Node("o", 1, 1, 4, IDENTITY)],
                 [Edge(0, 1, CONV, k, stride), Edge(1, 2, GAP_DENSE)], R=R + [1])
        run(g)


def test_few_channel_input_edges_are_staged():
    for cin, k in ((3, 3), (1, 3), (3, 1)):
        g = tiny("stem", [Node("in", 16, 16, cin, IDENTITY), Node("a", 16, 16, 64), Node("b", 16, 16, 64),
                          Node("o", 1, 1, 4, IDENTITY)],
                 [Edge(0, 1, CONV, k, 1), Edge(1, 2, CONV, 3, 1), Edge(0, 2, CONV, k, 1), Edge(1, 1, CONV, 3, 1),
                  Edge(2, 3, GAP_DENSE)], frames=4, R=[1, 1, 0, 1, 0])
        run(g)
        # the staged edge's activation box in an activation slot (0) / in the weight ring behind its weights (2)
        for stem_ring in (0, 2):
            parity.check_stepwise(g, "p", zero_bias=False, stem_ring=stem_ring)


def test_a_node_fed_by_a_staged_edge_only():
    # every K-block of node a travels in the weight ring: the activation ring stays empty for its tiles
    g = tiny("stem_only", [Node("in", 32, 32, 3, IDENTITY), Node("a", 32, 32, 64), Node("b", 32, 32, 128), Node("o", 1, 1, 4, IDENTITY)],
             [Edge(0, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 1), Edge(2, 3, GAP_DENSE)], batch=5, frames=4)
    for stem_ring in (0, 1, 2):
        parity.check_stepwise(g, "p", zero_bias=False, stem_ring=stem_ring)


@pytest.mark.parametrize("c,act_b", [(64, RELU), (32, IDENTITY)])
def test_two_narrow_nodes_that_share_a_source_run_as_one_plan(c, act_b):
    # a <- {in (staged), a}, b <- {a, b, in (1x1, staged)}, d <- {a, b}: a and b have the same shape, at most 64 channels
    # and both read a through a 3x3 filter from the previous frame, so b's weights take rows 64..127 of a's tiles
    g = tiny("fused", [Node("in", 24, 16, 3, IDENTITY), Node("a", 24, 16, c), Node("b", 24, 16, c, act_b), Node("d", 12, 8, 128),
                       Node("o", 1, 1, 4, IDENTITY)],
             [Edge(0, 1, CONV, 3, 1), Edge(1, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 1), Edge(2, 2, CONV, 3, 1), Edge(0, 2, CONV, 1, 1),
              Edge(1, 3, CONV, 3, 2), Edge(2, 3, CONV, 1, 2), Edge(3, 4, GAP_DENSE)], batch=5, frames=4)
    for fuse in (1, 0):
        parity.check_stepwise(g, "p", zero_bias=False, tc_fuse=fuse)
    parity.check_stepwise(g, "p", zero_bias=False, tc_fuse=1, tc_lists=1, stem_ring=2)
    # with a -> b inside the frame (R = 0) the two nodes are in different launch groups: nothing to fuse, same results
    g.patterns["q"] = [1, 1, 0, 1, 1, 1, 1, 1]
    parity.check_stepwise(g, "q", zero_bias=False)


def test_pooled_edge_and_recurrence():
    g = tiny("pool", [Node("in", 16, 16, 64, IDENTITY), Node("a", 8, 8, 128), Node("b", 8, 8, 128), Node("o", 1, 1, 4, IDENTITY)],
             [Edge(0, 1, CONV, 3, 1, 2), Edge(1, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 1), Edge(0, 2, CONV, 3, 2),
              Edge(2, 3, GAP_DENSE)], frames=4)
    run(g)


def test_rectangular_images_and_odd_batch():
    g = tiny("rect", [Node("in", 12, 20, 64, IDENTITY), Node("a", 12, 20, 64), Node("b", 6, 10, 64),
                      Node("o", 1, 1, 5, IDENTITY)],
             [Edge(0, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 2), Edge(2, 2, CONV, 3, 1), Edge(2, 3, GAP_DENSE)],
             batch=5, frames=4)
    run(g)


@pytest.mark.parametrize("name,kw", [
    ("c2", dict(batch=3, frames=6)),
    ("c3", dict(batch=2, frames=4, size=16)),
    ("c3", dict(batch=5, frames=3, size=32)),
    ("c4", dict(batch=2, frames=4, size=16)),
    ("c5", dict(batch=2, frames=4, size=16)),
])
def test_configs_reduced_tensor_cores(name, kw):
    g = build(name, **kw)
    for p in g.patterns:
        parity.check_stepwise(g, p, engine="auto", zero_bias=False)
        parity.check_stepwise(g, p, engine="auto", zero_bias=False, tc_pair=2)
        parity.check_run(g, p, engine="auto", graph_frames=2)
        parity.check_run(g, p, engine="auto", graph_frames=2, tc_pair=2, resident=False)


@pytest.mark.parametrize("batch", [1, 2, 7])
def test_pairs_with_ragged_batches_and_widths(batch):
    # lane 1 of the last pair falls outside the batch (sample pairs) or outside the image (column pairs)
    g = tiny("ragged", [Node("in", 20, 20, 64, IDENTITY), Node("a", 20, 20, 128), Node("b", 10, 10, 128), Node("c", 5, 5, 256),
                        Node("o", 1, 1, 4, IDENTITY)],
             [Edge(0, 1, CONV, 3, 1), Edge(1, 1, CONV, 3, 1), Edge(1, 2, CONV, 3, 2), Edge(2, 2, CONV, 3, 1), Edge(2, 3, CONV, 3, 2),
              Edge(0, 3, CONV, 1, 4), Edge(3, 4, GAP_DENSE)], batch=batch, frames=3)
    run(g)


@pytest.mark.parametrize("k", [0, 2, 6])
def test_paper_cifar10_networks_on_tensor_cores(k):
    # DSR0 / DSR2 / DSR6 (Sec. A, paragraph CIFAR10): receptive field 5 on the 3-channel input (75 columns, staged as two
    # K-blocks), 32- and 64-channel blocks with dense skips, stride-4 edges into the 4 x 4 x 512 node (four channel
    # tiles); every convolutional node runs on the tensor cores, only the dense output node does not
    from paper_1806_04965_b200 import Graph
    from workloads import graphs
    g = graphs.dsr(k, batch=3, frames=4)
    G = Graph(g.nodes, g.edges, g.patterns["streaming"], batch=g.batch, dtype="bf16")
    assert G.info["n_direct_nodes"] == 1 and G.info["n_tensor_core_nodes"] == len(g.nodes) - 2, G.info
    assert G.info["first_response_step"] == 4
    S = Graph(g.nodes, g.edges, g.patterns["sequential"], batch=0)
    assert S.info["first_response_step"] == 4 + k and S.info["inference_factor"] == 4 + k
    for p in g.patterns:
        parity.check_stepwise(g, p, zero_bias=False, tc_pair=1)
        parity.check_stepwise(g, p, zero_bias=False, tc_pair=2)
        parity.check_run(g, p, graph_frames=2)


def test_gtsrb_network_variant():
    # DSR4 without the H1 recurrence and with 43 classes (Sec. A, paragraph GTSRB)
    from workloads import graphs
    g = graphs.dsr(4, batch=2, frames=3, classes=43, h1_recurrence=False)
    parity.check_stepwise(g, "streaming", zero_bias=False)
