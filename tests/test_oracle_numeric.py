"""Pins for the numeric half of the oracle (oracle/frame_update.c): hand-computed
values, reductions to library routines, and invariants the paper states."""
import os
from types import SimpleNamespace as NS

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import frame_update as fu
from oracle import rollout_theory as rt
from workloads import data, graphs, rng

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
CONV, DENSE, GAP = 0, 1, 2


def node(h, w, c, act=1):
    return NS(h=h, w=w, c=c, act=act)


def edge(src, tgt, kind=CONV, k=3, stride=1, pool=0):
    return NS(src=src, tgt=tgt, kind=kind, k=k, stride=stride, pool=pool)


def randn(stream, shape):
    return rng.normal(4242, stream, int(np.prod(shape))).reshape(shape)


def one_edge(src_shape, tgt_shape, e, x, w, bias=None, act=0):
    """State of a target fed by a single within-frame edge, frame 1."""
    nodes = [node(*src_shape, act=0), node(*tgt_shape, act=act)]
    b = [np.zeros(src_shape[2]), np.zeros(tgt_shape[2]) if bias is None else bias]
    xs = np.stack([x, x])                                   # frames 0 and 1
    s = fu.rollout(nodes, [e], [0], x.shape[0], 1, {0: xs}, [w], b)
    return s[1][1]


def test_worked_example_matches_hand_computed_values():
    g = graphs.worked_example()
    x = np.array([1, 2, 0, 3, 1], dtype=np.float64).reshape(5, 1, 1, 1, 1)
    w = [np.array(v, dtype=np.float64).reshape(1, 1, 1, 1) for v in (1, 0.5, 2, -1)]
    b = [np.zeros(1), np.array([-0.5]), np.array([0.25])]
    rows = [l.split() for l in open(os.path.join(GOLDEN, "worked_example.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for row in rows:
        R = [int(v) for v in row[1:5]]
        vals = [float(v) for v in row[5:]]
        assert R == g.patterns[row[0]]
        s = fu.rollout(g.nodes, g.edges, R, 1, 4, {0: x}, w, b)
        got = []
        for t in range(1, 5):
            got += [s[1][t, 0, 0, 0, 0], s[2][t, 0, 0, 0, 0]]
        assert got == vals, (row[0], got, vals)
        assert s[1][0, 0, 0, 0, 0] == 0 and s[2][0, 0, 0, 0, 0] == 0        # zero initial state


def test_dense_edge_is_a_matrix_product():
    x = randn(1, (3, 2, 5, 4))                                # h != w, c_in != c_out
    w = randn(2, (7, 2, 5, 4))
    got = one_edge((2, 5, 4), (1, 1, 7), edge(0, 1, DENSE), x, w)
    want = x.reshape(3, -1) @ w.reshape(7, -1).T
    np.testing.assert_allclose(got.reshape(3, 7), want, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("k,stride,h,w", [(3, 1, 6, 9), (3, 2, 8, 12), (3, 4, 8, 16), (1, 1, 5, 7), (1, 2, 6, 8),
                                           (5, 1, 7, 6), (7, 4, 28, 28), (3, 8, 16, 16)])
def test_conv_edge_matches_library_convolution(k, stride, h, w):
    cin, cout, b = 3, 5, 2
    x = randn(10 + k, (b, h, w, cin))
    wt = randn(20 + k, (cout, k, k, cin))
    bias = randn(30, (cout,))
    p = (k - 1) // 2
    oh, ow = (h + 2 * p - k) // stride + 1, (w + 2 * p - k) // stride + 1
    got = one_edge((h, w, cin), (oh, ow, cout), edge(0, 1, CONV, k, stride), x, wt, bias=bias, act=1)
    ref = F.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2), torch.from_numpy(wt).permute(0, 3, 1, 2),
                   bias=torch.from_numpy(bias), stride=stride, padding=p)
    ref = torch.relu(ref).permute(0, 2, 3, 1).numpy()
    assert got.shape == ref.shape
    np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-11)


def test_paper_shape_arithmetic():
    # 28 -> 7 with receptive field 7 stride 4; 32 -> 32 with 5; 16 -> 4 with 3 stride 4 (paper Sec. A)
    for (n, k, s, out) in [(28, 7, 4, 7), (32, 5, 1, 32), (16, 3, 4, 4), (32, 3, 2, 16)]:
        assert (n + 2 * ((k - 1) // 2) - k) // s + 1 == out == n // s


def test_pointwise_conv_is_per_pixel_dense():
    x = randn(40, (2, 4, 5, 6))
    w = randn(41, (3, 1, 1, 6))
    got = one_edge((4, 5, 6), (4, 5, 3), edge(0, 1, CONV, 1, 1), x, w)
    want = np.einsum("bhwc,oc->bhwo", x, w[:, 0, 0, :])
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)


def test_strided_conv_is_subsampled_unit_stride_conv():
    x = randn(50, (1, 8, 12, 3))
    w = randn(51, (4, 3, 3, 3))
    full = one_edge((8, 12, 3), (8, 12, 4), edge(0, 1, CONV, 3, 1), x, w)
    for s in (2, 4):
        sub = one_edge((8, 12, 3), (8 // s, 12 // s, 4), edge(0, 1, CONV, 3, s), x, w)
        np.testing.assert_allclose(sub, full[:, ::s, ::s, :], rtol=1e-12, atol=1e-12)


def test_sum_over_in_edges_equals_one_conv_over_concatenation():
    # paper Sec. A: summing the outputs of several connections = one convolution on the concatenated inputs
    xa, xb = randn(60, (2, 6, 6, 3)), randn(61, (2, 6, 6, 5))
    wa, wb = randn(62, (4, 3, 3, 3)), randn(63, (4, 3, 3, 5))
    nodes = [node(6, 6, 3, 0), node(6, 6, 5, 0), node(6, 6, 4, 1)]
    bias = [np.zeros(3), np.zeros(5), randn(64, (4,))]
    s = fu.rollout(nodes, [edge(0, 2), edge(1, 2)], [0, 0], 2, 1,
                   {0: np.stack([xa, xa]), 1: np.stack([xb, xb])}, [wa, wb], bias)
    cat = one_edge((6, 6, 8), (6, 6, 4), edge(0, 1), np.concatenate([xa, xb], -1),
                   np.concatenate([wa, wb], -1), bias=bias[2], act=1)
    np.testing.assert_allclose(s[2][1], cat, rtol=1e-12, atol=1e-12)


def test_pooled_edge_equals_4x4_stride2_conv_with_box_filtered_weights():
    x = randn(70, (2, 8, 12, 3))
    w = randn(71, (4, 3, 3, 3))
    got = one_edge((8, 12, 3), (4, 6, 4), edge(0, 1, CONV, 3, 1, pool=2), x, w)
    # library route 1: conv then average pooling
    xt, wt = torch.from_numpy(x).permute(0, 3, 1, 2), torch.from_numpy(w).permute(0, 3, 1, 2)
    ref = F.avg_pool2d(F.conv2d(xt, wt, padding=1), 2).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-11)
    # route 2: a single 4x4 stride-2 pad-1 convolution whose kernel is the 3x3 one box-filtered by 2x2
    w4 = np.zeros((4, 4, 4, 3))
    for dy in (0, 1):
        for dx in (0, 1):
            w4[:, dy:dy + 3, dx:dx + 3, :] += 0.25 * w
    ref2 = F.conv2d(xt, torch.from_numpy(w4).permute(0, 3, 1, 2), stride=2, padding=1).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(got, ref2, rtol=1e-11, atol=1e-11)


def test_mean_dense_edge_equals_dense_with_replicated_scaled_weights():
    x = randn(80, (3, 4, 5, 6))
    w = randn(81, (7, 6))
    got = one_edge((4, 5, 6), (1, 1, 7), edge(0, 1, GAP), x, w)
    wrep = np.broadcast_to(w[:, None, None, :] / 20.0, (7, 4, 5, 6)).copy()
    want = one_edge((4, 5, 6), (1, 1, 7), edge(0, 1, DENSE), x, wrep)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(got.reshape(3, 7), x.mean(axis=(1, 2)) @ w.T, rtol=1e-12, atol=1e-12)


def test_relu_and_identity_and_bias_per_channel():
    x = randn(90, (2, 1, 1, 4))
    w = randn(91, (3, 1, 1, 4))
    b = np.array([10.0, -10.0, 0.5])
    lin = x.reshape(2, 4) @ w.reshape(3, 4).T + b
    got_id = one_edge((1, 1, 4), (1, 1, 3), edge(0, 1, DENSE), x, w, bias=b, act=0).reshape(2, 3)
    got_relu = one_edge((1, 1, 4), (1, 1, 3), edge(0, 1, DENSE), x, w, bias=b, act=1).reshape(2, 3)
    np.testing.assert_allclose(got_id, lin, rtol=1e-12)
    np.testing.assert_allclose(got_relu, np.maximum(lin, 0), rtol=1e-12)
    assert (got_id[:, 1] < 0).all() and (got_relu[:, 1] == 0).all()


def test_streaming_equals_sequential_on_skip_free_chain_with_constant_input():
    # paper Sec. 4: without skip or recurrent connections both rollouts are the same function;
    # with a constant input the streaming output from frame L on equals the sequential one, bit for bit
    L = 4
    g = graphs.ff_chain(L, width=6, batch=3, frames=10)
    W, B = data.make_weights(g), data.make_biases(g, zero=False)
    x0 = randn(100, (1, 3, 1, 1, 6))
    X = {0: np.repeat(x0, 11, axis=0)}
    s_str = fu.rollout_spec(g, "streaming", X, W, B)
    s_seq = fu.rollout_spec(g, "sequential", X, W, B)
    for t in range(1, 11):
        same = np.array_equal(s_str[L][t], s_seq[L][t])
        assert same == (t >= L), t
    assert np.abs(s_seq[L][1]).max() > 0
    # and with a changing input the streaming output at frame t is the sequential output for input frame t-L
    X2 = {0: randn(101, (11, 3, 1, 1, 6))}
    a = fu.rollout_spec(g, "streaming", X2, W, B)
    b = fu.rollout_spec(g, "sequential", X2, W, B)
    for t in range(L + 1, 11):
        assert np.array_equal(a[L][t], b[L][t - L])
        assert not np.array_equal(a[L][t], b[L][t])


def test_numeric_dependence_on_input_frames_matches_theory():
    g = graphs.mnist_net("S", batch=1, frames=5)
    es = [(e.src, e.tgt) for e in g.edges]
    W, B = data.make_weights(g), data.make_biases(g, zero=False)
    X = {0: np.abs(randn(110, (6, 1, 28, 28, 1)))}
    out = g.index("O")
    for pattern in ("streaming", "sequential"):
        base = fu.rollout_spec(g, pattern, X, W, B)[out][5]
        deps = []
        for f in range(6):
            X2 = {0: X[0].copy()}
            X2[0][f] += 1.0
            if not np.array_equal(fu.rollout_spec(g, pattern, X2, W, B)[out][5], base):
                deps.append(f)
        assert deps == rt.depends_on_input_frames(len(g.nodes), es, g.patterns[pattern], out, 5)


def test_resume_from_saved_states():
    # chaining windows (Sec. 4): the last frame of a window is frame 0 of the next, so 6 frames in one go equal 3 frames,
    # then 3 more frames started from the saved frame-3 states and fed input frames 3..6 - bit for bit, for a net with
    # recurrence and a skip, under both rollouts; and the restart really uses the saved states (zeros give other values)
    g = graphs.mnist_net("SR", batch=2, frames=6)
    W, B = data.make_weights(g), data.make_biases(g, zero=False)
    X = {0: np.abs(randn(120, (7, 2, 28, 28, 1)))}
    for pattern in ("streaming", "sequential"):
        full = fu.rollout_spec(g, pattern, X, W, B)
        first = fu.rollout_spec(g, pattern, {0: X[0][:4]}, W, B, frames=3)
        saved = {v: first[v][3] for v in range(1, len(g.nodes))}
        second = fu.rollout_spec(g, pattern, {0: X[0][3:]}, W, B, frames=3, initial_states=saved)
        cold = fu.rollout_spec(g, pattern, {0: X[0][3:]}, W, B, frames=3)
        for v in range(len(g.nodes)):
            assert np.array_equal(first[v][:4], full[v][:4])
            assert np.array_equal(second[v], full[v][3:])
        assert not np.array_equal(cold[3][1], full[3][4])


def test_edges_that_bridge_several_frames_equal_chains_of_copy_nodes():
    # Sec. 6: R(e) > 1 is covered by the theory through copy-nodes.  An edge with R(e) = d evaluated directly
    # (x_u of d frames earlier, nothing before frame 0) gives, bit for bit, what the chain u -> c_1 -> ... -> c_{d-1} -> v
    # of one-frame edges with identity copies gives; and the delay really shifts the response (a hand-checked case).
    g = graphs.mnist_net("SR", batch=2, frames=7)
    W, B = data.make_weights(g), data.make_biases(g, zero=False)
    X = {0: np.abs(randn(121, (8, 2, 28, 28, 1)))}
    delays = list(g.patterns["streaming"])
    skip = [i for i, e in enumerate(g.edges) if (e.src, e.tgt) == (1, 3)][0]          # H1 -> O
    rec = [i for i, e in enumerate(g.edges) if e.src == e.tgt][0]                    # H1 -> H1
    delays[skip], delays[rec] = 3, 2
    g.patterns["delayed"] = delays
    direct = fu.rollout_spec(g, "delayed", X, W, B)
    ex, ident = graphs.with_copy_nodes(g, delays)
    assert set(ex.patterns["p"]) <= {0, 1} and len(ex.nodes) == len(g.nodes) + 3 and len(ex.edges) == len(g.edges) + 3
    assert rt.is_valid(len(ex.nodes), [(e.src, e.tgt) for e in ex.edges], ex.patterns["p"])
    W_ex = list(W) + [np.eye(c).reshape(c, 1, 1, c) for c in ident]
    B_ex = list(B) + [np.zeros(n.c) for n in ex.nodes[len(g.nodes):]]
    chain = fu.rollout_spec(ex, "p", X, W_ex, B_ex)
    for v in range(len(g.nodes)):
        assert np.array_equal(direct[v], chain[v]), g.nodes[v].name
    assert not np.array_equal(direct[len(g.nodes) - 1], fu.rollout_spec(g, "streaming", X, W, B)[len(g.nodes) - 1])
    # hand-checked: in -> out, a dense identity edge that bridges 3 frames: out^t = in^(t-3), zero before
    nodes = [node(1, 1, 2, 0), node(1, 1, 2, 0)]
    x = np.arange(12, dtype=np.float64).reshape(6, 1, 1, 1, 2) + 1.0
    s = fu.rollout(nodes, [edge(0, 1, DENSE)], [3], 1, 5, {0: x}, [np.eye(2).reshape(2, 1, 1, 2)], [np.zeros(2), np.zeros(2)])
    assert s[1].reshape(6, 2).tolist() == [[0, 0], [0, 0], [0, 0], [1, 2], [3, 4], [5, 6]]


def test_bf16_rounding_switch():
    v = np.array([1.0, 1.00390625, 1.005859375, 1.0078125, -3.14159], dtype=np.float32)
    want = rng.round_to_bf16(v)
    assert want.tolist()[:4] == [1.0, 1.0, 1.0078125, 1.0078125]        # ties to even, then above the tie
    nodes = [node(1, 1, 5, 0), node(1, 1, 5, 0)]
    w = np.eye(5).reshape(5, 1, 1, 5)
    x = np.stack([v, v]).reshape(2, 1, 1, 1, 5).astype(np.float64)
    s = fu.rollout(nodes, [edge(0, 1, DENSE)], [0], 1, 1, {0: x}, [w], [np.zeros(5), np.zeros(5)],
                   round_states_bf16=True)
    assert s[1][1].reshape(5).tolist() == want.astype(np.float64).tolist()
    assert torch.tensor(v).to(torch.bfloat16).float().tolist() == want.tolist()


def test_generated_workloads_stay_in_range():
    # the weight scale keeps states finite and of order one over many frames of a recurrent graph
    g = graphs.build("c2", batch=2, frames=32)
    s = fu.rollout_spec(g, "streaming", data.make_inputs(g), data.make_weights(g), data.make_biases(g))
    for v in range(1, len(g.nodes)):
        m = np.abs(s[v][-1]).max()
        assert 1e-3 < m < 1e3, (v, m)
    g5 = graphs.build("c5", batch=1, frames=24, size=16)
    s5 = fu.rollout_spec(g5, "streaming", data.make_inputs(g5), data.make_weights(g5), data.make_biases(g5))
    for v in range(1, len(g5.nodes)):
        m = np.abs(s5[v][-1]).max()
        assert 1e-3 < m < 1e3, (v, m)
