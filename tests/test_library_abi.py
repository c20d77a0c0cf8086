"""CPU-side tests of the C-ABI library: it loads without a GPU, exports what the header declares,
and its graph compiler returns exactly the oracle's rollout-theory integers."""
import ctypes
import os
import re
from types import SimpleNamespace as NS

import pytest

from oracle import rollout_theory as rt
from paper_1806_04965_b200 import Graph, SrError, load_library
from workloads import graphs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def dense_graph(n, es):
    nodes = [NS(h=1, w=1, c=2, act=1) for _ in range(n)]
    edges = [NS(src=u, tgt=v, kind=1, k=1, stride=1, pool=0) for (u, v) in es]
    return nodes, edges


def test_library_exports_every_declared_symbol():
    lib = load_library()
    header = open(os.path.join(ROOT, "include", "sr_rollout.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(sr_[a-z_]+)\s*\(", header))
    assert {"sr_graph_create", "sr_rollout_step", "sr_rollout_run"} <= names and len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings():
    lib = load_library()
    for code in range(9):
        assert len(lib.sr_status_str(code)) > 0


def test_compiler_matches_oracle_on_all_small_networks():
    from tests.test_oracle_theory import NETS
    checked = 0
    for (n, es) in NETS:
        nodes, edges = dense_graph(n, es)
        for R in rt.all_patterns(len(es)):
            if not rt.is_valid(n, es, R):
                with pytest.raises(SrError) as ei:
                    Graph(nodes, edges, R, batch=0)
                assert ei.value.status == "SR_ERR_INVALID_ROLLOUT"
                continue
            G = Graph(nodes, edges, R, batch=0)
            lv = rt.frame_levels(n, es, R)
            assert G.levels() == lv
            assert G.info["inference_factor"] == rt.inference_factor(n, es, R) == G.info["n_groups"]
            assert G.info["n_inputs"] == len(rt.input_set(n, es))
            assert G.info["streaming_parallel"] == int(rt.equally_model_parallel(n, es, R, [1] * len(es)))
            assert (G.info["inference_factor"] == 1) == bool(G.info["streaming_parallel"])       # Theorem 1 a <=> b
            out = G.info["output_node"]
            fr = rt.first_response(n, es, R, out)
            if out in rt.input_set(n, es) or fr is None:
                assert G.info["first_response_frame"] == -1
            else:
                assert (G.info["first_response_frame"], G.info["first_response_step"]) == fr
            assert G.info["response_interval"] == rt.response_interval(n, es, R)
            checked += 1
    assert checked > 1000


def test_compiler_on_benchmark_graphs_and_paper_networks():
    specs = [graphs.build(c) for c in ("c1", "c2", "c3", "c4", "c5")] + [graphs.mnist_net(k) for k in ("FF", "S", "SR")]
    specs += [graphs.chain_with_shortcut(4 + k) for k in range(7)] + [graphs.worked_example()]
    specs += [graphs.dsr(k) for k in range(7)] + [graphs.dsr(4, classes=43, h1_recurrence=False)]
    for g in specs:
        es = [(e.src, e.tgt) for e in g.edges]
        for name, R in g.patterns.items():
            G = Graph(g.nodes, g.edges, R, batch=0)
            assert G.levels() == rt.frame_levels(len(g.nodes), es, R), (g.name, name)
            assert G.info["inference_factor"] == rt.inference_factor(len(g.nodes), es, R)
            assert (G.info["first_response_frame"], G.info["first_response_step"]) == \
                rt.first_response(len(g.nodes), es, R, G.info["output_node"]), (g.name, name)
            if name == "streaming":
                assert G.info["n_groups"] == 1
    # the paper's CIFAR10 nets themselves (Sec. 4): streaming answers after 4 update steps whatever the depth, the
    # sequential rollout after 4 + k; DSR2 has shortest path 4 and longest path 6
    for k in range(7):
        g = graphs.dsr(k)
        assert Graph(g.nodes, g.edges, g.patterns["streaming"]).info["first_response_step"] == 4
        assert Graph(g.nodes, g.edges, g.patterns["sequential"]).info["first_response_step"] == 4 + k
    sr = graphs.mnist_net("SR")
    assert Graph(sr.nodes, sr.edges, sr.patterns["sequential"]).info["inference_factor"] == 3   # paper Sec. 4
    assert Graph(sr.nodes, sr.edges, sr.patterns["streaming"]).info["inference_factor"] == 1


def test_error_codes():
    nodes, edges = dense_graph(2, [(0, 1)])
    with pytest.raises(SrError) as e:
        Graph(nodes, [], [], batch=0)
    assert e.value.status == "SR_ERR_NOT_A_NETWORK"
    with pytest.raises(SrError) as e:                       # node 2 hangs on its own loop: not input-connected
        n3, e3 = dense_graph(3, [(0, 1), (2, 2)])
        Graph(n3, e3, [1, 1], batch=0)
    assert e.value.status == "SR_ERR_NOT_A_NETWORK"
    with pytest.raises(SrError) as e:                       # self-loop inside a frame
        n2, e2 = dense_graph(2, [(0, 1), (1, 1)])
        Graph(n2, e2, [1, 0], batch=0)
    assert e.value.status == "SR_ERR_INVALID_ROLLOUT"
    with pytest.raises(SrError) as e:                       # 3x3 stride-2 conv cannot map 8x8 to 8x8
        nn = [NS(h=8, w=8, c=3, act=0), NS(h=8, w=8, c=4, act=1)]
        Graph(nn, [NS(src=0, tgt=1, kind=0, k=3, stride=2, pool=0)], [1], batch=0)
    assert e.value.status == "SR_ERR_SHAPE_MISMATCH"
    with pytest.raises(SrError) as e:
        Graph(nodes, [NS(src=0, tgt=5, kind=1, k=1, stride=1, pool=0)], [1], batch=0)
    assert e.value.status == "SR_ERR_INVALID_ARG"
    with pytest.raises(SrError) as e:
        Graph(nodes, edges, [2], batch=0)
    assert e.value.status == "SR_ERR_INVALID_ARG"


def test_theory_only_graph_refuses_device_calls():
    lib = load_library()
    nodes, edges = dense_graph(2, [(0, 1)])
    G = Graph(nodes, edges, [1], batch=0)
    n = ctypes.c_size_t()
    assert lib.sr_graph_workspace_bytes(G._h, ctypes.byref(n)) == 8            # SR_ERR_STATE
    assert lib.sr_rollout_step(G._h, None, None, None) == 8
    assert lib.sr_graph_info(None, None) == 1


def test_window_tableau_matches_the_oracle_for_every_window_size():
    # Eq. 4 for W = 1..4: the compiler's closed recursion against the oracle's iteration of the update step U on the
    # explicit window, on every valid pattern of the small networks and on the named graphs
    from tests.test_oracle_theory import NETS
    checked = 0
    cases = [(n, es, None) for (n, es) in NETS[:60]]
    for g in [graphs.worked_example(), graphs.mnist_net("SR"), graphs.dsr(2), graphs.build("c3", batch=1, frames=1)]:
        cases.append((len(g.nodes), [(e.src, e.tgt) for e in g.edges], g))
    for n, es, g in cases:
        patterns = list(g.patterns.values()) if g is not None else [R for R in rt.all_patterns(len(es)) if rt.is_valid(n, es, R)]
        for R in patterns:
            nodes, edges = (g.nodes, g.edges) if g is not None else dense_graph(n, es)
            G = Graph(nodes, edges, R, batch=0)
            for W in (1, 2, 3, 4):
                want, _ = rt.tableau_by_updates(n, es, R, W)
                got = G.window_tableau(W)
                for i in range(W + 1):
                    for v in range(n):
                        assert got[i][v] == want[(i, v)], (es, R, W, i, v)
                checked += 1
    assert checked > 300
    # frames of a recurrence-free network under the sequential rollout do not depend on each other: every frame has the
    # tableau of frame 1, so a whole window is F(R) update steps (Sec. 4, the GTSRB comparison)
    g = graphs.dsr(4, classes=43, h1_recurrence=False)
    G = Graph(g.nodes, g.edges, g.patterns["sequential"], batch=0)
    T = G.window_tableau(8)
    assert all(T[i] == T[1] for i in range(1, 9)) and max(T[8]) == G.info["inference_factor"] == 8
    S = Graph(g.nodes, g.edges, g.patterns["streaming"], batch=0)
    assert max(S.window_tableau(8)[8]) == 8 and S.window_tableau(8)[3][len(g.nodes) - 1] == 3
