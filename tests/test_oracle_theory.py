"""Pins for the theory half of the oracle: it is checked against what the paper
proves or prints, by brute force on small graphs, never against itself alone."""
import itertools
import os

import pytest

from oracle import rollout_theory as rt
from workloads import graphs, rng

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def printed():
    out = {}
    for line in open(os.path.join(GOLDEN, "printed_values.txt")):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = int(line[1])
    return out


def small_networks():
    """Every directed graph on <= 3 nodes with <= 5 edges that is a network, plus
    seeded random 4-node graphs with <= 6 edges."""
    nets = []
    for n in (2, 3):
        possible = [(u, v) for u in range(n) for v in range(n)]
        for m in range(1, 6):
            for es in itertools.combinations(possible, m):
                if rt.is_network(n, es):
                    nets.append((n, list(es)))
    possible = [(u, v) for u in range(4) for v in range(4)]
    picks = rng.bits64(123, 0, 4000)
    i, found = 0, 0
    while found < 120 and i < len(picks) - 8:
        m = 3 + int(picks[i] % 4)
        idx = sorted({int(picks[i + 1 + j] % 16) for j in range(m)})
        i += 8
        es = [possible[j] for j in idx]
        if rt.is_network(4, es):
            nets.append((4, es))
            found += 1
    return nets


NETS = small_networks()


def r0_subgraph_acyclic(n, es, R):
    sub = [e for (e, r) in zip(es, R) if r == 0]
    V = [(0, v) for v in range(n)]
    return rt._is_acyclic(V, [((0, u), (0, v)) for (u, v) in sub])


def test_enough_small_networks():
    assert len(NETS) > 200 and sum(1 for (n, _) in NETS if n == 4) >= 50
    assert any(any(u == v for (u, v) in es) for (_, es) in NETS)          # self-loops are covered


def test_input_set_and_network_definition():
    # Eq. (1) and the definition of a network
    assert rt.input_set(3, [(0, 1), (1, 2)]) == [0]
    assert rt.input_set(3, [(0, 1), (2, 1)]) == [0, 2]
    assert not rt.is_network(2, [])                                      # |E| = 0
    assert not rt.is_network(2, [(0, 1), (1, 0)])                        # no input node at all
    assert not rt.is_network(3, [(0, 1), (2, 2)])                        # node 2 only reachable from itself
    assert rt.is_network(3, [(0, 1), (1, 2), (2, 1), (1, 1)])


def test_window_definition_eq2():
    V, E = rt.rollout_window(2, [(0, 1), (1, 1)], [0, 1], 2)
    assert sorted(V) == [(i, v) for i in range(3) for v in range(2)]
    assert sorted(E) == sorted([((0, 0), (0, 1)), ((1, 0), (1, 1)), ((2, 0), (2, 1)),
                                ((0, 1), (1, 1)), ((1, 1), (2, 1))])


def test_validity_is_independent_of_W_and_equals_acyclic_R0_subgraph():
    for (n, es) in NETS:
        for R in rt.all_patterns(len(es)):
            v = [rt.is_valid(n, es, R, W) for W in (1, 2, 3)]
            assert v[0] == v[1] == v[2]
            assert v[0] == r0_subgraph_acyclic(n, es, R)


def test_streaming_always_valid_and_selfloops_force_one():
    for (n, es) in NETS:
        assert rt.is_valid(n, es, [1] * len(es))
        for R in rt.valid_patterns(n, es):
            for (e, (u, v)) in enumerate(es):
                if u == v:
                    assert R[e] == 1


def _edges_in_cycles(n, es):
    reach = [[False] * n for _ in range(n)]
    for (u, v) in es:
        reach[u][v] = True
    for k in range(n):
        for i in range(n):
            for j in range(n):
                reach[i][j] = reach[i][j] or (reach[i][k] and reach[k][j])
    return [e for (e, (u, v)) in enumerate(es) if u == v or reach[v][u]]


def _minimal_cycles(n, es):
    """All injective cycles as tuples of edge indices."""
    cycles = set()

    def walk(start, node, used_edges, used_nodes):
        for (e, (u, v)) in enumerate(es):
            if u != node or e in used_edges:
                continue
            if v == start:
                c = used_edges + [e]
                k = c.index(min(c))
                cycles.add(tuple(c[k:] + c[:k]))
            elif v not in used_nodes and v > start:
                walk(start, v, used_edges + [e], used_nodes | {v})

    for s in range(n):
        walk(s, s, [], {s})
    return [list(c) for c in cycles]


def test_lemma1_bounds():
    for (n, es) in NETS:
        count = len(rt.valid_patterns(n, es))
        n_rec = sum(1 for (u, v) in es if u == v)
        assert count <= 2 ** (len(es) - n_rec)
        n_forward = len(es) - len(_edges_in_cycles(n, es))
        assert n_forward >= 1
        assert 2 ** n_forward <= count
        cycles = _minimal_cycles(n, es)
        # every set of pairwise non-overlapping minimal cycles gives a lower bound
        for r in range(0, min(3, len(cycles)) + 1):
            for C in itertools.combinations(cycles, r):
                flat = [e for c in C for e in c]
                if len(flat) != len(set(flat)):
                    continue
                bound = 1
                for c in C:
                    bound *= 2 ** len(c) - 1
                assert 1 <= bound <= count


def test_lemma1_tight_on_worked_example():
    g = graphs.worked_example()
    es = [(e.src, e.tgt) for e in g.edges]
    assert len(rt.valid_patterns(3, es)) == 8 == 2 ** (len(es) - 1)


def test_tableau_two_definitions_agree_eq4_and_updates_converge():
    for (n, es) in NETS:
        for R in rt.valid_patterns(n, es):
            for W in (1, 2, 3):
                T_min, steps = rt.tableau_by_updates(n, es, R, W)        # also proves convergence to S_full
                T_max = rt.tableau_by_paths(n, es, R, W)
                assert T_min == T_max
                assert steps == max(T_min.values())
            if n <= 3:
                assert rt.tableau_by_path_enumeration(n, es, R, 3) == rt.tableau_by_paths(n, es, R, 3)


def test_invalid_pattern_never_reaches_full_state():
    with pytest.raises(RuntimeError):
        rt.tableau_by_updates(2, [(0, 1), (1, 1)], [1, 0], 1)


def test_window_edge_count():
    # all windows of size W have W*|E| edges outside frame 0, whatever the pattern
    for (n, es) in NETS[::7]:
        for R in rt.valid_patterns(n, es):
            for W in (1, 2, 4):
                _, E_W = rt.rollout_window(n, es, R, W)
                assert sum(1 for (_, b) in E_W if b[0] != 0) == W * len(es)


def test_theorem1_equivalences():
    for (n, es) in NETS:
        valid = rt.valid_patterns(n, es)
        stream = [1] * len(es)
        W = 3
        tabs = {tuple(R): rt.tableau_by_paths(n, es, R, W) for R in valid}
        best = {v: min(t[v] for t in tabs.values()) for v in tabs[tuple(stream)]}
        for R in valid:
            a = rt.equally_model_parallel(n, es, R, stream)
            b = rt.inference_factor(n, es, R) == 1
            c = all(tabs[tuple(R)][(i, v)] <= i for (i, v) in tabs[tuple(R)])
            d = all(tabs[tuple(R)][v] == best[v] for v in best)
            assert a == b == c == d, (n, es, R, a, b, c, d)


def test_closed_forms_feed_forward_chain():
    for L in (1, 3, 5):
        es = [(i, i + 1) for i in range(L)]
        W = L + 2
        Ts = rt.tableau_by_updates(L + 1, es, [1] * L, W)[0]
        Tq = rt.tableau_by_updates(L + 1, es, [0] * L, W)[0]
        for i in range(1, W + 1):
            for d in range(1, L + 1):
                assert Ts[(i, d)] == min(i, d)
                assert Tq[(i, d)] == d
        assert rt.first_response(L + 1, es, [1] * L, L) == (L, L)        # same first response time ...
        assert rt.first_response(L + 1, es, [0] * L, L) == (1, L)
        assert rt.response_interval(L + 1, es, [1] * L) == 1             # ... but more frequent outputs
        assert rt.response_interval(L + 1, es, [0] * L) == L


def test_printed_values_sr_network():
    p = printed()
    g = graphs.mnist_net("SR")
    es = [(e.src, e.tgt) for e in g.edges]
    n, out = len(g.nodes), g.index("O")
    assert rt.inference_factor(n, es, g.patterns["streaming"]) == p["sr_net_F_streaming"]
    assert rt.inference_factor(n, es, g.patterns["sequential"]) == p["sr_net_F_sequential"]
    fs = rt.first_response(n, es, g.patterns["streaming"], out)
    fq = rt.first_response(n, es, g.patterns["sequential"], out)
    assert fq[1] - fs[1] == p["sr_net_first_response_gain"]
    assert fs == (2, 2) and fq == (1, 3)
    assert rt.launch_groups(n, es, g.patterns["sequential"]) == [[1], [2], [3]]
    assert rt.launch_groups(n, es, g.patterns["streaming"]) == [[1, 2, 3]]


def test_printed_values_deep_chain():
    p = printed()
    firsts = []
    for k in range(0, 7):
        g = graphs.chain_with_shortcut(4 + k, p["dsr2_shortest_path"])
        es = [(e.src, e.tgt) for e in g.edges]
        n, out = len(g.nodes), len(g.nodes) - 1
        fs = rt.first_response(n, es, g.patterns["streaming"], out)
        fq = rt.first_response(n, es, g.patterns["sequential"], out)
        firsts.append((fs[1], fq[1]))
    assert [a for (a, _) in firsts] == [4] * 7                           # constant for streaming
    assert [b for (_, b) in firsts] == [4 + k for k in range(7)]         # grows linearly with depth for sequential
    k = p["dsr2_longest_path"] - p["dsr2_shortest_path"]
    assert firsts[k][1] - firsts[k][0] == p["dsr2_first_response_gain"]


def test_three_cycle_has_three_most_sequential_patterns():
    g = graphs.three_cycle_net()
    es = [(e.src, e.tgt) for e in g.edges]
    valid = rt.valid_patterns(len(g.nodes), es)
    most = max(R.count(0) for R in valid)
    assert sum(1 for R in valid if R.count(0) == most) == printed()["three_cycle_most_sequential"]
    assert len(valid) == 2 * (2 ** 3 - 1)                                # forward edge free, cycle: all but R = 0


def test_skip_network_integrates_two_frames_when_streaming():
    # S net: sequential classifies single images, streaming integrates over two input frames
    g = graphs.mnist_net("S")
    es = [(e.src, e.tgt) for e in g.edges]
    n, out = len(g.nodes), g.index("O")
    assert rt.depends_on_input_frames(n, es, g.patterns["sequential"], out, 5) == [5]
    assert rt.depends_on_input_frames(n, es, g.patterns["streaming"], out, 5) == [2, 3]
    gf = graphs.mnist_net("FF")
    ef = [(e.src, e.tgt) for e in gf.edges]
    assert rt.depends_on_input_frames(4, ef, gf.patterns["streaming"], 3, 5) == [2]
    # SR net after the streaming rollout uses the full network: frames 0 and 1 reach the output at frame 3
    gs = graphs.mnist_net("SR")
    esr = [(e.src, e.tgt) for e in gs.edges]
    assert rt.depends_on_input_frames(4, esr, gs.patterns["streaming"], 3, 3) == [0, 1]
    assert rt.depends_on_input_frames(4, esr, gs.patterns["sequential"], 3, 1) == [1]


def test_benchmark_patterns_are_valid():
    for name in ("c1", "c2", "c3", "c4", "c5"):
        g = graphs.build(name)
        es = [(e.src, e.tgt) for e in g.edges]
        assert rt.is_network(len(g.nodes), es)
        for pname, R in g.patterns.items():
            assert rt.is_valid(len(g.nodes), es, R), (name, pname)
        assert rt.inference_factor(len(g.nodes), es, g.patterns["streaming"]) == 1
        # the canonical sequential pattern is most-sequential: no further edge can be set to 0
        seq = g.patterns["sequential"]
        for e in range(len(es)):
            if seq[e] == 1:
                flipped = list(seq)
                flipped[e] = 0
                assert not rt.is_valid(len(g.nodes), es, flipped)
