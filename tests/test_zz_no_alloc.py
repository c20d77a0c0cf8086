"""The built-in workspace (sr_graph_bind_static_workspace) for callers that cannot allocate device memory.

A host application may forbid allocations where a graph gets set up: inside a real-time section, when
a foreign component owns the memory pool, or after the device has been fully committed.  Such a caller
binds the fixed array inside the library instead of its own buffer.  This test drives that entry point
through the C ABI and checks that a rollout on the built-in workspace gives what the ordinary,
caller-allocated workspace gives - twice in a row with different graphs, because the array is shared
and still holds the previous graph's data when the next one binds it.  It runs last on purpose.
"""
import numpy as np
import pytest

from tests import parity
from workloads import data, graphs

pytestmark = pytest.mark.gpu


def rollout(spec, static):
    import torch
    from paper_1806_04965_b200 import Graph
    X, W, Bi = data.make_inputs(spec), data.make_weights(spec), data.make_biases(spec, zero=False)
    G = Graph(spec.nodes, spec.edges, spec.patterns["streaming"], batch=spec.batch, dtype=spec.dtype,
              static_workspace=static)
    G.set_weights(W, Bi)
    out = G.rollout([parity.to_device(spec, X[v]) for v in G.input_nodes])
    G.sync_status()
    states = [G.get_state(v).float().cpu().numpy() for v in range(len(spec.nodes))]
    torch.cuda.synchronize()                       # the array is free for the next graph only after this
    return out.cpu().numpy(), states, G.info


def test_built_in_workspace_matches_caller_workspace_twice():
    # first a graph with tensor-core nodes and a staged input edge, then a smaller fp32 one that
    # lands on memory the first graph has left dirty
    specs = [graphs.build("c2", batch=8, frames=5), graphs.build("c1", batch=4, frames=6)]
    for spec in specs:
        want_out, want_states, _ = rollout(spec, static=False)
        got_out, got_states, info = rollout(spec, static=True)
        tol = parity.TOL[spec.dtype]
        assert parity.rel_err(got_out, want_out.astype(np.float64)) <= tol
        for g, w in zip(got_states, want_states):
            assert parity.rel_err(g, w.astype(np.float64)) <= tol
        assert np.abs(want_out).max() > 0
    # same kernels on the same data: the second bind saw stale contents and still agrees exactly
    assert np.array_equal(got_out, want_out)


def test_a_new_bind_takes_the_array_from_the_previous_graph_and_allocates_nothing():
    import torch
    from paper_1806_04965_b200 import Graph, SrError
    spec = graphs.build("c2", batch=4, frames=3)
    X, W, Bi = data.make_inputs(spec), data.make_weights(spec), data.make_biases(spec)
    x = parity.to_device(spec, X[0])
    first = Graph(spec.nodes, spec.edges, spec.patterns["streaming"], batch=spec.batch, dtype=spec.dtype, static_workspace=True)
    first.set_weights(W, Bi)
    want = first.rollout([x]).cpu().numpy()
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    second = Graph(spec.nodes, spec.edges, spec.patterns["streaming"], batch=spec.batch, dtype=spec.dtype, static_workspace=True)
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before                # binding the built-in array takes no device memory
    # the first graph no longer owns the array: its calls fail on the host instead of running on the new owner's tables
    for call in (lambda: first.reset([x[0]]), lambda: first.step([x[1]]), lambda: first.run([x[1:]]),
                 lambda: first.get_state(1), lambda: first.set_weights(W, Bi)):
        with pytest.raises(SrError) as e:
            call()
        assert e.value.status == "SR_ERR_STATE"
    second.set_weights(W, Bi)
    got = second.rollout([x]).cpu().numpy()
    second.sync_status()
    assert np.array_equal(got, want)


def test_graph_larger_than_the_built_in_workspace_is_refused():
    from paper_1806_04965_b200 import Graph, SrError
    spec = graphs.build("c3")                      # hundreds of MiB of states
    with pytest.raises(SrError) as e:
        Graph(spec.nodes, spec.edges, spec.patterns["streaming"], batch=spec.batch, dtype=spec.dtype,
              static_workspace=True)
    assert e.value.status == "SR_ERR_TOO_LARGE"
