"""Oracle, theory half: the paper's rollout definitions written out literally.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this module;
it exists so that tests and the benchmark's CPU baseline can check the CUDA
library against the paper.  Pure Python, explicit graphs, no shortcuts: every
function builds the rollout window R_W as a graph and works on that graph.

A network is given as (n_nodes, edges) with edges a list of (src, tgt) pairs;
parallel edges are allowed (the list index identifies an edge).  A rollout
pattern R is a list with one 0/1 entry per edge.

Definitions followed (paper Sec. 3):
  input set I_N ................ Eq. (1)
  network ...................... Definition "network" (input-connected, 0 < |E|)
  rollout window R_W ........... Eq. (2)
  valid pattern ................ R_W acyclic
  S_init, update step U ........ Eq. (3) and the definition of U that follows it
  inference tableau T .......... Eq. (4), both sides, computed independently
  inference factor F(R) ........ Eq. (5)
Response quantities under chained windows of size 1 (Sec. 4, "we conduct
inference on shallow rollouts (W = 1)"): see first_response().
"""
from __future__ import annotations

from itertools import product
from typing import Dict, List, Sequence, Tuple

EdgeList = Sequence[Tuple[int, int]]
WNode = Tuple[int, int]          # (frame, node)


# ----------------------------------------------------------------------------- Sec. 3, graphs
def input_set(n_nodes: int, edges: EdgeList) -> List[int]:
    """I_N: nodes without incoming edges, Eq. (1)."""
    return [v for v in range(n_nodes) if not any(t == v for (_, t) in edges)]


def is_input_connected(n_nodes: int, edges: EdgeList) -> bool:
    """Every node is the end of a path that starts in I_N (input nodes themselves
    are taken as connected: they are given, not computed)."""
    reached = set(input_set(n_nodes, edges))
    grew = True
    while grew:
        grew = False
        for (u, v) in edges:
            if u in reached and v not in reached:
                reached.add(v)
                grew = True
    return len(reached) == n_nodes


def is_network(n_nodes: int, edges: EdgeList) -> bool:
    """Definition "network": directed, input-connected, 0 < |E| < infinity."""
    return len(edges) > 0 and is_input_connected(n_nodes, edges)


# ----------------------------------------------------------------------------- Sec. 3, rollout windows
def rollout_window(n_nodes: int, edges: EdgeList, R: Sequence[int], W: int):
    """R_W = (V_W, E_W) of Eq. (2): V_W = {0..W} x V and ((i,u),(j,v)) in E_W iff
    (u,v) in E and j = i + R((u,v)).  Returns (V_W, E_W) as lists."""
    V_W = [(i, v) for i in range(W + 1) for v in range(n_nodes)]
    E_W = []
    for (e, (u, v)) in enumerate(edges):
        for i in range(W + 1):
            j = i + R[e]
            if j <= W:
                E_W.append(((i, u), (j, v)))
    return V_W, E_W


def _is_acyclic(V: List[WNode], E: List[Tuple[WNode, WNode]]) -> bool:
    succ: Dict[WNode, List[WNode]] = {v: [] for v in V}
    for (a, b) in E:
        succ[a].append(b)
    WHITE, GREY, BLACK = 0, 1, 2
    colour = {v: WHITE for v in V}
    for root in V:
        if colour[root] != WHITE:
            continue
        stack = [(root, iter(succ[root]))]
        colour[root] = GREY
        while stack:
            node, it = stack[-1]
            nxt = next(it, None)
            if nxt is None:
                colour[node] = BLACK
                stack.pop()
            elif colour[nxt] == GREY:
                return False
            elif colour[nxt] == WHITE:
                colour[nxt] = GREY
                stack.append((nxt, iter(succ[nxt])))
    return True


def is_valid(n_nodes: int, edges: EdgeList, R: Sequence[int], W: int = 1) -> bool:
    """A pattern is valid iff its rollout window is acyclic (for one, hence all, W)."""
    V_W, E_W = rollout_window(n_nodes, edges, R, W)
    return _is_acyclic(V_W, E_W)


def all_patterns(n_edges: int):
    return [list(p) for p in product((0, 1), repeat=n_edges)]


def valid_patterns(n_nodes: int, edges: EdgeList) -> List[List[int]]:
    return [R for R in all_patterns(len(edges)) if is_valid(n_nodes, edges, R)]


def equally_model_parallel(n_nodes: int, edges: EdgeList, R1: Sequence[int], R2: Sequence[int]) -> bool:
    """R1 = R2 on every edge that does not originate in the input set."""
    I = set(input_set(n_nodes, edges))
    return all(R1[e] == R2[e] for (e, (u, _)) in enumerate(edges) if u not in I)


# ----------------------------------------------------------------------------- Sec. 3, update states and tableau
def s_init(n_nodes: int, edges: EdgeList, W: int) -> Dict[WNode, int]:
    """Eq. (3): S_init((i,v)) = 1 iff v in I_N or i = 0."""
    I = set(input_set(n_nodes, edges))
    return {(i, v): int(v in I or i == 0) for i in range(W + 1) for v in range(n_nodes)}


def update_step(S: Dict[WNode, int], E_W) -> Dict[WNode, int]:
    """U(S)(v) = 1 if S(v) = 1 or every predecessor of v in E_W has S = 1."""
    preds: Dict[WNode, List[WNode]] = {v: [] for v in S}
    for (a, b) in E_W:
        preds[b].append(a)
    return {v: int(S[v] == 1 or all(S[u] == 1 for u in preds[v])) for v in S}


def tableau_by_updates(n_nodes: int, edges: EdgeList, R: Sequence[int], W: int, max_steps: int = 10_000):
    """Right-hand side of Eq. (4): the first n with U^n(S_init)(v) = 1.
    Returns (T, n_steps_to_full)."""
    _, E_W = rollout_window(n_nodes, edges, R, W)
    S = s_init(n_nodes, edges, W)
    T = {v: 0 for v in S if S[v] == 1}
    n = 0
    while not all(S.values()):
        n += 1
        if n > max_steps:
            raise RuntimeError("update steps do not reach the full state (invalid pattern?)")
        S2 = update_step(S, E_W)
        if S2 == S:
            raise RuntimeError("update step made no progress (invalid pattern?)")
        for v in S2:
            if S2[v] == 1 and S[v] == 0:
                T[v] = n
        S = S2
    return T, n


def tableau_by_paths(n_nodes: int, edges: EdgeList, R: Sequence[int], W: int) -> Dict[WNode, int]:
    """Left-hand side of Eq. (4): the longest path in R_W that ends at the node
    and whose first edge does not end in frame 0 (0 if there is none).  Every
    later edge of such a path ends in a frame >= 1 too, since no edge points
    back in time, so the recursion only has to skip edges that end in frame 0."""
    V_W, E_W = rollout_window(n_nodes, edges, R, W)
    preds: Dict[WNode, List[WNode]] = {v: [] for v in V_W}
    for (a, b) in E_W:
        preds[b].append(a)
    memo: Dict[WNode, int] = {}

    def longest(v: WNode, depth: int = 0) -> int:
        if v in memo:
            return memo[v]
        if depth > len(V_W):
            raise RuntimeError("cycle in rollout window")
        best = 0
        if v[0] != 0:
            for u in preds[v]:
                best = max(best, 1 + longest(u, depth + 1))
        memo[v] = best
        return best

    return {v: longest(v) for v in V_W}


def tableau_by_path_enumeration(n_nodes: int, edges: EdgeList, R: Sequence[int], W: int) -> Dict[WNode, int]:
    """Same quantity by listing every admissible path (tiny graphs only)."""
    V_W, E_W = rollout_window(n_nodes, edges, R, W)
    succ: Dict[WNode, List[WNode]] = {v: [] for v in V_W}
    for (a, b) in E_W:
        succ[a].append(b)
    best = {v: 0 for v in V_W}

    def walk(v: WNode, length: int):
        best[v] = max(best[v], length)
        for nxt in succ[v]:
            walk(nxt, length + 1)

    for (a, b) in E_W:               # first edge of the path
        if b[0] != 0:
            walk(b, 1)
    return best


def inference_factor(n_nodes: int, edges: EdgeList, R: Sequence[int]) -> int:
    """F(R) = max over V_1 of T_{R_1}, Eq. (5)."""
    T, _ = tableau_by_updates(n_nodes, edges, R, 1)
    return max(T.values())


def frame_levels(n_nodes: int, edges: EdgeList, R: Sequence[int]) -> List[int]:
    """T_{R_1}((1, v)) for every node v: the update step, inside one chained window
    of size 1, at which v is computed (0 for input nodes)."""
    T, _ = tableau_by_updates(n_nodes, edges, R, 1)
    return [T[(1, v)] for v in range(n_nodes)]


def launch_groups(n_nodes: int, edges: EdgeList, R: Sequence[int]) -> List[List[int]]:
    """Nodes computed together: group l holds the non-input nodes with level l, l = 1..F(R)."""
    lv = frame_levels(n_nodes, edges, R)
    return [[v for v in range(n_nodes) if lv[v] == l] for l in range(1, max(lv) + 1)]


# ----------------------------------------------------------------------------- Sec. 4, responses under chained W = 1 windows
def first_response(n_nodes: int, edges: EdgeList, R: Sequence[int], out_node: int):
    """(frame, update step) of the first output that depends on an input.

    Windows of size 1 are chained: frame 1 of a window becomes frame 0 of the
    next, every window costs F(R) update steps, and inside a window the output
    node is ready after T_{R_1}((1, out)) steps.  Frame-0 states are given
    (zero), never computed, so an edge that ends in frame 0 carries nothing.
    The first informative frame k is found by search in explicit windows: the
    smallest k such that (k, out) is reachable from some (j, u), u in I_N, using
    only edges that end in a frame >= 1.  Returns None if the output is never
    reached.
    """
    I = set(input_set(n_nodes, edges))
    F = inference_factor(n_nodes, edges, R)
    t_out = frame_levels(n_nodes, edges, R)[out_node]
    for W in range(1, 2 * n_nodes + 2):
        V_W, E_W = rollout_window(n_nodes, edges, R, W)
        reached = {(i, u) for (i, u) in V_W if u in I}
        grew = True
        while grew:
            grew = False
            for (a, b) in E_W:
                if b[0] >= 1 and a in reached and b not in reached:
                    reached.add(b)
                    grew = True
        hit = [i for i in range(1, W + 1) if (i, out_node) in reached and out_node not in I]
        if hit:
            k = min(hit)
            return k, (k - 1) * F + t_out
    return None


def response_interval(n_nodes: int, edges: EdgeList, R: Sequence[int]) -> int:
    """Update steps between consecutive outputs = F(R) (Sec. 4)."""
    return inference_factor(n_nodes, edges, R)


def depends_on_input_frames(n_nodes: int, edges: EdgeList, R: Sequence[int], out_node: int, frame: int) -> List[int]:
    """Which input frames the output at `frame` can depend on, in the explicit
    window R_frame with frame-0 states given (edges ending in frame 0 unused)."""
    I = set(input_set(n_nodes, edges))
    V_W, E_W = rollout_window(n_nodes, edges, R, frame)
    preds: Dict[WNode, List[WNode]] = {v: [] for v in V_W}
    for (a, b) in E_W:
        if b[0] >= 1:
            preds[b].append(a)
    seen, stack = set(), [(frame, out_node)]
    while stack:
        v = stack.pop()
        if v in seen:
            continue
        seen.add(v)
        stack.extend(preds[v])
    return sorted({i for (i, u) in seen if u in I})
