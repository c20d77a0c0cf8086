// Graph compiler: network and rollout-pattern validation, inference-tableau levels, launch groups
// and response quantities.  Host only, integers only.
//
// The closed forms used here follow from the paper's definitions (Sec. 3):
//  * R is valid iff the rollout window is acyclic.  No window edge points back in time and every
//    frame repeats the same within-frame edges, so a cycle can only consist of R = 0 edges of one
//    frame: R is valid iff the subgraph of R = 0 edges is acyclic.
//  * The tableau of the window of size 1 (Eq. 4) is the longest path ending at (1, v) whose first
//    edge does not end in frame 0.  Such a path lies in frame 1 except for a possible first edge
//    that bridges from frame 0, hence   level(v) = 0 for input nodes, else
//    level(v) = max(1, 1 + max over R = 0 in-edges (u, v) of level(u)),   F(R) = max_v level(v) (Eq. 5).
//  * Chained windows of size 1 (Sec. 4): frame-0 states are given, never computed, so information
//    enters only through edges that end in a frame >= 1.  Along a path from an input node the frame
//    index grows by R(e) per edge, and the first edge must leave frame 0 if it starts there; the
//    first informative frame is therefore the shortest path from an input node to the output node
//    with edge cost 1 on edges that leave an input node and R(e) elsewhere.
#include <algorithm>
#include <climits>
#include <deque>

#include "sr_internal.h"

static int conv_out(int n, int k, int s)
{
    const int p = (k - 1) / 2;
    return (n + 2 * p - k) / s + 1;
}

sr_status sr_compile(sr_graph* g, const sr_node_desc* nodes, int n_nodes, const sr_edge_desc* edges, int n_edges,
                     const uint8_t* R)
{
    if (!nodes || n_nodes <= 0 || n_edges < 0 || (n_edges > 0 && (!edges || !R))) return SR_ERR_INVALID_ARG;
    if (n_edges == 0) return SR_ERR_NOT_A_NETWORK;                       // 0 < |E|
    for (int v = 0; v < n_nodes; ++v) {
        const sr_node_desc& d = nodes[v];
        if (d.h <= 0 || d.w <= 0 || d.c <= 0 || (d.act != 0 && d.act != 1)) return SR_ERR_INVALID_ARG;
    }
    for (int e = 0; e < n_edges; ++e) {
        const sr_edge_desc& d = edges[e];
        if (d.src < 0 || d.src >= n_nodes || d.tgt < 0 || d.tgt >= n_nodes) return SR_ERR_INVALID_ARG;
        if (R[e] > 1) return SR_ERR_INVALID_ARG;
        if (d.kind < 0 || d.kind > 2) return SR_ERR_INVALID_ARG;
        if (d.kind == SR_EDGE_CONV && (d.k <= 0 || (d.k % 2) == 0 || d.stride <= 0 || (d.pool != 0 && d.pool != 2)))
            return SR_ERR_INVALID_ARG;
    }
    g->nodes.assign(n_nodes, SrHostNode());
    g->edges.assign(n_edges, SrHostEdge());
    for (int v = 0; v < n_nodes; ++v) g->nodes[v].d = nodes[v];
    for (int e = 0; e < n_edges; ++e) {
        g->edges[e].d = edges[e];
        g->edges[e].R = R[e];
        g->nodes[edges[e].tgt].in_edges.push_back(e);
    }
    // input set (Eq. 1) and input-connectedness
    g->input_nodes.clear();
    std::vector<char> reached(n_nodes, 0);
    std::deque<int> q;
    for (int v = 0; v < n_nodes; ++v) {
        g->nodes[v].is_input = g->nodes[v].in_edges.empty();
        if (g->nodes[v].is_input) {
            g->nodes[v].input_slot = (int)g->input_nodes.size();
            g->input_nodes.push_back(v);
            reached[v] = 1;
            q.push_back(v);
        }
    }
    while (!q.empty()) {
        const int u = q.front();
        q.pop_front();
        for (int e = 0; e < n_edges; ++e)
            if (edges[e].src == u && !reached[edges[e].tgt]) {
                reached[edges[e].tgt] = 1;
                q.push_back(edges[e].tgt);
            }
    }
    for (int v = 0; v < n_nodes; ++v)
        if (!reached[v]) return SR_ERR_NOT_A_NETWORK;
    // edge shapes
    for (int e = 0; e < n_edges; ++e) {
        SrHostEdge& he = g->edges[e];
        const sr_node_desc& s = nodes[he.d.src];
        const sr_node_desc& t = nodes[he.d.tgt];
        if (he.d.kind == SR_EDGE_CONV) {
            int oh = conv_out(s.h, he.d.k, he.d.stride), ow = conv_out(s.w, he.d.k, he.d.stride);
            he.k_eff = he.d.k;
            he.stride_eff = he.d.stride;
            he.pad_eff = (he.d.k - 1) / 2;
            if (he.d.pool == 2) {
                oh /= 2;
                ow /= 2;
                he.k_eff = he.d.k + he.d.stride;          // conv then 2x2 average = one conv, kernel k+s, stride 2s
                he.stride_eff = 2 * he.d.stride;
            }
            if (oh != t.h || ow != t.w || oh <= 0 || ow <= 0) return SR_ERR_SHAPE_MISMATCH;
            he.K = he.k_eff * he.k_eff * s.c;
        } else {
            if (t.h != 1 || t.w != 1) return SR_ERR_SHAPE_MISMATCH;
            he.K = (he.d.kind == SR_EDGE_DENSE) ? s.h * s.w * s.c : s.c;
        }
    }
    // validity of R: Kahn's algorithm on the R = 0 subgraph; the peeling order also yields the levels
    std::vector<int> indeg0(n_nodes, 0), level(n_nodes, 0);
    for (int e = 0; e < n_edges; ++e)
        if (R[e] == 0) indeg0[edges[e].tgt]++;
    for (int v = 0; v < n_nodes; ++v) {
        level[v] = g->nodes[v].is_input ? 0 : 1;
        if (indeg0[v] == 0) q.push_back(v);
    }
    int peeled = 0;
    while (!q.empty()) {
        const int u = q.front();
        q.pop_front();
        ++peeled;
        for (int e = 0; e < n_edges; ++e) {
            if (R[e] != 0 || edges[e].src != u) continue;
            const int v = edges[e].tgt;
            level[v] = std::max(level[v], level[u] + 1);
            if (--indeg0[v] == 0) q.push_back(v);
        }
    }
    if (peeled != n_nodes) return SR_ERR_INVALID_ROLLOUT;
    int F = 0;
    for (int v = 0; v < n_nodes; ++v) {
        g->nodes[v].level = level[v];
        F = std::max(F, level[v]);
    }
    g->groups.assign(F, std::vector<int>());
    for (int v = 0; v < n_nodes; ++v)
        if (level[v] > 0) g->groups[level[v] - 1].push_back(v);
    // output node
    int out = n_nodes - 1;
    for (int v = n_nodes - 1; v >= 0; --v) {
        bool has_out = false;
        for (int e = 0; e < n_edges; ++e)
            if (edges[e].src == v && edges[e].tgt != v) has_out = true;
        if (!has_out && !g->nodes[v].is_input) {
            out = v;
            break;
        }
    }
    // first informative frame: 0-1 shortest path from the input set
    std::vector<int> dist(n_nodes, INT_MAX);
    std::deque<int> dq;
    for (int v : g->input_nodes) {
        dist[v] = 0;
        dq.push_back(v);
    }
    while (!dq.empty()) {
        const int u = dq.front();
        dq.pop_front();
        for (int e = 0; e < n_edges; ++e) {
            if (edges[e].src != u) continue;
            const int cost = g->nodes[u].is_input ? 1 : (int)R[e];
            const int v = edges[e].tgt;
            if (dist[u] + cost < dist[v]) {
                dist[v] = dist[u] + cost;
                if (cost == 0) dq.push_front(v); else dq.push_back(v);
            }
        }
    }
    bool par = true;
    for (int e = 0; e < n_edges; ++e)
        if (!g->nodes[edges[e].src].is_input && R[e] != 1) par = false;
    sr_info& I = g->info;
    I = sr_info{};
    I.n_nodes = n_nodes;
    I.n_edges = n_edges;
    I.n_inputs = (int)g->input_nodes.size();
    I.inference_factor = F;
    I.n_groups = F;
    I.streaming_parallel = par ? 1 : 0;
    I.output_node = out;
    const bool informative = !g->nodes[out].is_input && dist[out] != INT_MAX;
    I.first_response_frame = informative ? std::max(1, dist[out]) : -1;
    I.first_response_step = informative ? (I.first_response_frame - 1) * F + level[out] : -1;
    I.response_interval = F;
    return SR_OK;
}

// Inference tableau of the rollout window of size W (Eq. 4): T((i, v)) for i = 0..W, row-major [W + 1][n_nodes].
// Frame 0 and the input nodes are given (T = 0); every other node of the window becomes computable one update step
// after the last of its predecessors ((i - R(e), u) for every edge e = (u, v)), which is also the length of the longest
// admissible path that ends in it.  Frames are visited in increasing order and, inside a frame, nodes in increasing
// level, so every predecessor is final when it is read.
void sr_window_tableau(const sr_graph* g, int W, int32_t* T)
{
    const int n = (int)g->nodes.size();
    std::vector<int> order;
    for (const std::vector<int>& grp : g->groups)
        for (int v : grp) order.push_back(v);
    for (int v = 0; v < n; ++v) T[v] = 0;
    for (int i = 1; i <= W; ++i) {
        for (int v = 0; v < n; ++v) T[(size_t)i * n + v] = 0;
        for (int v : order) {
            int t = 0;
            for (int e : g->nodes[v].in_edges) {
                const SrHostEdge& he = g->edges[e];
                t = std::max(t, T[(size_t)(i - he.R) * n + he.d.src]);
            }
            T[(size_t)i * n + v] = t + 1;
        }
    }
}
