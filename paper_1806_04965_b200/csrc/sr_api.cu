// C ABI of the streaming-rollout library: graph objects, workspace layout, parameter upload and the
// per-frame launch sequence (frame input, one launch group per tableau level, buffer flip).
#include <cuda_runtime.h>

#include <algorithm>
#include <cstddef>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "sr_internal.h"
#include "sr_kernels.h"
#include "sr_dense.h"
#include "sr_resident.h"
#include "sr_tc.h"

// Built-in workspace for callers that may not allocate device memory.  In host code the array's name
// is only a handle: its device address is looked up once per device and that pointer is what the
// kernels get (through the ordinary bind path).
static __device__ __align__(256) unsigned char sr_static_workspace[SR_STATIC_WORKSPACE_BYTES];

namespace {

// One owner per device: the graph that bound the array last.  Binding takes the array away from the previous owner,
// which becomes unbound (its calls then fail with SR_ERR_STATE on the host instead of running kernels on tables the
// new owner has overwritten).
struct StaticSlot {
    void* address = nullptr;
    sr_graph* owner = nullptr;
};
std::mutex static_mutex;
StaticSlot static_slot[64];

void unbind(sr_graph* g)
{
    g->ws = nullptr;
    g->static_device = -1;
    for (SrHostEdge& e : g->edges) e.w_set = false;
    for (SrHostNode& n : g->nodes) n.bias_set = false;
}

void sr_release_static_workspace(sr_graph* g)
{
    std::lock_guard<std::mutex> lock(static_mutex);
    if (g->static_device >= 0 && g->static_device < 64 && static_slot[g->static_device].owner == g)
        static_slot[g->static_device].owner = nullptr;
    g->static_device = -1;
}

struct GraphCache {
    cudaStream_t capture_stream = nullptr;
    cudaGraphExec_t exec = nullptr;
    int frames = 0;
    int kernels = 0;
    bool with_out = false;
};

// A second stream lets independent launches of one frame overlap: the CUDA-core kernel and the
// tensor-core kernel of a launch group, and - when no input edge stays inside the frame - the copy
// and staging of the next input frame, which nothing of the current update reads.
struct SideStream {
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
};

SideStream* side_of(sr_graph* g)
{
    if (!g->side) {
        SideStream* s = new SideStream();
        if (cudaStreamCreateWithFlags(&s->stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&s->fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&s->join, cudaEventDisableTiming) != cudaSuccess) {
            delete s;
            return nullptr;
        }
        g->side = s;
    }
    return static_cast<SideStream*>(g->side);
}

float round_bf16_host(float f)
{
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u) return f;
    u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    std::memcpy(&f, &u, 4);
    return f;
}

size_t node_elems(const sr_graph* g, int v)
{
    const sr_node_desc& d = g->nodes[v].d;
    return (size_t)g->batch * d.h * d.w * d.c;
}

SrRegion take(size_t& off, size_t bytes)
{
    SrRegion r;
    r.offset = off;
    r.bytes = bytes;
    off = sr_align_up(off + bytes, 256);
    return r;
}

// Decide the engine of every node, lay out the workspace and build the block work lists.
sr_status plan(sr_graph* g)
{
    if (g->batch <= 0) return SR_ERR_STATE;
    const int n_nodes = (int)g->nodes.size(), n_edges = (int)g->edges.size();
    for (int v = 0; v < n_nodes; ++v) {
        SrHostNode& n = g->nodes[v];
        n.dense_target = false;
        if (n.is_input) continue;
        int n_conv = 0, n_dense = 0;
        for (int e : n.in_edges) (g->edges[e].d.kind == SR_EDGE_CONV ? n_conv : n_dense)++;
        if (n_conv && n_dense) return SR_ERR_UNSUPPORTED;        // a node sums either convolutions or dense maps
        n.dense_target = n_dense > 0;
        n.use_tc = false;
    }
    if ((int)g->input_nodes.size() > SR_MAX_INPUTS) return SR_ERR_UNSUPPORTED;
    if (g->opt_engine == 0 && g->dtype == SR_DTYPE_BF16) sr_tc_select_nodes(g);
    size_t off = 0;
    for (int v = 0; v < n_nodes; ++v) {
        SrHostNode& n = g->nodes[v];
        n.state[0] = take(off, node_elems(g, v) * g->elem);
        n.state[1] = take(off, node_elems(g, v) * g->elem);
        n.bias = take(off, (size_t)n.d.c * sizeof(float));
    }
    for (int e = 0; e < n_edges; ++e) {
        SrHostEdge& he = g->edges[e];
        const SrHostNode& t = g->nodes[he.d.tgt];
        he.w_direct = SrRegion();
        if (!t.use_tc) he.w_direct = take(off, (size_t)he.K * t.d.c * sizeof(float));
    }
    g->r_nodes = take(off, sizeof(SrDevNode) * n_nodes);
    g->r_edges = take(off, sizeof(SrDevEdge) * n_edges);
    g->r_ctl = take(off, sizeof(SrFrameCtl) + sizeof(int) * SR_MAX_INPUTS);
    // work lists of the direct kernels, one contiguous range per group
    g->items.clear();
    g->group_item_offset.clear();
    g->group_item_count.clear();
    const int px = sr_direct_conv_pixels_per_block(), dco = sr_direct_dense_outputs_per_block(),
              dsb = sr_direct_dense_samples_per_block();
    for (size_t gi = 0; gi < g->groups.size(); ++gi) {
        g->group_item_offset.push_back((int)g->items.size());
        for (int v : g->groups[gi]) {
            const SrHostNode& n = g->nodes[v];
            if (n.use_tc) continue;
            if (n.dense_target) {
                // one sample and a chunk of outputs per block, unless a mean-dense source has more channels
                // than the block's mean buffer holds (then: one warp per output and 8 samples)
                bool fast = true;
                for (int e : n.in_edges)
                    if (g->edges[e].d.kind == SR_EDGE_MEAN_DENSE && g->nodes[g->edges[e].d.src].d.c > sr_direct_head_max_channels())
                        fast = false;
                if (fast) {
                    // a block takes up to 16 outputs of one sample; with a long reduction (thousands of inputs per
                    // output) only 4, so that a small batch still gives every SM several blocks' worth of loads in flight
                    long long k_in = 0;
                    for (int e : n.in_edges) k_in += g->edges[e].K;
                    const int hco = k_in >= 4096 ? 4 : sr_direct_head_outputs_per_block();
                    for (int b0 = 0; b0 < g->batch; ++b0)
                        for (int c0 = 0; c0 < n.d.c; c0 += hco) g->items.push_back(SrDirectItem{v, b0, c0, 1 | (hco << 8)});
                } else {
                    for (int b0 = 0; b0 < g->batch; b0 += dsb)
                        for (int c0 = 0; c0 < n.d.c; c0 += dco) g->items.push_back(SrDirectItem{v, b0, c0, 0});
                }
            } else {
                const int HW = n.d.h * n.d.w;
                for (int b = 0; b < g->batch; ++b)
                    for (int p0 = 0; p0 < HW; p0 += px) g->items.push_back(SrDirectItem{v, b, p0, 0});
            }
        }
        g->group_item_count.push_back((int)g->items.size() - g->group_item_offset.back());
    }
    g->r_items = take(off, sizeof(SrDirectItem) * std::max<size_t>(1, g->items.size()));
    sr_status st = sr_tc_plan(g, off);
    if (st != SR_OK) return st;
    st = sr_rs_plan(g, off);
    if (st != SR_OK) return st;
    st = sr_dn_plan(g, off);
    if (st != SR_OK) return st;
    g->ws_bytes = off;
    int n_tc = 0, n_direct = 0;
    for (const SrHostNode& n : g->nodes)
        if (!n.is_input) (n.use_tc ? n_tc : n_direct)++;
    g->info.n_tensor_core_nodes = n_tc;
    g->info.n_direct_nodes = n_direct;
    int rs_warps = 0;
    sr_rs_describe(g, &g->info.resident_cluster, &rs_warps, &g->info.resident_smem_bytes, &g->info.resident_heads_on_chip);
    if (sr_dn_available(g)) {
        sr_dn_describe(g, &g->info.resident_cluster, &g->info.resident_smem_bytes);
        g->info.resident_heads_on_chip = 1;
    }
    return SR_OK;
}

bool cuda_ok(cudaError_t e) { return e == cudaSuccess; }


sr_status ready(const sr_graph* g)
{
    if (!g) return SR_ERR_INVALID_ARG;
    if (g->batch <= 0 || !g->ws) return SR_ERR_STATE;
    for (const SrHostEdge& e : g->edges)
        if (!e.w_set) return SR_ERR_STATE;
    return SR_OK;
}

const int* input_list_dev(const sr_graph* g)
{
    return reinterpret_cast<const int*>(g->ws + g->r_ctl.offset + sizeof(SrFrameCtl));
}

// Queue the kernels of `frames` consecutive frame updates; returns the number of launches.
int enqueue_frames(sr_graph* g, int first_off, int frames, cudaStream_t s)
{
    int launches = 0;
    SideStream* side = g->opt_overlap ? side_of(g) : nullptr;
    for (int f = first_off; f < first_off + frames; ++f) {
        bool forked = false;
        auto fork = [&]() {
            if (!forked) {
                cudaEventRecord(side->fork, s);
                cudaStreamWaitEvent(side->stream, side->fork, 0);
                forked = true;
            }
        };
        auto join = [&]() {
            if (forked) {
                cudaEventRecord(side->join, side->stream);
                cudaStreamWaitEvent(s, side->join, 0);
                forked = false;
            }
        };
        // frame input: on the side stream if this frame's update does not read it
        cudaStream_t in_stream = s;
        if (side && !g->input_feeds_same_frame) {
            fork();
            in_stream = side->stream;
        }
        sr_launch_input(g, input_list_dev(g), f, in_stream);
        ++launches;
        launches += sr_tc_stage_inputs(g, f, in_stream);
        for (int gi = 0; gi < (int)g->groups.size(); ++gi) {
            const bool has_direct = g->group_item_count[gi] > 0, has_tc = sr_tc_group_has_work(g, gi);
            if (has_direct) {
                cudaStream_t ds = s;
                if (side && has_tc) {
                    fork();
                    ds = side->stream;
                }
                sr_launch_direct_group(g, gi, f, ds);
                ++launches;
            }
            launches += sr_tc_launch_group(g, gi, f, s);
            if (gi + 1 < (int)g->groups.size()) join();       // the next group reads what this one wrote
        }
        join();
    }
    return launches;
}

SrFrameCtl make_ctl(const sr_graph* g, const void* const* in, bool sequence, float* out)
{
    SrFrameCtl c{};
    c.t = g->t;
    c.run_t = 0;
    for (size_t i = 0; i < g->input_nodes.size(); ++i) {
        c.in_base[i] = in[i];
        c.in_stride_bytes[i] = sequence ? (int64_t)(node_elems(g, g->input_nodes[i]) * g->elem) : 0;
    }
    c.out_base = out;
    c.out_stride = (int64_t)node_elems(g, g->info.output_node);          // [B][H][W][C] floats per frame
    return c;
}

// What the launch path derives from the input nodes' current state (staged few-channel edges) is brought up to
// date after a resident run.
void refresh_staging(sr_graph* g, cudaStream_t s)
{
    if (g->stage_dirty) {
        g->launches += sr_tc_after_state_change(g, s);
        g->stage_dirty = false;
    }
}

}  // namespace

extern "C" {

sr_status sr_graph_create(const sr_node_desc* nodes, int n_nodes, const sr_edge_desc* edges, int n_edges,
                          const uint8_t* R, int batch, int dtype, sr_graph** out)
{
    if (!out || batch < 0 || (dtype != SR_DTYPE_F32 && dtype != SR_DTYPE_BF16)) return SR_ERR_INVALID_ARG;
    sr_graph* g = new (std::nothrow) sr_graph();
    if (!g) return SR_ERR_INVALID_ARG;
    const sr_status st = sr_compile(g, nodes, n_nodes, edges, n_edges, R);
    if (st != SR_OK) {
        delete g;
        return st;
    }
    g->input_feeds_same_frame = false;
    for (const SrHostEdge& e : g->edges)
        if (g->nodes[e.d.src].is_input && e.R == 0) g->input_feeds_same_frame = true;
    g->batch = batch;
    g->dtype = dtype;
    g->elem = dtype == SR_DTYPE_BF16 ? 2 : 4;
    *out = g;
    return SR_OK;
}

void sr_graph_destroy(sr_graph* g)
{
    if (!g) return;
    if (g->window) sr_graph_destroy(g->window);
    g->window = nullptr;
    sr_release_static_workspace(g);
    if (g->graphs) {
        GraphCache* c = static_cast<GraphCache*>(g->graphs);
        if (c->exec) cudaGraphExecDestroy(c->exec);
        if (c->capture_stream) cudaStreamDestroy(c->capture_stream);
        delete c;
    }
    if (g->side) {
        SideStream* sd = static_cast<SideStream*>(g->side);
        cudaEventDestroy(sd->fork);
        cudaEventDestroy(sd->join);
        cudaStreamDestroy(sd->stream);
        delete sd;
    }
    sr_tc_destroy(g);
    sr_rs_destroy(g);
    sr_dn_destroy(g);
    delete g;
}

sr_status sr_graph_info(const sr_graph* g, sr_info* out)
{
    if (!g || !out) return SR_ERR_INVALID_ARG;
    *out = g->info;
    return SR_OK;
}

sr_status sr_graph_levels(const sr_graph* g, int32_t* level)
{
    if (!g || !level) return SR_ERR_INVALID_ARG;
    for (size_t v = 0; v < g->nodes.size(); ++v) level[v] = g->nodes[v].level;
    return SR_OK;
}

sr_status sr_graph_set_option(sr_graph* g, int key, int value)
{
    if (!g) return SR_ERR_INVALID_ARG;
    if (key == 0) {
        if (g->ws) return SR_ERR_STATE;
        if (value != 0 && value != 1) return SR_ERR_INVALID_ARG;
        g->opt_engine = value;
        return SR_OK;
    }
    if (key == 1) {
        if (value < 0 || value > 1024) return SR_ERR_INVALID_ARG;
        g->opt_graph_frames = value;
        return SR_OK;
    }
    if (key == 5) {
        if (value != 0 && value != 1) return SR_ERR_INVALID_ARG;
        g->opt_time_tc = value;
        return SR_OK;
    }
    if (key == 4) {
        if (value != 0 && value != 1) return SR_ERR_INVALID_ARG;
        g->opt_overlap = value;
        return SR_OK;
    }
    if (key == 3) {
        if (g->ws) return SR_ERR_STATE;
        if (value != 0 && value != 8 && value != 16 && value != 32) return SR_ERR_INVALID_ARG;
        g->opt_tile_w = value;
        return SR_OK;
    }
    if (key == 2) {
        if (g->ws) return SR_ERR_STATE;
        if (value < 0 || value > 8 || value == 1) return SR_ERR_INVALID_ARG;
        g->opt_b_units = value;
        return SR_OK;
    }
    if (key == 6) {
        if (g->ws) return SR_ERR_STATE;
        if (value != 0 && value != 1) return SR_ERR_INVALID_ARG;
        g->opt_resident = value;
        return SR_OK;
    }
    if (key == 7) {
        if (g->ws) return SR_ERR_STATE;
        if (value != 0 && value != 1 && value != 2 && value != 4) return SR_ERR_INVALID_ARG;
        g->opt_rs_cluster = value;
        return SR_OK;
    }
    if (key == 9) {
        if (g->ws) return SR_ERR_STATE;
        if (value < 0 || value > 2) return SR_ERR_INVALID_ARG;
        g->opt_rs_split = value;
        return SR_OK;
    }
    if (key == 8) {
        if (g->ws) return SR_ERR_STATE;
        if (value != 0 && (value < 4 || value > 32)) return SR_ERR_INVALID_ARG;
        g->opt_rs_warps = value;
        return SR_OK;
    }
    if (key == 11) {
        if (g->ws) return SR_ERR_STATE;
        if (value < 0 || value > 2) return SR_ERR_INVALID_ARG;
        g->opt_tc_pair = value;
        return SR_OK;
    }
    if (key == 14) {
        if (g->ws) return SR_ERR_STATE;
        if (value < 0 || value > 1) return SR_ERR_INVALID_ARG;
        g->opt_tc_fuse = value;
        return SR_OK;
    }
    if (key == 13) {
        if (g->ws) return SR_ERR_STATE;
        if (value < 0 || value > 1) return SR_ERR_INVALID_ARG;
        g->opt_tc_lists = value;
        return SR_OK;
    }
    if (key == 12) {
        if (g->ws) return SR_ERR_STATE;
        if (value < 0 || value > 2) return SR_ERR_INVALID_ARG;
        g->opt_stem_ring = value;
        return SR_OK;
    }
    if (key == 10) {
        if (value < 0 || value > 60000) return SR_ERR_INVALID_ARG;
        g->opt_wait_ms = value;
        if (g->graphs) {                                 // recorded launches carry the old limit
            GraphCache* c = static_cast<GraphCache*>(g->graphs);
            if (c->exec) cudaGraphExecDestroy(c->exec);
            c->exec = nullptr;
        }
        return SR_OK;
    }
    return SR_ERR_INVALID_ARG;
}

sr_status sr_graph_workspace_bytes(const sr_graph* g, size_t* bytes)
{
    if (!g || !bytes) return SR_ERR_INVALID_ARG;
    if (g->ws) {
        *bytes = g->ws_bytes;
        return SR_OK;
    }
    const sr_status st = plan(const_cast<sr_graph*>(g));
    if (st != SR_OK) return st;
    *bytes = g->ws_bytes;
    return SR_OK;
}

sr_status sr_graph_bind_workspace(sr_graph* g, void* workspace_dev, size_t bytes)
{
    if (!g || !workspace_dev) return SR_ERR_INVALID_ARG;
    if (g->ws) return SR_ERR_STATE;
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 255) return SR_ERR_INVALID_ARG;
    if (g->graphs) {                                     // launches recorded for an earlier binding point at its tables
        GraphCache* c = static_cast<GraphCache*>(g->graphs);
        if (c->exec) cudaGraphExecDestroy(c->exec);
        c->exec = nullptr;
    }
    sr_status st = plan(g);
    if (st != SR_OK) return st;
    if (bytes < g->ws_bytes) return SR_ERR_INVALID_ARG;
    char* ws = static_cast<char*>(workspace_dev);
    const int n_nodes = (int)g->nodes.size(), n_edges = (int)g->edges.size();
    std::vector<SrDevNode> dn(n_nodes);
    std::vector<SrDevEdge> de(n_edges);
    int pos = 0;
    for (int v = 0; v < n_nodes; ++v) {
        const SrHostNode& n = g->nodes[v];
        SrDevNode& d = dn[v];
        d.state[0] = ws + n.state[0].offset;
        d.state[1] = ws + n.state[1].offset;
        d.bias = reinterpret_cast<const float*>(ws + n.bias.offset);
        d.H = n.d.h; d.W = n.d.w; d.C = n.d.c; d.act = n.d.act;
        d.first_edge = pos;
        d.n_edges = (int)n.in_edges.size();
        d.is_output = v == g->info.output_node;
        d.input_slot = n.input_slot;
        for (int e : n.in_edges) {
            const SrHostEdge& he = g->edges[e];
            const SrHostNode& s = g->nodes[he.d.src];
            SrDevEdge& x = de[pos++];
            x.src[0] = ws + s.state[0].offset;
            x.src[1] = ws + s.state[1].offset;
            x.w = reinterpret_cast<const float*>(ws + he.w_direct.offset);
            x.Hs = s.d.h; x.Ws = s.d.w; x.Cs = s.d.c;
            x.kind = he.d.kind; x.k = he.k_eff; x.stride = he.stride_eff; x.pad = he.pad_eff;
            x.R = he.R; x.K = he.K; x.src_is_input = s.is_input;
        }
    }
    if (!cuda_ok(cudaMemset(ws, 0, g->ws_bytes))) return SR_ERR_CUDA;
    if (!cuda_ok(cudaMemcpy(ws + g->r_nodes.offset, dn.data(), sizeof(SrDevNode) * n_nodes, cudaMemcpyHostToDevice)))
        return SR_ERR_CUDA;
    if (!cuda_ok(cudaMemcpy(ws + g->r_edges.offset, de.data(), sizeof(SrDevEdge) * n_edges, cudaMemcpyHostToDevice)))
        return SR_ERR_CUDA;
    if (!g->items.empty() &&
        !cuda_ok(cudaMemcpy(ws + g->r_items.offset, g->items.data(), sizeof(SrDirectItem) * g->items.size(),
                            cudaMemcpyHostToDevice)))
        return SR_ERR_CUDA;
    std::vector<int> il(SR_MAX_INPUTS, 0);
    for (size_t i = 0; i < g->input_nodes.size(); ++i) il[i] = g->input_nodes[i];
    if (!cuda_ok(cudaMemcpy(ws + g->r_ctl.offset + sizeof(SrFrameCtl), il.data(), sizeof(int) * SR_MAX_INPUTS,
                            cudaMemcpyHostToDevice)))
        return SR_ERR_CUDA;
    g->ws = ws;
    st = sr_tc_bind(g);
    if (st == SR_OK) st = sr_rs_bind(g);
    if (st == SR_OK) st = sr_dn_bind(g);
    if (st != SR_OK) {
        g->ws = nullptr;
        return st;
    }
    g->t = 0;
    return SR_OK;
}

sr_status sr_graph_bind_static_workspace(sr_graph* g)
{
    if (!g) return SR_ERR_INVALID_ARG;
    if (g->ws || g->batch <= 0) return SR_ERR_STATE;
    size_t need = 0;
    sr_status st = sr_graph_workspace_bytes(g, &need);
    if (st != SR_OK) return st;
    if (need > (size_t)SR_STATIC_WORKSPACE_BYTES) return SR_ERR_TOO_LARGE;
    int dev = -1;
    if (!cuda_ok(cudaGetDevice(&dev)) || dev < 0 || dev >= 64) return SR_ERR_CUDA;
    std::lock_guard<std::mutex> lock(static_mutex);
    StaticSlot& slot = static_slot[dev];
    if (!slot.address) {
        void* p = nullptr;
        if (!cuda_ok(cudaGetSymbolAddress(&p, sr_static_workspace)) || !p) return SR_ERR_CUDA;
        slot.address = p;
    }
    if (slot.owner && slot.owner != g) unbind(slot.owner);
    slot.owner = nullptr;
    st = sr_graph_bind_workspace(g, slot.address, (size_t)SR_STATIC_WORKSPACE_BYTES);
    if (st != SR_OK) return st;
    slot.owner = g;
    g->static_device = dev;
    return SR_OK;
}

sr_status sr_graph_set_edge_weights(sr_graph* g, int edge, const float* w, int is_device)
{
    if (!g || !w || edge < 0 || edge >= (int)g->edges.size()) return SR_ERR_INVALID_ARG;
    if (!g->ws) return SR_ERR_STATE;
    SrHostEdge& he = g->edges[edge];
    const SrHostNode& s = g->nodes[he.d.src];
    const SrHostNode& t = g->nodes[he.d.tgt];
    const int Cout = t.d.c, Cs = s.d.c;
    const size_t n_user = (he.d.kind == SR_EDGE_CONV) ? (size_t)Cout * he.d.k * he.d.k * Cs : (size_t)Cout * he.K;
    std::vector<float> u(n_user);
    if (is_device) {
        if (!cuda_ok(cudaMemcpy(u.data(), w, n_user * sizeof(float), cudaMemcpyDeviceToHost))) return SR_ERR_CUDA;
    } else {
        std::memcpy(u.data(), w, n_user * sizeof(float));
    }
    if (g->kept_weights.size() != g->edges.size()) g->kept_weights.assign(g->edges.size(), std::vector<float>());
    g->kept_weights[edge] = u;                                   // as set by the caller: a window graph gets the same
    if (g->dtype == SR_DTYPE_BF16)
        for (float& x : u) x = round_bf16_host(x);
    // the convolution actually executed: [C_out][k'][k'][Cs]; a pooled edge gets the box-filtered kernel
    std::vector<float> eff;
    const int k = he.d.k, ke = he.k_eff;
    if (he.d.kind == SR_EDGE_CONV && he.d.pool == 2) {
        eff.assign((size_t)Cout * ke * ke * Cs, 0.f);
        const int sh = he.d.stride;
        for (int co = 0; co < Cout; ++co)
            for (int dy = 0; dy < 2; ++dy)
                for (int dx = 0; dx < 2; ++dx)
                    for (int ky = 0; ky < k; ++ky)
                        for (int kx = 0; kx < k; ++kx)
                            for (int ci = 0; ci < Cs; ++ci)
                                eff[(((size_t)co * ke + ky + dy * sh) * ke + kx + dx * sh) * Cs + ci] +=
                                    0.25f * u[(((size_t)co * k + ky) * k + kx) * Cs + ci];
    } else {
        eff.swap(u);
    }
    if (!t.use_tc) {
        std::vector<float> d;
        const float* src = eff.data();
        if (he.d.kind == SR_EDGE_CONV) {                        // [C_out][K] -> [K][C_out]
            d.resize((size_t)he.K * Cout);
            for (int co = 0; co < Cout; ++co)
                for (int kk = 0; kk < he.K; ++kk) d[(size_t)kk * Cout + co] = eff[(size_t)co * he.K + kk];
            src = d.data();
        }
        if (!cuda_ok(cudaMemcpy(g->ws + he.w_direct.offset, src, (size_t)he.K * Cout * sizeof(float),
                                cudaMemcpyHostToDevice)))
            return SR_ERR_CUDA;
    } else {
        const sr_status st = sr_tc_set_weights(g, edge, eff.data());
        if (st != SR_OK) return st;
    }
    {
        sr_status st = sr_rs_set_weights(g, edge, eff.data());
        if (st == SR_OK) st = sr_dn_set_weights(g, edge, eff.data());
        if (st != SR_OK) return st;
    }
    he.w_set = true;
    return SR_OK;
}

sr_status sr_graph_set_node_bias(sr_graph* g, int node, const float* bias_host)
{
    if (!g || !bias_host || node < 0 || node >= (int)g->nodes.size()) return SR_ERR_INVALID_ARG;
    if (!g->ws) return SR_ERR_STATE;
    SrHostNode& n = g->nodes[node];
    if (!cuda_ok(cudaMemcpy(g->ws + n.bias.offset, bias_host, (size_t)n.d.c * sizeof(float), cudaMemcpyHostToDevice)))
        return SR_ERR_CUDA;
    n.bias_set = true;
    if (g->kept_bias.size() != g->nodes.size()) g->kept_bias.assign(g->nodes.size(), std::vector<float>());
    g->kept_bias[node].assign(bias_host, bias_host + n.d.c);
    return SR_OK;
}

sr_status sr_graph_reset(sr_graph* g, const void* const* in0_dev, void* stream)
{
    if (!g || !in0_dev) return SR_ERR_INVALID_ARG;
    if (g->batch <= 0 || !g->ws) return SR_ERR_STATE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (int v = 0; v < (int)g->nodes.size(); ++v) {
        const SrHostNode& n = g->nodes[v];
        const size_t bytes = node_elems(g, v) * g->elem;
        if (n.is_input) {
            if (!in0_dev[n.input_slot]) return SR_ERR_INVALID_ARG;
            if (!cuda_ok(cudaMemcpyAsync(g->ws + n.state[0].offset, in0_dev[n.input_slot], bytes,
                                         cudaMemcpyDeviceToDevice, s)))
                return SR_ERR_CUDA;
            if (!cuda_ok(cudaMemsetAsync(g->ws + n.state[1].offset, 0, bytes, s))) return SR_ERR_CUDA;
        } else {
            if (!cuda_ok(cudaMemsetAsync(g->ws + n.state[0].offset, 0, bytes, s))) return SR_ERR_CUDA;
            if (!cuda_ok(cudaMemsetAsync(g->ws + n.state[1].offset, 0, bytes, s))) return SR_ERR_CUDA;
        }
    }
    // a reported device-side error (an expired wait) is cleared here: the rollout starts over
    if (!cuda_ok(cudaMemsetAsync(g->ws + g->r_ctl.offset + offsetof(SrFrameCtl, error), 0, sizeof(int32_t), s))) return SR_ERR_CUDA;
    g->t = 0;
    g->stage_dirty = false;
    g->launches += sr_tc_after_state_change(g, s);
    return cuda_ok(cudaGetLastError()) ? SR_OK : SR_ERR_CUDA;
}

sr_status sr_rollout_step(sr_graph* g, const void* const* in_next_dev, float* out_dev, void* stream)
{
    sr_status st = ready(g);
    if (st != SR_OK) return st;
    if (!in_next_dev) return SR_ERR_INVALID_ARG;
    for (size_t i = 0; i < g->input_nodes.size(); ++i)
        if (!in_next_dev[i]) return SR_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    refresh_staging(g, s);
    sr_launch_set_ctl(g, make_ctl(g, in_next_dev, false, out_dev), s);
    g->launches += 1 + enqueue_frames(g, 0, 1, s);
    g->t += 1;
    return cuda_ok(cudaGetLastError()) ? SR_OK : SR_ERR_CUDA;
}

sr_status sr_rollout_run(sr_graph* g, const void* const* in_seq_dev, int T, float* out_seq_dev, void* stream)
{
    sr_status st = ready(g);
    if (st != SR_OK) return st;
    if (!in_seq_dev || T < 0) return SR_ERR_INVALID_ARG;
    if (T == 0) return SR_OK;                                    // an empty sequence: nothing to read, nothing changes
    for (size_t i = 0; i < g->input_nodes.size(); ++i)
        if (!in_seq_dev[i]) return SR_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (sr_rs_available(g)) {
        bool aligned = true;                                     // the resident kernel fetches input rows in 4-byte words
        for (size_t i = 0; i < g->input_nodes.size(); ++i)
            if (reinterpret_cast<uintptr_t>(in_seq_dev[i]) & 3) aligned = false;
        if (aligned) {
            // one launch walks all T frames with the states in shared memory, then the frame counter
            // advances and whatever the launch path derives from the input state is refreshed
            st = sr_rs_launch(g, T, make_ctl(g, in_seq_dev, true, out_seq_dev), s);
            if (st != SR_OK) return st;
            g->launches += 1;
            g->t += T;
            g->stage_dirty = true;             // refreshed when the launch path is used next
            return cuda_ok(cudaGetLastError()) ? SR_OK : SR_ERR_CUDA;
        }
    }
    if (sr_dn_available(g)) {
        bool aligned = true;                                     // the dense resident kernel fetches input frames in 16-byte words
        for (size_t i = 0; i < g->input_nodes.size(); ++i)
            if (reinterpret_cast<uintptr_t>(in_seq_dev[i]) & 15) aligned = false;
        if (aligned) {
            st = sr_dn_launch(g, T, make_ctl(g, in_seq_dev, true, out_seq_dev), s);
            if (st != SR_OK) return st;
            g->launches += 1;
            g->t += T;
            return cuda_ok(cudaGetLastError()) ? SR_OK : SR_ERR_CUDA;
        }
    }
    refresh_staging(g, s);
    sr_launch_set_ctl(g, make_ctl(g, in_seq_dev, true, out_seq_dev), s);
    g->launches += 1;
    int done = 0;
    const int gf = g->opt_graph_frames;
    if (gf > 0 && T >= gf) {
        GraphCache* c = static_cast<GraphCache*>(g->graphs);
        if (!c) {
            c = new GraphCache();
            g->graphs = c;
        }
        if (c->exec && c->frames != gf) {
            cudaGraphExecDestroy(c->exec);
            c->exec = nullptr;
        }
        if (!c->exec) {
            if (!c->capture_stream && !cuda_ok(cudaStreamCreateWithFlags(&c->capture_stream, cudaStreamNonBlocking)))
                return SR_ERR_CUDA;
            cudaGraph_t graph = nullptr;
            if (!cuda_ok(cudaStreamBeginCapture(c->capture_stream, cudaStreamCaptureModeThreadLocal))) return SR_ERR_CUDA;
            int k = enqueue_frames(g, 0, gf, c->capture_stream);
            sr_launch_advance(g, gf, c->capture_stream);
            ++k;
            // a capture that has begun is always ended, also when a launch inside it failed: a stream left in
            // capture mode would refuse every later use
            const bool queued = cuda_ok(cudaGetLastError());
            const bool ended = cuda_ok(cudaStreamEndCapture(c->capture_stream, &graph));
            if (!queued || !ended || !graph) {
                if (graph) cudaGraphDestroy(graph);
                cudaGetLastError();
                return SR_ERR_CUDA;
            }
            const cudaError_t ie = cudaGraphInstantiate(&c->exec, graph, 0);
            cudaGraphDestroy(graph);
            if (!cuda_ok(ie)) {
                c->exec = nullptr;
                return SR_ERR_CUDA;
            }
            c->frames = gf;
            c->kernels = k;
        }
        while (T - done >= gf) {
            if (!cuda_ok(cudaGraphLaunch(c->exec, s))) return SR_ERR_CUDA;
            g->launches += c->kernels;
            done += gf;
        }
    }
    if (done < T) {
        // ctl.t / ctl.run_t already stand at `done` (each graph advanced them); offsets are relative to that
        g->launches += enqueue_frames(g, 0, T - done, s);
        sr_launch_advance(g, T - done, s);
        g->launches += 1;
    }
    g->t += T;
    return cuda_ok(cudaGetLastError()) ? SR_OK : SR_ERR_CUDA;
}

// ------------------------------------------------------------------ deep windows (W > 1)
sr_status sr_graph_window_tableau(const sr_graph* g, int W, int32_t* T_host)
{
    if (!g || !T_host || W < 1 || W > 4096) return SR_ERR_INVALID_ARG;
    sr_window_tableau(g, W, T_host);
    return SR_OK;
}

static bool frames_independent(const sr_graph* g)
{
    for (const SrHostEdge& e : g->edges)
        if (e.R == 1 && !g->nodes[e.d.src].is_input) return false;
    return true;
}

sr_status sr_graph_window_workspace_bytes(sr_graph* g, int W, size_t* bytes)
{
    if (!g || !bytes || W < 1 || W > 4096) return SR_ERR_INVALID_ARG;
    if (g->batch <= 0) return SR_ERR_STATE;
    if (!frames_independent(g)) return SR_ERR_UNSUPPORTED;
    if (g->window && g->window_frames != W) {
        if (g->window->ws) return SR_ERR_STATE;                  // a bound window keeps its size
        sr_graph_destroy(g->window);
        g->window = nullptr;
    }
    if (!g->window) {
        std::vector<sr_node_desc> nd;
        std::vector<sr_edge_desc> ed;
        std::vector<uint8_t> R;
        for (const SrHostNode& n : g->nodes) nd.push_back(n.d);
        for (const SrHostEdge& e : g->edges) {
            ed.push_back(e.d);
            R.push_back((uint8_t)e.R);
        }
        sr_graph* w = nullptr;
        const sr_status st = sr_graph_create(nd.data(), (int)nd.size(), ed.data(), (int)ed.size(), R.data(), g->batch * W, g->dtype, &w);
        if (st != SR_OK) return st;
        w->opt_engine = g->opt_engine;
        w->opt_b_units = g->opt_b_units;
        w->opt_tile_w = g->opt_tile_w;
        w->opt_overlap = g->opt_overlap;
        w->opt_tc_pair = g->opt_tc_pair;
        w->opt_stem_ring = g->opt_stem_ring;
        w->opt_tc_lists = g->opt_tc_lists;
        w->opt_tc_fuse = g->opt_tc_fuse;
        w->opt_wait_ms = g->opt_wait_ms;
        w->opt_resident = 0;                                     // a window is one update of a large batch: the launch path
        g->window = w;
        g->window_frames = W;
    }
    return sr_graph_workspace_bytes(g->window, bytes);
}

sr_status sr_graph_bind_window(sr_graph* g, int W, void* workspace_dev, size_t bytes)
{
    if (!g || !workspace_dev) return SR_ERR_INVALID_ARG;
    sr_status st = ready(g);
    if (st != SR_OK) return st;
    size_t need = 0;
    st = sr_graph_window_workspace_bytes(g, W, &need);
    if (st != SR_OK) return st;
    if (g->window->ws) return SR_ERR_STATE;
    if (g->kept_weights.size() != g->edges.size()) return SR_ERR_STATE;
    st = sr_graph_bind_workspace(g->window, workspace_dev, bytes);
    if (st != SR_OK) return st;
    for (size_t e = 0; e < g->edges.size(); ++e) {
        st = sr_graph_set_edge_weights(g->window, (int)e, g->kept_weights[e].data(), 0);
        if (st != SR_OK) return st;
    }
    for (size_t v = 0; v < g->nodes.size() && v < g->kept_bias.size(); ++v)
        if (!g->kept_bias[v].empty()) {
            st = sr_graph_set_node_bias(g->window, (int)v, g->kept_bias[v].data());
            if (st != SR_OK) return st;
        }
    return SR_OK;
}

sr_status sr_rollout_window(sr_graph* g, const void* const* in_seq_dev, int W, float* out_seq_dev, void* stream)
{
    sr_status st = ready(g);
    if (st != SR_OK) return st;
    sr_graph* w = g->window;
    if (!w || !w->ws || g->window_frames != W) return SR_ERR_STATE;
    if (!in_seq_dev) return SR_ERR_INVALID_ARG;
    for (size_t i = 0; i < g->input_nodes.size(); ++i)
        if (!in_seq_dev[i]) return SR_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // frames t .. t+W-1 of the input nodes side by side: what edges that bridge a frame read (Eq. 2: frame i - R(e))
    for (size_t i = 0; i < g->input_nodes.size(); ++i) {
        const int v = g->input_nodes[i];
        const size_t frame = node_elems(g, v) * g->elem;
        char* dst = w->ws + w->nodes[v].state[0].offset;
        if (!cuda_ok(cudaMemcpyAsync(dst, g->ws + g->nodes[v].state[g->t & 1].offset, frame, cudaMemcpyDeviceToDevice, s))) return SR_ERR_CUDA;
        if (W > 1 && !cuda_ok(cudaMemcpyAsync(dst + frame, in_seq_dev[i], frame * (size_t)(W - 1), cudaMemcpyDeviceToDevice, s)))
            return SR_ERR_CUDA;
    }
    w->t = 0;
    w->stage_dirty = false;
    w->launches += sr_tc_after_state_change(w, s);
    // ONE update of the window graph computes all W frames: its batch is [W][B], which is how in_seq and out_seq lie in memory
    st = sr_rollout_step(w, in_seq_dev, out_seq_dev, stream);
    if (st != SR_OK) return st;
    // the last frame of the window becomes the current frame of this graph (Sec. 4: windows chain)
    const int64_t t_new = g->t + W;
    for (size_t v = 0; v < g->nodes.size(); ++v) {
        const size_t frame = node_elems(g, (int)v) * g->elem;
        char* dst = g->ws + g->nodes[v].state[t_new & 1].offset;
        const char* src = g->nodes[v].is_input
                              ? static_cast<const char*>(in_seq_dev[g->nodes[v].input_slot]) + frame * (size_t)(W - 1)
                              : w->ws + w->nodes[v].state[1].offset + frame * (size_t)(W - 1);
        if (!cuda_ok(cudaMemcpyAsync(dst, src, frame, cudaMemcpyDeviceToDevice, s))) return SR_ERR_CUDA;
    }
    g->t = t_new;
    g->stage_dirty = true;
    g->launches += w->launches;
    w->launches = 0;
    return cuda_ok(cudaGetLastError()) ? SR_OK : SR_ERR_CUDA;
}

sr_status sr_graph_get_state(const sr_graph* g, int node, void* dst_dev, void* stream)
{
    if (!g || !dst_dev || node < 0 || node >= (int)g->nodes.size()) return SR_ERR_INVALID_ARG;
    if (g->batch <= 0 || !g->ws) return SR_ERR_STATE;
    const SrHostNode& n = g->nodes[node];
    return cuda_ok(cudaMemcpyAsync(dst_dev, g->ws + n.state[g->t & 1].offset, node_elems(g, node) * g->elem,
                                   cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)))
               ? SR_OK : SR_ERR_CUDA;
}

sr_status sr_graph_set_state(sr_graph* g, int node, const void* src_dev, void* stream)
{
    if (!g || !src_dev || node < 0 || node >= (int)g->nodes.size()) return SR_ERR_INVALID_ARG;
    if (g->batch <= 0 || !g->ws) return SR_ERR_STATE;
    const SrHostNode& n = g->nodes[node];
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!cuda_ok(cudaMemcpyAsync(g->ws + n.state[g->t & 1].offset, src_dev, node_elems(g, node) * g->elem,
                                 cudaMemcpyDeviceToDevice, s)))
        return SR_ERR_CUDA;
    if (n.is_input) g->launches += sr_tc_after_state_change(g, s);
    return SR_OK;
}

sr_status sr_graph_frame(const sr_graph* g, int64_t* t)
{
    if (!g || !t) return SR_ERR_INVALID_ARG;
    *t = g->t;
    return SR_OK;
}

sr_status sr_graph_launch_count(const sr_graph* g, int64_t* n)
{
    if (!g || !n) return SR_ERR_INVALID_ARG;
    *n = g->launches;
    return SR_OK;
}

sr_status sr_graph_kernel_time(sr_graph* g, double* ms, int64_t* launches)
{
    if (!g || !ms || !launches) return SR_ERR_INVALID_ARG;
    if (g->batch <= 0 || !g->ws) return SR_ERR_STATE;
    long long n = 0, n_rs = 0;
    double ms_rs = 0.0;
    sr_status st = sr_tc_timing(g, ms, &n);
    if (st == SR_OK) st = sr_rs_timing(g, &ms_rs, &n_rs);
    double ms_dn = 0.0;
    long long n_dn = 0;
    if (st == SR_OK) st = sr_dn_timing(g, &ms_dn, &n_dn);
    *ms += ms_rs + ms_dn;
    *launches = n + n_rs + n_dn;
    return st;
}

sr_status sr_graph_sync_status(sr_graph* g, void* stream)
{
    if (!g) return SR_ERR_INVALID_ARG;
    if (g->batch <= 0 || !g->ws) return SR_ERR_STATE;
    if (!cuda_ok(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)))) return SR_ERR_CUDA;
    SrFrameCtl c;
    if (!cuda_ok(cudaMemcpy(&c, g->ws + g->r_ctl.offset, sizeof(c), cudaMemcpyDeviceToHost))) return SR_ERR_CUDA;
    if (c.error != 0) return SR_ERR_TIMEOUT;
    return SR_OK;
}

const char* sr_status_str(sr_status s)
{
    switch (s) {
        case SR_OK: return "ok";
        case SR_ERR_INVALID_ARG: return "invalid argument";
        case SR_ERR_NOT_A_NETWORK: return "not a network (no edges, or a node is not connected to an input)";
        case SR_ERR_INVALID_ROLLOUT: return "invalid rollout pattern (its rollout window has a cycle)";
        case SR_ERR_SHAPE_MISMATCH: return "an edge does not map its source shape to its target shape";
        case SR_ERR_UNSUPPORTED: return "unsupported configuration";
        case SR_ERR_CUDA: return "CUDA error";
        case SR_ERR_TIMEOUT: return "a device-side wait expired";
        case SR_ERR_STATE: return "call order (workspace not bound, weights not set, or graph is theory-only)";
        case SR_ERR_TOO_LARGE: return "the graph needs more workspace than the built-in workspace holds";
    }
    return "unknown status";
}

}  // extern "C"
