// Internal structures of the streaming-rollout library: host-side graph, device-side tables.
#pragma once
#include <cstddef>
#include <cstdint>
#include <string>
#include <vector>

#include "../../include/sr_rollout.h"

#define SR_MAX_INPUTS 4

// ------------------------------------------------------------------ tables read by the kernels
// One incoming edge of a node, as the CUDA-core ("direct") kernels see it.  A pooled edge
// (conv k, stride s, then 2x2 average) is stored as the single convolution it equals:
// kernel k+s, stride 2s, same padding, box-filtered weights.
struct SrDevEdge {
    const void* src[2];     // source state, frame parity 0 / 1
    const float* w;         // conv: [k*k*Cs][C_out] (K-major rows, channels contiguous); dense: [C_out][K]
    int32_t Hs, Ws, Cs;     // source shape
    int32_t kind, k, stride, pad;
    int32_t R;              // 1: read frame t, 0: read frame t+1 (Eq. 2)
    int32_t K;              // reduction length of this edge
    int32_t src_is_input;
};

struct SrDevNode {
    void* state[2];
    const float* bias;
    int32_t H, W, C, act;
    int32_t first_edge, n_edges;     // range in the SrDevEdge table
    int32_t is_output;
    int32_t input_slot;              // >= 0 for input nodes: index into SrFrameCtl::in_base
};

// One block's work in a grouped direct launch.
struct SrDirectItem {
    int32_t node;        // index into the SrDevNode table
    int32_t b0;          // first sample (dense nodes: sample chunk)
    int32_t p0;          // first pixel (conv nodes) or first output channel (dense nodes)
    int32_t pad_;
};

// Frame control block in device memory: lets a recorded launch sequence be replayed for later frames.
struct SrFrameCtl {
    int64_t t;                            // frame updates completed since reset
    int64_t run_t;                        // frame updates completed inside the current step / run call
    const void* in_base[SR_MAX_INPUTS];   // frame used by update run_t is in_base + run_t * in_stride_bytes
    int64_t in_stride_bytes[SR_MAX_INPUTS];
    float* out_base;                      // output of update run_t goes to out_base + run_t * out_stride (floats); may be null
    int64_t out_stride;
    int32_t error;                        // first device-side error code (0 = none)
    int32_t pad_;
};

// ------------------------------------------------------------------ host-side graph
struct SrRegion { size_t offset = 0, bytes = 0; };

struct SrHostNode {
    sr_node_desc d;
    bool is_input = false;
    int level = 0;
    int input_slot = -1;
    std::vector<int> in_edges;
    bool dense_target = false;     // all incoming edges are dense / mean-dense
    bool use_tc = false;
    SrRegion state[2], bias;
    bool bias_set = false;
};

struct SrHostEdge {
    sr_edge_desc d;
    int R = 1;
    // the convolution actually executed (pooled edges are rewritten)
    int k_eff = 0, stride_eff = 0, pad_eff = 0, K = 0;
    SrRegion w_direct;
    bool w_set = false;
};

struct sr_graph {
    std::vector<SrHostNode> nodes;
    std::vector<SrHostEdge> edges;
    int batch = 0, dtype = 0, elem = 4;
    sr_info info{};
    std::vector<int> input_nodes;
    std::vector<std::vector<int>> groups;          // groups[l-1] = nodes of level l
    // options
    int opt_engine = 0, opt_graph_frames = 0, opt_b_units = 0, opt_tile_w = 0, opt_overlap = 1, opt_time_tc = 0;
    int opt_tc_fuse = 1;                           // two nodes of at most 64 channels that share a source run as one 128-row plan
    int opt_tc_lists = 0;                          // tensor-core work items: 1 = a list per CTA made on the host, 0 = the same plus a shared list of the smallest items
    int opt_stem_ring = 1;                         // activation boxes of staged few-channel edges travel in the weight ring
    int opt_tc_pair = 0;                           // tensor-core work items: 0 / 1 = single pixel tiles, 2 = pairs of tiles wherever the geometry allows
    int opt_wait_ms = 1000;                        // limit of every device-side wait; 0 = expire at once (test hook)
    int opt_resident = 1, opt_rs_cluster = 0, opt_rs_warps = 0, opt_rs_split = 0;   // 16-channel work units: 0 never, 1 always, 2 by cost
    // workspace
    size_t ws_bytes = 0;
    char* ws = nullptr;
    SrRegion r_nodes, r_edges, r_ctl, r_items;
    std::vector<SrRegion> r_group_items;           // per group
    std::vector<int> group_item_count;
    std::vector<SrDirectItem> items;
    std::vector<int> group_item_offset;
    // dynamic state
    int64_t t = 0;
    int64_t launches = 0;
    void* tc = nullptr;                            // tensor-core engine state (opaque here)
    void* rs = nullptr;                            // resident engine state (opaque here)
    void* dn = nullptr;                            // dense resident engine state (opaque here)
    std::vector<unsigned char> dn_headers;         // its per-rank table images, uploaded when a workspace is bound
    void* graphs = nullptr;                        // CUDA-graph cache (opaque here)
    void* side = nullptr;                          // side stream and fork / join events (opaque here)
    bool input_feeds_same_frame = false;           // some edge that leaves an input node has R = 0
    // deep-window mode: a second graph of the same network whose batch holds the W frames of a window side by side
    sr_graph* window = nullptr;
    int window_frames = 0;
    std::vector<std::vector<float>> kept_weights;  // the parameters as the caller set them (host copies), for that graph
    std::vector<std::vector<float>> kept_bias;
    int static_device = -1;                        // >= 0: bound to the built-in workspace of that device
    bool stage_dirty = false;                      // the resident kernel ran: staged copies of the input state are stale
};

// sr_compile.cpp
sr_status sr_compile(sr_graph* g, const sr_node_desc* nodes, int n_nodes, const sr_edge_desc* edges, int n_edges,
                     const uint8_t* R);

void sr_window_tableau(const sr_graph* g, int W, int32_t* T /* [W + 1][n_nodes] */);

inline size_t sr_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
