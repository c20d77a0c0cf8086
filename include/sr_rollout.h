/*
 * sr_rollout.h - C ABI of the streaming-rollout frame-update library (CUDA, sm_100a).
 *
 * The objects are the paper's (arXiv 1806.04965):
 *   - a network is a directed, input-connected graph N = (V, E) with 0 < |E|
 *     (Sec. 3, Definition "network"); nodes are layers, edges are transformations;
 *   - a rollout pattern is a map R : E -> {0, 1}; R(e) = 1 lets edge e bridge one
 *     frame ("stream"), R(e) = 0 keeps it inside a frame (Sec. 3, Definition
 *     "rollout pattern and window", Eq. 2); R is valid iff its rollout window is acyclic;
 *   - the streaming rollout is R = 1 on every edge; patterns that agree with it on
 *     all edges not leaving an input node update a whole frame in ONE step
 *     (Theorem 1 a <=> b), i.e. in one launch group;
 *   - a node is updated as  x_v = sigma( b_v + sum_{e in SRC_v} f_e(theta_e, x_src(e)) )
 *     (Sec. A1.2), where the source state is taken from frame t+1-R(e) (Eq. 2);
 *   - inference chains rollout windows of size W = 1: frame 1 of a window becomes
 *     frame 0 of the next (Sec. 4 and Sec. 5), so two state buffers per node suffice.
 *
 * Conventions of every call
 *   - returns an sr_status; never throws, never aborts; out-parameters are left
 *     untouched on error;
 *   - pointers named *_dev are DEVICE pointers, *_host are HOST pointers; the
 *     caller owns every buffer it passes and keeps it alive until the work queued
 *     on `stream` has finished;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream);
 *     reset / step / run / get_state / set_state are asynchronous on that stream;
 *   - the library allocates no device memory: the caller provides one workspace
 *     (sr_graph_workspace_bytes / sr_graph_bind_workspace) in which the library
 *     places states, packed weights, biases and its launch tables;
 *   - layouts: state / frame [B][H][W][C]; conv weight [C_out][k][k][C_in]; dense
 *     weight [C_out][H][W][C_in] (source flattened in H, W, C order); mean-dense
 *     weight [C_out][C_in]; bias [C];
 *   - element type of states and input frames: float (dtype 0) or bfloat16 bit
 *     patterns (dtype 1).  Weights and biases are always passed as float; in
 *     bfloat16 mode weights are rounded to bfloat16 (nearest even) when stored.
 *     Outputs (`out_dev`, `out_seq_dev`) are always float and have the output node's full shape,
 *     [B][H][W][C] per frame ([B][C] for a dense output node, whose H = W = 1).
 */
#ifndef SR_ROLLOUT_H
#define SR_ROLLOUT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sr_graph sr_graph;          /* opaque; owned by the library */

typedef enum {
    SR_OK = 0,
    SR_ERR_INVALID_ARG = 1,        /* null pointer, index out of range, bad size                      */
    SR_ERR_NOT_A_NETWORK = 2,      /* |E| = 0 or not input-connected (Sec. 3, Definition "network")   */
    SR_ERR_INVALID_ROLLOUT = 3,    /* the rollout window of R has a cycle (Sec. 3, validity)          */
    SR_ERR_SHAPE_MISMATCH = 4,     /* an edge does not map its source shape to its target shape       */
    SR_ERR_UNSUPPORTED = 5,        /* a combination this library does not implement                   */
    SR_ERR_CUDA = 6,               /* a CUDA runtime or driver call failed                            */
    SR_ERR_TIMEOUT = 7,            /* a bounded device-side wait expired                              */
    SR_ERR_STATE = 8,              /* call order: workspace not bound, weights missing, ...           */
    SR_ERR_TOO_LARGE = 9           /* the graph needs more than the built-in workspace holds          */
} sr_status;

/* A node (layer).  Dense nodes have h = w = 1.  act: 0 identity, 1 ReLU (the sigma of Sec. A1.2).
 * Whether a node is an input is derived: it has no incoming edge (Eq. 1). */
typedef struct { int32_t h, w, c, act; } sr_node_desc;

/* An edge (transformation f_e, Sec. A1.2).
 *   kind 0  convolution (cross-correlation) k x k, stride `stride`, zero padding (k-1)/2 on every side,
 *           output size floor((n + 2p - k)/stride) + 1; pool = 2 appends a 2x2 stride-2 average, 0 none;
 *   kind 1  dense over the flattened source;
 *   kind 2  mean over h, w of the source followed by dense over channels. */
typedef struct { int32_t src, tgt, kind, k, stride, pool; } sr_edge_desc;

enum { SR_EDGE_CONV = 0, SR_EDGE_DENSE = 1, SR_EDGE_MEAN_DENSE = 2 };
enum { SR_DTYPE_F32 = 0, SR_DTYPE_BF16 = 1 };

/* Rollout-theory quantities of a compiled graph (all integers, exact). */
typedef struct {
    int32_t n_nodes, n_edges, n_inputs;
    int32_t inference_factor;          /* F(R), Eq. 5 = number of launch groups per frame                */
    int32_t n_groups;                  /* same number; kept separate for readability at call sites        */
    int32_t streaming_parallel;        /* 1 iff R equals the streaming rollout on all edges that do not
                                          leave an input node (Theorem 1 a), which is iff F(R) = 1        */
    int32_t output_node;               /* the node whose state is copied to `out`: the highest-index node
                                          without an outgoing edge to another node (else the last node)   */
    int32_t first_response_frame;      /* first frame whose output depends on an input, windows of size 1
                                          chained (Sec. 4); -1 if the output never depends on an input    */
    int32_t first_response_step;       /* (first_response_frame - 1) * F(R) + level(output_node)          */
    int32_t response_interval;         /* update steps between outputs = F(R) (Sec. 4)                    */
    int32_t n_tensor_core_nodes;       /* nodes updated by the tcgen05 implicit-GEMM kernel               */
    int32_t n_direct_nodes;            /* nodes updated by the CUDA-core kernels                          */
    int32_t resident_cluster;          /* CTAs per sequence of the shared-memory-resident kernel that
                                          sr_rollout_run uses for this graph; 0 = it does not apply       */
    int32_t resident_smem_bytes;       /* shared memory per CTA of that kernel                            */
    int32_t resident_heads_on_chip;    /* 1 if the dense / mean-dense weights are resident as well, 0 if they
                                          are read from global memory every frame                         */
} sr_info;

/*
 * Compile a network and a rollout pattern (Sec. 3).  Validates the graph (network definition, edge
 * shapes) and the pattern (acyclic rollout window), computes the inference tableau of the window of
 * size 1 (Eq. 4): level(v) = T((1, v)), and from it the launch groups of a frame: group l holds the
 * nodes with level l, l = 1..F(R).  Pure host work; needs no GPU.
 *   nodes, edges : host arrays, copied.      R : host array, n_edges entries, each 0 or 1.
 *   batch        : B >= 1, or 0 for a theory-only graph (info and levels only; no device calls allowed).
 *   dtype        : SR_DTYPE_F32 or SR_DTYPE_BF16.
 * Errors: INVALID_ARG, NOT_A_NETWORK, SHAPE_MISMATCH, INVALID_ROLLOUT, UNSUPPORTED.
 */
sr_status sr_graph_create(const sr_node_desc* nodes, int n_nodes, const sr_edge_desc* edges, int n_edges,
                          const uint8_t* R, int batch, int dtype, sr_graph** out);
void sr_graph_destroy(sr_graph* g);

sr_status sr_graph_info(const sr_graph* g, sr_info* out);
/* level[v] = T_{R_1}((1, v)) (Eq. 4): 0 for input nodes, else the update step inside a frame. */
sr_status sr_graph_levels(const sr_graph* g, int32_t* level_host /* n_nodes */);

/* Bytes of device memory the graph needs; the caller allocates them (256-byte aligned) and binds them.
 * Binding uploads the launch tables (synchronous copies) and zeroes the states. */
sr_status sr_graph_workspace_bytes(const sr_graph* g, size_t* bytes);
sr_status sr_graph_bind_workspace(sr_graph* g, void* workspace_dev, size_t bytes);

/*
 * Bind the library's built-in workspace instead of a caller-allocated one.  (The paper has no
 * counterpart; this exists for deployment.)
 *
 * Who needs it: code that is not allowed to allocate device memory at the point where it sets a graph
 * up - a plugin that runs inside a host application's real-time or stream-ordered section, a process
 * whose memory pool is owned and sized by another component, a late start-up phase after the device
 * has been handed over fully committed.  Such a caller cannot produce the buffer that
 * sr_graph_bind_workspace wants.  This call needs none: the workspace is a fixed array of
 * SR_STATIC_WORKSPACE_BYTES that lives in the library's device image, so every GPU that loads the
 * library holds that much memory until the process exits, whether or not this call is ever made.
 *
 * Behaviour
 *   - allocates no device memory (no cudaMalloc / cudaFree, no allocating library call); inputs and
 *     outputs are still the caller's buffers, passed to reset / step / run as before.  Host-side objects are
 *     still created later, as for any graph: the first step / run creates a stream and two events, and
 *     sr_rollout_run with CUDA graphs enabled instantiates a graph;
 *   - the first call on a device looks the array's address up for that device (the device must be
 *     current) and remembers it; make that first call before any stream capture begins;
 *   - a graph whose sr_graph_workspace_bytes exceeds SR_STATIC_WORKSPACE_BYTES is refused with
 *     SR_ERR_TOO_LARGE and stays unbound;
 *   - all graphs bound this way share the one array.  It still holds what the previous user left, so
 *     binding clears the part the new graph uses (states start at zero) and parameters must be set
 *     again.  Only one such graph may be in use at a time: work of two graphs bound to the built-in
 *     workspace that overlaps on the GPU (different streams, or a new bind while an older graph's work
 *     is still queued) races on the same memory.  Synchronise before handing the array to the next graph;
 *   - the array has one owner per device, the graph that bound it last.  A new bind takes it away from the
 *     previous owner, which becomes unbound: its reset / step / run / get_state / set_state / parameter calls
 *     return SR_ERR_STATE until it is bound again (to either kind of workspace) and given its parameters
 *     again.  Concurrent binds from several host threads are serialised by the library.
 * Otherwise identical to sr_graph_bind_workspace: same kernels, same results.
 * Errors: INVALID_ARG, STATE (already bound, or theory-only graph), TOO_LARGE, CUDA.
 */
#define SR_STATIC_WORKSPACE_BYTES (32u * 1024u * 1024u)
sr_status sr_graph_bind_static_workspace(sr_graph* g);

/* Parameters theta_e and b_v (Sec. A1.2).  `w` holds floats in the layout given above, on the host
 * (is_device = 0) or on the device (is_device = 1).  Synchronous.  Needs a bound workspace. */
sr_status sr_graph_set_edge_weights(sr_graph* g, int edge, const float* w, int is_device);
sr_status sr_graph_set_node_bias(sr_graph* g, int node, const float* bias_host);

/* Options.  key 0 "engine": 0 = tensor cores where a node qualifies (default), 1 = CUDA-core kernels only.
 *           key 1 "frames per CUDA graph" used by sr_rollout_run: 0 = plain launches, n >= 1 = graphs
 *                  of n frames (default 0).
 *           key 2 "weight ring": weight boxes the tensor-core kernel keeps in flight in shared memory
 *                  (2..8; 0 = default); the rest of the shared memory holds activation boxes.
 *           key 3 "tile width": width in pixels (8, 16 or 32; 0 = default) of the 128-pixel output tiles of
 *                  nodes that have a stride-1 k x k incoming edge (narrow tiles reload less halo, wide
 *                  tiles read longer contiguous runs).
 *           key 4 "overlap": 1 (default) runs independent launches of a frame on a second, library-owned
 *                  stream (the CUDA-core and the tensor-core kernel of a group; the next frame's input
 *                  copy when no input edge has R = 0), joined before the frame ends; 0 = one stream.
 *           key 5 "kernel timing": 1 brackets every tensor-core group launch and every resident launch with CUDA
 *                  events on the launching stream (plain launches only, not inside CUDA graphs); read with
 *                  sr_graph_kernel_time.
 *           key 6 "resident": 1 (default) lets sr_rollout_run use the resident kernel when the network qualifies
 *                  (bfloat16; per-sequence states and convolution weights fit in the shared memory of a
 *                  thread-block cluster): one cluster per sequence walks all T frames in one launch with
 *                  the states on chip; 0 = always the per-frame launch path.  sr_rollout_step always uses
 *                  the launch path.
 *           key 7 "resident cluster size": CTAs per sequence, 1, 2 or 4; 0 (default) = chosen by the library.
 *           key 8 "resident warps": warps per CTA of the resident kernel, 4..32; 0 = default.
 *           key 9 "resident tile width": 0 (default) = 16-pixel x 32-channel work units only, 1 = 16-channel units for
 *                  every convolutional node, 2 = 16-channel units for the nodes whose 32-channel unit would be the
 *                  longest dependent chain of a frame (more, shorter units; they load the activations twice).
 *           key 10 "device wait limit": milliseconds (1..60000, default 1000) after which a wait inside a kernel (on a
 *                  shared-memory barrier, on a descriptor queue) gives up; the kernel then records an error, waits
 *                  for its own copies in flight, frees its tensor memory and returns, and sr_graph_sync_status
 *                  reports SR_ERR_TIMEOUT.  0 is a test hook: every tensor-core launch reports the error at once and
 *                  returns before it touches a barrier, a copy or an MMA.  May be set at any time.
 *           key 11 "tile pairs": the tensor-core kernel's work item is a pair of neighbouring pixel tiles that share every
 *                  weight box (half the weight traffic, twice the work per item).  0 (default) and 1 = single tiles,
 *                  2 = pairs wherever the geometry allows.
 *           key 12 "staged boxes in the weight ring": the activation box of a staged few-channel input edge (two MMAs'
 *                  worth of work) is fetched into the tensor-core kernel's weight ring together with its weights, so
 *                  that it does not hold one of the few large activation slots.  1 (default) = in launch groups whose
 *                  weight ring has at least four slots, 2 = wherever the box fits a weight slot, 0 = never.
 *           key 13 "work lists": how the tensor-core kernel's persistent CTAs get their work items.  1 = one list per
 *                  CTA, balanced on the host by estimated cost; 0 (default) = the same for the larger items, while
 *                  the smallest ones (a fifth of the work of a launch with many items) form one shared list that
 *                  every CTA takes from when its own list is done (a device-wide counter).
 *           key 14 "fused nodes": 1 (default) = two convolutional nodes of one launch group that have the same shape,
 *                  at most 64 channels (a multiple of 32) each and an incoming edge from the same source with the
 *                  same filter geometry and the same R (or of which one has two K-blocks of reduction at most)
 *                  run as ONE tensor-core work item per pixel tile: the second
 *                  node's weights fill the otherwise empty rows 64..127 of the M = 128 instruction, and the shared
 *                  source is read and multiplied once for both.  0 = every node on its own.  Results are identical.
 * Must be set before sr_graph_workspace_bytes / sr_graph_bind_workspace (engine, weight ring, tile width, tile pairs,
 * staged boxes, work lists, fused nodes, resident keys) / before the first run (graphs). */
sr_status sr_graph_set_option(sr_graph* g, int key, int value);

/*
 * Frame 0 (Sec. A "Training details", Eq. 3): every non-input state := 0; input node i := in0_dev[i]
 * (one device pointer per input node, in increasing node order, each [B][H][W][C] of the graph dtype).
 * The frame counter returns to 0 and a device-side error recorded earlier (SR_ERR_TIMEOUT) is cleared.
 */
sr_status sr_graph_reset(sr_graph* g, const void* const* in0_dev, void* stream);

/*
 * One frame update t -> t+1 (Sec. 4: one chained window of size 1): input nodes take the caller's
 * frame t+1; then, group by group, every node v of the group gets
 *     x_v^{t+1} = sigma_v( b_v + sum_e f_e(theta_e, x_src(e)^{t+1-R(e)}) )
 * and the buffers flip.  A streaming pattern runs ONE group.  If out_dev is not NULL it receives the
 * output node's new state as float [B][H][W][C_out] ([B][C_out] for a dense output node).
 */
sr_status sr_rollout_step(sr_graph* g, const void* const* in_next_dev, float* out_dev, void* stream);

/*
 * T frame updates without host round trips in between: in_seq_dev[i] points to the T frames
 * t+1..t+T of input node i, [T][B][H][W][C]; out_seq_dev (may be NULL) receives T frames of the output node's
 * shape, [T][B][H][W][C_out] floats.
 * Equivalent to T calls of sr_rollout_step.
 */
sr_status sr_rollout_run(sr_graph* g, const void* const* in_seq_dev, int T, float* out_seq_dev, void* stream);

/*
 * Deep rollout windows, W > 1 (Sec. 3, Definition "rollout pattern and window", Eq. 2; inference tableau, Eq. 4).
 *
 * sr_graph_window_tableau: T((i, v)) of the window of size W for i = 0..W, row-major [W + 1][n_nodes] on the host: the
 * update step at which node v of frame i becomes computable when the whole window is evaluated at once (0 for frame
 * 0 and for input nodes).  All nodes with the same value form one update step.  Pure host work; any valid pattern.
 *
 * sr_rollout_window: evaluates the W frame updates t+1 .. t+W as ONE window instead of W chained windows of size 1.
 * Implemented for patterns whose frames do not depend on each other - every edge that bridges a frame leaves an
 * input node (e.g. the sequential rollout of a network without recurrence) -, where T((i, v)) = level(v) for every
 * frame i: level by level, the nodes of ALL W frames are updated in one launch group over a batch of W * B samples
 * (the equal-compute comparison of Sec. 4, where a deep window classifies its first frames side by side).  Other patterns
 * return SR_ERR_UNSUPPORTED.  in_seq_dev / out_seq_dev as for sr_rollout_run; afterwards the graph stands at frame
 * t + W and can be stepped on.  Results equal those of W calls of sr_rollout_step.
 * The window needs a workspace of its own (states of all W frames): ask for its size, allocate, bind; binding copies
 * the parameters set so far, so set weights and biases first (later changes do not reach the window).
 * Errors: INVALID_ARG, STATE (not bound, parameters missing, other W than bound), UNSUPPORTED, CUDA.
 */
sr_status sr_graph_window_tableau(const sr_graph* g, int W, int32_t* T_host);
sr_status sr_graph_window_workspace_bytes(sr_graph* g, int W, size_t* bytes);
sr_status sr_graph_bind_window(sr_graph* g, int W, void* workspace_dev, size_t bytes);
sr_status sr_rollout_window(sr_graph* g, const void* const* in_seq_dev, int W, float* out_seq_dev, void* stream);

/* Copy the current (frame t) state of a node out of / into the graph, [B][H][W][C] of the graph dtype.
 * Restoring all states and continuing to step resumes a rollout (Sec. 5: the next window starts
 * from the last frame of the previous one). */
sr_status sr_graph_get_state(const sr_graph* g, int node, void* dst_dev, void* stream);
sr_status sr_graph_set_state(sr_graph* g, int node, const void* src_dev, void* stream);

/* Frames computed since the last reset (host-side count of queued updates). */
sr_status sr_graph_frame(const sr_graph* g, int64_t* t);
/* Kernels launched by this graph so far (counts launches inside replayed CUDA graphs as well). */
sr_status sr_graph_launch_count(const sr_graph* g, int64_t* n);
/* Sum of the event-timed durations (milliseconds) and the number of tensor-core group launches and resident
 * launches since the previous call (option key 5); waits for those launches to finish. */
sr_status sr_graph_kernel_time(sr_graph* g, double* ms, int64_t* launches);
/* Synchronises `stream` and reports SR_ERR_CUDA / SR_ERR_TIMEOUT if queued work failed.  A recorded time-out stays
 * recorded, and is reported by every later call, until sr_graph_reset starts the rollout over. */
sr_status sr_graph_sync_status(sr_graph* g, void* stream);

const char* sr_status_str(sr_status s);

#ifdef __cplusplus
}
#endif
#endif /* SR_ROLLOUT_H */
