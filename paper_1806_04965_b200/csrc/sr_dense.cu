// Dense resident engine: the frame update  x_v = sigma(b_v + sum_e W_e x_src(e))  (paper Sec. A1.2) of a small network
// whose edges are all dense, in fp32, for all T frames of a run in ONE launch.
//
// Such a network (the paper's H2 / O layers, a tiny MLP) moves a few hundred kilobytes of weights per frame and does a
// million multiply-adds: launched frame by frame it is pure launch latency.  Here a cluster of eight CTAs keeps ALL
// weights in shared memory, split by output rows, and walks the frames of eight sequences by itself:
//   - every CTA holds a full copy of every node state of its eight sequences (two buffers by frame parity; input
//     nodes three, because the next input frame is fetched with cp.async while the current update still reads the
//     previous one);
//   - a work unit is two output rows of one node; a warp takes a unit, its lanes stride over the reduction index with
//     16-byte loads (one weight vector per row, one state vector per sequence), shuffles sum the lanes (halving the
//     number of values per step), and the results (bias, ReLU) are written into the state copies of ALL eight CTAs
//     through distributed shared memory; warps never wait for each other inside a level.  (Measured alternatives:
//     eight-row jobs whose reduction index is split over warps, with partial sums through shared memory, need two
//     block-wide barriers per level and came out slower, 5.2 / 10.3 us per frame against 4.6 / 6.4 for the streaming /
//     sequential rollout of the 784-128-128-10 network.)
//   - a tableau level (Eq. 4) ends at a cluster barrier; a streaming frame has one.
// The sums run in a fixed order, so results are reproducible bit for bit.  There is no spin-wait: the only
// synchronisation is the hardware cluster barrier, reached by every thread the same number of times.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <vector>

#include "sr_dense.h"

namespace {

constexpr int kDnMaxNodes = 16, kDnMaxEdges = 32, kDnMaxLevels = 16, kDnMaxUnits = 64;
constexpr int kDnCluster = 8;          // CTAs per cluster
constexpr int kDnSamples = 8;          // sequences per cluster
constexpr int kDnWarps = 16;
constexpr int kDnSmemMax = 220 * 1024;

struct DnNode {
    float* gstate[2];                  // state buffers in global memory, [B][C], by frame parity
    const float* bias;
    int32_t C, Cpad, act, is_input, input_slot, is_output;
    int32_t buf[3];                    // float offsets of the shared-memory state buffers: frame f lives in buf[f % 3] (input
                                       // nodes) or buf[f & 1] (others)
    int32_t bias_off;                  // float offset of the node's bias copy in shared memory
};

struct DnEdge { int32_t src, tgt, R, Kpad; };

struct DnUnit { int32_t node, row0, nrows, rel_row; };      // two rows of a node; rel_row: row0 relative to the rank's first row

struct DnBlobHdr {                     // head of a rank's blob; the rank's weight slices follow
    int32_t n_units, pad_[3];
    int32_t level_begin[kDnMaxLevels + 1];                   // units of level l: [level_begin[l-1], level_begin[l])
    int32_t pad2_[3];
    int32_t w_off[kDnMaxEdges];                              // float offset of the rank's slice of every edge's weights
    DnUnit units[kDnMaxUnits];
};
static_assert(sizeof(DnBlobHdr) % 16 == 0, "the weights that follow are read with 16-byte loads");

struct DnParams {
    int32_t n_nodes, n_edges, n_levels, B;
    int32_t blob_bytes, hdr_floats, total_floats, pad_;
    const unsigned char* blobs;        // kDnCluster blobs of blob_bytes each
    DnNode nodes[kDnMaxNodes];
    DnEdge edges[kDnMaxEdges];
    int32_t first_edge[kDnMaxNodes + 1];                     // edges are sorted by target node
};

__device__ __forceinline__ void dn_cp_async16(void* dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void dn_cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void dn_st_cluster(const float* local, uint32_t rank, float v)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((uint32_t)__cvta_generic_to_shared(local)), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

// Fetch `n` floats (a multiple of 4, 16-byte aligned on both sides) with cp.async.
__device__ __forceinline__ void dn_fetch(float* dst, const float* src, int n, int tid, int nthr)
{
    for (int i = tid * 4; i < n; i += nthr * 4) dn_cp_async16(dst + i, src + i);
}

__global__ void __launch_bounds__(kDnWarps * 32, 1)
sr_dense_kernel(const DnParams P, SrFrameCtl* __restrict__ ctl_out, const SrFrameCtl init, int T)
{
    extern __shared__ __align__(16) float dn_smem[];
    const int tid = threadIdx.x, nthr = blockDim.x, warp = tid >> 5, lane = tid & 31;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int b0 = (int)(blockIdx.x / kDnCluster) * kDnSamples;
    const int nb = min(kDnSamples, P.B - b0);
    const DnBlobHdr* H = reinterpret_cast<const DnBlobHdr*>(dn_smem);
    const float* wsm = dn_smem + P.hdr_floats;

    // this rank's tables and weight slices, and zeros in every state buffer (padding columns and unused sequences stay zero)
    {
        const float* blob = reinterpret_cast<const float*>(P.blobs + (size_t)rank * P.blob_bytes);
        dn_fetch(dn_smem, blob, P.blob_bytes / 4, tid, nthr);
        for (int i = P.blob_bytes / 4 + tid; i < P.total_floats; i += nthr) dn_smem[i] = 0.f;
    }
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    // frame t of every node from the state buffers in global memory (relative frame 0)
    const long long t0 = init.t, run0 = init.run_t;
    const int par0 = (int)(t0 & 1);
    for (int v = 0; v < P.n_nodes; ++v) {
        const DnNode& nd = P.nodes[v];
        const float* gsrc = nd.gstate[par0] + (size_t)b0 * nd.C;
        float* dst = dn_smem + nd.buf[0];
        if (nd.Cpad == nd.C) dn_fetch(dst, gsrc, nb * nd.C, tid, nthr);                  // rows are contiguous: 16-byte copies
        else
            for (int i = tid; i < nb * nd.C; i += nthr) dst[(i / nd.C) * nd.Cpad + (i % nd.C)] = gsrc[i];
        if (!nd.is_input)
            for (int i = tid; i < nd.C; i += nthr) dn_smem[nd.bias_off + i] = nd.bias[i];
    }
    // relative frame 1 of the input nodes is on its way while the cluster assembles
    auto fetch_inputs = [&](int k) {
        for (int v = 0; v < P.n_nodes; ++v) {
            const DnNode& nd = P.nodes[v];
            if (!nd.is_input) continue;
            const float* src = reinterpret_cast<const float*>(static_cast<const char*>(init.in_base[nd.input_slot]) +
                                                               (run0 + k - 1) * init.in_stride_bytes[nd.input_slot]) + (size_t)b0 * nd.C;
            dn_fetch(dn_smem + nd.buf[k % 3], src, nb * nd.C, tid, nthr);     // input nodes have Cpad == C
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    fetch_inputs(1);
    dn_cluster_sync();                                       // every CTA of the cluster has its buffers in place before remote writes start

    for (int f = 0; f < T; ++f) {                            // relative frame f -> f + 1
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        if (f + 1 < T) fetch_inputs(f + 2);
        for (int l = 1; l <= P.n_levels; ++l) {
            for (int u = H->level_begin[l - 1] + warp; u < H->level_begin[l]; u += kDnWarps) {
                const DnUnit un = H->units[u];
                const DnNode& nd = P.nodes[un.node];
                float acc0[kDnSamples], acc1[kDnSamples];
#pragma unroll
                for (int b = 0; b < kDnSamples; ++b) acc0[b] = acc1[b] = 0.f;
                for (int e = P.first_edge[un.node]; e < P.first_edge[un.node + 1]; ++e) {
                    const DnEdge ed = P.edges[e];
                    const DnNode& sn = P.nodes[ed.src];
                    const int sf = f + 1 - ed.R;                                  // Eq. 2: the source frame
                    const float* xs = dn_smem + (sn.is_input ? sn.buf[sf % 3] : sn.buf[sf & 1]);
                    const float* w0 = wsm + H->w_off[e] + (size_t)un.rel_row * ed.Kpad;
                    const float* w1 = un.nrows > 1 ? w0 + ed.Kpad : w0;
                    for (int k = lane * 4; k < ed.Kpad; k += 128) {
                        const float4 a = *reinterpret_cast<const float4*>(w0 + k);
                        const float4 c = *reinterpret_cast<const float4*>(w1 + k);
#pragma unroll
                        for (int b = 0; b < kDnSamples; ++b) {
                            const float4 x = *reinterpret_cast<const float4*>(xs + b * sn.Cpad + k);
                            acc0[b] = fmaf(a.w, x.w, fmaf(a.z, x.z, fmaf(a.y, x.y, fmaf(a.x, x.x, acc0[b]))));
                            acc1[b] = fmaf(c.w, x.w, fmaf(c.z, x.z, fmaf(c.y, x.y, fmaf(c.x, x.x, acc1[b]))));
                        }
                    }
                }
                // Sum over the lanes by halving: in the step with distance d a lane keeps the half of its values that
                // matches its bit d and adds the partner's; after distances 16, 8, 4, 2 lane L holds value L >> 1
                // (row (L >> 4), sequence (L >> 1) & 7), and the step with distance 1 completes it in both lanes of a pair.
                float v8[8], v4[4], v2[2], v1;
                {
                    const bool up = (lane & 16) != 0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float keep = up ? acc1[j] : acc0[j], send = up ? acc0[j] : acc1[j];
                        v8[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
                    }
                }
                {
                    const bool up = (lane & 8) != 0;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float keep = up ? v8[j + 4] : v8[j], send = up ? v8[j] : v8[j + 4];
                        v4[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
                    }
                }
                {
                    const bool up = (lane & 4) != 0;
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const float keep = up ? v4[j + 2] : v4[j], send = up ? v4[j] : v4[j + 2];
                        v2[j] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
                    }
                }
                {
                    const bool up = (lane & 2) != 0;
                    const float keep = up ? v2[1] : v2[0], send = up ? v2[0] : v2[1];
                    v1 = keep + __shfl_xor_sync(0xffffffffu, send, 2);
                }
                v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
                const int r = lane >> 4, b = (lane >> 1) & 7;
                if (r < un.nrows) {
                    const int row = un.row0 + r;
                    float z = v1 + dn_smem[nd.bias_off + row];
                    if (nd.act == 1) z = fmaxf(z, 0.f);
                    const float* cell = dn_smem + nd.buf[(f + 1) & 1] + b * nd.Cpad + row;
                    const uint32_t q = (uint32_t)(lane & 1) * 4u;              // the two lanes of a pair serve four ranks each
#pragma unroll
                    for (uint32_t k = 0; k < 4; ++k) dn_st_cluster(cell, q + k, z);
                    if (nd.is_output && init.out_base && (lane & 1) == 0 && b < nb)
                        init.out_base[(run0 + f) * init.out_stride + (long long)(b0 + b) * nd.C + row] = z;
                }
            }
            dn_cluster_sync();                               // the level is complete in every CTA's copy
        }
    }

    if (blockIdx.x == 0 && tid == 0) {
        SrFrameCtl c = init;
        c.t += T;
        c.run_t += T;
        c.error = ctl_out->error;
        *ctl_out = c;
    }
    // relative frame T back to the state buffers in global memory (parity of t + T); rank 0 holds a full copy
    if (rank == 0) {
        const int parT = (int)((t0 + T) & 1);
        for (int v = 0; v < P.n_nodes; ++v) {
            const DnNode& nd = P.nodes[v];
            const float* src = dn_smem + (nd.is_input ? nd.buf[T % 3] : nd.buf[T & 1]);
            float* gdst = nd.gstate[parT] + (size_t)b0 * nd.C;
            if (nd.Cpad == nd.C)
                for (int i = tid * 4; i < nb * nd.C; i += nthr * 4) *reinterpret_cast<float4*>(gdst + i) = *reinterpret_cast<const float4*>(src + i);
            else
                for (int i = tid; i < nb * nd.C; i += nthr) gdst[i] = src[(i / nd.C) * nd.Cpad + (i % nd.C)];
        }
    }
}

// ------------------------------------------------------------------------------------------ host side
struct DnEngine {
    DnParams P{};
    std::vector<int> edge_of_host;                 // host edge -> index in P.edges
    std::vector<int> row_lo;                       // [node][rank] first row of the rank's slice, kDnCluster + 1 entries per node
    std::vector<std::vector<int>> w_off;           // [rank][edge]
    SrRegion r_blobs;
    int smem_bytes = 0;
    bool attr_set = false;
    std::vector<cudaEvent_t> ev;
    size_t ev_used = 0;
};

DnEngine* dn_of(const sr_graph* g) { return static_cast<DnEngine*>(g->dn); }

}  // namespace

void sr_dn_destroy(sr_graph* g)
{
    if (DnEngine* E = dn_of(g))
        for (cudaEvent_t e : E->ev) cudaEventDestroy(e);
    delete dn_of(g);
    g->dn = nullptr;
}

bool sr_dn_available(const sr_graph* g) { return g->dn != nullptr; }

void sr_dn_describe(const sr_graph* g, int* cluster_size, int* smem_bytes)
{
    const DnEngine* E = dn_of(g);
    *cluster_size = E ? kDnCluster : 0;
    *smem_bytes = E ? E->smem_bytes : 0;
}

// The engine applies to fp32 graphs in which every node is a vector (h = w = 1) and every edge dense, small enough for
// the shared memory of a cluster.  Rows of every node are split evenly over the ranks.
sr_status sr_dn_plan(sr_graph* g, size_t& offset)
{
    sr_dn_destroy(g);
    if (!g->opt_resident || g->opt_engine != 0 || g->dtype != SR_DTYPE_F32) return SR_OK;
    const int n_nodes = (int)g->nodes.size(), n_edges = (int)g->edges.size();
    if (n_nodes > kDnMaxNodes || n_edges > kDnMaxEdges || (int)g->groups.size() > kDnMaxLevels || g->groups.empty()) return SR_OK;
    if ((int)g->input_nodes.size() > SR_MAX_INPUTS) return SR_OK;
    for (const SrHostNode& n : g->nodes) {
        if (n.d.h != 1 || n.d.w != 1) return SR_OK;
        if (n.is_input && n.d.c % 4 != 0) return SR_OK;
    }
    for (const SrHostEdge& e : g->edges)
        if (e.d.kind == SR_EDGE_CONV) return SR_OK;
    DnEngine* E = new DnEngine();
    DnParams& P = E->P;
    P.n_nodes = n_nodes;
    P.n_edges = n_edges;
    P.n_levels = (int)g->groups.size();
    P.B = g->batch;
    // edges sorted by target
    E->edge_of_host.assign(n_edges, -1);
    int pos = 0;
    for (int v = 0; v < n_nodes; ++v) {
        P.first_edge[v] = pos;
        for (int e : g->nodes[v].in_edges) {
            const SrHostEdge& he = g->edges[e];
            const int Kpad = (g->nodes[he.d.src].d.c + 3) / 4 * 4;
            P.edges[pos] = DnEdge{he.d.src, he.d.tgt, he.R, Kpad};
            E->edge_of_host[e] = pos++;
        }
    }
    P.first_edge[n_nodes] = pos;
    // row slices and weight offsets per rank; units (two rows of a node each, longest reduction first inside a level)
    E->row_lo.assign((size_t)n_nodes * (kDnCluster + 1), 0);
    E->w_off.assign(kDnCluster, std::vector<int>(kDnMaxEdges, 0));
    int max_w = 0;
    std::vector<DnBlobHdr> hdrs(kDnCluster);
    for (int v = 0; v < n_nodes; ++v)
        for (int r = 0; r <= kDnCluster; ++r) E->row_lo[(size_t)v * (kDnCluster + 1) + r] = g->nodes[v].d.c * r / kDnCluster;
    for (int r = 0; r < kDnCluster; ++r) {
        DnBlobHdr& h = hdrs[r];
        std::memset(&h, 0, sizeof(h));
        int w = 0;
        for (int e = 0; e < n_edges; ++e) {
            const int v = P.edges[e].tgt;
            const int rows = E->row_lo[(size_t)v * (kDnCluster + 1) + r + 1] - E->row_lo[(size_t)v * (kDnCluster + 1) + r];
            E->w_off[r][e] = w;
            h.w_off[e] = w;
            w += rows * P.edges[e].Kpad;
        }
        max_w = std::max(max_w, w);
        int n_units = 0;
        bool fits = true;
        for (int l = 1; l <= P.n_levels && fits; ++l) {
            std::vector<std::pair<long long, DnUnit>> lv;
            for (int v : g->groups[l - 1]) {
                long long K = 0;
                for (int e = P.first_edge[v]; e < P.first_edge[v + 1]; ++e) K += P.edges[e].Kpad;
                const int lo = E->row_lo[(size_t)v * (kDnCluster + 1) + r], hi = E->row_lo[(size_t)v * (kDnCluster + 1) + r + 1];
                for (int row = lo; row < hi; row += 2) lv.push_back({K, DnUnit{v, row, std::min(2, hi - row), row - lo}});
            }
            std::stable_sort(lv.begin(), lv.end(), [](const auto& a, const auto& b) { return a.first > b.first; });
            for (auto& u : lv) {
                if (n_units >= kDnMaxUnits) { fits = false; break; }
                h.units[n_units++] = u.second;
            }
            h.level_begin[l] = n_units;
        }
        for (int l = P.n_levels + 1; l <= kDnMaxLevels; ++l) h.level_begin[l] = n_units;
        h.n_units = n_units;
        if (!fits) {
            delete E;
            return SR_OK;
        }
    }
    // shared-memory layout in floats: header, weights, state buffers
    int off = (int)(sizeof(DnBlobHdr) / 4);
    P.hdr_floats = off;
    off += (max_w + 3) / 4 * 4;
    P.blob_bytes = off * 4;
    for (int v = 0; v < n_nodes; ++v) {
        const SrHostNode& n = g->nodes[v];
        DnNode& d = P.nodes[v];
        d.C = n.d.c;
        d.Cpad = (n.d.c + 3) / 4 * 4;
        d.act = n.d.act;
        d.is_input = n.is_input ? 1 : 0;
        d.input_slot = n.input_slot;
        d.is_output = v == g->info.output_node ? 1 : 0;
        for (int i = 0; i < (n.is_input ? 3 : 2); ++i) {
            d.buf[i] = off;
            off += kDnSamples * d.Cpad;
        }
        d.bias_off = off;
        if (!n.is_input) off += d.Cpad;
    }
    P.total_floats = off;
    E->smem_bytes = off * 4;
    if (E->smem_bytes > kDnSmemMax) {
        delete E;
        return SR_OK;
    }
    E->r_blobs.offset = offset;
    E->r_blobs.bytes = (size_t)kDnCluster * P.blob_bytes;
    offset = sr_align_up(offset + E->r_blobs.bytes, 256);
    g->dn = E;
    // the per-rank table images; they go to the workspace when one is bound
    g->dn_headers.assign((size_t)kDnCluster * sizeof(DnBlobHdr), 0);
    for (int r = 0; r < kDnCluster; ++r) std::memcpy(g->dn_headers.data() + (size_t)r * sizeof(DnBlobHdr), &hdrs[r], sizeof(DnBlobHdr));
    return SR_OK;
}

sr_status sr_dn_bind(sr_graph* g)
{
    DnEngine* E = dn_of(g);
    if (!E) return SR_OK;
    DnParams& P = E->P;
    char* ws = g->ws;
    P.blobs = reinterpret_cast<const unsigned char*>(ws + E->r_blobs.offset);
    for (int v = 0; v < P.n_nodes; ++v) {
        const SrHostNode& n = g->nodes[v];
        P.nodes[v].gstate[0] = reinterpret_cast<float*>(ws + n.state[0].offset);
        P.nodes[v].gstate[1] = reinterpret_cast<float*>(ws + n.state[1].offset);
        P.nodes[v].bias = reinterpret_cast<const float*>(ws + n.bias.offset);
    }
    // the workspace was zeroed by the caller of bind: weights start at zero, headers go in now
    for (int r = 0; r < kDnCluster; ++r)
        if (cudaMemcpy(ws + E->r_blobs.offset + (size_t)r * P.blob_bytes, g->dn_headers.data() + (size_t)r * sizeof(DnBlobHdr),
                       sizeof(DnBlobHdr), cudaMemcpyHostToDevice) != cudaSuccess)
            return SR_ERR_CUDA;
    return SR_OK;
}

sr_status sr_dn_set_weights(sr_graph* g, int edge, const float* w)
{
    DnEngine* E = dn_of(g);
    if (!E) return SR_OK;
    const DnParams& P = E->P;
    const int e = E->edge_of_host[edge];
    const SrHostEdge& he = g->edges[edge];
    const int v = he.d.tgt, K = he.K, Kpad = P.edges[e].Kpad;
    for (int r = 0; r < kDnCluster; ++r) {
        const int lo = E->row_lo[(size_t)v * (kDnCluster + 1) + r], hi = E->row_lo[(size_t)v * (kDnCluster + 1) + r + 1];
        if (hi <= lo) continue;
        std::vector<float> h((size_t)(hi - lo) * Kpad, 0.f);
        for (int row = lo; row < hi; ++row)
            std::memcpy(&h[(size_t)(row - lo) * Kpad], w + (size_t)row * K, sizeof(float) * K);
        char* dst = g->ws + E->r_blobs.offset + (size_t)r * P.blob_bytes + sizeof(DnBlobHdr) + (size_t)E->w_off[r][e] * 4;
        if (cudaMemcpy(dst, h.data(), h.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) return SR_ERR_CUDA;
    }
    return SR_OK;
}

sr_status sr_dn_launch(sr_graph* g, int T, const SrFrameCtl& init, cudaStream_t s)
{
    DnEngine* E = dn_of(g);
    if (!E) return SR_ERR_STATE;
    if (!E->attr_set) {
        if (cudaFuncSetAttribute(sr_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, E->smem_bytes) != cudaSuccess) return SR_ERR_CUDA;
        E->attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)((g->batch + kDnSamples - 1) / kDnSamples * kDnCluster));
    cfg.blockDim = dim3((unsigned)(kDnWarps * 32));
    cfg.dynamicSmemBytes = (size_t)E->smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)kDnCluster;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    SrFrameCtl* ctl = reinterpret_cast<SrFrameCtl*>(g->ws + g->r_ctl.offset);
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    bool timed = g->opt_time_tc != 0 && cudaStreamIsCapturing(s, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone;
    if (timed && E->ev_used + 2 > E->ev.size()) {
        if (E->ev.size() >= 4096) timed = false;
        for (int i = 0; timed && i < 2; ++i) {
            cudaEvent_t e = nullptr;
            if (cudaEventCreate(&e) != cudaSuccess) timed = false;
            else E->ev.push_back(e);
        }
        if (E->ev_used + 2 > E->ev.size()) timed = false;
    }
    if (timed) cudaEventRecord(E->ev[E->ev_used], s);
    if (cudaLaunchKernelEx(&cfg, sr_dense_kernel, E->P, ctl, init, T) != cudaSuccess) return SR_ERR_CUDA;
    if (timed) {
        cudaEventRecord(E->ev[E->ev_used + 1], s);
        E->ev_used += 2;
    }
    return SR_OK;
}

sr_status sr_dn_timing(sr_graph* g, double* ms, long long* launches)
{
    DnEngine* E = dn_of(g);
    *ms = 0.0;
    *launches = 0;
    if (!E) return SR_OK;
    for (size_t i = 0; i + 1 < E->ev_used; i += 2) {
        if (cudaEventSynchronize(E->ev[i + 1]) != cudaSuccess) return SR_ERR_CUDA;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, E->ev[i], E->ev[i + 1]) != cudaSuccess) return SR_ERR_CUDA;
        *ms += t;
        *launches += 1;
    }
    E->ev_used = 0;
    return SR_OK;
}
