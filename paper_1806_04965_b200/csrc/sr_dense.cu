// Dense resident engine: the frame update  x_v = sigma(b_v + sum_e W_e x_src(e))  (paper Sec. A1.2) of a small network
// whose edges are all dense, in fp32, for all T frames of a run in ONE launch.
//
// Such a network (the paper's H2 / O layers, a tiny MLP) moves a few hundred kilobytes of weights per frame and does a
// million multiply-adds: launched frame by frame it is pure launch latency.  Here a cluster of eight or sixteen CTAs
// keeps ALL weights in shared memory, split by output rows, and walks the frames of eight sequences by itself:
//   - every CTA holds a full copy of every node state of its eight sequences (two buffers by frame parity; input
//     nodes three, because the next input frame is fetched with cp.async while the current update still reads the
//     previous one);
//   - a work unit is up to four output rows of one node; a warp takes a unit, its lanes stride over the reduction
//     index with 16-byte loads (one weight vector per row, one state vector per sequence: 12 loads feed 128
//     multiply-adds; what bounds a frame is the shared-memory bandwidth, and two-row units needed 10 loads per 64),
//     shuffles sum the lanes (halving the number of values per step until a group of four lanes holds the four
//     rows of one sequence), and the results (bias, ReLU) are written as one 16-byte word into the state copies of
//     ALL CTAs of the cluster through distributed shared memory; warps never wait for each other inside a level.
//     (Measured alternatives, both slower: eight-row jobs whose reduction index is split over warps with two
//     block-wide barriers per level; four-row units cut along the reduction index into parts on up to fourteen warps
//     that hand their partial sums to the unit's first part through shared memory and a named barrier, 3.1 against
//     2.8 us per frame: the shared-memory traffic stays the same and every part pays the reduction over the lanes.)
//   - units are given to the warps longest first (host side); the warps left without a unit in the first level fetch
//     the next input frame;
//   - a tableau level (Eq. 4) ends at a cluster barrier; a streaming frame has one.
// The sums run in a fixed order, so results are reproducible bit for bit.  There is no spin-wait: the only
// synchronisation is the hardware cluster barrier, reached by every thread the same number of times.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstddef>
#include <cstring>
#include <vector>

#include "sr_dense.h"

namespace {

constexpr int kDnMaxNodes = 16, kDnMaxEdges = 32, kDnMaxLevels = 16, kDnMaxUnits = 128;
constexpr int kDnMaxCluster = 16;      // CTAs per cluster: 8, or 16 (a non-portable size) for rollouts with one level per frame
constexpr int kDnSamples = 8;          // sequences per cluster
constexpr int kDnWarps = 16;
constexpr int kDnRows = 4;             // output rows per work unit
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

// One incoming edge of a work unit, ready to use (32 bytes): where the unit's weight rows start (floats from the
// rank's first weight), the padded reduction length = row pitch of the weights, the row pitch of the source state,
// the frames the edge looks back (Eq. 2), and the source's shared-memory buffers (three for an input node).
struct DnTerm { int32_t w_off, Kpad, xp, R, n_buf, buf[3]; };
static_assert(sizeof(DnTerm) == 32, "read as two 16-byte words");

// Up to four rows of a node with everything a warp needs (48 bytes).  nrows = 0: no unit (a gap in a warp's list).
struct DnUnit {
    int32_t nrows, row0, term0, n_terms;
    int32_t bias_off, Cpad, C, flags;                        // flags: 1 = ReLU, 2 = the output node
    int32_t buf[2], pad_[2];                                 // the node's two shared-memory buffers by frame parity
};
static_assert(sizeof(DnUnit) == 48, "read as three 16-byte words");

constexpr int kDnMaxTerms = 256;

struct DnBlobHdr {                     // head of a rank's blob; the rank's weight slices follow
    int32_t n_units, fetch_warp0, pad_[2];                   // fetch_warp0: first of the warps that fetch input frames
    int32_t level_begin[kDnMaxLevels + 1];                   // units of level l: [level_begin[l-1], level_begin[l]); warp w
    int32_t pad2_[3];                                        // takes entries w, w + 16, ... of a level
    DnUnit units[kDnMaxUnits];
    DnTerm terms[kDnMaxTerms];
};
static_assert(sizeof(DnBlobHdr) % 16 == 0, "the weights that follow are read with 16-byte loads");
static_assert(offsetof(DnBlobHdr, units) % 16 == 0 && offsetof(DnBlobHdr, terms) % 16 == 0, "tables are read with 16-byte loads");

struct DnParams {
    int32_t n_nodes, n_edges, n_levels, B;
    int32_t blob_bytes, hdr_floats, total_floats, pad_;
    const unsigned char* blobs;        // one blob of blob_bytes per rank of the cluster
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
__device__ __forceinline__ uint32_t dn_map_rank(const float* local, uint32_t rank)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((uint32_t)__cvta_generic_to_shared(local)), "r"(rank));
    return remote;
}
__device__ __forceinline__ void dn_st_cluster(const float* local, uint32_t rank, float v)
{
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(dn_map_rank(local, rank)), "f"(v) : "memory");
}
__device__ __forceinline__ void dn_st_cluster4(const float* local, uint32_t rank, const float (&v)[4])
{
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dn_map_rank(local, rank)), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]) : "memory");
}

// Fetch `n` floats (a multiple of 4, 16-byte aligned on both sides) with cp.async.
__device__ __forceinline__ void dn_fetch(float* dst, const float* src, int n, int tid, int nthr)
{
    for (int i = tid * 4; i < n; i += nthr * 4) dn_cp_async16(dst + i, src + i);
}

// acc[r][b0 + b] += a[r] . x[b] for four sequences, the four components of the vectors added in the order x, y, z, w.
// Written component by component so that consecutive multiply-adds are independent of each other.
template <int R>
__device__ __forceinline__ void dn_fma4(float (&acc)[R][kDnSamples], const float4 (&a)[R], const float4 (&x)[4], int b0)
{
#pragma unroll
    for (int b = 0; b < 4; ++b)
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r][b0 + b] = fmaf(a[r].x, x[b].x, acc[r][b0 + b]);
#pragma unroll
    for (int b = 0; b < 4; ++b)
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r][b0 + b] = fmaf(a[r].y, x[b].y, acc[r][b0 + b]);
#pragma unroll
    for (int b = 0; b < 4; ++b)
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r][b0 + b] = fmaf(a[r].z, x[b].z, acc[r][b0 + b]);
#pragma unroll
    for (int b = 0; b < 4; ++b)
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r][b0 + b] = fmaf(a[r].w, x[b].w, acc[r][b0 + b]);
}

// One work unit: up to R rows of a node for the eight sequences of the cluster, relative frame f -> f + 1.
// The loads of a reduction step are issued ahead of the multiply-adds that use them: the weights and the first four
// sequences of step i + 1 while the last four sequences of step i are still being multiplied.
template <int R, int CL>
__device__ __forceinline__ void dn_unit(const DnBlobHdr* H, const DnUnit& un, float* dn_smem, const float* wsm,
                                        const SrFrameCtl& init, int f, int lane, int b0, int nb, long long run0)
{
    float acc[R][kDnSamples];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int b = 0; b < kDnSamples; ++b) acc[r][b] = 0.f;
    for (int ti = un.term0; ti < un.term0 + un.n_terms; ++ti) {
        const DnTerm tm = H->terms[ti];
        const int sf = f + 1 - tm.R;                                  // Eq. 2: the source frame
        const int bi = tm.n_buf == 3 ? sf % 3 : (sf & 1);
        const float* xs = dn_smem + (bi == 0 ? tm.buf[0] : (bi == 1 ? tm.buf[1] : tm.buf[2])) + lane * 4;
        const float* w0 = wsm + tm.w_off + lane * 4;
        int ro[R];                                                    // rows the unit does not have repeat row 0 (their sums are dropped)
#pragma unroll
        for (int r = 0; r < R; ++r) ro[r] = r < un.nrows ? r * tm.Kpad : 0;
        const int xp = tm.xp, n_k = tm.Kpad - lane * 4;               // this lane's steps: k = 0, 128, ... < n_k
        if (n_k <= 0) continue;
        float4 a[R], xa[4], xb[4];
#pragma unroll
        for (int r = 0; r < R; ++r) a[r] = *reinterpret_cast<const float4*>(w0 + ro[r]);
#pragma unroll
        for (int b = 0; b < 4; ++b) xa[b] = *reinterpret_cast<const float4*>(xs + b * xp);
        for (int k = 0; k < n_k; k += 128) {
#pragma unroll
            for (int b = 0; b < 4; ++b) xb[b] = *reinterpret_cast<const float4*>(xs + (b + 4) * xp + k);
            dn_fma4<R>(acc, a, xa, 0);
            float4 an[R];
            const int kn = k + 128 < n_k ? k + 128 : k;               // the last step re-reads itself (no branch)
#pragma unroll
            for (int r = 0; r < R; ++r) an[r] = *reinterpret_cast<const float4*>(w0 + ro[r] + kn);
#pragma unroll
            for (int b = 0; b < 4; ++b) xa[b] = *reinterpret_cast<const float4*>(xs + b * xp + kn);
            dn_fma4<R>(acc, a, xb, 4);
#pragma unroll
            for (int r = 0; r < R; ++r) a[r] = an[r];
        }
    }
    // Sum over the lanes by halving: in the step with distance d a lane keeps the half of its sequences that matches
    // its bit d and adds the partner's; after distances 16, 8 and 4 lane L holds the R rows of sequence L >> 2, summed
    // over the lanes that share L's two low bits; distances 2 and 1 complete the sums in all four lanes of a group.
    float v16[R][4], v8[R][2], z[R];
    {
        const bool up = (lane & 16) != 0;
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float keep = up ? acc[r][j + 4] : acc[r][j], send = up ? acc[r][j] : acc[r][j + 4];
                v16[r][j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
            }
    }
    {
        const bool up = (lane & 8) != 0;
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const float keep = up ? v16[r][j + 2] : v16[r][j], send = up ? v16[r][j] : v16[r][j + 2];
                v8[r][j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
            }
    }
    {
        const bool up = (lane & 4) != 0;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float keep = up ? v8[r][1] : v8[r][0], send = up ? v8[r][0] : v8[r][1];
            z[r] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) z[r] += __shfl_xor_sync(0xffffffffu, z[r], 2);
#pragma unroll
    for (int r = 0; r < R; ++r) z[r] += __shfl_xor_sync(0xffffffffu, z[r], 1);
    const int b = lane >> 2;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        z[r] += dn_smem[un.bias_off + un.row0 + (r < un.nrows ? r : 0)];
        if (un.flags & 1) z[r] = fmaxf(z[r], 0.f);
    }
    const float* cell = dn_smem + (((f + 1) & 1) ? un.buf[1] : un.buf[0]) + b * un.Cpad + un.row0;
    constexpr uint32_t kPerLane = CL / 4;                             // the four lanes of a group serve a quarter of the ranks each
    const uint32_t q = (uint32_t)(lane & 3) * kPerLane;
    if (R == 4 && un.nrows == 4 && (un.row0 & 3) == 0) {
        const float z4[4] = {z[0], z[1], z[2 % R], z[3 % R]};
#pragma unroll
        for (uint32_t i = 0; i < kPerLane; ++i) dn_st_cluster4(cell, q + i, z4);
    } else {
#pragma unroll
        for (int r = 0; r < R; ++r)
            if (r < un.nrows) {
#pragma unroll
                for (uint32_t i = 0; i < kPerLane; ++i) dn_st_cluster(cell + r, q + i, z[r]);
            }
    }
    if ((un.flags & 2) && init.out_base && (lane & 3) == 0 && b < nb) {
        float* o = init.out_base + (run0 + f) * init.out_stride + (long long)(b0 + b) * un.C + un.row0;
#pragma unroll
        for (int r = 0; r < R; ++r)
            if (r < un.nrows) o[r] = z[r];
    }
}

template <int CL>
__global__ void __launch_bounds__(kDnWarps * 32, 1)
sr_dense_kernel(const DnParams P, SrFrameCtl* __restrict__ ctl_out, const SrFrameCtl init, int T)
{
    extern __shared__ __align__(16) float dn_smem[];
    // the input nodes as the fetching warps need them: first float of this cluster's sequences in the caller's frame 0
    // of the run, floats from one frame to the next, floats per frame, the three shared-memory buffers
    __shared__ const float* in_src[SR_MAX_INPUTS];
    __shared__ long long in_step[SR_MAX_INPUTS];
    __shared__ int in_len[SR_MAX_INPUTS], in_buf[SR_MAX_INPUTS][3], n_in;
    const int tid = threadIdx.x, nthr = blockDim.x, warp = tid >> 5, lane = tid & 31;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int b0 = (int)(blockIdx.x / CL) * kDnSamples;
    const int nb = min(kDnSamples, P.B - b0);
    const DnBlobHdr* H = reinterpret_cast<const DnBlobHdr*>(dn_smem);
    const float* wsm = dn_smem + P.hdr_floats;

    // this rank's tables and weight slices, and zeros in every state buffer (padding columns and unused sequences stay zero)
    {
        const float* blob = reinterpret_cast<const float*>(P.blobs + (size_t)rank * P.blob_bytes);
        dn_fetch(dn_smem, blob, P.blob_bytes / 4, tid, nthr);
        for (int i = P.blob_bytes / 4 + tid; i < P.total_floats; i += nthr) dn_smem[i] = 0.f;
    }
    const long long t0 = init.t, run0 = init.run_t;
    if (tid == 0) {
        int n = 0;
        for (int v = 0; v < P.n_nodes; ++v) {
            const DnNode& nd = P.nodes[v];
            if (!nd.is_input) continue;
            in_src[n] = reinterpret_cast<const float*>(static_cast<const char*>(init.in_base[nd.input_slot]) + run0 * init.in_stride_bytes[nd.input_slot]) + (size_t)b0 * nd.C;
            in_step[n] = init.in_stride_bytes[nd.input_slot] / 4;
            in_len[n] = nb * nd.C;                           // input nodes have Cpad == C
            for (int i = 0; i < 3; ++i) in_buf[n][i] = nd.buf[i];
            ++n;
        }
        n_in = n;
    }
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    // frame t of every node from the state buffers in global memory (relative frame 0)
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
    // Input frame k of the run (relative frame k) -> buffer k % 3, by the warps from fetch_warp0 on.
    const int f_tid = tid - H->fetch_warp0 * 32, f_nthr = nthr - H->fetch_warp0 * 32;
    auto fetch_inputs = [&](int k) {
        if (f_tid < 0) return;
        for (int i = 0; i < n_in; ++i) dn_fetch(dn_smem + in_buf[i][k % 3], in_src[i] + (k - 1) * in_step[i], in_len[i], f_tid, f_nthr);
    };
    fetch_inputs(1);
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
    dn_cluster_sync();                                       // every CTA of the cluster has its buffers in place before remote writes start

    for (int f = 0; f < T; ++f) {                            // relative frame f -> f + 1
        // the input frame after the next one is on its way during this update; it has landed, and is made visible
        // to the whole CTA, at the cluster barrier that ends the update
        if (f + 1 < T) fetch_inputs(f + 2);
        asm volatile("cp.async.commit_group;" ::: "memory");
        for (int l = 1; l <= P.n_levels; ++l) {
            for (int u = H->level_begin[l - 1] + warp; u < H->level_begin[l]; u += kDnWarps) {
                const DnUnit un = H->units[u];
                if (un.nrows == 0) continue;
                if (un.nrows > 2) dn_unit<4, CL>(H, un, dn_smem, wsm, init, f, lane, b0, nb, run0);
                else dn_unit<2, CL>(H, un, dn_smem, wsm, init, f, lane, b0, nb, run0);
            }
            if (l == P.n_levels) asm volatile("cp.async.wait_group 0;" ::: "memory");
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
    // relative frame T back to the state buffers in global memory (parity of t + T); every rank holds a full copy and
    // writes its share of it
    {
        const int parT = (int)((t0 + T) & 1);
        const int gtid = (int)rank * nthr + tid, gthr = CL * nthr;
        for (int v = 0; v < P.n_nodes; ++v) {
            const DnNode& nd = P.nodes[v];
            const float* src = dn_smem + (nd.is_input ? nd.buf[T % 3] : nd.buf[T & 1]);
            float* gdst = nd.gstate[parT] + (size_t)b0 * nd.C;
            if (nd.Cpad == nd.C)
                for (int i = gtid * 4; i < nb * nd.C; i += gthr * 4) *reinterpret_cast<float4*>(gdst + i) = *reinterpret_cast<const float4*>(src + i);
            else
                for (int i = gtid; i < nb * nd.C; i += gthr) gdst[i] = src[(i / nd.C) * nd.Cpad + (i % nd.C)];
        }
    }
}

// ------------------------------------------------------------------------------------------ host side
struct DnEngine {
    DnParams P{};
    std::vector<int> edge_of_host;                 // host edge -> index in P.edges
    int cluster = 8;                               // CTAs per cluster
    std::vector<int> row_lo;                       // [node][rank] first row of the rank's slice, cluster + 1 entries per node
    std::vector<std::vector<int>> w_off;           // [rank][edge]
    std::vector<DnBlobHdr> hdrs;                   // per rank
    SrRegion r_blobs;
    int smem_bytes = 0;
    bool attr_set = false;
    std::vector<cudaEvent_t> ev;
    size_t ev_used = 0;
};

DnEngine* dn_of(const sr_graph* g) { return static_cast<DnEngine*>(g->dn); }

typedef void (*DnKernel)(const DnParams, SrFrameCtl*, const SrFrameCtl, int);

bool dn_prepare(DnKernel kernel, int cluster, int smem_bytes)
{
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess) return false;
    if (cluster > 8 && cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) return false;
    return true;
}

// Can at least one cluster of this size and shared-memory footprint be resident on the device?
bool dn_cluster_fits(int cluster, int smem_bytes)
{
    DnKernel kernel = cluster == 16 ? sr_dense_kernel<16> : sr_dense_kernel<8>;
    if (!dn_prepare(kernel, cluster, smem_bytes)) { cudaGetLastError(); return false; }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)cluster);
    cfg.blockDim = dim3((unsigned)(kDnWarps * 32));
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)cluster;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) { cudaGetLastError(); return false; }
    return n >= 1;
}

// Plans the engine for a cluster of CL CTAs: rows of every node split evenly over the ranks.  Null if it does not fit.
DnEngine* dn_build(const sr_graph* g, int CL)
{
    const int n_nodes = (int)g->nodes.size(), n_edges = (int)g->edges.size();
    DnEngine* E = new DnEngine();
    DnParams& P = E->P;
    E->cluster = CL;
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
    // row slices and weight offsets per rank
    E->row_lo.assign((size_t)n_nodes * (CL + 1), 0);
    E->w_off.assign(CL, std::vector<int>(kDnMaxEdges, 0));
    int max_w = 0;
    for (int v = 0; v < n_nodes; ++v)
        for (int r = 0; r <= CL; ++r) E->row_lo[(size_t)v * (CL + 1) + r] = g->nodes[v].d.c * r / CL;
    for (int r = 0; r < CL; ++r) {
        int w = 0;
        for (int e = 0; e < n_edges; ++e) {
            const int v = P.edges[e].tgt;
            const int rows = E->row_lo[(size_t)v * (CL + 1) + r + 1] - E->row_lo[(size_t)v * (CL + 1) + r];
            E->w_off[r][e] = w;
            w += rows * P.edges[e].Kpad;
        }
        max_w = std::max(max_w, w);
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
        return nullptr;
    }
    // Per rank: units (up to four rows of a node each) with their terms (one per incoming edge).  The units of a level
    // go longest first onto the warp with the least work so far; warp w's i-th unit of the level is entry
    // level_begin + 16 i + w (gaps have nrows = 0).
    std::vector<DnBlobHdr>& hdrs = E->hdrs;
    hdrs.assign(CL, DnBlobHdr{});
    for (int r = 0; r < CL; ++r) {
        DnBlobHdr& h = hdrs[r];
        std::memset(&h, 0, sizeof(h));
        int n_units = 0, n_terms = 0;
        bool fits = true;
        for (int l = 1; l <= P.n_levels && fits; ++l) {
            std::vector<std::pair<long long, DnUnit>> lv;
            for (int v : g->groups[l - 1]) {
                const DnNode& d = P.nodes[v];
                long long K = 0;
                for (int e = P.first_edge[v]; e < P.first_edge[v + 1]; ++e) K += P.edges[e].Kpad;
                const int lo = E->row_lo[(size_t)v * (CL + 1) + r], hi = E->row_lo[(size_t)v * (CL + 1) + r + 1];
                for (int row = lo; row < hi && fits; row += kDnRows) {
                    const int nr = std::min(kDnRows, hi - row), n_e = P.first_edge[v + 1] - P.first_edge[v];
                    if (n_terms + n_e > kDnMaxTerms) { fits = false; break; }
                    DnUnit u{};
                    u.nrows = nr;
                    u.row0 = row;
                    u.term0 = n_terms;
                    u.n_terms = n_e;
                    u.bias_off = d.bias_off;
                    u.Cpad = d.Cpad;
                    u.C = d.C;
                    u.flags = (d.act == 1 ? 1 : 0) | (d.is_output ? 2 : 0);
                    u.buf[0] = d.buf[0];
                    u.buf[1] = d.buf[1];
                    for (int e = P.first_edge[v]; e < P.first_edge[v + 1]; ++e) {
                        const DnNode& sn = P.nodes[P.edges[e].src];
                        DnTerm& tm = h.terms[n_terms++];
                        tm.w_off = E->w_off[r][e] + (row - lo) * P.edges[e].Kpad;
                        tm.Kpad = P.edges[e].Kpad;
                        tm.xp = sn.Cpad;
                        tm.R = P.edges[e].R;
                        tm.n_buf = sn.is_input ? 3 : 2;
                        for (int i = 0; i < 3; ++i) tm.buf[i] = sn.buf[i < tm.n_buf ? i : 0];
                    }
                    lv.push_back({K * (4 + (nr > 2 ? 4 : 2)) + 256, u});     // loads per step + reduction and stores
                }
            }
            if (!fits) break;
            std::stable_sort(lv.begin(), lv.end(), [](const auto& a, const auto& b) { return a.first > b.first; });
            std::vector<std::vector<DnUnit>> of_warp(kDnWarps);
            std::vector<long long> load(kDnWarps, 0);
            for (auto& u : lv) {
                // a warp issues through scheduler (warp % 4): the least loaded scheduler first, then its least loaded warp
                long long sched[4] = {0, 0, 0, 0};
                for (int w = 0; w < kDnWarps; ++w) sched[w & 3] += load[w];
                int w = 0;
                for (int c = 1; c < kDnWarps; ++c)
                    if (sched[c & 3] < sched[w & 3] || (sched[c & 3] == sched[w & 3] && load[c] < load[w])) w = c;
                of_warp[w].push_back(u.second);
                load[w] += u.first;
            }
            size_t rounds = 0;
            for (auto& q : of_warp) rounds = std::max(rounds, q.size());
            if (n_units + (int)rounds * kDnWarps > kDnMaxUnits) { fits = false; break; }
            for (size_t i = 0; i < rounds; ++i)
                for (int w = 0; w < kDnWarps; ++w) h.units[n_units++] = i < of_warp[w].size() ? of_warp[w][i] : DnUnit{};
            h.level_begin[l] = n_units;
            if (l == 1) {
                // warps without a unit in the first level fetch the input frames, if there are at least four of them
                int last = -1;
                for (int w = 0; w < kDnWarps; ++w)
                    if (!of_warp[w].empty()) last = w;
                h.fetch_warp0 = last + 1 <= kDnWarps - 4 ? last + 1 : 0;
            }
        }
        for (int l = P.n_levels + 1; l <= kDnMaxLevels; ++l) h.level_begin[l] = n_units;
        h.n_units = n_units;
        if (!fits) {
            delete E;
            return nullptr;
        }
    }
    return E;
}

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
    *cluster_size = E ? E->cluster : 0;
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
    // With one level per frame (the streaming rollout) a frame is one round of work units and one cluster barrier:
    // sixteen CTAs (a non-portable cluster size) halve the units of each CTA (measured on the 784-128-128-10 network:
    // 2.8 against 3.2 us per frame), while with several levels per frame the costlier barrier of the larger cluster
    // outweighs that (6.2 against 5.7).  The larger cluster is used only if the device can hold one.
    DnEngine* E = nullptr;
    if (g->groups.size() == 1) {
        E = dn_build(g, kDnMaxCluster);
        if (E && !dn_cluster_fits(kDnMaxCluster, E->smem_bytes)) {
            delete E;
            E = nullptr;
        }
    }
    if (!E) E = dn_build(g, 8);
    if (!E) return SR_OK;
    const int CL = E->cluster;
    DnParams& P = E->P;
    E->r_blobs.offset = offset;
    E->r_blobs.bytes = (size_t)CL * P.blob_bytes;
    offset = sr_align_up(offset + E->r_blobs.bytes, 256);
    g->dn = E;
    // the per-rank table images; they go to the workspace when one is bound
    g->dn_headers.assign((size_t)CL * sizeof(DnBlobHdr), 0);
    for (int r = 0; r < CL; ++r) std::memcpy(g->dn_headers.data() + (size_t)r * sizeof(DnBlobHdr), &E->hdrs[r], sizeof(DnBlobHdr));
    return SR_OK;
}

sr_status sr_dn_bind(sr_graph* g)
{
    DnEngine* E = dn_of(g);
    if (!E) return SR_OK;
    DnParams& P = E->P;
    const int CL = E->cluster;
    char* ws = g->ws;
    P.blobs = reinterpret_cast<const unsigned char*>(ws + E->r_blobs.offset);
    for (int v = 0; v < P.n_nodes; ++v) {
        const SrHostNode& n = g->nodes[v];
        P.nodes[v].gstate[0] = reinterpret_cast<float*>(ws + n.state[0].offset);
        P.nodes[v].gstate[1] = reinterpret_cast<float*>(ws + n.state[1].offset);
        P.nodes[v].bias = reinterpret_cast<const float*>(ws + n.bias.offset);
    }
    // the workspace was zeroed by the caller of bind: weights start at zero, headers go in now
    for (int r = 0; r < CL; ++r)
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
    const int CL = E->cluster;
    const int e = E->edge_of_host[edge];
    const SrHostEdge& he = g->edges[edge];
    const int v = he.d.tgt, K = he.K, Kpad = P.edges[e].Kpad;
    for (int r = 0; r < CL; ++r) {
        const int lo = E->row_lo[(size_t)v * (CL + 1) + r], hi = E->row_lo[(size_t)v * (CL + 1) + r + 1];
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
    const int CL = E->cluster;
    auto kernel = CL == 16 ? sr_dense_kernel<16> : sr_dense_kernel<8>;
    if (!E->attr_set) {
        if (!dn_prepare(kernel, CL, E->smem_bytes)) return SR_ERR_CUDA;
        E->attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)((g->batch + kDnSamples - 1) / kDnSamples * CL));
    cfg.blockDim = dim3((unsigned)(kDnWarps * 32));
    cfg.dynamicSmemBytes = (size_t)E->smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)CL;
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
    if (cudaLaunchKernelEx(&cfg, kernel, E->P, ctl, init, T) != cudaSuccess) return SR_ERR_CUDA;
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
