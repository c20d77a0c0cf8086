// Resident engine of the frame update
//     x_v^{t+1} = sigma_v( b_v + sum_e f_e(theta_e, x_src(e)^{t+1-R(e)}) )        (paper Sec. A1.2, Eq. 2)
// for networks whose per-sample state fits in shared memory.
//
// The sequences of a batch are independent (the paper's rollouts couple nodes and frames, never
// samples), so ONE thread-block cluster owns ONE sequence and walks all T frames of a run with every
// node state, every convolution weight and the rollout tables resident in shared memory.  Nothing but
// the next input frame and the output crosses HBM per frame, and no launch or device-wide barrier
// separates frames: a frame ends at a cluster barrier (a block barrier for a cluster of one).
//   * The CTAs of a cluster split every node by image rows; a CTA keeps its own rows plus the halo
//     rows its convolutions read, and the owner of a row writes it into the neighbour's halo through
//     distributed shared memory as part of its epilogue.
//   * A frame of a streaming rollout is one level: all (node, 16-pixel, 32-channel) units of the CTA
//     are spread over its warps by estimated cost once, on the host.  Sequential and hybrid patterns
//     run their F(R) tableau levels (Eq. 4, Eq. 5) with a barrier after each.
//   * A unit is an implicit GEMM on mma.sync m16n8k16 (bf16 in, fp32 accumulate): the A rows are
//     gathered by ldmatrix straight from the NHWC state (one row address per lane = one pixel of one
//     filter tap; out-of-image taps point at a zero line), the B fragments come from weights packed
//     per k-step in ldmatrix order.  The sum over incoming edges is one accumulator walked over the
//     k-steps of all edges (the concatenated-convolution view of Sec. A).  Tiles of 16 pixels of ONE
//     sample are far below the size the tcgen05 pipe needs to pay off (an instruction with M = 128
//     costs >= 110 cycles however few columns it has), which is why this engine uses the warp-level
//     tensor path and the batch-tiled tcgen05 kernel serves the large networks.
//   * Few-channel edges (C_in * k * k <= 64, the first layer of an image network) build their A
//     fragments from scalar shared-memory loads through a small per-edge lookup table.
//   * Dense and mean-dense heads run on CUDA cores: every warp reduces a slice of the flattened
//     source into a slot, slots of all CTAs are summed in a fixed order after the barrier.
// State layout in shared memory: [row][col][C] bf16 in 16-byte chunks, chunk q stored at
// (q & ~7) | ((q ^ (q >> 3)) & 7) so that the eight row addresses of an ldmatrix phase fall into
// different bank groups for unit-stride and stride-2 taps.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstddef>
#include <cstring>
#include <vector>

#include "sr_internal.h"
#include "sr_resident.h"

namespace {

constexpr int kRsMaxCluster = 4;
constexpr int kRsSmemMax = 232448 - 128;      // 227 KiB per CTA minus the kernel's static shared memory
constexpr int kRsMaxWarps = 32;
constexpr int kRsDenseUnitChunks = 64;        // 16-byte chunks of the source per dense unit
constexpr int kRsMaxDenseC = 64;
constexpr int kRsFinalizeWarp = 0;            // sums the dense slots after a level's barrier
constexpr int kRsFetchWarp = 1;               // fetches the next input frame

enum { RS_INPUT = 0, RS_CONV = 1, RS_DENSE = 2 };
enum { RS_E_MMA = 0, RS_E_GATHER = 1, RS_E_DENSE = 2, RS_E_MEAN = 3 };
enum { RS_U_CONV = 0, RS_U_DENSE = 1 };

// The first five 16-byte groups of RsNode and the first three of RsEdge are what a work unit needs; the unit
// fetches them with 128-bit loads (a quarter of the shared-memory instructions of field-by-field reads, which
// matter: the kernel is bound by the shared-memory pipe).  The static_asserts below pin the layout.
struct RsNode {
    int32_t kind, W, C, slo;                 // [slo, shi) rows stored by this CTA (own + halo)
    int32_t shi, buf[3];                     // byte offsets of the state buffers in shared memory (inputs rotate over in_nb)
    int32_t in_nb, in_tail, act, buf_bytes;
    int32_t n_edges, first_edge, pix_off, bias_off;   // pix_off: table of the CTA's own pixels
    int32_t w_off, ksteps, up_slo, dn_slo;   // up_slo / dn_slo: first stored row of the previous / next CTA of the cluster
    int32_t H, level, lo, hi;                // level: 0-based tableau level; [lo, hi) rows owned by this CTA
    int32_t is_output, input_slot, in_pitch, in_pt;   // input nodes: zero-padded plain layout [top pad + rows + bottom
    int32_t in_ple, in_wpr, in_magic, in_lead;        // pad][in_pitch] (+ a zero tail), see rs_input_fetch
    int32_t up_lo, up_hi, dn_lo, dn_hi;      // own rows that the previous / next CTA of the cluster also stores
    int32_t slot_off, n_slots, has_consumers, pad0;
    char* gstate[2];                         // the node's two state buffers in global memory
};
static_assert(offsetof(RsNode, kind) == 0 && offsetof(RsNode, shi) == 16 && offsetof(RsNode, in_nb) == 32 &&
              offsetof(RsNode, n_edges) == 48 && offsetof(RsNode, w_off) == 64 && sizeof(RsNode) % 16 == 0, "RsNode layout");

struct RsEdge {
    int32_t src, type, k, stride;
    int32_t pad, R, ksteps, lut_off;
    int32_t g_const, g_ys, g_xs, Kreal;      // few-channel edge: element offset of the window of output pixel (0, 0) and
                                             // its step per output row / column; Kreal = k * k * C_in
    int32_t wd_off, wd_ld, n_chunks, x_chunk0;   // dense: weights in shared memory at wd_off (row pitch wd_ld elements) or < 0;
                                                 // first source chunk of this CTA's slice
    int32_t wchunk_mod;                      // mean-dense: chunks per pixel
    float scale;
    int32_t pad_a, pad_b;
    const char* wd_global;                   // dense weights in global memory, already at this CTA's slice
    int64_t wd_gld;                          // row pitch there, in elements
};
static_assert(offsetof(RsEdge, src) == 0 && offsetof(RsEdge, pad) == 16 && offsetof(RsEdge, g_const) == 32 &&
              sizeof(RsEdge) % 16 == 0, "RsEdge layout");

struct RsUnit { int32_t kind, node, a, b, c, d; };
struct RsCopy { const char* src; int32_t dst, bytes; };

struct RsHeader {
    int32_t n_nodes, n_edges, n_levels, n_warps;
    int32_t off_nodes, off_edges, off_units, off_ubegin;
    int32_t off_copies, n_copies, zero_off, smem_bytes;
    int32_t dense_level_mask, sync_after_finalize, blob_bytes, pad_;
};

// ------------------------------------------------------------------------------------------------ device helpers
__device__ __forceinline__ uint32_t rs_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t rs_swz(uint32_t q) { return (q & ~7u) | ((q ^ (q >> 3)) & 7u); }

__device__ __forceinline__ void rs_ldsm4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

__device__ __forceinline__ void rs_mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t rs_cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

__device__ __forceinline__ uint32_t rs_mapa(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}

__device__ __forceinline__ void rs_st_cluster_u32(uint32_t addr, uint32_t v)
{
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

__device__ __forceinline__ void rs_st_cluster_v4(uint32_t addr, const uint32_t (&v)[4])
{
    asm volatile("st.shared::cluster.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]) : "memory");
}

__device__ __forceinline__ void rs_st_cluster_v2(uint32_t addr, uint32_t v0, uint32_t v1)
{
    asm volatile("st.shared::cluster.v2.u32 [%0], {%1,%2};" ::"r"(addr), "r"(v0), "r"(v1) : "memory");
}

__device__ __forceinline__ void rs_cp_async4(uint32_t dst, const void* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}

__device__ __forceinline__ void rs_cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

__device__ __forceinline__ void rs_cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// End of a level: every warp of every CTA of the cluster has finished its units; their shared-memory
// writes (local and remote) are visible afterwards.
__device__ __forceinline__ void rs_level_barrier(int cs)
{
    if (cs > 1) {
        __syncwarp();
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    } else {
        __syncthreads();
    }
}

struct RsCtx {
    unsigned char* smem;
    uint32_t sbase;
    const RsHeader* H;
    const RsNode* nodes;
    const RsEdge* edges;
    uint32_t rank;
    int cs, lane;
};

// Rows [slo, shi) of an input frame from global memory into the node's zero-padded buffer: 4-byte words, word i
// belongs to row i / in_wpr (by multiplication with in_magic = ceil(2^20 / in_wpr), checked on the host).
__device__ __forceinline__ void rs_input_fetch(const RsCtx& cx, const RsNode& nd, const char* g, int bufoff, int tid, int nthr)
{
    const int wpr = nd.in_wpr, nw = (nd.shi - nd.slo) * wpr, magic = nd.in_magic, pt = nd.in_pt, pitch = nd.in_pitch, ple = nd.in_ple;
    for (int i = tid; i < nw; i += nthr) {
        const int row = (int)(((unsigned)i * (unsigned)magic) >> 20), col = i - row * wpr;
        rs_cp_async4(cx.sbase + bufoff + (((row + pt) * pitch + ple) << 1) + col * 4, g + (size_t)i * 4);
    }
}

// Operand fragments of G consecutive k-steps (16 source channels each) of one filter tap for a tile of NB * 16
// output channels.
template <int G, int NB>
struct RsFrag {
    uint32_t a[G][4], b[G][NB][4];
};

template <int G, int NB>
__device__ __forceinline__ void rs_mma_group(float (&acc)[2 * NB][4], const RsFrag<G, NB>& fr)
{
#pragma unroll
    for (int i = 0; i < G; ++i)
#pragma unroll
        for (int nt = 0; nt < 2 * NB; ++nt)
            rs_mma(acc[nt], fr.a[i], fr.b[i][nt >> 1][(nt & 1) * 2], fr.b[i][nt >> 1][(nt & 1) * 2 + 1]);
}

// All taps of a K x K edge whose source has NC16 * 16 channels (2 or 4: at most one 128-byte line per pixel).
// First the A address of every tap (independent arithmetic, nothing waits on anything), then a pure
// load / multiply-add sequence in groups of two k-steps, the loads of a group issued before the
// multiply-adds of the previous one; no branch inside (a conditional load into registers that live across
// groups makes the compiler copy the whole fragment set at every merge).  Chunk q of the swizzled buffer
// lives at q ^ ((q >> 3) & 7); the k-steps of a tap read chunks q, q + 2, q + 4, q + 6 of one line, i.e. the
// first address XOR 32, 64, 96 (the zero line used by out-of-image taps is 128 bytes long, so the XOR applies
// to it as well).  `rowm` / `colm`: this lane's valid filter rows / columns; q00: the lane's chunk index at
// tap (0, 0); the weights of the unit's k-steps are contiguous, 1 KiB each (constant offsets after unrolling).
template <int K, int NC16, int NB>
__device__ __forceinline__ void rs_mma_edge_unrolled(float (&acc)[2 * NB][4], uint32_t rowm, uint32_t colm, int q00, int qrow, int nch,
                                                     uint32_t sb, uint32_t zaddr, uint32_t waddr)
{
    constexpr int GPT = NC16 / 2, S = K * K * GPT;          // groups of two k-steps per tap, groups in all
    uint32_t ad[K * K];
#pragma unroll
    for (int ky = 0; ky < K; ++ky)
#pragma unroll
        for (int kx = 0; kx < K; ++kx) {
            const uint32_t q = (uint32_t)(q00 + ky * qrow + kx * nch);
            const bool ok = ((rowm >> ky) & 1u) && ((colm >> kx) & 1u);
            ad[ky * K + kx] = ok ? sb + ((q ^ ((q >> 3) & 7u)) << 4) : zaddr;
        }
    RsFrag<2, NB> f0, f1;
    auto load = [&](RsFrag<2, NB>& fr, int s) {
        const uint32_t a0 = ad[s / GPT] ^ (uint32_t)((s % GPT) * 64);
        rs_ldsm4(fr.a[0], a0);
        rs_ldsm4(fr.a[1], a0 ^ 32u);
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < NB; ++j) rs_ldsm4(fr.b[i][j], waddr + s * 2048 + i * 1024 + j * 512);
    };
    load(f0, 0);
#pragma unroll
    for (int s = 0; s < S; s += 2) {
        if (s + 1 < S) load(f1, s + 1);
        rs_mma_group<2, NB>(acc, f0);
        if (s + 2 < S) load(f0, s + 2);
        if (s + 1 < S) rs_mma_group<2, NB>(acc, f1);
    }
}

// The same for any filter size and channel count (not unrolled).
template <int NB>
__device__ __forceinline__ void rs_mma_edge_generic(float (&acc)[2 * NB][4], int k, int nc16, uint32_t rowm, uint32_t colm, uint32_t anym,
                                                    int q00, int qrow, int nch, uint32_t sb, uint32_t zaddr, uint32_t waddr)
{
    int tap = 0;
    for (int ky = 0; ky < k; ++ky) {
        const bool rv = (rowm >> ky) & 1u;
        int q0 = q00 + ky * qrow;
        for (int kx = 0; kx < k; ++kx, ++tap, q0 += nch, waddr += nc16 * 1024) {
            if (!((anym >> (tap & 31)) & 1u)) continue;
            const bool ok = rv && ((colm >> kx) & 1u);
            for (int c = 0; c < nc16; ++c) {
                RsFrag<1, NB> fr;
                const uint32_t q = (uint32_t)(q0 + 2 * c);
                rs_ldsm4(fr.a[0], ok ? sb + ((q ^ ((q >> 3) & 7u)) << 4) : zaddr);
#pragma unroll
                for (int j = 0; j < NB; ++j) rs_ldsm4(fr.b[0][j], waddr + c * 1024 + j * 512);
                rs_mma_group<1, NB>(acc, fr);
            }
        }
    }
}

// One (16 pixels x NB * 16 channels) tile of a convolutional node: all k-steps of all incoming edges into one
// accumulator, then bias, activation, bf16 cast and the stores into the next frame's buffer (own copy and,
// for halo rows, the neighbour's).  `f` is the frame index relative to the start of the run: the update
// computes relative frame f + 1.  n0 is the first channel of the 32-channel block; a 16-channel tile (NB = 1)
// takes n-tiles 2 * half, 2 * half + 1 of the block.  Table fields are copied to registers before the loops
// that use them.
template <int NB>
__device__ __forceinline__ void rs_conv_unit(const RsCtx& cx, const RsNode& nd, int j0, int n0, int half, int f)
{
    const int lane = cx.lane;
    const uint4* np = reinterpret_cast<const uint4*>(&nd);
    const uint4 nq0 = np[0], nq3 = np[3], nq4 = np[4];
    const int W = (int)nq0.y, C = (int)nq0.z, nslo = (int)nq0.w, n_edges = (int)nq3.x, first_edge = (int)nq3.y;
    const uint32_t zaddr = cx.sbase + cx.H->zero_off;
    // Column c of n-tile nt of a block holds output channel n0 + (c >> 1) * 8 + nt * 2 + (c & 1) (the host packs the
    // weights that way), so a lane's accumulator columns are consecutive channels: n0 + tq * 8 .. + 7 for a
    // 32-channel tile (one 16-byte chunk per pixel), the lower or upper four of them for a 16-channel tile.
    // The accumulators start at the bias.
    float acc[2 * NB][4];
    {
        const float* bias = reinterpret_cast<const float*>(cx.smem + nq3.w) + n0 + (lane & 3) * 8 + (NB == 1 ? half * 4 : 0);
        const float4 bl = *reinterpret_cast<const float4*>(bias);
        acc[0][0] = acc[0][2] = bl.x; acc[0][1] = acc[0][3] = bl.y;
        acc[1][0] = acc[1][2] = bl.z; acc[1][1] = acc[1][3] = bl.w;
        if (NB == 2) {
            const float4 bh = *reinterpret_cast<const float4*>(bias + 4);
            acc[2 * NB - 2][0] = acc[2 * NB - 2][2] = bh.x; acc[2 * NB - 2][1] = acc[2 * NB - 2][3] = bh.y;
            acc[2 * NB - 1][0] = acc[2 * NB - 1][2] = bh.z; acc[2 * NB - 1][1] = acc[2 * NB - 1][3] = bh.w;
        }
    }
    // the pixel whose row address this lane supplies to ldmatrix, and the 8-channel half it points at
    // (table entry: bit 31 / 30 = the previous / next CTA keeps the pixel's row as halo, row << 15 | column;
    // padded to a multiple of 16 pixels with 0xFFFFFFFF)
    const uint32_t* pix = reinterpret_cast<const uint32_t*>(cx.smem + nq3.z);
    const uint32_t tl = pix[j0 + (lane & 15)];
    const bool vl = tl != 0xFFFFFFFFu;
    const int oyl = (int)((tl >> 15) & 0x7FFFu), oxl = (int)(tl & 0x7FFFu);
    const int khalf = lane >> 4;
    const int g = lane >> 2, tq = lane & 3;       // accumulator rows g and g + 8, columns 2 * tq, 2 * tq + 1 of every n-tile
    // the packed weights of this unit's 32 channels: 1 KiB per k-step, k-steps of all edges in order
    uint32_t waddr = cx.sbase + nq4.x + (uint32_t)(n0 >> 5) * nq4.y * 1024u + lane * 16 + (NB == 1 ? half * 512 : 0);
    for (int ei = 0; ei < n_edges; ++ei) {
        const RsEdge& e = cx.edges[first_edge + ei];
        const uint4* ep = reinterpret_cast<const uint4*>(&e);
        const uint4 eq0 = ep[0], eq1 = ep[1];
        const int etype = (int)eq0.y, k = (int)eq0.z, stride = (int)eq0.w, pad = (int)eq1.x, ksteps = (int)eq1.z, lut_off = (int)eq1.w;
        const RsNode& sn = cx.nodes[eq0.x];
        const uint4* sp = reinterpret_cast<const uint4*>(&sn);
        const uint4 sq0 = sp[0], sq1 = sp[1];
        const int fb = f + 1 - (int)eq1.y;                            // relative frame of the source state (Eq. 2)
        int sbuf = (fb & 1) ? (int)sq1.z : (int)sq1.y;
        if (sq0.x == RS_INPUT) {
            const int bi = fb % sn.in_nb;
            sbuf = bi == 0 ? (int)sq1.y : bi == 1 ? (int)sq1.z : (int)sq1.w;
        }
        const int Ws = (int)sq0.y, Cs = (int)sq0.z, slo = (int)sq0.w, shi = (int)sq1.x;
        (void)Cs;
        if (etype == RS_E_MMA) {
            const uint32_t sb = cx.sbase + sbuf;
            const int nch = Cs >> 3, nc16 = Cs >> 4;
            const int iy0 = oyl * stride - pad, ix0 = oxl * stride - pad;
            uint32_t rowm = 0, colm = 0;
            for (int t = 0; t < k; ++t) {
                rowm |= (uint32_t)(vl && iy0 + t >= slo && iy0 + t < shi) << t;    // stored rows cover every in-image row read
                colm |= (uint32_t)((unsigned)(ix0 + t) < (unsigned)Ws) << t;
            }
            const int q00 = ((iy0 - slo) * Ws + ix0) * nch + khalf, qrow = Ws * nch;
            const int sel = (k == 3 ? 0 : k == 1 ? 4 : 8) + (nc16 == 2 ? 0 : nc16 == 4 ? 1 : 3);
            switch (sel) {
                case 0: rs_mma_edge_unrolled<3, 2, NB>(acc, rowm, colm, q00, qrow, nch, sb, zaddr, waddr); break;
                case 1: rs_mma_edge_unrolled<3, 4, NB>(acc, rowm, colm, q00, qrow, nch, sb, zaddr, waddr); break;
                case 4: rs_mma_edge_unrolled<1, 2, NB>(acc, rowm, colm, q00, qrow, nch, sb, zaddr, waddr); break;
                case 5: rs_mma_edge_unrolled<1, 4, NB>(acc, rowm, colm, q00, qrow, nch, sb, zaddr, waddr); break;
                default: {
                    // other filter sizes and channel counts: a plain loop; taps no lane of the warp needs are skipped
                    uint32_t anym = 0xFFFFFFFFu;
                    if (k * k <= 32) {
                        uint32_t m = 0;
                        for (int t = 0; t < k; ++t)
                            if ((rowm >> t) & 1u) m |= colm << (t * k);
                        anym = __reduce_or_sync(0xffffffffu, m);
                    }
                    rs_mma_edge_generic<NB>(acc, k, nc16, rowm, colm, anym, q00, qrow, nch, sb, zaddr, waddr);
                    break;
                }
            }
            waddr += (uint32_t)ksteps * 1024u;
        } else {
            // few-channel edge (source = an input node, stored zero-padded): A fragments from scalar loads; the
            // table gives the offset of every k index inside a pixel's window, so no bounds are checked
            const uint16_t* src = reinterpret_cast<const uint16_t*>(cx.smem + sbuf);
            const uint32_t* lut = reinterpret_cast<const uint32_t*>(cx.smem + lut_off);
            const uint4 eq2 = ep[2];
            const int g_const = (int)eq2.x, g_ys = (int)eq2.y, g_xs = (int)eq2.z, tail = sn.in_tail;
            int base[2];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const uint32_t t = pix[j0 + g + 8 * r];
                base[r] = t != 0xFFFFFFFFu ? g_const + (int)((t >> 15) & 0x7FFFu) * g_ys + (int)(t & 0x7FFFu) * g_xs : tail;
            }
            for (int ks = 0; ks < ksteps; ++ks) {
                uint32_t a[4];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint2 L = *reinterpret_cast<const uint2*>(lut + ks * 16 + h * 8 + 2 * tq);
#pragma unroll
                    for (int r = 0; r < 2; ++r)
                        a[h * 2 + r] = (uint32_t)src[base[r] + (int)L.x] | ((uint32_t)src[base[r] + (int)L.y] << 16);
                }
#pragma unroll
                for (int j = 0; j < NB; ++j) {
                    uint32_t bj[4];
                    rs_ldsm4(bj, waddr + j * 512);
                    rs_mma(acc[2 * j], a, bj[0], bj[1]);
                    rs_mma(acc[2 * j + 1], a, bj[2], bj[3]);
                }
                waddr += 1024;
            }
        }
    }
    // epilogue: activation, bf16, one 16-byte (8-byte for a 16-channel tile) store per pixel, and one into the
    // neighbour's halo where the pixel table says so
    const uint32_t nchd = (uint32_t)(C >> 3), ch = (uint32_t)((n0 >> 3) + tq), sub = NB == 1 ? (uint32_t)half * 8u : 0u;
    const uint4 nq1 = np[1], nq2 = np[2], nq4e = np[4];      // fetched here, not kept in registers across the main loop
    const uint32_t dbuf = ((f + 1) & 1) ? nq1.z : nq1.y, buf_bytes = nq2.w;
    const bool relu = nq2.z == 1;
    const int d_up = (nslo - (int)nq4e.z) * W, d_dn = (nslo - (int)nq4e.w) * W;
    auto put = [&](uint32_t off, const uint32_t (&pk)[4], int peer) {
        if (off >= buf_bytes) return;
        if (peer < 0) {
            if (NB == 2) *reinterpret_cast<uint4*>(cx.smem + dbuf + off) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            else *reinterpret_cast<uint2*>(cx.smem + dbuf + off + sub) = make_uint2(pk[0], pk[1]);
        } else {
            const uint32_t ra = rs_mapa(cx.sbase + dbuf + off + sub, (uint32_t)peer);
            if (NB == 2) rs_st_cluster_v4(ra, pk);
            else rs_st_cluster_v2(ra, pk[0], pk[1]);
        }
    };
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const uint32_t t = pix[j0 + g + 8 * r];
        if (t == 0xFFFFFFFFu) continue;
        const int y = (int)((t >> 15) & 0x7FFFu), x = (int)(t & 0x7FFFu);
        uint32_t pk[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int nt = 0; nt < 2 * NB; ++nt) {
            __nv_bfloat162 v = __floats2bfloat162_rn(acc[nt][2 * r], acc[nt][2 * r + 1]);
            if (relu) v = __hmax2(v, __floats2bfloat162_rn(0.f, 0.f));
            pk[nt] = *reinterpret_cast<const uint32_t*>(&v);
        }
        const int lin = (y - nslo) * W + x;
        put(rs_swz((uint32_t)lin * nchd + ch) * 16u, pk, -1);
        if (t & 0x80000000u) put(rs_swz((uint32_t)(lin + d_up) * nchd + ch) * 16u, pk, (int)cx.rank - 1);   // halo of the previous CTA
        if (t & 0x40000000u) put(rs_swz((uint32_t)(lin + d_dn) * nchd + ch) * 16u, pk, (int)cx.rank + 1);   // of the next one
    }
}

__device__ __forceinline__ void rs_unpack8(const uint4& q, float (&v)[8])
{
    v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xFFFF0000u);
    v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xFFFF0000u);
    v[4] = __uint_as_float(q.z << 16); v[5] = __uint_as_float(q.z & 0xFFFF0000u);
    v[6] = __uint_as_float(q.w << 16); v[7] = __uint_as_float(q.w & 0xFFFF0000u);
}

// A slice of a dense / mean-dense edge: this warp's partial dot products of the 16-byte chunks
// [c_begin, c_end) of the CTA's part of the source with the matching weight columns, for every output,
// written to slot `slot` of the target node in every CTA of the cluster.
__device__ __forceinline__ void rs_dense_unit(const RsCtx& cx, const RsNode& nd, const RsEdge& e, int c_begin, int c_end,
                                              int slot, int f)
{
    const int lane = cx.lane;
    const RsNode& sn = cx.nodes[e.src];
    const int fb = f + 1 - e.R;
    const unsigned char* xb = cx.smem + sn.buf[fb & 1];
    const bool swz = sn.kind == RS_CONV;
    const char* wb = e.wd_off >= 0 ? reinterpret_cast<const char*>(cx.smem + e.wd_off) : e.wd_global;
    const long long ld = e.wd_off >= 0 ? (long long)e.wd_ld : (long long)e.wd_gld;
    const uint32_t slot_base = (uint32_t)nd.slot_off + (uint32_t)((((f + 1) & 1) * nd.n_slots + slot) * nd.C) * 4u;
    const int C = nd.C, wmod = e.wchunk_mod, x0 = e.x_chunk0;
    const float scale = e.scale;
    for (int ob = 0; ob < C; ob += 16) {
        float acc[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[j] = 0.f;
        for (int cl = c_begin + lane; cl < c_end; cl += 32) {
            const uint32_t q = (uint32_t)(x0 + cl);
            const uint4 xq = *reinterpret_cast<const uint4*>(xb + (swz ? rs_swz(q) : q) * 16u);
            float x[8];
            rs_unpack8(xq, x);
            const int wc = wmod ? cl % wmod : cl;
            const char* wp = wb + ((long long)ob * ld + (long long)wc * 8) * 2;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if (ob + j < C) {
                    const uint4 wq = *reinterpret_cast<const uint4*>(wp + (long long)j * ld * 2);
                    float w[8];
                    rs_unpack8(wq, w);
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[j] = fmaf(w[i], x[i], acc[j]);
                }
            }
        }
        // reduce-scatter over the warp: every step halves the values a lane keeps and adds the partner's copy of
        // them (16 shuffles for 16 outputs instead of 80); lane l ends with the total of output ob + (l & 15)
        float v8[8], v4[4], v2[2];
        const bool h3 = lane & 8, h2 = lane & 4, h1 = lane & 2, h0 = lane & 1;
#pragma unroll
        for (int i = 0; i < 8; ++i) v8[i] = (h3 ? acc[i + 8] : acc[i]) + __shfl_xor_sync(0xffffffffu, h3 ? acc[i] : acc[i + 8], 8);
#pragma unroll
        for (int i = 0; i < 4; ++i) v4[i] = (h2 ? v8[i + 4] : v8[i]) + __shfl_xor_sync(0xffffffffu, h2 ? v8[i] : v8[i + 4], 4);
#pragma unroll
        for (int i = 0; i < 2; ++i) v2[i] = (h1 ? v4[i + 2] : v4[i]) + __shfl_xor_sync(0xffffffffu, h1 ? v4[i] : v4[i + 2], 2);
        float v = (h0 ? v2[1] : v2[0]) + __shfl_xor_sync(0xffffffffu, h0 ? v2[0] : v2[1], 1);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        if (lane < 16 && ob + lane < C) {
            v *= scale;
            const uint32_t a = cx.sbase + slot_base + (uint32_t)(ob + lane) * 4u;
            if (cx.cs > 1) {
                for (int r = 0; r < cx.cs; ++r) rs_st_cluster_u32(rs_mapa(a, (uint32_t)r), __float_as_uint(v));
            } else {
                *reinterpret_cast<float*>(cx.smem + slot_base + (uint32_t)(ob + lane) * 4u) = v;
            }
        }
    }
}

// The kernel body.  It is instantiated for 16, 24 and 32 warps per CTA (128, 80 and 64 registers per thread: the
// code needs about 80, the compiler uses whatever the bound leaves), see the wrappers below.
__device__ __forceinline__ void rs_kernel_body(const unsigned char* __restrict__ blobs, int blob_stride, SrFrameCtl* __restrict__ ctl_out,
                                               const SrFrameCtl& init, int T, int cs)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, nthr = blockDim.x;
    const uint32_t rank = cs > 1 ? rs_cluster_rank() : 0u;
    const int b = blockIdx.x / cs;                                    // the sequence this cluster rolls out
    {
        const uint4* src = reinterpret_cast<const uint4*>(blobs + (size_t)rank * blob_stride);
        const int n16 = reinterpret_cast<const RsHeader*>(src)->blob_bytes >> 4;
        for (int i = tid; i < n16; i += nthr) reinterpret_cast<uint4*>(smem)[i] = src[i];
    }
    __syncthreads();
    RsCtx cx;
    cx.smem = smem;
    cx.sbase = rs_smem_u32(smem);
    cx.H = reinterpret_cast<const RsHeader*>(smem);
    cx.nodes = reinterpret_cast<const RsNode*>(smem + cx.H->off_nodes);
    cx.edges = reinterpret_cast<const RsEdge*>(smem + cx.H->off_edges);
    cx.rank = rank;
    cx.cs = cs;
    cx.lane = tid & 31;
    const RsHeader& H = *cx.H;
    const RsUnit* units = reinterpret_cast<const RsUnit*>(smem + H.off_units);
    const int32_t* ubegin = reinterpret_cast<const int32_t*>(smem + H.off_ubegin);
    const int warp = tid >> 5;
    if (tid < 32) reinterpret_cast<uint32_t*>(smem + H.zero_off)[tid] = 0u;
    // the input buffers' padding stays zero for the whole run
    for (int v = 0; v < H.n_nodes; ++v) {
        const RsNode& nd = cx.nodes[v];
        if (nd.kind != RS_INPUT) continue;
        for (int k = 0; k < nd.in_nb; ++k)
            for (int i = tid; i < (nd.buf_bytes >> 2); i += nthr) reinterpret_cast<uint32_t*>(smem + nd.buf[k])[i] = 0u;
    }
    __syncthreads();
    // parameters: packed convolution weights, dense weight slices, biases
    {
        const RsCopy* cp = reinterpret_cast<const RsCopy*>(smem + H.off_copies);
        // every cluster reads the same parameter blocks: each starts at a different 2 KiB-aligned place inside a
        // block, so that at any moment the clusters pull different lines out of L2
        for (int c = 0; c < H.n_copies; ++c) {
            const int bytes = cp[c].bytes;
            const int rot = (int)(((unsigned)b * 2048u) % (unsigned)bytes) & ~15;
            for (int i = tid * 16; i < bytes; i += nthr * 16) {
                int j = i + rot;
                if (j >= bytes) j -= bytes;
                rs_cp_async16(cx.sbase + cp[c].dst + j, cp[c].src + j);
            }
        }
    }
    // frame t of every node (relative frame 0), and the first input frame of the run (relative frame 1)
    // `init` is the frame control block of this run (frame counter, the caller's input sequences and output);
    // the block in global memory is brought up to date at the end, for the launches that follow
    const SrFrameCtl* const ctl = &init;
    const long long t0 = ctl->t, run0 = ctl->run_t, out_stride = ctl->out_stride;
    float* const out_base = ctl->out_base;
    const int par0 = (int)(t0 & 1);
    for (int v = 0; v < H.n_nodes; ++v) {
        const RsNode& nd = cx.nodes[v];
        if (nd.kind == RS_DENSE) {
            const uint16_t* g = reinterpret_cast<const uint16_t*>(nd.gstate[par0]) + (size_t)b * nd.C;
            for (int i = tid; i < nd.C; i += nthr) reinterpret_cast<uint16_t*>(smem + nd.buf[0])[i] = g[i];
        } else if (nd.kind == RS_CONV) {
            const int nq = (nd.shi - nd.slo) * nd.W * (nd.C >> 3);
            const char* g = nd.gstate[par0] + ((size_t)b * nd.H + nd.slo) * nd.W * nd.C * 2;
            for (int q = tid; q < nq; q += nthr) rs_cp_async16(cx.sbase + nd.buf[0] + rs_swz((uint32_t)q) * 16u, g + (size_t)q * 16);
        } else {
            // relative frame 0 from the state buffer; frames 1 .. in_lead - 1 from the caller's sequence
            const size_t row0 = ((size_t)b * nd.H + nd.slo) * nd.W * nd.C * 2;
            rs_input_fetch(cx, nd, nd.gstate[par0] + row0, nd.buf[0], tid, nthr);
            for (int k = 1; k < nd.in_lead && k <= T; ++k)
                rs_input_fetch(cx, nd, static_cast<const char*>(ctl->in_base[nd.input_slot]) +
                                           (run0 + k - 1) * ctl->in_stride_bytes[nd.input_slot] + row0, nd.buf[k % nd.in_nb], tid, nthr);
        }
    }
    __shared__ const char* in_ptr[SR_MAX_INPUTS];      // the caller's frame sequences, read once
    __shared__ long long in_stride[SR_MAX_INPUTS];
    if (tid < SR_MAX_INPUTS) {
        in_stride[tid] = ctl->in_stride_bytes[tid];
        in_ptr[tid] = static_cast<const char*>(ctl->in_base[tid]) + run0 * ctl->in_stride_bytes[tid];
    }
    rs_cp_async_wait_all();
    rs_level_barrier(cs);             // also: every CTA of the cluster runs before any remote store is issued

    for (int f = 0; f < T; ++f) {
        // the input frame a later update reads (relative frame f + in_lead), fetched by one warp while this update
        // computes (the host gave that warp fewer units)
        if (warp == kRsFetchWarp) {
            for (int v = 0; v < H.n_nodes; ++v) {
                const RsNode& nd = cx.nodes[v];
                if (nd.kind != RS_INPUT || f + nd.in_lead > T) continue;
                const int fr = f + nd.in_lead;
                rs_input_fetch(cx, nd, in_ptr[nd.input_slot] + (size_t)(fr - 1) * in_stride[nd.input_slot] +
                                           ((size_t)b * nd.H + nd.slo) * nd.W * nd.C * 2, nd.buf[fr % nd.in_nb], cx.lane, 32);
            }
        }
        for (int l = 0; l < H.n_levels; ++l) {
            const int ub = ubegin[l * H.n_warps + warp], ue = ubegin[l * H.n_warps + warp + 1];
            for (int u = ub; u < ue; ++u) {
                const RsUnit& un = units[u];
                const RsNode& nd = cx.nodes[un.node];
                if (un.kind == RS_U_CONV) {
                    if (un.c == 2) rs_conv_unit<2>(cx, nd, un.a, un.b, 0, f);
                    else rs_conv_unit<1>(cx, nd, un.a, un.b, un.c, f);
                }
                else rs_dense_unit(cx, nd, cx.edges[un.a], un.b, un.c, un.d, f);
            }
            if (l == H.n_levels - 1) rs_cp_async_wait_all();
            rs_level_barrier(cs);
            if ((H.dense_level_mask >> l) & 1) {
                // dense nodes of this level: fixed-order sum of the slots (the bias is slot-independent), activation
                if (warp == kRsFinalizeWarp) {
                    for (int v = 0; v < H.n_nodes; ++v) {
                        const RsNode& nd = cx.nodes[v];
                        if (nd.kind != RS_DENSE || nd.level != l) continue;
                        const int C = nd.C, n_slots = nd.n_slots;
                        const float* slots = reinterpret_cast<const float*>(smem + nd.slot_off) + ((f + 1) & 1) * n_slots * C;
                        const float* bias = reinterpret_cast<const float*>(smem + nd.bias_off);
                        for (int o = cx.lane; o < C; o += 32) {
                            float z = 0.f;
                            for (int s = 0; s < n_slots; ++s) z += slots[s * C + o];
                            z += bias[o];
                            if (nd.act == 1) z = fmaxf(z, 0.f);
                            reinterpret_cast<__nv_bfloat16*>(smem + nd.buf[(f + 1) & 1])[o] = __float2bfloat16_rn(z);
                            if (nd.is_output && rank == 0 && out_base) out_base[(run0 + f) * out_stride + (long long)b * C + o] = z;
                        }
                    }
                }
                if (H.sync_after_finalize) __syncthreads();
            }
        }
    }

    if (blockIdx.x == 0 && tid == 0) {
        SrFrameCtl c = init;
        c.t += T;
        c.run_t += T;
        c.error = ctl_out->error;
        *ctl_out = c;
    }
    // relative frame T back to the state buffers in global memory (parity of t + T)
    const int parT = (int)((t0 + T) & 1);
    for (int v = 0; v < H.n_nodes; ++v) {
        const RsNode& nd = cx.nodes[v];
        if (nd.kind == RS_DENSE) {
            if (rank == 0) {
                uint16_t* g = reinterpret_cast<uint16_t*>(nd.gstate[parT]) + (size_t)b * nd.C;
                for (int i = tid; i < nd.C; i += nthr) g[i] = reinterpret_cast<const uint16_t*>(smem + nd.buf[T & 1])[i];
            }
        } else if (nd.kind == RS_CONV) {
            const int nch = nd.C >> 3, nq = (nd.hi - nd.lo) * nd.W * nch, q0 = (nd.lo - nd.slo) * nd.W * nch;
            char* g = nd.gstate[parT] + ((size_t)b * nd.H + nd.lo) * nd.W * nd.C * 2;
            for (int q = tid; q < nq; q += nthr)
                *reinterpret_cast<uint4*>(g + (size_t)q * 16) =
                    *reinterpret_cast<const uint4*>(smem + nd.buf[T & 1] + rs_swz((uint32_t)(q + q0)) * 16u);
        } else {
            const int wpr = nd.in_wpr, nw = (nd.hi - nd.lo) * wpr, r0 = nd.lo - nd.slo + nd.in_pt;
            char* g = nd.gstate[parT] + ((size_t)b * nd.H + nd.lo) * nd.W * nd.C * 2;
            const unsigned char* sbuf = smem + nd.buf[T % nd.in_nb];
            for (int i = tid; i < nw; i += nthr) {
                const int row = (int)(((unsigned)i * (unsigned)nd.in_magic) >> 20), col = i - row * wpr;
                reinterpret_cast<uint32_t*>(g)[i] =
                    *reinterpret_cast<const uint32_t*>(sbuf + (((row + r0) * nd.in_pitch + nd.in_ple) << 1) + col * 4);
            }
        }
    }
}

template <int MAXT>
__global__ void __launch_bounds__(MAXT, 1)
sr_resident_kernel(const unsigned char* __restrict__ blobs, int blob_stride, SrFrameCtl* __restrict__ ctl_out,
                   const __grid_constant__ SrFrameCtl init, int T, int cs)
{
    rs_kernel_body(blobs, blob_stride, ctl_out, init, T, cs);
}

// ------------------------------------------------------------------------------------------------ host side
struct RsPlanNode {
    int kind = RS_INPUT;
    int lo[kRsMaxCluster + 1] = {0}, slo[kRsMaxCluster] = {0}, shi[kRsMaxCluster] = {0};
    int buf[3] = {0, 0, 0}, buf_bytes = 0, bias_off = 0, w_off = 0, slot_off = 0, n_slots = 0, pix_off = 0, pix_entries = 0;
    int first_edge = 0, ksteps = 0;
    size_t w_global = 0;            // byte offset of the packed weights inside the convolution-weight region
    bool has_consumers = false;
    // input nodes: zero-padded buffer geometry (elements), buffers in rotation and how far ahead frames are fetched
    int in_pitch = 0, in_pt = 0, in_pb = 0, in_ple = 0, in_tail_len = 0, in_wpr = 0, in_magic = 0, in_nb = 3, in_lead = 2;
};

struct RsPlanEdge {
    int host_edge = -1, type = RS_E_MMA, ksteps = 0, ks0 = 0, lut_off = 0, Kreal = 0;
    size_t wd_global = 0;           // dense: byte offset inside the dense-weight region
    int wd_off[kRsMaxCluster] = {-1, -1, -1, -1};
};

struct RsOffsets { int nodes = 0, edges = 0, units = 0, ubegin = 0, copies = 0; };   // table offsets inside a rank's blob

struct RsEngine {
    int cs = 1, warps = 16, smem_bytes = 0, blob_bytes = 0, n_levels = 1;
    RsOffsets offs;                             // written by rs_layout, read when the blobs are filled
    std::vector<RsPlanNode> pn;
    std::vector<RsPlanEdge> pe;                 // ordered by target node, then by the node's in-edge order
    std::vector<int> pe_of_host_edge;
    std::vector<std::vector<RsUnit>> units;     // per rank, sorted by (level, warp)
    std::vector<std::vector<int>> ubegin;       // per rank
    std::vector<std::vector<uint32_t>> luts;    // per plan edge (gather edges only)
    int zero_off = 0;
    bool dense_in_smem = false;
    SrRegion r_blobs, r_wconv, r_wdense;
    bool attr_set = false;
    std::vector<cudaEvent_t> ev;                // pairs bracketing timed launches (option "kernel timing")
    size_t ev_used = 0;
};

int rs_row_lo(int H, int r, int cs) { return (H * r + cs / 2) / cs; }
int rs_up16(int x) { return (x + 15) / 16 * 16; }
int rs_up128(int x) { return (x + 127) / 128 * 128; }

// Lays the engine out for a cluster of `cs` CTAs; false if the network does not fit.
bool rs_layout(const sr_graph* g, RsEngine& E, int cs, int warps)
{
    const int n_nodes = (int)g->nodes.size();
    E.cs = cs;
    E.warps = warps;
    E.n_levels = (int)g->groups.size();
    // row ownership and stored ranges
    for (int v = 0; v < n_nodes; ++v) {
        RsPlanNode& p = E.pn[v];
        const sr_node_desc& d = g->nodes[v].d;
        if (p.kind == RS_DENSE) {
            for (int r = 0; r <= cs; ++r) p.lo[r] = r == 0 ? 0 : 1;
            for (int r = 0; r < cs; ++r) {
                p.slo[r] = 0;
                p.shi[r] = 1;
            }
            continue;
        }
        if (d.h < cs) return false;
        for (int r = 0; r <= cs; ++r) p.lo[r] = rs_row_lo(d.h, r, cs);
        for (int r = 0; r < cs; ++r) {
            p.slo[r] = p.lo[r];
            p.shi[r] = p.lo[r + 1];
        }
    }
    for (const RsPlanEdge& pe : E.pe) {
        const SrHostEdge& he = g->edges[pe.host_edge];
        if (he.d.kind != SR_EDGE_CONV) continue;
        RsPlanNode& s = E.pn[he.d.src];
        const RsPlanNode& t = E.pn[he.d.tgt];
        const int Hs = g->nodes[he.d.src].d.h;
        for (int r = 0; r < cs; ++r) {
            const int clo = t.lo[r], chi = t.lo[r + 1];
            if (chi <= clo) continue;
            const int need_lo = std::max(0, he.stride_eff * clo - he.pad_eff);
            const int need_hi = std::min(Hs, he.stride_eff * (chi - 1) - he.pad_eff + he.k_eff);
            s.slo[r] = std::min(s.slo[r], need_lo);
            s.shi[r] = std::max(s.shi[r], need_hi);
        }
    }
    // a halo row must belong to a direct neighbour (its owner mirrors it there)
    for (int v = 0; v < n_nodes; ++v) {
        const RsPlanNode& p = E.pn[v];
        if (p.kind == RS_DENSE) continue;
        for (int r = 0; r < cs; ++r) {
            if (r > 0 && p.slo[r] < p.lo[r - 1]) return false;
            if (r + 1 < cs && p.shi[r] > p.lo[r + 2]) return false;
        }
    }
    // units per rank
    E.units.assign(cs, std::vector<RsUnit>());
    E.ubegin.assign(cs, std::vector<int>());
    std::vector<int> slot_count(n_nodes, 0);
    struct Cand { RsUnit u; int level; long cost; };
    std::vector<std::vector<Cand>> cand(cs);
    // which nodes are cut into 16-channel tiles: those whose 32-channel tile alone would take more than half of a
    // warp's fair share of its level
    std::vector<char> split(n_nodes, 0);
    if (g->opt_rs_split != 0) {
        std::vector<long> level_cost(E.n_levels, 0), unit_cost(n_nodes, 0);
        for (int v = 0; v < n_nodes; ++v) {
            const RsPlanNode& p = E.pn[v];
            const SrHostNode& hn = g->nodes[v];
            if (p.kind == RS_INPUT) continue;
            long c = 1700, units = 0;
            if (p.kind == RS_CONV) {
                for (int ei = 0; ei < (int)hn.in_edges.size(); ++ei) {
                    const RsPlanEdge& pe = E.pe[p.first_edge + ei];
                    c += (long)pe.ksteps * (pe.type == RS_E_MMA ? 160 : 400);
                }
                units = (long)(((p.lo[1] - p.lo[0]) * hn.d.w + 15) / 16) * (hn.d.c / 32);
            } else {
                c = 5000;
                units = 4;
            }
            unit_cost[v] = c;
            level_cost[hn.level - 1] += c * units;
        }
        for (int v = 0; v < n_nodes; ++v)
            if (E.pn[v].kind == RS_CONV && (g->opt_rs_split == 1 || unit_cost[v] * 2 * warps > level_cost[g->nodes[v].level - 1]))
                split[v] = 1;
    }
    for (int v = 0; v < n_nodes; ++v) {
        const RsPlanNode& p = E.pn[v];
        const SrHostNode& hn = g->nodes[v];
        if (p.kind == RS_INPUT) continue;
        const int level = hn.level - 1;
        if (p.kind == RS_CONV) {
            // estimated cycles of a unit while all warps of the CTA are busy (measured on B200 with 16 warps: the
            // warps of a scheduler share its tensor pipe and the CTA's shared-memory pipe)
            long cost = 1700;
            for (int ei = 0; ei < (int)hn.in_edges.size(); ++ei) {
                const RsPlanEdge& pe = E.pe[p.first_edge + ei];
                cost += (long)pe.ksteps * (pe.type == RS_E_MMA ? 160 : 400);
            }
            // a unit is a 16-pixel x 32-channel tile (c = 2), or, for nodes with many k-steps when the CTA has more
            // warps than such tiles, its two 16-channel halves (c = 0, 1): they load the A operand twice but halve the
            // longest dependent chain of a frame
            for (int r = 0; r < cs; ++r) {
                const int npix = (p.lo[r + 1] - p.lo[r]) * hn.d.w;
                for (int j0 = 0; j0 < npix; j0 += 16)
                    for (int n0 = 0; n0 < hn.d.c; n0 += 32) {
                        if (split[v]) {
                            cand[r].push_back(Cand{RsUnit{RS_U_CONV, v, j0, n0, 0, 0}, level, 1400 + (cost - 1700) * 6 / 10});
                            cand[r].push_back(Cand{RsUnit{RS_U_CONV, v, j0, n0, 1, 0}, level, 1400 + (cost - 1700) * 6 / 10});
                        } else {
                            cand[r].push_back(Cand{RsUnit{RS_U_CONV, v, j0, n0, 2, 0}, level, cost});
                        }
                    }
            }
        } else {
            for (int ei = 0; ei < (int)hn.in_edges.size(); ++ei) {
                const SrHostEdge& he = g->edges[hn.in_edges[ei]];
                const RsPlanNode& sp = E.pn[he.d.src];
                const sr_node_desc& sd = g->nodes[he.d.src].d;
                for (int r = 0; r < cs; ++r) {
                    int n = 0;
                    if (sp.kind == RS_CONV) n = (sp.lo[r + 1] - sp.lo[r]) * sd.w * (sd.c / 8);
                    else if (r == 0) n = sd.c / 8;
                    if (n == 0) continue;
                    const int parts = (n + kRsDenseUnitChunks - 1) / kRsDenseUnitChunks;
                    const int per = (n + parts - 1) / parts;
                    for (int c0 = 0; c0 < n; c0 += per) {
                        const int c1 = std::min(n, c0 + per);
                        const long cost = 2200 + (long)((c1 - c0 + 31) / 32) * 250 * hn.d.c;
                        cand[r].push_back(Cand{RsUnit{RS_U_DENSE, v, p.first_edge + ei, c0, c1, slot_count[v]++}, level, cost});
                    }
                }
            }
        }
    }
    for (int v = 0; v < n_nodes; ++v) E.pn[v].n_slots = slot_count[v];
    for (int r = 0; r < cs; ++r) {
        // longest-processing-time-first: level by level, to the least loaded scheduler partition
        // (warp id mod 4), then to its least loaded warp
        std::vector<std::vector<std::vector<RsUnit>>> lists(E.n_levels, std::vector<std::vector<RsUnit>>(warps));
        for (int l = 0; l < E.n_levels; ++l) {
            std::vector<Cand> cs_l;
            for (const Cand& c : cand[r])
                if (c.level == l) cs_l.push_back(c);
            std::stable_sort(cs_l.begin(), cs_l.end(), [](const Cand& a, const Cand& b) { return a.cost > b.cost; });
            std::vector<long> wl(warps, 0), pl(4, 0);
            // fixed duties: the slot sums of the dense nodes of this level, the input fetch (last level's barrier waits for it)
            bool dense_here = false;
            for (int v = 0; v < n_nodes; ++v)
                if (E.pn[v].kind == RS_DENSE && g->nodes[v].level - 1 == l) dense_here = true;
            if (dense_here && kRsFinalizeWarp < warps) {
                wl[kRsFinalizeWarp] += 3500;
                pl[kRsFinalizeWarp % 4] += 3500;
            }
            if (l == 0 && kRsFetchWarp < warps) {
                wl[kRsFetchWarp] += 2500;
                pl[kRsFetchWarp % 4] += 2500;
            }
            for (const Cand& c : cs_l) {
                int bp = 0;
                for (int p = 1; p < std::min(4, warps); ++p)
                    if (pl[p] < pl[bp]) bp = p;
                int bw = bp;
                for (int w = bp; w < warps; w += 4)
                    if (wl[w] < wl[bw]) bw = w;
                wl[bw] += c.cost;
                pl[bp] += c.cost;
                lists[l][bw].push_back(c.u);
            }
        }
        for (int l = 0; l < E.n_levels; ++l)
            for (int w = 0; w < warps; ++w) {
                E.ubegin[r].push_back((int)E.units[r].size());
                for (const RsUnit& u : lists[l][w]) E.units[r].push_back(u);
            }
        E.ubegin[r].push_back((int)E.units[r].size());
    }
    // tables
    size_t max_units = 0;
    for (int r = 0; r < cs; ++r) max_units = std::max(max_units, E.units[r].size());
    int off = (int)sizeof(RsHeader);
    auto take = [&](int bytes, int align) {
        off = (off + align - 1) / align * align;
        const int o = off;
        off += bytes;
        return o;
    };
    const int off_nodes = take((int)sizeof(RsNode) * n_nodes, 16);
    const int off_edges = take((int)sizeof(RsEdge) * (int)E.pe.size(), 16);
    const int off_units = take((int)(sizeof(RsUnit) * std::max<size_t>(1, max_units)), 16);
    const int off_ubegin = take((int)sizeof(int32_t) * (E.n_levels * warps + 1), 16);
    int n_copies = 0;
    for (int v = 0; v < n_nodes; ++v)
        if (E.pn[v].kind != RS_INPUT) n_copies += 1 + (E.pn[v].kind == RS_CONV ? 1 : 0);
    int dense_rows = 0;
    for (const RsPlanEdge& pe : E.pe) {
        const SrHostEdge& he = g->edges[pe.host_edge];
        if (he.d.kind != SR_EDGE_CONV) dense_rows += g->nodes[he.d.tgt].d.c;
    }
    const int off_copies = take((int)sizeof(RsCopy) * (n_copies + dense_rows), 16);
    for (size_t i = 0; i < E.pe.size(); ++i)
        if (E.pe[i].type == RS_E_GATHER) E.pe[i].lut_off = take((int)E.luts[i].size() * 4, 16);
    for (int v = 0; v < n_nodes; ++v) {
        RsPlanNode& p = E.pn[v];
        if (p.kind != RS_CONV) continue;
        int npix = 0;
        for (int r = 0; r < cs; ++r) npix = std::max(npix, (p.lo[r + 1] - p.lo[r]) * g->nodes[v].d.w);
        p.pix_entries = (npix + 15) / 16 * 16;
        p.pix_off = take(p.pix_entries * 4, 16);
    }
    E.blob_bytes = rs_up16(off);
    off = E.blob_bytes;
    E.zero_off = take(128, 128);
    for (int v = 0; v < n_nodes; ++v) {
        RsPlanNode& p = E.pn[v];
        const sr_node_desc& d = g->nodes[v].d;
        if (p.kind != RS_INPUT) p.bias_off = take(rs_up16(d.c * 4), 16);
        if (p.kind == RS_DENSE) p.slot_off = take(2 * std::max(1, p.n_slots) * d.c * 4, 16);
    }
    for (int v = 0; v < n_nodes; ++v) {
        RsPlanNode& p = E.pn[v];
        const sr_node_desc& d = g->nodes[v].d;
        int rows = 0;
        for (int r = 0; r < cs; ++r) rows = std::max(rows, p.shi[r] - p.slo[r]);
        if (p.kind == RS_DENSE) p.buf_bytes = rs_up16(d.c * 2);
        else if (p.kind == RS_INPUT) p.buf_bytes = rs_up16(((p.in_pt + rows + p.in_pb) * p.in_pitch + p.in_tail_len) * 2);
        else p.buf_bytes = rs_up128(rows * d.w * d.c * 2);
        const int nb = p.kind == RS_INPUT ? p.in_nb : 2;
        for (int i = 0; i < nb; ++i) p.buf[i] = take(p.buf_bytes, 128);
    }
    for (int v = 0; v < n_nodes; ++v) {
        RsPlanNode& p = E.pn[v];
        if (p.kind == RS_CONV) p.w_off = take(p.ksteps * (g->nodes[v].d.c / 32) * 1024, 128);
    }
    if (off > kRsSmemMax) return false;
    // dense weights in shared memory if every slice fits, else they are read from global memory (L2)
    const int before_dense = off;
    E.dense_in_smem = true;
    for (RsPlanEdge& pe : E.pe) {
        const SrHostEdge& he = g->edges[pe.host_edge];
        if (he.d.kind == SR_EDGE_CONV) continue;
        const RsPlanNode& sp = E.pn[he.d.src];
        const sr_node_desc& sd = g->nodes[he.d.src].d;
        const int Cout = g->nodes[he.d.tgt].d.c;
        int max_slice = 0;
        for (int r = 0; r < cs; ++r) {
            int n = 0;
            if (he.d.kind == SR_EDGE_MEAN_DENSE) n = sd.c;
            else if (sp.kind == RS_CONV) n = (sp.lo[r + 1] - sp.lo[r]) * sd.w * sd.c;
            else n = r == 0 ? sd.c : 0;
            max_slice = std::max(max_slice, n);
        }
        const int o = take(Cout * max_slice * 2, 16);
        for (int r = 0; r < cs; ++r) pe.wd_off[r] = o;
    }
    if (off > kRsSmemMax) {
        off = before_dense;
        E.dense_in_smem = false;
        for (RsPlanEdge& pe : E.pe)
            for (int r = 0; r < kRsMaxCluster; ++r) pe.wd_off[r] = -1;
    }
    E.smem_bytes = rs_up128(off);
    E.offs.nodes = off_nodes;
    E.offs.edges = off_edges;
    E.offs.units = off_units;
    E.offs.ubegin = off_ubegin;
    E.offs.copies = off_copies;
    return true;
}

RsEngine* rs_of(const sr_graph* g) { return static_cast<RsEngine*>(g->rs); }

}  // namespace

void sr_rs_destroy(sr_graph* g)
{
    if (RsEngine* E = rs_of(g))
        for (cudaEvent_t e : E->ev) cudaEventDestroy(e);
    delete rs_of(g);
    g->rs = nullptr;
}

bool sr_rs_available(const sr_graph* g) { return g->rs != nullptr; }

void sr_rs_describe(const sr_graph* g, int* cluster_size, int* warps, int* smem_bytes, int* heads_on_chip)
{
    const RsEngine* E = rs_of(g);
    *cluster_size = E ? E->cs : 0;
    *warps = E ? E->warps : 0;
    *smem_bytes = E ? E->smem_bytes : 0;
    *heads_on_chip = E && E->dense_in_smem ? 1 : 0;
}

sr_status sr_rs_plan(sr_graph* g, size_t& offset)
{
    sr_rs_destroy(g);
    if (!g->opt_resident || g->opt_engine != 0 || g->dtype != SR_DTYPE_BF16) return SR_OK;
    const int n_nodes = (int)g->nodes.size(), n_edges = (int)g->edges.size();
    if (n_nodes > 32 || n_edges > 64 || g->groups.size() > 30 || g->groups.empty()) return SR_OK;
    if ((int)g->input_nodes.size() > SR_MAX_INPUTS) return SR_OK;
    RsEngine* E = new RsEngine();
    E->pn.assign(n_nodes, RsPlanNode());
    E->pe_of_host_edge.assign(n_edges, -1);
    bool ok = true;
    // node kinds
    for (int v = 0; v < n_nodes && ok; ++v) {
        const SrHostNode& n = g->nodes[v];
        RsPlanNode& p = E->pn[v];
        if (n.is_input) {
            p.kind = RS_INPUT;
            if ((n.d.w * n.d.c) % 2 != 0) ok = false;
        } else if (n.dense_target) {
            p.kind = RS_DENSE;
            if (n.d.c > kRsMaxDenseC) ok = false;
        } else {
            p.kind = RS_CONV;
            if (n.d.c % 32 != 0 || n.d.c > 256) ok = false;
        }
    }
    if (ok && E->pn[g->info.output_node].kind != RS_DENSE) ok = false;
    // edges, grouped by target
    for (int v = 0; v < n_nodes && ok; ++v) {
        const SrHostNode& n = g->nodes[v];
        RsPlanNode& p = E->pn[v];
        p.first_edge = (int)E->pe.size();
        int ks = 0;
        for (int e : n.in_edges) {
            const SrHostEdge& he = g->edges[e];
            const RsPlanNode& sp = E->pn[he.d.src];
            const sr_node_desc& sd = g->nodes[he.d.src].d;
            RsPlanEdge pe;
            pe.host_edge = e;
            if (he.d.kind == SR_EDGE_CONV) {
                if (p.kind != RS_CONV || sp.kind == RS_DENSE || he.k_eff > 15) ok = false;
                if (sp.kind == RS_CONV) {
                    pe.type = RS_E_MMA;
                    pe.ksteps = he.k_eff * he.k_eff * (sd.c / 16);
                } else {
                    // input nodes are stored unswizzled and read by the table-driven path
                    pe.type = RS_E_GATHER;
                    pe.Kreal = he.k_eff * he.k_eff * sd.c;
                    if (pe.Kreal > 64 || sd.c > 255) ok = false;
                    pe.ksteps = (pe.Kreal + 15) / 16;
                }
                pe.ks0 = ks;
                ks += pe.ksteps;
            } else {
                if (p.kind != RS_DENSE || sp.kind == RS_INPUT || sd.c % 8 != 0) ok = false;
                pe.type = he.d.kind == SR_EDGE_DENSE ? RS_E_DENSE : RS_E_MEAN;
                if (sp.kind == RS_DENSE && pe.type == RS_E_MEAN) pe.type = RS_E_DENSE;   // mean over one pixel
            }
            E->pe_of_host_edge[e] = (int)E->pe.size();
            E->pe.push_back(pe);
            E->pn[he.d.src].has_consumers = true;
        }
        p.ksteps = ks;
    }
    if (!ok) {
        delete E;
        return SR_OK;
    }
    // input nodes are kept zero-padded (top / bottom rows, left / right columns as wide as any consumer's filter
    // reaches) so that the few-channel path never checks bounds
    for (int v = 0; v < n_nodes && ok; ++v) {
        RsPlanNode& p = E->pn[v];
        if (p.kind != RS_INPUT) continue;
        const sr_node_desc& d = g->nodes[v].d;
        int pt = 0, pb = 0, kmax = 1;
        bool has0 = false, has1 = false;
        for (const RsPlanEdge& pe : E->pe) {
            const SrHostEdge& he = g->edges[pe.host_edge];
            if (he.d.src != v) continue;
            pt = std::max(pt, he.pad_eff);
            pb = std::max(pb, he.k_eff - 1 - he.pad_eff);
            kmax = std::max(kmax, he.k_eff);
            (he.R ? has1 : has0) = true;
        }
        p.in_pt = pt;
        p.in_pb = pb;
        p.in_ple = (pt * d.c + 1) / 2 * 2;
        p.in_pitch = (p.in_ple + d.w * d.c + pb * d.c + 1) / 2 * 2;
        p.in_tail_len = ((kmax - 1) * p.in_pitch + kmax * d.c + 1) / 2 * 2;
        p.in_wpr = d.w * d.c / 2;
        p.in_magic = ((1 << 20) + p.in_wpr - 1) / p.in_wpr;
        p.in_nb = (has0 && has1) ? 3 : 2;
        p.in_lead = has0 ? 2 : 1;
        const int nw = d.h * p.in_wpr;
        if (nw > 8192) ok = false;
        for (int i = 0; i < nw && ok; ++i)
            if ((int)(((unsigned)i * (unsigned)p.in_magic) >> 20) != i / p.in_wpr) ok = false;
    }
    if (!ok) {
        delete E;
        return SR_OK;
    }
    // lookup tables of the few-channel edges: the offset of every k index (filter row, column, channel) inside a
    // pixel's window of the padded source; padded k indices point at the window's first element (their weights are 0)
    E->luts.assign(E->pe.size(), std::vector<uint32_t>());
    for (size_t i = 0; i < E->pe.size(); ++i) {
        const RsPlanEdge& pe = E->pe[i];
        if (pe.type != RS_E_GATHER) continue;
        const SrHostEdge& he = g->edges[pe.host_edge];
        const int Cs = g->nodes[he.d.src].d.c, P = E->pn[he.d.src].in_pitch;
        std::vector<uint32_t>& L = E->luts[i];
        L.assign((size_t)pe.ksteps * 16, 0u);
        for (int kk = 0; kk < pe.Kreal; ++kk) {
            const int tap = kk / Cs, ci = kk % Cs;
            L[kk] = (uint32_t)((tap / he.k_eff) * P + (tap % he.k_eff) * Cs + ci);
        }
    }
    // cluster size: the largest that still gives every sequence its own cluster in one wave, else the
    // smallest that fits
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    std::vector<int> order;
    if (g->opt_rs_cluster > 0) {
        order.push_back(g->opt_rs_cluster);
    } else {
        for (int c = kRsMaxCluster; c >= 1; c >>= 1)
            if (g->batch * c <= sms) order.push_back(c);
        for (int c = 1; c <= kRsMaxCluster; c <<= 1)
            if (g->batch * c > sms) order.push_back(c);
    }
    // 24 warps (80 registers each) hide the shared-memory latencies best on B200; with 32 the 64-register build spills
    const int warps = std::min(kRsMaxWarps, g->opt_rs_warps > 0 ? g->opt_rs_warps : 24);
    bool placed = false;
    for (int c : order)
        if (rs_layout(g, *E, c, warps)) {
            placed = true;
            break;
        }
    if (!placed) {
        delete E;
        return SR_OK;
    }
    // workspace regions: per-rank tables, packed convolution weights, dense weights
    auto take = [&](size_t bytes) {
        SrRegion r;
        r.offset = offset;
        r.bytes = bytes;
        offset = sr_align_up(offset + bytes, 256);
        return r;
    };
    size_t wconv = 0, wdense = 0;
    for (int v = 0; v < n_nodes; ++v) {
        RsPlanNode& p = E->pn[v];
        if (p.kind != RS_CONV) continue;
        p.w_global = wconv;
        wconv += (size_t)p.ksteps * (g->nodes[v].d.c / 32) * 1024;
    }
    for (RsPlanEdge& pe : E->pe) {
        const SrHostEdge& he = g->edges[pe.host_edge];
        if (he.d.kind == SR_EDGE_CONV) continue;
        pe.wd_global = wdense;
        wdense += sr_align_up((size_t)g->nodes[he.d.tgt].d.c * he.K * 2, 16);
    }
    E->r_blobs = take((size_t)E->cs * E->blob_bytes);
    E->r_wconv = take(std::max<size_t>(16, wconv));
    E->r_wdense = take(std::max<size_t>(16, wdense));
    g->rs = E;
    return SR_OK;
}

sr_status sr_rs_bind(sr_graph* g)
{
    RsEngine* Ep = rs_of(g);
    if (!Ep) return SR_OK;
    RsEngine& E = *Ep;
    const int n_nodes = (int)g->nodes.size();
    const RsOffsets O = E.offs;
    for (int r = 0; r < E.cs; ++r) {
        std::vector<unsigned char> blob((size_t)E.blob_bytes, 0);
        RsHeader* H = reinterpret_cast<RsHeader*>(blob.data());
        RsNode* nodes = reinterpret_cast<RsNode*>(blob.data() + O.nodes);
        RsEdge* edges = reinterpret_cast<RsEdge*>(blob.data() + O.edges);
        RsUnit* units = reinterpret_cast<RsUnit*>(blob.data() + O.units);
        int32_t* ubegin = reinterpret_cast<int32_t*>(blob.data() + O.ubegin);
        RsCopy* copies = reinterpret_cast<RsCopy*>(blob.data() + O.copies);
        int n_copies = 0, dense_mask = 0, sync_after = 0;
        for (int v = 0; v < n_nodes; ++v) {
            const SrHostNode& hn = g->nodes[v];
            const RsPlanNode& p = E.pn[v];
            RsNode& d = nodes[v];
            d.kind = p.kind;
            d.H = hn.d.h; d.W = hn.d.w; d.C = hn.d.c; d.act = hn.d.act;
            d.level = hn.level - 1;
            d.lo = p.lo[r]; d.hi = p.lo[r + 1];
            d.slo = p.slo[r]; d.shi = p.shi[r];
            d.is_output = v == g->info.output_node;
            d.input_slot = hn.input_slot;
            for (int i = 0; i < 3; ++i) d.buf[i] = p.buf[i];
            d.bias_off = p.bias_off;
            d.w_off = p.w_off;
            d.first_edge = p.first_edge;
            d.n_edges = (int)hn.in_edges.size();
            d.buf_bytes = p.buf_bytes;
            d.ksteps = p.ksteps;
            d.up_lo = d.up_hi = d.up_slo = d.dn_lo = d.dn_hi = d.dn_slo = 0;
            if (p.kind != RS_DENSE) {
                if (r > 0) {
                    d.up_lo = d.lo;
                    d.up_hi = std::min(d.hi, p.shi[r - 1]);
                    d.up_slo = p.slo[r - 1];
                }
                if (r + 1 < E.cs) {
                    d.dn_lo = std::max(d.lo, p.slo[r + 1]);
                    d.dn_hi = d.hi;
                    d.dn_slo = p.slo[r + 1];
                }
            }
            d.slot_off = p.slot_off;
            d.n_slots = p.n_slots;
            d.has_consumers = p.has_consumers;
            d.in_pitch = p.in_pitch; d.in_pt = p.in_pt; d.in_ple = p.in_ple; d.in_wpr = p.in_wpr; d.in_magic = p.in_magic;
            d.in_nb = p.in_nb; d.in_lead = p.in_lead;
            d.in_tail = 0;
            if (p.kind == RS_INPUT) {
                int rows = 0;
                for (int rr = 0; rr < E.cs; ++rr) rows = std::max(rows, p.shi[rr] - p.slo[rr]);
                d.in_tail = (p.in_pt + rows + p.in_pb) * p.in_pitch;
            }
            d.pix_off = p.pix_off;
            if (p.kind == RS_CONV) {
                uint32_t* pix = reinterpret_cast<uint32_t*>(blob.data() + p.pix_off);
                const int npix = (d.hi - d.lo) * d.W;
                for (int j = 0; j < p.pix_entries; ++j) {
                    const int y = d.lo + j / d.W, x = j % d.W;
                    const uint32_t up = (r > 0 && y >= d.up_lo && y < d.up_hi) ? 0x80000000u : 0u;
                    const uint32_t dn = (r + 1 < E.cs && y >= d.dn_lo && y < d.dn_hi) ? 0x40000000u : 0u;
                    pix[j] = j < npix ? (up | dn | ((uint32_t)y << 15) | (uint32_t)x) : 0xFFFFFFFFu;
                }
            }
            d.gstate[0] = g->ws + hn.state[0].offset;
            d.gstate[1] = g->ws + hn.state[1].offset;
            if (p.kind == RS_DENSE) {
                dense_mask |= 1 << d.level;
                if (p.has_consumers) sync_after = 1;
            }
            if (p.kind != RS_INPUT) copies[n_copies++] = RsCopy{g->ws + hn.bias.offset, p.bias_off, rs_up16(hn.d.c * 4)};
            if (p.kind == RS_CONV)
                copies[n_copies++] = RsCopy{g->ws + E.r_wconv.offset + p.w_global, p.w_off, p.ksteps * (hn.d.c / 32) * 1024};
        }
        for (size_t i = 0; i < E.pe.size(); ++i) {
            const RsPlanEdge& pe = E.pe[i];
            const SrHostEdge& he = g->edges[pe.host_edge];
            const RsPlanNode& sp = E.pn[he.d.src];
            const sr_node_desc& sd = g->nodes[he.d.src].d;
            RsEdge& d = edges[i];
            d.src = he.d.src;
            d.type = pe.type;
            d.k = he.k_eff; d.stride = he.stride_eff; d.pad = he.pad_eff;
            d.R = he.R;
            d.ksteps = pe.ksteps;
            d.lut_off = pe.lut_off;
            d.Kreal = pe.Kreal;
            d.wd_off = -1; d.wd_ld = 0; d.n_chunks = 0; d.x_chunk0 = 0; d.wchunk_mod = 0;
            d.scale = 1.f;
            d.wd_global = nullptr;
            d.wd_gld = 0;
            d.g_const = d.g_ys = d.g_xs = 0;
            if (pe.type == RS_E_GATHER) {
                d.g_const = (-he.pad_eff - sp.slo[r] + sp.in_pt) * sp.in_pitch + sp.in_ple - he.pad_eff * sd.c;
                d.g_ys = he.stride_eff * sp.in_pitch;
                d.g_xs = he.stride_eff * sd.c;
            }
            if (pe.type == RS_E_GATHER)
                std::memcpy(blob.data() + pe.lut_off, E.luts[i].data(), E.luts[i].size() * 4);
            if (he.d.kind != SR_EDGE_CONV) {
                const int Cout = g->nodes[he.d.tgt].d.c;
                const int nch = sd.c / 8;
                int k_begin = 0, k_len = 0;          // this rank's slice of the flattened source, in elements
                if (sp.kind == RS_CONV) {
                    k_begin = sp.lo[r] * sd.w * sd.c;
                    k_len = (sp.lo[r + 1] - sp.lo[r]) * sd.w * sd.c;
                    d.x_chunk0 = (sp.lo[r] - sp.slo[r]) * sd.w * nch;
                } else if (r == 0) {
                    k_len = sd.c;
                }
                d.n_chunks = k_len / 8;
                const char* wg = g->ws + E.r_wdense.offset + pe.wd_global;
                if (pe.type == RS_E_MEAN) {
                    d.wchunk_mod = nch;
                    d.scale = 1.f / (float)(sd.h * sd.w);
                    d.wd_global = wg;
                    d.wd_gld = sd.c;
                    if (pe.wd_off[r] >= 0) {
                        d.wd_off = pe.wd_off[r];
                        d.wd_ld = sd.c;
                        for (int o = 0; o < Cout; ++o)
                            copies[n_copies++] = RsCopy{wg + (size_t)o * sd.c * 2, d.wd_off + o * sd.c * 2, sd.c * 2};
                    }
                } else {
                    d.wd_global = wg + (size_t)k_begin * 2;
                    d.wd_gld = he.K;
                    if (pe.wd_off[r] >= 0 && k_len > 0) {
                        d.wd_off = pe.wd_off[r];
                        d.wd_ld = k_len;
                        for (int o = 0; o < Cout; ++o)
                            copies[n_copies++] =
                                RsCopy{wg + ((size_t)o * he.K + k_begin) * 2, d.wd_off + o * k_len * 2, k_len * 2};
                    }
                }
            }
        }
        std::memcpy(units, E.units[r].data(), sizeof(RsUnit) * E.units[r].size());
        std::memcpy(ubegin, E.ubegin[r].data(), sizeof(int32_t) * E.ubegin[r].size());
        H->n_nodes = n_nodes;
        H->n_edges = (int)E.pe.size();
        H->n_levels = E.n_levels;
        H->n_warps = E.warps;
        H->off_nodes = O.nodes; H->off_edges = O.edges; H->off_units = O.units; H->off_ubegin = O.ubegin;
        H->off_copies = O.copies;
        H->n_copies = n_copies;
        H->zero_off = E.zero_off;
        H->smem_bytes = E.smem_bytes;
        H->dense_level_mask = dense_mask;
        H->sync_after_finalize = sync_after;
        H->blob_bytes = E.blob_bytes;
        if (cudaMemcpy(g->ws + E.r_blobs.offset + (size_t)r * E.blob_bytes, blob.data(), blob.size(), cudaMemcpyHostToDevice) !=
            cudaSuccess)
            return SR_ERR_CUDA;
    }
    return SR_OK;
}

sr_status sr_rs_set_weights(sr_graph* g, int edge, const float* w_eff)
{
    RsEngine* Ep = rs_of(g);
    if (!Ep) return SR_OK;
    RsEngine& E = *Ep;
    const RsPlanEdge& pe = E.pe[E.pe_of_host_edge[edge]];
    const SrHostEdge& he = g->edges[edge];
    const int Cout = g->nodes[he.d.tgt].d.c, Cs = g->nodes[he.d.src].d.c;
    auto bf16 = [](float f) {
        uint32_t u;
        std::memcpy(&u, &f, 4);
        if ((u & 0x7F800000u) != 0x7F800000u) u += 0x7FFFu + ((u >> 16) & 1u);
        return (uint16_t)(u >> 16);
    };
    if (he.d.kind == SR_EDGE_CONV) {
        // ldmatrix order: per k-step and 32 output channels two 512-byte blocks; lane l of a block holds 8
        // consecutive k, starting at k = ((l >> 3) & 1) * 8, of column (l & 7) of n-tile hb * 2 + (l >> 4).
        // Column c of n-tile nt is output channel (c >> 1) * 8 + nt * 2 + (c & 1) of the 32, which makes the
        // eight accumulator columns of a lane consecutive channels
        const int nb = Cout / 32, nc16 = Cs / 16;
        std::vector<uint16_t> pk((size_t)pe.ksteps * nb * 512, 0);
        for (int ks = 0; ks < pe.ksteps; ++ks)
            for (int b = 0; b < nb; ++b)
                for (int hb = 0; hb < 2; ++hb)
                    for (int l = 0; l < 32; ++l) {
                        const int nt = hb * 2 + (l >> 4), col = l & 7, kh = (l >> 3) & 1;
                        const int n = b * 32 + (col >> 1) * 8 + nt * 2 + (col & 1);
                        for (int j = 0; j < 8; ++j) {
                            float w = 0.f;
                            if (pe.type == RS_E_MMA) {
                                const int tap = ks / nc16, c = (ks % nc16) * 16 + kh * 8 + j;
                                w = w_eff[(size_t)n * he.K + (size_t)tap * Cs + c];
                            } else {
                                const int kk = ks * 16 + kh * 8 + j;
                                if (kk < pe.Kreal) w = w_eff[(size_t)n * he.K + kk];
                            }
                            pk[(((size_t)b * pe.ksteps + ks) * 2 + hb) * 256 + l * 8 + j] = bf16(w);
                        }
                    }
        // in the node's region the 32-channel blocks are outermost, then the k-steps of all edges in order
        const RsPlanNode& p = E.pn[he.d.tgt];
        for (int b = 0; b < nb; ++b) {
            char* dst = g->ws + E.r_wconv.offset + p.w_global + ((size_t)b * p.ksteps + pe.ks0) * 1024;
            if (cudaMemcpy(dst, pk.data() + (size_t)b * pe.ksteps * 512, (size_t)pe.ksteps * 1024, cudaMemcpyHostToDevice) != cudaSuccess)
                return SR_ERR_CUDA;
        }
    } else {
        std::vector<uint16_t> pk((size_t)Cout * he.K);
        for (size_t i = 0; i < pk.size(); ++i) pk[i] = bf16(w_eff[i]);
        if (cudaMemcpy(g->ws + E.r_wdense.offset + pe.wd_global, pk.data(), pk.size() * 2, cudaMemcpyHostToDevice) != cudaSuccess)
            return SR_ERR_CUDA;
    }
    return SR_OK;
}

sr_status sr_rs_launch(sr_graph* g, int T, const SrFrameCtl& init, cudaStream_t s)
{
    RsEngine* E = rs_of(g);
    if (!E) return SR_ERR_STATE;
    if (!E->attr_set) {
        if (cudaFuncSetAttribute(sr_resident_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize, E->smem_bytes) != cudaSuccess ||
            cudaFuncSetAttribute(sr_resident_kernel<768>, cudaFuncAttributeMaxDynamicSharedMemorySize, E->smem_bytes) != cudaSuccess ||
            cudaFuncSetAttribute(sr_resident_kernel<1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, E->smem_bytes) != cudaSuccess)
            return SR_ERR_CUDA;
        E->attr_set = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(g->batch * E->cs));
    cfg.blockDim = dim3((unsigned)(E->warps * 32));
    cfg.dynamicSmemBytes = (size_t)E->smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)E->cs;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = E->cs > 1 ? 1 : 0;
    const unsigned char* blobs = reinterpret_cast<const unsigned char*>(g->ws + E->r_blobs.offset);
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
    cudaError_t le;
    if (E->warps <= 16) le = cudaLaunchKernelEx(&cfg, sr_resident_kernel<512>, blobs, E->blob_bytes, ctl, init, T, E->cs);
    else if (E->warps <= 24) le = cudaLaunchKernelEx(&cfg, sr_resident_kernel<768>, blobs, E->blob_bytes, ctl, init, T, E->cs);
    else le = cudaLaunchKernelEx(&cfg, sr_resident_kernel<1024>, blobs, E->blob_bytes, ctl, init, T, E->cs);
    if (le != cudaSuccess) return SR_ERR_CUDA;
    if (timed) {
        cudaEventRecord(E->ev[E->ev_used + 1], s);
        E->ev_used += 2;
    }
    return SR_OK;
}

// Sum of the event-timed durations of the resident launches since the last call (synchronises).
sr_status sr_rs_timing(sr_graph* g, double* ms, long long* launches)
{
    RsEngine* E = rs_of(g);
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
