// Tensor-core engine: the node update  x_v = sigma(b_v + sum_e f_e(theta_e, x_src(e)))  (paper Sec. A1.2)
// for all convolutional nodes of one launch group as ONE grouped implicit GEMM on tcgen05 / TMEM.
//
// The sum over the incoming edges of a node is one convolution over the concatenated sources (paper
// Sec. A notes the equivalence): the K loop of an output tile simply walks the K-blocks of every
// incoming edge, tap by tap, into one TMEM accumulator.
//
// GEMM shape.  D[c_out][pixel] = sum_k W[c_out][k] * X[pixel][k]: the weights are the M operand
// (128 rows per instruction, one tile per 128 output channels), up to 256 output pixels are the N operand.
// Measured on B200, one tcgen05.mma of M = 128 costs about 110 cycles however small N is and 128
// cycles at N = 256, and a tcgen05.commit is only free if about eight MMAs lie between commits; so
// every instruction is given N = 256 pixels and commits come once per eight MMAs.
//
// Operands.  K-block = one filter tap x up to 64 input channels.  Activation tiles come straight from
// the NHWC state of the source node through 4-D TMA boxes (zero fill outside the image = zero
// padding); a stride-s edge reads one of s*s residue-class views of the source, so every tap is again
// a dense box.  The node's weight matrix [C_out][K] (K-major) keeps its columns in the order the K loop
// walks them, so that consecutive K-blocks of equal width are one 3-D tensor and a weight group of two
// K-blocks is ONE TMA copy.  Few-channel input edges (C_in = 1 or 3) are staged per frame into an im2col
// tensor with K padded to 16/32/64 so that they are ordinary K-blocks.
//
// Pixel tile.  A tile is tb samples x th rows x tw columns (tw a multiple of 8, so an image row of
// the tile is a whole number of swizzle atoms).  Every activation box holds th + sep rows per sample
// (sep = k - 1 of the node's stride-1 k x k edges), and the N columns of the GEMM are the rows of
// that stacked box: column n = (b * (th + sep) + r) * tw + x.  Columns with r >= th are never stored.
// This makes the k taps of one filter column row-shifted windows of ONE box: the box is loaded once
// per filter column and the shared-memory descriptor of tap ky just starts ky * tw rows further down
// (with 8-wide tiles the taps of a filter row share the box as well).
//
// Work items.  An item is one pixel tile of one plan (a node, or two narrow nodes fused, see TcNode);
// optionally a PAIR of neighbouring tiles ("lanes") that share every weight box (lane 0 accumulates in
// TMEM columns 0..255, lane 1 in 256..511).  The persistent CTAs take the items from one shared list.
//
// Warp roles in a CTA of 384 threads: warp 0 = weight producer (and keeper of the item queue); warp 3 =
// activation producer; warp 2 = scout (all barrier waits and address arithmetic; publishes one 16-byte
// burst descriptor per eight or so MMAs); warp 1 = MMA issuer (owns TMEM; reads descriptors and issues,
// nothing else); warps 4..11 = epilogue (TMEM lane = output channel; bias, ReLU, bf16, NHWC stores in
// which a warp writes 32 consecutive channels of one pixel).  Every wait is bounded; on expiry the kernel
// records an error in the frame control block, waits for its own copies, frees TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <map>
#include <tuple>
#include <vector>

#include "sr_tc.h"

namespace {

constexpr int kMaxCols = 256;                         // pixels (N of the MMA) per lane
constexpr int kThreads = 384;
constexpr int kEpiWarps = 8;                          // warps 4..11
constexpr int kFifo = 16;                             // burst descriptors in flight between scout and issuer
constexpr int kMaxA = 4;                              // activation ring depth
constexpr int kMaxW = 8;                              // weight ring depth (one weight group per slot)
// Dynamic shared memory of a CTA.  With the 24 KiB of static shared memory this leaves about 20 KiB of the SM's 228 KiB
// free: the other kernels of a frame (input staging, dense heads: up to 7.4 KiB per block) run on a second stream beside
// the persistent CTAs, and measured on B200 they queue behind them, frame after frame, once less than about 10 KiB of
// the SM's shared-memory partition is left (a 117 us frame then takes 170 us).
constexpr int kSmemBudget = 184 * 1024;
constexpr int kMaxNodeKb = 128;                       // K-blocks per node the shared-memory tables hold

// One weight group (consecutive K-blocks of equal channel-block width, fetched by ONE copy) as the weight producer
// sees it (16 bytes).  A thread that waits for a slot, arms the barrier and starts a copy gets through about one
// copy per 420 cycles (measured on B200), so copies must be large: a group, not a K-block.
// The K-block of a staged few-channel edge is two MMAs long, and its activation box would hold one of the two or three
// large activation slots for that short time only to keep the next filter's box from being requested early.  Such a
// box travels in the weight ring instead: the group is then the block's weights followed by its activation box.
struct TcKbWeight {
    uint16_t blk;           // index of the group's first K-block in its tensor map (a run of equally wide blocks)
    uint16_t w_map;         // tensor map of that run: dims (channels of a block, output channels, blocks)
    uint16_t w_bytes16;     // (bytes of the whole group, the activation box included) / 16
    uint16_t x_off16;       // (offset of the activation box inside the slot) / 16; 0 = the group has none
    uint16_t x_map0, x_map1;// tensor map of that box for source frame parity 0 / 1
    uint8_t c0_16;          // (first channel of the box) / 16
    uint8_t flags;          // 1: the edge reads frame t (R = 1), else frame t+1
    uint16_t pad_;
};
static_assert(sizeof(TcKbWeight) == 16, "copied as one 16-byte word");

// One activation box of a node's reduction as the activation producer sees it (16 bytes); only the K-blocks that
// open a fresh box have one.
struct TcKbAct {
    uint16_t x_map0, x_map1;// tensor map of the activation box for source frame parity 0 / 1
    uint16_t x_bytes16;     // (bytes of the activation box) / 16
    int8_t qx, qy;          // box origin relative to the tile origin (columns, rows)
    uint8_t c0_16;          // (first channel of the box) / 16
    uint8_t flags;          // 1: the edge reads frame t (R = 1), else frame t+1
    uint8_t pad_[6];
};
static_assert(sizeof(TcKbAct) == 16, "copied as one 16-byte word");

// One burst (= one weight group: one or two K-blocks of equal descriptor state) as the scout sees it (8 bytes).  The
// scout is a single thread whose every shared-memory access or barrier probe costs tens to hundreds of cycles, so
// everything that can be worked out on the host is.
struct TcBurst {
    uint16_t xa_off16;      // (byte offset of the first block's operand window inside its activation slot) / 16
    uint16_t xb_off16;      // two blocks: the same for the second block; one block: for lane 1's window of that block
    uint8_t flags;          // 1 / 2: the first / second block opens a fresh activation slot; 4 / 8: the first / second
                            // block is the last reader of its slot; 16: the burst has two blocks; 32: the activation
                            // box lies in the burst's weight slot (xa_off16 counts from the start of that slot)
    uint8_t state;          // descriptor state of the burst: index into the node's state table
    uint16_t pad_;
};
static_assert(sizeof(TcBurst) == 8, "copied as one 8-byte word");

// Descriptor state shared by consecutive bursts of a node (16 bytes).
struct TcState {
    uint32_t desc_hi;       // upper word of the weight descriptors (swizzle, SBO, version)
    uint32_t x_hi;          // upper word of the activation descriptors (SBO = one image row of the box)
    uint16_t n_k16;         // MMA steps (K = 16 each) per K-block
    uint16_t w_step16;      // (bytes of one block's weights) / 16
    uint32_t pad_;
};
static_assert(sizeof(TcState) == 16, "read as one 16-byte word");

// A plan can cover TWO nodes of at most 64 channels each that have the same shape: an M = 128 instruction on a
// 64-channel node is half empty, so the second node's weights take rows 64..127 and every K-block of a source both
// read (same filter geometry, same frame) serves both.  TMEM lanes 64..127 then belong to the second node.  Nodes are
// paired if they share a source, or if one of them has next to no reduction of its own.
struct TcNode {
    void* state[2];
    const float* bias;
    void* state2[2];                // the second node of a fused plan (fused != 0)
    const float* bias2;
    int32_t act2, fused;
    int32_t H, W, C, act;
    int32_t tw, th, tb, sep;        // geometry of one lane's tile (see the file comment)
    int32_t n_cols;                 // N of the MMA: stacked rows of a lane's tile, rounded up to 32
    int32_t l1_dw, l1_db;           // where lane 1's tile lies relative to lane 0's: columns, samples
    int32_t first_state, pad_;      // first entry of the node in the state table
    int32_t first_act, n_act;       // range in the activation-box table
    int32_t first_wg, n_wg;         // range in the weight-group table and in the burst table (one burst per group)
};

struct TcTile { int32_t node, b0, h0, w0, m0, lanes, pad_[2]; };   // m0: first output channel; lanes: 1 or 2 pixel tiles

struct TcStem {             // a few-channel input edge staged as im2col rows
    const void* src[2];
    void* dst[2];
    int32_t Hs, Ws, Cs, Ho, Wo, k, stride, pad, Kp, K;
};

// ------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait.  Returns false if the limit expired or another role already gave up.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit)
{
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 32; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, limit);
}
// Wait for a copy this thread started itself, before the CTA gives up its shared memory.  It has its own limit and
// does not look at the abort flag: after another role gave up, the copies in flight still have to land.
__device__ __noinline__ void mbar_wait_drain(uint32_t bar, uint32_t parity, long long limit)
{
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > limit) return;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void* map, uint32_t bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
// Ask for a box to be brought into L2 (no shared memory, no barrier: fire and forget).
__device__ __forceinline__ void tma_prefetch_4d(const void* map, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void* map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w)
{
    asm volatile("st.volatile.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.volatile.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
// Same with the descriptors given as (address word, shared upper word).
__device__ __forceinline__ void tc_mma_bf16_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                                 uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }


// ------------------------------------------------------------------------------------------ the kernel
// Burst descriptors (scout -> issuer): 16 bytes, written and read as one 128-bit access.
//   x : bits 0-15 sequence number; 16 kind (1 = state); 29 stop
//       burst: 17-18 K-blocks in the burst (1 or 2); 19 first MMA of each lane overwrites its accumulator;
//              20-21 lanes to issue; 22-23 lanes whose accumulator is complete after this burst; 24-27 activation
//              slots to hand back; 28 hand the weight slot of the burst back
//       state: 17-19 K = 16 steps per K-block; 20 / 21 accumulator of lane 0 / 1; 22-27 MMA columns / 8
//   y, z, w (burst): lower descriptor words, ready to use: y the weights of the (first) K-block.  A burst of ONE
//       K-block applies it to every lane named: z = lane 0's activation window, w = lane 1's.  A burst of TWO
//       K-blocks belongs to a single tile (lane 0's accumulator): z = first block's window, w = second block's, whose
//       weights lie one block further on in the slot (the step is part of the state).
//       w bits 24-31 repeat the low sequence bits (a torn read would show).
//   y, z (state): upper descriptor words of the weight and of the activation operand; w bits 0-15: the weight step / 16
constexpr uint32_t kDescState = 1u << 16, kDescStop = 1u << 29;

// Work items.  CTA c walks column c of a matrix of items made on the host (longest first onto the least loaded CTA);
// every role of the CTA works out the column's entries by itself, so the roles stay decoupled.  The kernel ends when
// its slowest CTA ends, and the cost of an item is only an estimate: measured on B200 such lists left that CTA 2-8 %
// above the mean.  So (sched != nullptr) the matrix holds only the larger items, and the smallest ones, a fifth of the
// work, form ONE shared list behind it from which every CTA takes, by a device-wide counter, when its own column is
// done: the weight producer asks the counter two items ahead and keeps the answers in a small queue in shared memory
// that the other roles read.  (ALL items in one shared list balanced the largest workload as well, but cost 3-8 % on
// workloads and rollouts with many small launches, where a role could no longer run ahead of the weight producer.)
constexpr int kTileQ = 8;                              // queue entries; no role is ever that many items ahead of the epilogue

// Index of this CTA's it-th item in the tile table, or -1 when there is none (any more).  own_len: the length of the
// CTA's column, -1 while the role has not reached its end.
__device__ __forceinline__ int tc_item(int it, int& own_len, const TcTile* __restrict__ tiles, int n_own, int n_tiles, const int* sched,
                                       const volatile int* tile_q, const volatile int* tile_n, volatile int* abort_flag, long long limit)
{
    if (own_len < 0) {
        const long long idx = (long long)blockIdx.x + (long long)it * gridDim.x;
        if (idx < n_own && tiles[idx].node >= 0) return (int)idx;
        own_len = it;
    }
    if (!sched || n_own >= n_tiles) return -1;
    const int j = it - own_len;                        // position in the CTA's share of the shared list
    if (*tile_n <= j) {
        const long long t0 = clock64();
        while (*tile_n <= j) {
            if (*abort_flag) return -1;
            if (clock64() - t0 > limit) {
                *abort_flag = 1;
                return -1;
            }
        }
    }
    __threadfence_block();
    return tile_q[j & (kTileQ - 1)];
}

__global__ void __launch_bounds__(kThreads, 2)
sr_tc_group_kernel(const CUtensorMap* __restrict__ maps, const TcNode* __restrict__ nodes,
                   const TcKbWeight* __restrict__ kb_weight, const TcKbAct* __restrict__ kb_act, const TcBurst* __restrict__ bursts, const TcState* __restrict__ states,
                   const TcTile* __restrict__ tiles, int n_tiles, SrFrameCtl* __restrict__ ctl, int t_off, int B,
                   int n_a, int a_slot, int n_w, int w_slot, int tmem_cols, long long wait_limit, int* sched, int n_own)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * kMaxA + 2 * kMaxW + 4];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int epi_stop;
    __shared__ uint4 w_tab[kMaxNodeKb];                    // K-block records of the weight producer's current node,
    __shared__ uint4 a_tab[kMaxNodeKb];                    // of the activation producer's
    __shared__ uint2 m_tab[kMaxNodeKb];                    // and the burst records of the scout's
    __shared__ __align__(16) uint16_t epi_buf[kEpiWarps][32 * 32];   // per epilogue warp: 32 pixels x 32 channels, bf16
    __shared__ int pix_off[2 * kMaxCols];                  // element offset of every pixel of both lanes, -1 = not stored
    __shared__ __align__(16) uint4 fifo[kFifo];            // burst descriptors, scout -> issuer
    __shared__ volatile uint32_t fifo_read;                // descriptors the issuer has taken
    __shared__ volatile int tile_q[kTileQ];                // items taken from the shared list (indices into the tile table, -1 = end)
    __shared__ volatile int tile_n;                        // how many of them so far
    __shared__ volatile int epi_items;                     // items of the shared list the epilogue has finished
    __shared__ volatile int epi_ti;                        // the epilogue's current item

    // A wait limit of zero (a host-side test hook) means "every wait has already expired": report it and return
    // before any barrier, tensor memory, copy or MMA is touched.
    if (wait_limit <= 0) {
        if (threadIdx.x == 0) atomicExch(&ctl->error, 1);
        return;
    }
    // weight ring first: an M = 128 instruction on a node with fewer than 128 output channels reads
    // rows past its weight box, which then still lie inside this allocation
    const uint32_t w_ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_ring = w_ring + (uint32_t)(n_w * w_slot);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t bar_afull = smem_u32(&bars[0]), bar_aempty = smem_u32(&bars[kMaxA]);
    const uint32_t bar_wfull = smem_u32(&bars[2 * kMaxA]), bar_wempty = smem_u32(&bars[2 * kMaxA + kMaxW]);
    const uint32_t bar_tfull = smem_u32(&bars[2 * kMaxA + 2 * kMaxW]), bar_tempty = bar_tfull + 16;

    if (threadIdx.x < kFifo) fifo[threadIdx.x] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        epi_stop = 0;
        fifo_read = 0;
        tile_n = 0;
        epi_items = 0;
        for (int s = 0; s < n_a; ++s) {
            mbar_init(bar_afull + 8 * s, 1);
            mbar_init(bar_aempty + 8 * s, 1);
        }
        for (int s = 0; s < n_w; ++s) {
            mbar_init(bar_wfull + 8 * s, 1);
            mbar_init(bar_wempty + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, kEpiWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    volatile int* abortp = &abort_flag;

    const long long t = ctl->t + t_off;                     // this launch computes frame t+1 from frame t
    const int prev = (int)(t & 1), cur = prev ^ 1;

    if (warp == 0) {
        // ---------------------------------------------------------------- weight producer
        // The three feeding roles (weights, activations, scout) walk the same work list independently.  At every
        // change of node the whole warp copies its view of the node's K-block table into shared memory; lane 0 then
        // runs out of shared memory.  Both rings are plain rings: slot after slot, one phase bit per lap.  Weights and
        // activations have a producer each, so that an activation box (needed once per filter) is requested as soon
        // as its slot is free and not only when the weight ring has advanced to it.
        int cached_node = -1;
        uint32_t w_nxt = 0, w_ph = 0, w_used = 0, w_par = 0;  // next slot, phase; slots filled, parity of the latest fill
        bool ok = true;
        // Items of the shared list: the counter is asked two items ahead, BEFORE this item's copies are issued, and its
        // answer (a round trip through the L2, microseconds) is put into the queue after them, so that the copies never
        // wait for it.  (Only a CTA whose own column is shorter than three items has to wait for its first answers.)
        int n_fetched = 0, v_next = 0, own_len = -1, col_len = -1, probed = 0;
        bool q_end = false, asked = false;
        auto put = [&](int v) {                                           // append one item (or the end mark) to the queue
            if (n_fetched - epi_items >= kTileQ) {
                const long long t0 = clock64();
                while (n_fetched - epi_items >= kTileQ)
                    if (abort_flag || clock64() - t0 > wait_limit) { abort_flag = 1; ok = false; return; }
            }
            tile_q[n_fetched & (kTileQ - 1)] = v < n_tiles ? v : -1;
            q_end = v >= n_tiles;
            __threadfence_block();
            tile_n = ++n_fetched;
        };
        for (int it = 0;; ++it) {
            int ti = -1;
            if (lane == 0) {
                asked = false;
                if (sched && n_own < n_tiles) {
                    // where does the own column end?  (looked up two items ahead)
                    while (col_len < 0 && probed <= it + 2) {
                        const long long idx = (long long)blockIdx.x + (long long)probed * gridDim.x;
                        if (idx >= n_own || tiles[idx].node < 0) col_len = probed;
                        else ++probed;
                    }
                    if (col_len >= 0) {
                        const int need = it + 3 - col_len;                // entries of the shared list that should be in the queue
                        while (!q_end && ok && n_fetched < need - 2) put(n_own + atomicAdd(sched, 1));   // needed right now
                        asked = !q_end && ok && n_fetched < need;
                        if (asked) v_next = n_own + atomicAdd(sched, 1);
                    }
                }
                if (ok) ti = tc_item(it, own_len, tiles, n_own, n_tiles, sched, tile_q, &tile_n, abortp, wait_limit);
            }
            ti = __shfl_sync(0xffffffffu, ti, 0);
            if (ti < 0) break;
            const TcTile tl = tiles[ti];
            if (tl.node < 0) break;                                   // the rest of this CTA's column of the work list is padding
            const int first_wg = nodes[tl.node].first_wg, n_wg = nodes[tl.node].n_wg;
            if (tl.node != cached_node) {
                __syncwarp();
                for (int i = lane; i < n_wg; i += 32) w_tab[i] = reinterpret_cast<const uint4*>(kb_weight)[first_wg + i];
                cached_node = tl.node;
                __syncwarp();
            }
            if (lane == 0) {
                const TcKbWeight* tab = reinterpret_cast<const TcKbWeight*>(w_tab);
                for (int kb = 0; kb < n_wg; ++kb) {
                    const TcKbWeight k = tab[kb];
                    const uint32_t s = w_nxt;
                    if (!mbar_wait(bar_wempty + 8 * s, w_ph ^ 1, abortp, wait_limit)) { ok = false; break; }
                    w_used |= 1u << s;
                    w_par = (w_par & ~(1u << s)) | (w_ph << s);
                    if (++w_nxt == (uint32_t)n_w) { w_nxt = 0; w_ph ^= 1; }
                    mbar_expect_tx(bar_wfull + 8 * s, (uint32_t)k.w_bytes16 << 4);
                    tma_load_3d(w_ring + s * w_slot, &maps[k.w_map], bar_wfull + 8 * s, 0, tl.m0, (int)k.blk);
                    if (k.x_off16) {                                      // a staged edge's activation box rides along
                        const int par = (k.flags & 1) ? prev : cur;
                        tma_load_4d(w_ring + s * w_slot + ((uint32_t)k.x_off16 << 4), &maps[par ? k.x_map1 : k.x_map0], bar_wfull + 8 * s,
                                    (int)k.c0_16 << 4, tl.w0, tl.h0, tl.b0);
                    }
                }
                if (asked && ok) put(v_next);                             // the counter's answer: the next item
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
        }
        if (lane == 0)                       // every copy this thread started must have landed before the CTA may exit
            for (uint32_t v = 0; v < (uint32_t)n_w; ++v)
                if ((w_used >> v) & 1) mbar_wait_drain(bar_wfull + 8 * v, (w_par >> v) & 1, wait_limit);
    } else if (warp == 3) {
        // ---------------------------------------------------------------- activation producer
        int cached_node = -1;
        uint32_t a_nxt = 0, a_ph = 0, a_used = 0, a_par = 0;
        bool ok = true;
        int own_len = -1;
        for (int it = 0;; ++it) {
            int ti = lane == 0 ? tc_item(it, own_len, tiles, n_own, n_tiles, sched, tile_q, &tile_n, abortp, wait_limit) : 0;
            ti = __shfl_sync(0xffffffffu, ti, 0);
            if (ti < 0) break;
            const TcTile tl = tiles[ti];
            if (tl.node < 0) break;
            const int first_act = nodes[tl.node].first_act, n_act = nodes[tl.node].n_act;
            if (tl.node != cached_node) {
                __syncwarp();
                for (int i = lane; i < n_act; i += 32) a_tab[i] = reinterpret_cast<const uint4*>(kb_act)[first_act + i];
                cached_node = tl.node;
                __syncwarp();
            }
            if (lane == 0) {
                const TcKbAct* tab = reinterpret_cast<const TcKbAct*>(a_tab);
                // With two or three slots a box is requested only about one filter ahead of its use, and a box that
                // comes from DRAM takes longer than that.  So every request is accompanied by an L2 prefetch of the
                // box two further on (of the next work item when this one ends, if it belongs to the same node).
                TcTile nx = tl;                                       // the next work item, looked up when its boxes come into reach
                nx.node = -1;
                bool nx_seen = false;
                for (int i = 0; i < n_act; ++i) {
                    const TcKbAct k = tab[i];
                    {
                        const int j = i + 2 < n_act ? i + 2 : i + 2 - n_act;
                        const bool here = i + 2 < n_act;
                        if (!here && !nx_seen) {
                            const long long idx = (long long)blockIdx.x + (long long)(it + 1) * gridDim.x;
                            if (own_len < 0 && idx < n_own) {             // the next entry of the own column (may be padding)
                                nx = tiles[idx];
                                nx_seen = nx.node >= 0;
                            }
                            if (!nx_seen && sched && n_own < n_tiles) {   // else the next answer of the counter, if it is there
                                const int j = it + 1 - (own_len < 0 ? it + 1 : own_len);
                                if (tile_n > j) {
                                    const int nti = tile_q[j & (kTileQ - 1)];
                                    if (nti >= 0) nx = tiles[nti];
                                    nx_seen = true;
                                }
                            }
                        }
                        if ((here || nx.node == tl.node) && j < n_act) {
                            const TcKbAct p = tab[j];
                            const TcTile& pt = here ? tl : nx;
                            const int par = (p.flags & 1) ? prev : cur;
                            tma_prefetch_4d(&maps[par ? p.x_map1 : p.x_map0], (int)p.c0_16 << 4, pt.w0 + p.qx, pt.h0 + p.qy, pt.b0);
                        }
                    }
                    const uint32_t s = a_nxt;
                    if (!mbar_wait(bar_aempty + 8 * s, a_ph ^ 1, abortp, wait_limit)) { ok = false; break; }
                    a_used |= 1u << s;
                    a_par = (a_par & ~(1u << s)) | (a_ph << s);
                    if (++a_nxt == (uint32_t)n_a) { a_nxt = 0; a_ph ^= 1; }
                    mbar_expect_tx(bar_afull + 8 * s, (uint32_t)k.x_bytes16 << 4);
                    const int par = (k.flags & 1) ? prev : cur;
                    tma_load_4d(a_ring + s * a_slot, &maps[par ? k.x_map1 : k.x_map0], bar_afull + 8 * s, (int)k.c0_16 << 4,
                                tl.w0 + k.qx, tl.h0 + k.qy, tl.b0);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
        }
        if (lane == 0)
            for (uint32_t v = 0; v < (uint32_t)n_a; ++v)
                if ((a_used >> v) & 1) mbar_wait_drain(bar_afull + 8 * v, (a_par >> v) & 1, wait_limit);
    } else if (warp == 2) {
        // ---------------------------------------------------------------- scout
        int cached_node = -1;
        uint32_t a_nxt = 0, a_ph = 0, w_nxt = 0, w_ph = 0;    // next slot of each ring and the phase of its barriers
        uint32_t n_pub = 0, a_cur = 0, a_base16 = 0;          // descriptors published, activation slot in use and its address / 16
        uint32_t cur_state = 0xFFFFFFFFu, w_hi = 0, x_hi = 0, nk = 0, w_step = 0;   // descriptor state of the current burst
        uint32_t st_w_hi = 0xFFFFFFFFu, st_x_hi = 0xFFFFFFFFu, st_misc = 0xFFFFFFFFu;   // state the issuer holds
        uint32_t uses0 = 0, uses1 = 0;                        // tiles each accumulator has served
        bool ok = true;
        // hand one descriptor to the issuer; never overwrites a descriptor not yet taken
        uint32_t seen_read = 0;                               // the issuer's progress as last looked up
        auto publish = [&](uint32_t x, uint32_t y, uint32_t z, uint32_t w) -> bool {
            ++n_pub;
            if (n_pub - seen_read >= (uint32_t)kFifo) {
                const long long t0 = clock64();
                while (n_pub - (seen_read = fifo_read) >= (uint32_t)kFifo)
                    if (abort_flag || clock64() - t0 > wait_limit) { abort_flag = 1; return false; }
            }
            st_shared_v4(smem_u32(&fifo[n_pub & (kFifo - 1)]), (n_pub & 0xFFFFu) | x, y, z, (w & 0x00FFFFFFu) | (n_pub << 24));
            return true;
        };
        int own_len = -1;
        for (int it = 0;; ++it) {
            int ti = lane == 0 ? tc_item(it, own_len, tiles, n_own, n_tiles, sched, tile_q, &tile_n, abortp, wait_limit) : 0;
            ti = __shfl_sync(0xffffffffu, ti, 0);
            if (ti < 0) break;
            const TcTile tl = tiles[ti];
            if (tl.node < 0) break;
            const int first_wg = nodes[tl.node].first_wg, n_bursts = nodes[tl.node].n_wg, first_state = nodes[tl.node].first_state;
            const uint32_t ncols8 = (uint32_t)nodes[tl.node].n_cols >> 3;
            if (tl.node != cached_node) {
                __syncwarp();
                for (int i = lane; i < n_bursts; i += 32) m_tab[i] = reinterpret_cast<const uint2*>(bursts)[first_wg + i];
                cached_node = tl.node;
                cur_state = 0xFFFFFFFFu;
                __syncwarp();
            }
            if (lane == 0 && ok) {
                {
                    // ------------------------------------------------------ scout
                    // Measured: whatever the issuing thread executes between two tcgen05.mma costs tensor-pipe
                    // time one for one (a probe of a ready barrier ~165 cycles, a shared-memory load ~110, a
                    // commit ~50), except for ~200 cycles per burst of >= 8 MMAs.  So this thread does all the
                    // waiting and address arithmetic and hands the issuer one 16-byte descriptor per burst: one
                    // weight box applied to both lanes of a pair, or two boxes applied to a single tile (8 MMAs
                    // at 64 channels per K-block either way).
                    const uint32_t lanes = (uint32_t)tl.lanes;
                    const uint32_t acc0 = lanes == 2 ? 0u : ((tmem_cols >= 512 && uses0 > uses1) ? 1u : 0u);
                    const uint32_t lane_all = lanes == 2 ? 3u : 1u;
                    int kb = 0;
                    const int n_kb = n_bursts;
                    bool first = true;
                    while (kb < n_kb && ok) {
                        const uint2 rec = m_tab[kb];
                        ++kb;
                        const uint32_t fl = rec.y & 0xFFu, st = (rec.y >> 8) & 0xFFu;
                        if (st != cur_state) {
                            const uint4 sv = __ldg(reinterpret_cast<const uint4*>(states) + first_state + st);
                            w_hi = sv.x;
                            x_hi = sv.y;
                            nk = sv.z & 0xFFFFu;
                            w_step = sv.z >> 16;
                            cur_state = st;
                        }
                        uint32_t act_mask = 0;
                        if (fl & 1u) {
                            a_cur = a_nxt;
                            if (!mbar_wait(bar_afull + 8 * a_cur, a_ph, abortp, wait_limit)) { ok = false; break; }
                            if (++a_nxt == (uint32_t)n_a) { a_nxt = 0; a_ph ^= 1; }
                            a_base16 = (a_ring + a_cur * a_slot) >> 4;
                        }
                        // the window of the first block: in the activation slot, or (a staged edge) in the weight slot
                        const uint32_t x_base16 = (fl & 32u) ? (w_ring + w_nxt * w_slot) >> 4 : a_base16;
                        const uint32_t z = ((x_base16 + (rec.x & 0xFFFFu)) & 0x3FFFu) | 0x10000u;
                        if (fl & 4u) act_mask |= 1u << a_cur;
                        if (fl & 2u) {
                            a_cur = a_nxt;
                            if (!mbar_wait(bar_afull + 8 * a_cur, a_ph, abortp, wait_limit)) { ok = false; break; }
                            if (++a_nxt == (uint32_t)n_a) { a_nxt = 0; a_ph ^= 1; }
                            a_base16 = (a_ring + a_cur * a_slot) >> 4;
                        }
                        const uint32_t w = ((a_base16 + (rec.x >> 16)) & 0x3FFFu) | 0x10000u;
                        if (fl & 8u) act_mask |= 1u << a_cur;
                        if (!mbar_wait(bar_wfull + 8 * w_nxt, w_ph, abortp, wait_limit)) { ok = false; break; }
                        const uint32_t y = (((w_ring + w_nxt * w_slot) >> 4) & 0x3FFFu) | 0x10000u;
                        if (++w_nxt == (uint32_t)n_w) { w_nxt = 0; w_ph ^= 1; }
                        const uint32_t nt = (fl & 16u) ? 2u : 1u;
                        const uint32_t misc = nk | (acc0 << 3) | (1u << 4) | (ncols8 << 5) | (w_step << 11);
                        if (w_hi != st_w_hi || x_hi != st_x_hi || misc != st_misc) {
                            if (!publish(kDescState | ((misc & 0x7FFu) << 17), w_hi, x_hi, w_step)) { ok = false; break; }
                            st_w_hi = w_hi; st_x_hi = x_hi; st_misc = misc;
                        }
                        const uint32_t last = kb == n_kb ? 1u : 0u;
                        const uint32_t base = nt << 17;
                        if (first) {
                            // the accumulators come back from the epilogue one after the other (lane 0's first): lane 0
                            // starts as soon as its own is free
                            if (!mbar_wait(bar_tempty + 8 * acc0, ((acc0 ? uses1 : uses0) & 1) ^ 1, abortp, wait_limit)) { ok = false; break; }
                            if (lanes == 2) {
                                if (!publish(base | (1u << 19) | (1u << 20) | (last << 22), y, z, w)) { ok = false; break; }
                                if (!mbar_wait(bar_tempty + 8, (uses1 & 1) ^ 1, abortp, wait_limit)) { ok = false; break; }
                                if (!publish(base | (1u << 19) | (2u << 20) | ((last * 2u) << 22) | (act_mask << 24) | (1u << 28), y, z, w)) { ok = false; break; }
                            } else {
                                if (!publish(base | (1u << 19) | (1u << 20) | (last << 22) | (act_mask << 24) | (1u << 28), y, z, w)) { ok = false; break; }
                            }
                            first = false;
                        } else {
                            if (!publish(base | (lane_all << 20) | ((last * lane_all) << 22) | (act_mask << 24) | (1u << 28), y, z, w)) { ok = false; break; }
                        }
                    }
                    if (lanes == 2) { ++uses0; ++uses1; }
                    else if (acc0 == 0) ++uses0;
                    else ++uses1;
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
        }
        if (lane == 0) {
            ++n_pub;                                                                // tell the issuer to stop (this slot may be
            st_shared_v4(smem_u32(&fifo[n_pub & (kFifo - 1)]), (n_pub & 0xFFFFu) | kDescStop, 0, 0, n_pub << 24);   // taken only after an abort)
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        // One thread; it reads burst descriptors and issues, nothing else (see the scout).
        if (lane == 0) {
            uint32_t n = 0, w_hi = 0, x_hi = 0, idesc = 0, nk = 0, acc_of[2] = {0u, 1u}, w_rel = 0, w_step = 0;
            for (;;) {
                ++n;
                const uint32_t e = smem_u32(&fifo[n & (kFifo - 1)]);
                uint4 q = ld_shared_v4(e);
                if ((q.x & 0xFFFFu) != (n & 0xFFFFu) || (q.w >> 24) != (n & 0xFFu)) {
                    const long long t0 = clock64();
                    bool give_up = false;
                    for (;;) {
                        q = ld_shared_v4(e);
                        if ((q.x & 0xFFFFu) == (n & 0xFFFFu) && (q.w >> 24) == (n & 0xFFu)) break;
                        if (abort_flag || clock64() - t0 > wait_limit) { give_up = true; break; }
                    }
                    if (give_up) { abort_flag = 1; break; }
                }
                const uint32_t fl = q.x;
                fifo_read = n;
                if (fl & kDescStop) break;
                if (fl & kDescState) {
                    const uint32_t misc = fl >> 17;
                    nk = misc & 7u;
                    acc_of[0] = (misc >> 3) & 1u;
                    acc_of[1] = (misc >> 4) & 1u;
                    // instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128 output channels, N = pixels
                    idesc = (1u << 4) | (1u << 7) | (1u << 10) | (((misc >> 5) & 63u) << 17) | ((uint32_t)(128 >> 4) << 24);
                    w_hi = q.y;
                    x_hi = q.z;
                    w_step = q.w & 0xFFFFu;
                    continue;
                }
                const uint32_t first = fl & (1u << 19);
                const uint32_t xw = q.w & 0x1FFFFu;
                if (first) tc_fence_after();                             // the accumulator was just handed back
                // a K = 16 step moves both operands 32 bytes along K: +2 in the descriptors' address field
                if (((fl >> 17) & 3u) == 2u) {
                    // two K-blocks of a single tile
                    const uint32_t d_tmem = tmem_base + acc_of[0] * 256, wb = q.y + w_step;
                    if (nk == 4) {
                        tc_mma_bf16_lohi(d_tmem, q.y, w_hi, q.z, x_hi, idesc, first ? 0u : 1u);
                        tc_mma_bf16_lohi(d_tmem, q.y + 2, w_hi, q.z + 2, x_hi, idesc, 1u);
                        tc_mma_bf16_lohi(d_tmem, q.y + 4, w_hi, q.z + 4, x_hi, idesc, 1u);
                        tc_mma_bf16_lohi(d_tmem, q.y + 6, w_hi, q.z + 6, x_hi, idesc, 1u);
                        tc_mma_bf16_lohi(d_tmem, wb, w_hi, xw, x_hi, idesc, 1u);
                        tc_mma_bf16_lohi(d_tmem, wb + 2, w_hi, xw + 2, x_hi, idesc, 1u);
                        tc_mma_bf16_lohi(d_tmem, wb + 4, w_hi, xw + 4, x_hi, idesc, 1u);
                        tc_mma_bf16_lohi(d_tmem, wb + 6, w_hi, xw + 6, x_hi, idesc, 1u);
                    } else {
                        uint32_t accum = first ? 0u : 1u;
                        for (uint32_t j = 0; j < nk; ++j) {
                            tc_mma_bf16_lohi(d_tmem, q.y + 2 * j, w_hi, q.z + 2 * j, x_hi, idesc, accum);
                            accum = 1u;
                        }
                        for (uint32_t j = 0; j < nk; ++j) tc_mma_bf16_lohi(d_tmem, wb + 2 * j, w_hi, xw + 2 * j, x_hi, idesc, 1u);
                    }
                    if ((fl >> 22) & 1u) tc_commit(bar_tfull + 8 * acc_of[0]);
                } else {
#pragma unroll
                    for (uint32_t l = 0; l < 2; ++l) {
                        if (!((fl >> (20 + l)) & 1u)) continue;
                        const uint32_t d_tmem = tmem_base + acc_of[l] * 256;
                        const uint32_t xa = l == 0 ? q.z : xw;
                        if (nk == 4) {
                            tc_mma_bf16_lohi(d_tmem, q.y, w_hi, xa, x_hi, idesc, first ? 0u : 1u);
                            tc_mma_bf16_lohi(d_tmem, q.y + 2, w_hi, xa + 2, x_hi, idesc, 1u);
                            tc_mma_bf16_lohi(d_tmem, q.y + 4, w_hi, xa + 4, x_hi, idesc, 1u);
                            tc_mma_bf16_lohi(d_tmem, q.y + 6, w_hi, xa + 6, x_hi, idesc, 1u);
                        } else {
                            uint32_t accum = first ? 0u : 1u;
                            for (uint32_t j = 0; j < nk; ++j) {
                                tc_mma_bf16_lohi(d_tmem, q.y + 2 * j, w_hi, xa + 2 * j, x_hi, idesc, accum);
                                accum = 1u;
                            }
                        }
                        if ((fl >> (22 + l)) & 1u) tc_commit(bar_tfull + 8 * acc_of[l]);   // this lane's accumulator is complete
                    }
                }
                if (fl & (1u << 28)) {                                   // hand the weight slot of this burst back (ring order)
                    tc_commit(bar_wempty + 8 * w_rel);
                    if (++w_rel == (uint32_t)n_w) w_rel = 0;
                }
                uint32_t m = (fl >> 24) & 15u;
                while (m) {                                              // activation slots this burst read last
                    const uint32_t sl = __ffs(m) - 1;
                    tc_commit(bar_aempty + 8 * sl);
                    m &= m - 1;
                }
            }
        }
    } else if (warp >= 4) {
        // ---------------------------------------------------------------- epilogue (warps 4..11)
        // TMEM lane = output channel, TMEM column = pixel.  Two warps share each quarter of the 128 lanes and take
        // alternate 32-column chunks.  A warp turns 32 channels x 32 pixels into NHWC order through a 2 KiB
        // shared-memory buffer: every thread writes its channel of 32 pixels (bias, ReLU, bf16), then reads back
        // 8 consecutive channels of one pixel and stores them as one 16-byte word, so a pixel's 32 channels leave
        // the warp as one 64-byte run.  The element offset of every pixel of the work item (or -1 for separator
        // rows and pixels outside the image) is tabulated once per item.  Lane 0's accumulator is drained first and
        // handed back first.
        const int ew = warp - 4, quarter = ew & 3, half = ew >> 2;      // TMEM lanes 32*quarter .. +31 belong to this warp
        const int et = threadIdx.x - 128;                               // 0..255 among the epilogue threads
        uint16_t* tbuf = &epi_buf[ew][0];
        uint32_t uses0 = 0, uses1 = 0;
        bool ok = true;
        // one thread looks the next item up (before the barrier that ends the current one): one answer for all eight warps
        int own_len = -1;
        if (et == 0) epi_ti = tc_item(0, own_len, tiles, n_own, n_tiles, sched, tile_q, &tile_n, abortp, wait_limit);
        asm volatile("bar.sync 1, 256;" ::: "memory");
        for (int it = 0;; ++it) {
            const int ti = epi_ti;
            if (ti < 0) break;
            const TcTile tl = tiles[ti];
            if (tl.node < 0) break;
            const TcNode nd = nodes[tl.node];
            const int rows = nd.th + nd.sep;
            for (int idx = et; idx < tl.lanes * kMaxCols; idx += kEpiWarps * 32) {
                const int l = idx >> 8, n = idx & (kMaxCols - 1);
                int off = -1;
                if (n < nd.n_cols) {
                    const int x = n % nd.tw, q = n / nd.tw, r = q % rows, bi = q / rows;
                    const int b = tl.b0 + bi + l * nd.l1_db, y = tl.h0 + r, xx = tl.w0 + x + l * nd.l1_dw;
                    if (r < nd.th && bi < nd.tb && b < B && y < nd.H && xx < nd.W) off = (int)((((size_t)b * nd.H + y) * nd.W + xx) * nd.C);
                }
                pix_off[idx] = off;
            }
            if (!ok) abort_flag = 1;
            if (et == 0) epi_stop = abort_flag;                      // one decision for all eight warps
            asm volatile("bar.sync 1, 256;" ::: "memory");           // the offset table is complete
            if (epi_stop) break;
            const uint32_t acc0 = tl.lanes == 2 ? 0u : ((tmem_cols >= 512 && uses0 > uses1) ? 1u : 0u);
            const bool second = nd.fused && quarter >= 2;           // this warp's TMEM lanes belong to the plan's second node
            __nv_bfloat16* out = static_cast<__nv_bfloat16*>(second ? nd.state2[cur] : nd.state[cur]);
            const int co_w = nd.fused ? (quarter & 1) * 32 : tl.m0 + quarter * 32;   // first channel of this warp
            const int co = co_w + lane;                             // TMEM lane = output channel
            const float bias = co < nd.C ? __ldg((second ? nd.bias2 : nd.bias) + co) : 0.f;
            const int act = second ? nd.act2 : nd.act;
            const bool gvalid = co_w + (lane & 3) * 8 < nd.C;       // this thread's group of 8 channels exists
            for (int l = 0; l < tl.lanes && ok; ++l) {
                const uint32_t acc = l == 0 ? acc0 : 1u;
                if (!mbar_wait(bar_tfull + 8 * acc, (acc ? uses1 : uses0) & 1, abortp, wait_limit)) ok = false;
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * 256;
                const int* poff = pix_off + l * kMaxCols;
                for (int c0 = half * 32; c0 < nd.n_cols; c0 += 64) {
                    uint32_t v[32];
                    tc_ld32(taddr + c0, v);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        float z = __uint_as_float(v[j]) + bias;
                        if (act == 1) z = fmaxf(z, 0.f);
                        const __nv_bfloat16 hz = __float2bfloat16_rn(z);
                        tbuf[j * 32 + lane] = *reinterpret_cast<const uint16_t*>(&hz);
                    }
                    __syncwarp();
#pragma unroll
                    for (int pass = 0; pass < 4; ++pass) {
                        const int p = pass * 8 + (lane >> 2);
                        const int o = poff[c0 + p];
                        if (o >= 0 && gvalid) {
                            const uint4 w = *reinterpret_cast<const uint4*>(tbuf + p * 32 + (lane & 3) * 8);
                            *reinterpret_cast<uint4*>(out + (size_t)o + co_w + (lane & 3) * 8) = w;
                        }
                    }
                    __syncwarp();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
            }
            if (et == 0) {
                if (own_len >= 0) epi_items = it + 1 - own_len;
                epi_ti = tc_item(it + 1, own_len, tiles, n_own, n_tiles, sched, tile_q, &tile_n, abortp, wait_limit);
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");           // everybody is done with the offset table
            if (tl.lanes == 2) { ++uses0; ++uses1; }
            else if (acc0 == 0) ++uses0;
            else ++uses1;
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&ctl->error, 1);
    if (threadIdx.x == 0 && sched && n_own < n_tiles) {
        // the CTA that leaves last (none takes an item any more) puts the counters back for the next launch
        __threadfence();
        if (atomicAdd(sched + 1, 1) == (int)gridDim.x - 1) {
            sched[0] = 0;
            sched[1] = 0;
            __threadfence();
        }
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// Few-channel input edges: row (b, oy, ox) of the staged tensor holds the k*k*C_in receptive field
// of that output pixel (zero outside the image, zero padded to Kp), so the edge becomes a K-block.
__global__ void sr_tc_stage_kernel(const TcStem* __restrict__ stems, int n_stems, const SrFrameCtl* __restrict__ ctl,
                                   int t_off, int fixed_parity, int B)
{
    __shared__ int tap_off[128];    // offset of element kk relative to the (unpadded) window origin, -1 = padding
    __shared__ short tap_dy[128], tap_dx[128];
    const int cur = fixed_parity >= 0 ? fixed_parity : (int)((ctl->t + t_off + 1) & 1);
    for (int si = 0; si < n_stems; ++si) {
        const TcStem st = stems[si];
        __syncthreads();
        if (threadIdx.x < 128) {
            const int kk = threadIdx.x;
            if (kk < st.K) {
                const int ci = kk % st.Cs, tap = kk / st.Cs, kx = tap % st.k, ky = tap / st.k;
                tap_dy[kk] = (short)(ky - st.pad);
                tap_dx[kk] = (short)(kx - st.pad);
                tap_off[kk] = ((ky - st.pad) * st.Ws + (kx - st.pad)) * st.Cs + ci;
            } else {
                tap_dy[kk] = tap_dx[kk] = 0;
                tap_off[kk] = -1;
            }
        }
        __syncthreads();
        const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(st.src[cur]);
        __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(st.dst[cur]);
        const int chunks = st.Kp / 8;
        const size_t n_pix = (size_t)B * st.Ho * st.Wo;
        for (size_t p = (size_t)blockIdx.x * blockDim.x + threadIdx.x; p < n_pix; p += (size_t)gridDim.x * blockDim.x) {
            const int ox = (int)(p % st.Wo);
            const size_t r = p / st.Wo;
            const int oy = (int)(r % st.Ho);
            const int b = (int)(r / st.Ho);
            const int y0 = oy * st.stride, x0 = ox * st.stride;
            const __nv_bfloat16* base = src + (((size_t)b * st.Hs + y0) * st.Ws + x0) * st.Cs;
            for (int c = 0; c < chunks; ++c) {
                __align__(16) __nv_bfloat16 v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int kk = c * 8 + j;
                    const int iy = y0 + tap_dy[kk], ix = x0 + tap_dx[kk];
                    const bool ok = kk < st.K && iy >= 0 && iy < st.Hs && ix >= 0 && ix < st.Ws;
                    v[j] = ok ? base[tap_off[kk]] : __float2bfloat16_rn(0.f);
                }
                reinterpret_cast<uint4*>(dst)[p * chunks + c] = *reinterpret_cast<const uint4*>(v);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------ host side
struct KbHost {
    int edge;
    bool stem;
    int stem_index;
    int ky, kx, c0, bk;
    int k_off;
    bool x_load;       // loads a fresh activation box (else: reuses the box loaded earlier for this channel block)
    int x_shift;       // pixels by which this tap's window is shifted inside the box
    int x_width;       // pixels per image row of the box (lane width, plus the pixel range of the taps it serves)
    bool x_release;
    int box_qy = 0, box_qx = 0, box_ry = 0, box_rx = 0;   // origin and residue class of the box (loading block)
    int src_col = 0;   // first column of this block in the edge's own weight matrix [C_out][k * k * C_in]
    int run = 0;       // run of equally wide K-blocks this block belongs to, and its index inside the run
    int blk = 0;
    bool w_first = false, w_last = false;   // first / last block of a weight group
    int w_off = 0;     // byte offset of this block's weights inside the group's slot
    bool in_wring = false;   // a staged edge whose activation box travels in the weight ring, behind the block's weights
    int box_off = 0;         // byte offset of that box inside the slot
    int row_off = 0;         // first row of `edge`'s weights in the plan's weight matrix (64: the second node of a fused plan)
    int edge2 = -1;          // fused plan: the second node's edge that shares this block (its weights take rows 64..127)
};

// Consecutive K-blocks of equal channel-block width: one 3-D view (channels of a block, output channels, blocks) of
// the node's weight matrix, whose columns are stored in the order the K loop walks them.
struct WRun { int bk, first_col, n_blocks; };
// what the MMAs of one K-block need (host-side; folded into burst records and descriptor states at bind time)
struct KmHost {
    uint32_t desc_hi = 0, x_off16 = 0, x_l1off16 = 0, x_sbo16 = 0, n_k16 = 0, w_step16 = 0;
    bool x_load = false, x_release = false, in_wring = false;
};
struct WGroup { int run, blk, n, bytes; };

struct NodePlan {
    int node;
    int node2 = -1;                 // the second node of a fused plan
    int rows_total(const sr_graph* g) const { return node2 >= 0 ? 128 : g->nodes[node].d.c; }   // rows of the weight matrix
    int tw, th, tb, sep, n_cols;
    bool one_box;                   // tw == 8: one activation box per channel block serves all k x k taps
    int pair;                       // 0: single tiles; 1: lane 1 is the tile tw columns to the right; 2: the next tb samples
    bool stem_ring;                 // boxes of staged edges travel in the weight ring
    int k_total;                    // columns of the concatenated weight matrix
    std::vector<KbHost> kbs;
    std::vector<WRun> runs;
    std::vector<WGroup> wgroups;
    SrRegion wcat;
    int lane_w() const { return pair == 1 ? 2 * tw : tw; }           // columns of the activation box that hold pixels
    int box_tb() const { return pair == 2 ? 2 * tb : tb; }           // samples of the activation box
};

struct StemPlan {
    int edge;
    int Kp;
    SrRegion buf[2];
};

struct TcEngine {
    std::vector<NodePlan> nodes;                 // tensor-core nodes
    std::vector<int> node_of;                    // graph node -> index in nodes, or -1
    std::vector<StemPlan> stems;
    std::vector<int> stem_of_edge;
    std::vector<std::vector<TcTile>> group_tiles;
    std::vector<int> group_tile_offset, group_a_slot, group_n_a, group_n_w, group_w_slot, group_grid, group_ctas_per_sm, group_n_own;
    SrRegion r_maps, r_nodes, r_kb_weight, r_kb_act, r_bursts, r_states, r_tiles, r_stems, r_sched;
    int n_maps = 0, n_kbs = 0, n_tiles = 0;
    int sm_count = 148;
    // optional timing of the group launches with CUDA events on the launching stream
    std::vector<cudaEvent_t> ev;             // pairs: start, stop
    size_t ev_used = 0;
    double timed_ms = 0.0;
    long long timed_launches = 0;
};

TcEngine* eng(const sr_graph* g) { return static_cast<TcEngine*>(g->tc); }

int block_k(int cs) { return cs % 64 == 0 ? 64 : (cs % 32 == 0 ? 32 : 16); }
int stem_kp(int K) { return K <= 16 ? 16 : (K <= 32 ? 32 : (K <= 64 ? 64 : 128)); }
bool is_stem(const sr_graph* g, const SrHostEdge& e)
{
    const SrHostNode& s = g->nodes[e.d.src];
    return s.is_input && (s.d.c % 16) != 0 && e.K <= 128;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

CUtensorMapSwizzle swizzle_of(int bk)
{
    return bk == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : (bk == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

uint32_t desc_hi_of(int bk)
{
    const uint32_t sbo = (uint32_t)(8 * bk * 2) >> 4;                    // 8 rows of bk bf16
    const uint32_t layout = bk == 64 ? 2u : (bk == 32 ? 4u : 6u);        // 128B / 64B / 32B swizzle
    return sbo | (1u << 14) | (layout << 29);
}

// Pick the pixel tile of a node: tw in {8, 16, 32} columns, th rows, tb samples, such that the stacked
// rows N = tb * (th + sep) * tw - sep * tw fit 256 MMA columns.  The cost of a tile is the time of its
// MMAs (about max(110, N/2) cycles each); the best shape computes the image with the least total cost.
void choose_tile(int H, int W, int B, int sep, int forced_tw, NodePlan& P)
{
    double best = 1e30;
    for (int tw = 8; tw <= 32; tw *= 2) {
        if (forced_tw > 0 && tw != forced_tw && !(forced_tw > 8 && tw == 8 && forced_tw > (W + 7) / 8 * 8)) continue;
        if (tw > 8 && tw > (W + 7) / 8 * 8) continue;
        const int th = std::min(H, kMaxCols / tw);
        int tb = 1;
        if (th == H) tb = std::max(1, std::min(B, (kMaxCols + sep * tw) / ((th + sep) * tw)));
        const int n = tb * (th + sep) * tw - sep * tw;
        const int n_cols = (n + 31) / 32 * 32;
        if (n_cols > kMaxCols) continue;
        const double tiles = (double)((W + tw - 1) / tw) * ((H + th - 1) / th) * ((B + tb - 1) / tb);
        const double cost = tiles * std::max(110.0, n_cols / 2.0) + tiles * 1e-3 * tw;      // tie: narrower tile, less halo
        if (cost < best) {
            best = cost;
            P.tw = tw; P.th = th; P.tb = tb; P.n_cols = n_cols;
        }
    }
}

void tap_q(int tap, int pad, int st, int& q, int& r)
{
    const int a = tap - pad;
    q = (a >= 0) ? a / st : -((-a + st - 1) / st);
    r = a - q * st;
}

// Do two edges read the same source through the same filter geometry in the same frame?  (Staged edges are not shared.)
bool same_source(const sr_graph* g, int e1, int e2)
{
    const SrHostEdge& a = g->edges[e1];
    const SrHostEdge& b = g->edges[e2];
    return a.d.src == b.d.src && a.d.kind == SR_EDGE_CONV && b.d.kind == SR_EDGE_CONV && a.k_eff == b.k_eff &&
           a.stride_eff == b.stride_eff && a.pad_eff == b.pad_eff && a.d.pool == b.d.pool && a.K == b.K && a.R == b.R &&
           !is_stem(g, a) && !is_stem(g, b);
}

// The K-blocks of a plan for its tile geometry and pairing mode (the stems' staging buffers exist already).
void build_kblocks(const sr_graph* g, const TcEngine* E, NodePlan& P)
{
    const SrHostNode& n = g->nodes[P.node];
    P.kbs.clear();
    // one_box: every class of an edge gets a box as wide as the widest class of the node needs, so that all
    // K-blocks of equal channel-block width share one activation descriptor state
    // the incoming edges of the plan: of its node and, fused, of its second node; an edge of the second node that
    // reads the same source through the same filter geometry in the same frame shares the first node's K-blocks
    struct Ent { int e, e2, row_off; };
    std::vector<Ent> ents;
    for (int e : n.in_edges) ents.push_back(Ent{e, -1, 0});
    if (P.node2 >= 0)
        for (int e2 : g->nodes[P.node2].in_edges) {
            int m = -1;
            for (size_t i = 0; i < ents.size() && m < 0; ++i)
                if (ents[i].row_off == 0 && ents[i].e2 < 0 && same_source(g, ents[i].e, e2)) m = (int)i;
            if (m >= 0) ents[m].e2 = e2;
            else ents.push_back(Ent{e2, -1, 64});
        }
    int span = 0;
    if (P.one_box)
        for (const Ent& en : ents) {
            const int e = en.e;
            const SrHostEdge& he = g->edges[e];
            if (is_stem(g, he)) continue;
            for (int r0 = 0; r0 < he.stride_eff; ++r0) {
                int lo = 1 << 20, hi = -(1 << 20);
                for (int t = 0; t < he.k_eff; ++t) {
                    int q, r;
                    tap_q(t, he.pad_eff, he.stride_eff, q, r);
                    if (r == r0) { lo = std::min(lo, q); hi = std::max(hi, q); }
                }
                if (hi >= lo) span = std::max(span, hi - lo);
            }
        }
    // The order of the reduction is free (a sum): edges with wider channel blocks come first, so that K-blocks of
    // equal width form one run each and a run's weights are one 3-D tensor.
    auto width_of = [&](int e) {
        const SrHostEdge& he = g->edges[e];
        return is_stem(g, he) ? std::min(64, E->stems[E->stem_of_edge[e]].Kp) : block_k(g->nodes[he.d.src].d.c);
    };
    std::stable_sort(ents.begin(), ents.end(), [&](const Ent& a, const Ent& b) { return width_of(a.e) > width_of(b.e); });
    const int rows = std::min(P.rows_total(g), 128);
    for (const Ent& en : ents) {
        const int e = en.e;
        const SrHostEdge& he = g->edges[e];
        const SrHostNode& s = g->nodes[he.d.src];
        if (is_stem(g, he)) {
            // a staged edge: its im2col rows are one K-block of 16 / 32 / 64 columns, or two of 64
            const int si = E->stem_of_edge[e], Kp = E->stems[si].Kp, bk = std::min(64, Kp);
            for (int c0 = 0; c0 < Kp; c0 += bk) {
                KbHost kb{e, true, si, 0, 0, c0, bk, 0, true, 0, P.lane_w(), true};
                kb.src_col = c0;
                kb.row_off = en.row_off;
                // weights, then the box, if both fit the weight slot that full-width groups need anyway (32 KiB)
                const size_t w_bytes = sr_align_up((size_t)rows * bk * 2, 1024);
                const size_t box_bytes = (size_t)kb.x_width * (P.th + P.sep) * P.box_tb() * bk * 2;
                if (P.pair == 0 && P.stem_ring && w_bytes + box_bytes <= 32 * 1024) {
                    kb.in_wring = true;
                    kb.box_off = (int)w_bytes;
                }
                P.kbs.push_back(kb);
            }
        } else {
            // Taps whose input pixels fall into the same residue class of the stride read the same view of the
            // source, shifted by whole pixels: they share ONE activation box and differ only in where their window
            // starts inside it (rows always; pixels too when the tile is 8 wide, because then the 8-pixel groups of
            // the operand are simply one box row apart, whatever the row length).
            const int bk = block_k(s.d.c), k = he.k_eff, st = he.stride_eff;
            struct Tap { int ky, kx, qy, qx; };
            std::map<std::tuple<int, int, int>, std::vector<Tap>> classes;      // (ry, rx, qx or 0) -> taps
            for (int ky = 0; ky < k; ++ky)
                for (int kx = 0; kx < k; ++kx) {
                    int qy, ry, qx, rx;
                    tap_q(ky, he.pad_eff, st, qy, ry);
                    tap_q(kx, he.pad_eff, st, qx, rx);
                    classes[std::make_tuple(ry, rx, P.one_box ? 0 : qx)].push_back(Tap{ky, kx, qy, qx});
                }
            for (int c0 = 0; c0 < s.d.c; c0 += bk)
                for (auto& cl : classes) {
                    const std::vector<Tap>& taps = cl.second;
                    int qy0 = 1 << 20, qx0 = 1 << 20;
                    for (const Tap& t : taps) { qy0 = std::min(qy0, t.qy); qx0 = std::min(qx0, t.qx); }
                    const int bw = P.lane_w() + span;
                    for (size_t i = 0; i < taps.size(); ++i) {
                        const Tap& t = taps[i];
                        // the first tap of the class carries the box origin (qy0, qx0)
                        KbHost kb{e, false, -1, t.ky, t.kx, c0, bk, 0,
                                  i == 0, (t.qy - qy0) * bw + (t.qx - qx0), bw, i + 1 == taps.size()};
                        kb.src_col = (t.ky * k + t.kx) * s.d.c + c0;
                        kb.row_off = en.row_off;
                        kb.edge2 = en.e2;
                        kb.box_qy = qy0;
                        kb.box_qx = qx0;
                        kb.box_ry = std::get<0>(cl.first);
                        kb.box_rx = std::get<1>(cl.first);
                        P.kbs.push_back(kb);
                    }
                }
        }
    }
    // columns in loop order; runs of equal block width; weight groups: up to two blocks of a run when tiles are single,
    // one when they come in pairs (a pair already gives eight MMAs per block), never two blocks that each open a
    // fresh activation box (the ring may have only two slots)
    P.runs.clear();
    P.wgroups.clear();
    const int per_group = P.pair ? 1 : 2;
    int k_off = 0;
    for (size_t i = 0; i < P.kbs.size(); ++i) {
        KbHost& kb = P.kbs[i];
        kb.k_off = k_off;
        k_off += kb.bk;
        if (P.runs.empty() || P.runs.back().bk != kb.bk) P.runs.push_back(WRun{kb.bk, kb.k_off, 0});
        kb.run = (int)P.runs.size() - 1;
        kb.blk = P.runs.back().n_blocks++;
        bool open = P.wgroups.empty() || P.wgroups.back().run != kb.run || P.wgroups.back().n >= per_group || kb.in_wring ||
                    (i > 0 && P.kbs[i - 1].in_wring);
        if (!open && kb.x_load) {
            bool had_load = false;
            for (int j = 0; j < P.wgroups.back().n; ++j) had_load |= P.kbs[i - 1 - j].x_load;
            open = had_load;
        }
        if (open) {
            if (i > 0) P.kbs[i - 1].w_last = true;
            P.wgroups.push_back(WGroup{kb.run, kb.blk, 0, 0});
            kb.w_first = true;
        }
        kb.w_off = P.wgroups.back().bytes;
        P.wgroups.back().n += 1;
        P.wgroups.back().bytes += rows * kb.bk * 2;
        if (kb.in_wring) P.wgroups.back().bytes = kb.box_off + kb.x_width * (P.th + P.sep) * P.box_tb() * kb.bk * 2;
    }
    if (!P.kbs.empty()) P.kbs.back().w_last = true;
    P.k_total = k_off;
}

// Pixels by which lane 1's operand window lies behind lane 0's inside a box of row length x_width.
int lane1_shift_px(const NodePlan& P, int x_width)
{
    if (P.pair == 1) return P.tw;
    if (P.pair == 2) return P.tb * (P.th + P.sep) * x_width;
    return 0;
}

int act_slot_bytes(const NodePlan& P)
{
    int a_slot = 1024;
    for (const KbHost& kb : P.kbs) {
        if (kb.in_wring) continue;
        const size_t box_px = (size_t)kb.x_width * (P.th + P.sep) * P.box_tb();
        // the last 8-pixel group a window reads: shift + (n_cols / 8 - 1) rows of the box + 8 pixels
        const size_t reach_px = (size_t)kb.x_shift + lane1_shift_px(P, kb.x_width) + (size_t)(P.n_cols / 8 - 1) * (kb.x_width * 8 / P.tw) + 8;
        a_slot = std::max(a_slot, (int)sr_align_up(std::max(box_px, reach_px) * kb.bk * 2, 1024));
    }
    return a_slot;
}

int weight_slot_bytes(const sr_graph*, const NodePlan& P)
{
    int w = 1024;
    for (const WGroup& wg : P.wgroups) w = std::max(w, (int)sr_align_up((size_t)wg.bytes, 1024));
    return w;
}

std::vector<TcTile> node_tiles(const sr_graph* g, const NodePlan& P, int node_index)
{
    const SrHostNode& n = g->nodes[P.node];
    std::vector<TcTile> out;
    const int db = P.tb * (P.pair == 2 ? 2 : 1), dw = P.tw * (P.pair == 1 ? 2 : 1);
    for (int b0 = 0; b0 < g->batch; b0 += db)
        for (int h0 = 0; h0 < n.d.h; h0 += P.th)
            for (int w0 = 0; w0 < n.d.w; w0 += dw)
                for (int m0 = 0; m0 < P.rows_total(g); m0 += 128) {
                    int lanes = 1;
                    if (P.pair == 1 && w0 + P.tw < n.d.w) lanes = 2;
                    if (P.pair == 2 && b0 + P.tb < g->batch) lanes = 2;
                    out.push_back(TcTile{node_index, b0, h0, w0, m0, lanes, {0, 0}});
                }
    return out;
}

}  // namespace

// A node goes to the tensor cores if it sums convolutions only, has at least 16 output channels in
// multiples of 8, and every incoming edge either has C_in % 16 == 0 or is a few-channel input edge.
void sr_tc_select_nodes(sr_graph* g)
{
    for (size_t v = 0; v < g->nodes.size(); ++v) {
        SrHostNode& n = g->nodes[v];
        n.use_tc = false;
        if (n.is_input || n.dense_target || (int)v == g->info.output_node) continue;
        if (n.d.c % 8 != 0 || n.d.c < 16 || n.d.c > 1024) continue;
        bool ok = true;
        int n_blocks = 0;
        for (int e : n.in_edges) {
            const SrHostEdge& he = g->edges[e];
            const SrHostNode& s = g->nodes[he.d.src];
            if (he.d.kind != SR_EDGE_CONV) ok = false;
            else if (s.d.c % 16 != 0 && !is_stem(g, he)) ok = false;
            else if (he.k_eff > 8) ok = false;
            else n_blocks += is_stem(g, he) ? 2 : he.k_eff * he.k_eff * (s.d.c / block_k(s.d.c));
        }
        if (ok && n_blocks >= 1 && n_blocks <= kMaxNodeKb) n.use_tc = true;
    }
}

sr_status sr_tc_plan(sr_graph* g, size_t& off)
{
    sr_tc_destroy(g);
    bool any = false;
    for (const SrHostNode& n : g->nodes) any |= n.use_tc;
    if (!any) return SR_OK;
    TcEngine* E = new TcEngine();
    g->tc = E;
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&E->sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (E->sm_count <= 0) E->sm_count = 148;
    E->node_of.assign(g->nodes.size(), -1);
    E->stem_of_edge.assign(g->edges.size(), -1);
    auto take = [&](size_t bytes) {
        SrRegion r;
        r.offset = off;
        r.bytes = bytes;
        off = sr_align_up(off + bytes, 1024);
        return r;
    };
    // Fused plans: two nodes of one launch group with the same shape and at most 64 channels (a multiple of 32) each,
    // which share at least one source or of which one is fed by next to nothing (see TcNode).
    std::vector<int> partner(g->nodes.size(), -1), leader(g->nodes.size(), -1);
    if (g->opt_tc_fuse)
        for (const std::vector<int>& grp : g->groups)
            for (size_t i = 0; i < grp.size(); ++i) {
                const int a = grp[i];
                const SrHostNode& na = g->nodes[a];
                if (!na.use_tc || partner[a] >= 0 || leader[a] >= 0 || na.d.c > 64 || na.d.c % 32 != 0) continue;
                for (size_t j = i + 1; j < grp.size() && partner[a] < 0; ++j) {
                    const int b = grp[j];
                    const SrHostNode& nb = g->nodes[b];
                    if (!nb.use_tc || partner[b] >= 0 || leader[b] >= 0 || nb.d.c != na.d.c || nb.d.h != na.d.h || nb.d.w != na.d.w) continue;
                    int shared = 0, blocks = 0, blocks_a = 0, blocks_b = 0;
                    for (int ea : na.in_edges) {
                        const SrHostEdge& he = g->edges[ea];
                        blocks_a += is_stem(g, he) ? 2 : he.k_eff * he.k_eff * (g->nodes[he.d.src].d.c / block_k(g->nodes[he.d.src].d.c));
                    }
                    blocks = blocks_a;
                    for (int eb : nb.in_edges) {
                        const SrHostEdge& he = g->edges[eb];
                        bool sh = false;
                        for (int ea : na.in_edges) sh |= same_source(g, ea, eb);
                        const int nb_e = is_stem(g, he) ? 2 : he.k_eff * he.k_eff * (g->nodes[he.d.src].d.c / block_k(g->nodes[he.d.src].d.c));
                        blocks_b += nb_e;
                        if (sh) ++shared;
                        else blocks += nb_e;
                    }
                    // without a shared source the fused plan issues as many MMAs as the two nodes; it still pays when one
                    // of them has next to no reduction (a node fed by a staged edge only): its tiles are all epilogue,
                    // which then runs beside the other node's MMAs
                    const bool tiny = std::min(blocks_a, blocks_b) <= 2;
                    if ((shared > 0 || tiny) && blocks <= kMaxNodeKb) {
                        partner[a] = b;
                        leader[b] = a;
                    }
                }
            }
    // tile geometry and staging buffers
    for (size_t v = 0; v < g->nodes.size(); ++v) {
        const SrHostNode& n = g->nodes[v];
        if (!n.use_tc) continue;
        if (leader[v] >= 0) continue;                     // the second node of a fused plan: its leader's plan covers it
        NodePlan P{};
        P.node = (int)v;
        P.node2 = partner[v];
        // sep: how many image rows the taps that share one activation box are apart at most
        P.sep = 0;
        std::vector<int> in_edges(n.in_edges.begin(), n.in_edges.end());
        if (P.node2 >= 0) in_edges.insert(in_edges.end(), g->nodes[P.node2].in_edges.begin(), g->nodes[P.node2].in_edges.end());
        for (int e : in_edges) {
            const SrHostEdge& he = g->edges[e];
            if (is_stem(g, he)) {
                StemPlan S;
                S.edge = e;
                S.Kp = stem_kp(he.K);
                const size_t bytes = (size_t)g->batch * n.d.h * n.d.w * S.Kp * 2;
                S.buf[0] = take(bytes);
                S.buf[1] = take(bytes);
                E->stem_of_edge[e] = (int)E->stems.size();
                E->stems.push_back(S);
                continue;
            }
            for (int r0 = 0; r0 < he.stride_eff; ++r0) {
                int lo = 1 << 20, hi = -(1 << 20);
                for (int t = 0; t < he.k_eff; ++t) {
                    int q, r;
                    tap_q(t, he.pad_eff, he.stride_eff, q, r);
                    if (r == r0) { lo = std::min(lo, q); hi = std::max(hi, q); }
                }
                if (hi >= lo) P.sep = std::max(P.sep, hi - lo);
            }
        }
        choose_tile(n.d.h, n.d.w, g->batch, P.sep, g->opt_tile_w, P);
        P.one_box = P.tw == 8;
        P.pair = 0;
        E->node_of[v] = (int)E->nodes.size();
        E->nodes.push_back(P);
    }
    for (size_t v = 0; v < g->nodes.size(); ++v)
        if (leader[v] >= 0) E->node_of[v] = E->node_of[leader[v]];
    // per launch group: pairing, K-blocks, work list (largest reduction first), ring geometry
    E->group_tiles.assign(g->groups.size(), {});
    int n_tiles = 0;
    for (size_t gi = 0; gi < g->groups.size(); ++gi) {
        std::vector<int> members;
        for (int v : g->groups[gi])
            if (E->node_of[v] >= 0 && leader[v] < 0) members.push_back(E->node_of[v]);
        // Pairs halve the weight traffic but double the size of a work item, expose the epilogue (both accumulators
        // are busy) and leave room for fewer weight slots; with copies issued group-wise the L2 keeps single tiles
        // fed, so pairs are used on request only.  Option "pair": 0 / 1 = single tiles, 2 = pairs wherever the
        // geometry allows.
        bool pair = g->opt_tc_pair == 2;
        // The box of a staged edge takes a weight slot for the two MMAs it feeds; that pays where the weight ring is
        // deep (launch groups of nodes with few output channels: small weight groups), not where it has three slots.
        bool stem_ring = g->opt_stem_ring != 0;
        int a_slot = 1024, w_slot = 1024, n_a = 2, n_w = 2, per_sm = 1;
        for (int attempt = 0; attempt < 3; ++attempt) {
            a_slot = 1024;
            w_slot = 1024;
            for (int ni : members) {
                NodePlan& P = E->nodes[ni];
                const SrHostNode& n = g->nodes[P.node];
                P.pair = 0;
                P.stem_ring = stem_ring;
                if (pair) {
                    if (P.tw == 8 && n.d.w > P.tw) P.pair = 1;
                    else if (P.th == n.d.h && g->batch > P.tb) P.pair = 2;
                }
                build_kblocks(g, E, P);
                a_slot = std::max(a_slot, act_slot_bytes(P));
                w_slot = std::max(w_slot, weight_slot_bytes(g, P));
            }
            // two activation slots (a box usually serves a whole filter, and its producer runs ahead on its own), the
            // weight ring as deep as it gets; more activation slots only once the weight ring is full
            const int avail = kSmemBudget - 1024;
            const int w_max = g->opt_b_units > 0 ? std::min(kMaxW, std::max(2, g->opt_b_units)) : kMaxW;
            n_a = 2;
            while (n_a < kMaxA && (n_a + 1) * a_slot + w_max * w_slot <= avail) ++n_a;
            n_w = std::min(w_max, (avail - n_a * a_slot) / w_slot);
            if (stem_ring && g->opt_stem_ring == 1 && n_w < 4) {
                stem_ring = false;
                continue;
            }
            if (n_w >= 3 || !pair) break;
            pair = false;                                  // the paired boxes do not leave room for a weight ring: single tiles
        }
        if (!members.empty() && n_w < 2) return SR_ERR_UNSUPPORTED;
        // Small launches (a few tiles per SM) are bound by the latency of one tile, not by throughput: give every
        // CTA the smallest rings and one accumulator, so that two CTAs share an SM and twice as many tiles are in flight.
        std::vector<std::pair<long long, TcTile>> tl;
        for (int ni : members) {
            const NodePlan& P = E->nodes[ni];
            long long mma_cycles = 0;                        // one lane's MMAs: about max(110, N / 2) cycles each
            for (const KbHost& kb : P.kbs) mma_cycles += (long long)(kb.bk / 16) * std::max(110, P.n_cols / 2);
            for (const TcTile& t : node_tiles(g, P, ni))
                tl.push_back({mma_cycles * t.lanes + (t.lanes == 2 ? 6000 : 1500), t});    // plus start-up and exposed epilogue
        }
        if (!pair && (int)tl.size() <= 4 * E->sm_count && 2 * a_slot + 3 * w_slot + 1024 <= 88 * 1024) {
            per_sm = 2;
            n_a = 2;
            n_w = std::min(kMaxW, (88 * 1024 - 1024 - 2 * a_slot) / w_slot);
        }
        // Work lists: the items go, longest first, to the CTA with the least work so far; CTA c walks column c of a
        // matrix with one row per round (entries of node -1 pad the shorter columns).  Unless the lists are asked to be
        // static, the smallest items - a fifth of the work, if the launch has more than two items per CTA - stay out of
        // the matrix and follow it as one shared list (see the kernel).
        std::stable_sort(tl.begin(), tl.end(), [](const auto& a, const auto& b) { return a.first > b.first; });
        const int grid = (int)std::min<size_t>(tl.size(), (size_t)E->sm_count * per_sm);
        std::vector<std::vector<TcTile>> lists(std::max(grid, 1));
        size_t n_matrix = tl.size();
        if (g->opt_tc_lists == 0 && tl.size() > 2 * (size_t)grid) {
            long long total = 0, tail = 0;
            for (auto& it : tl) total += it.first;
            while (n_matrix > (size_t)grid && (tail + tl[n_matrix - 1].first) * 5 <= total) tail += tl[--n_matrix].first;
        }
        {
            std::vector<std::pair<long long, int>> heap;     // (-load, cta): the standard heap keeps the largest on top
            for (int c = 0; c < grid; ++c) heap.push_back({0, -c});
            std::make_heap(heap.begin(), heap.end());
            for (size_t i = 0; i < n_matrix; ++i) {
                std::pop_heap(heap.begin(), heap.end());
                std::pair<long long, int> top = heap.back();
                lists[-top.second].push_back(tl[i].second);
                top.first -= tl[i].first;
                heap.back() = top;
                std::push_heap(heap.begin(), heap.end());
            }
            size_t n_rows = 0;
            for (auto& l : lists) n_rows = std::max(n_rows, l.size());
            for (size_t r = 0; r < n_rows; ++r)
                for (int c = 0; c < grid; ++c)
                    E->group_tiles[gi].push_back(r < lists[c].size() ? lists[c][r] : TcTile{-1, 0, 0, 0, 0, 0, {0, 0}});
        }
        E->group_n_own.push_back((int)E->group_tiles[gi].size());
        for (size_t i = n_matrix; i < tl.size(); ++i) E->group_tiles[gi].push_back(tl[i].second);
        E->group_grid.push_back(grid);
        E->group_tile_offset.push_back(n_tiles);
        n_tiles += (int)E->group_tiles[gi].size();
        E->group_ctas_per_sm.push_back(per_sm);
        E->group_a_slot.push_back(a_slot);
        E->group_n_a.push_back(n_a);
        E->group_n_w.push_back(n_w);
        E->group_w_slot.push_back(w_slot);
    }
    int n_kbs = 0;
    for (NodePlan& P : E->nodes) {
        n_kbs += (int)P.kbs.size();
        P.wcat = take((size_t)P.rows_total(g) * P.k_total * 2);
    }
    E->n_tiles = n_tiles;
    E->n_kbs = n_kbs;
    // upper bound on distinct tensor maps: two parities per K-block plus one weight map per (node, bk)
    E->r_maps = take(sizeof(CUtensorMap) * (size_t)(4 * n_kbs + 1));
    E->r_nodes = take(sizeof(TcNode) * E->nodes.size());
    E->r_kb_weight = take(sizeof(TcKbWeight) * (size_t)std::max(1, n_kbs));
    E->r_kb_act = take(sizeof(TcKbAct) * (size_t)std::max(1, n_kbs));
    E->r_bursts = take(sizeof(TcBurst) * (size_t)std::max(1, n_kbs));
    E->r_states = take(sizeof(TcState) * (size_t)std::max(1, n_kbs));
    E->r_tiles = take(sizeof(TcTile) * (size_t)std::max(1, n_tiles));
    E->r_stems = take(sizeof(TcStem) * std::max<size_t>(1, E->stems.size()));
    E->r_sched = take(256);                          // the shared list's counters: next item, CTAs that have left
    return SR_OK;
}

sr_status sr_tc_bind(sr_graph* g)
{
    TcEngine* E = eng(g);
    if (!E) return SR_OK;
    EncodeTiledFn encode = encode_fn();
    if (!encode) return SR_ERR_CUDA;
    if (cudaFuncSetAttribute(sr_tc_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) != cudaSuccess)
        return SR_ERR_CUDA;
    // Always the largest shared-memory partition: otherwise the SM is configured with the smallest partition that holds
    // this kernel's CTA, which can leave a few hundred bytes, and the frame's other kernels cannot run beside it.
    if (cudaFuncSetAttribute(sr_tc_group_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess)
        return SR_ERR_CUDA;
    char* ws = g->ws;
    std::vector<CUtensorMap> maps;
    std::map<std::tuple<uintptr_t, int, int, int, int, int, int, int, int>, int> cache;
    // 4-D activation view: dims (C, W', H', B), box (bk, tw, rows, tb)
    auto act_map = [&](char* base, int C, int Wv, int Hv, size_t stride_w, size_t stride_h, size_t stride_b, int bk,
                       int tw, int rows, int tb) -> int {
        auto key = std::make_tuple((uintptr_t)base, C, Wv, Hv, (int)stride_w, bk, tw, rows, tb);
        auto it = cache.find(key);
        if (it != cache.end()) return it->second;
        if (tw > 256 || rows > 256 || tb > 256) return -1;
        CUtensorMap m;
        cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)Wv, (cuuint64_t)Hv, (cuuint64_t)g->batch};
        cuuint64_t strides[3] = {(cuuint64_t)stride_w, (cuuint64_t)stride_h, (cuuint64_t)stride_b};
        cuuint32_t box[4] = {(cuuint32_t)bk, (cuuint32_t)tw, (cuuint32_t)rows, (cuuint32_t)tb};
        cuuint32_t es[4] = {1, 1, 1, 1};
        if (encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   swizzle_of(bk), CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return -1;
        maps.push_back(m);
        cache[key] = (int)maps.size() - 1;
        return (int)maps.size() - 1;
    };
    std::vector<TcNode> dn;
    std::vector<TcKbWeight> dw;
    std::vector<TcKbAct> da;
    std::vector<TcBurst> db;
    std::vector<TcState> ds;
    for (const NodePlan& P : E->nodes) {
        const SrHostNode& n = g->nodes[P.node];
        TcNode d{};
        d.state[0] = ws + n.state[0].offset;
        d.state[1] = ws + n.state[1].offset;
        d.bias = reinterpret_cast<const float*>(ws + n.bias.offset);
        d.H = n.d.h; d.W = n.d.w; d.C = n.d.c; d.act = n.d.act;
        if (P.node2 >= 0) {
            const SrHostNode& n2 = g->nodes[P.node2];
            d.state2[0] = ws + n2.state[0].offset;
            d.state2[1] = ws + n2.state[1].offset;
            d.bias2 = reinterpret_cast<const float*>(ws + n2.bias.offset);
            d.act2 = n2.d.act;
            d.fused = 1;
        }
        d.tw = P.tw; d.th = P.th; d.tb = P.tb; d.sep = P.sep;
        d.n_cols = P.n_cols;
        d.l1_dw = P.pair == 1 ? P.tw : 0;
        d.l1_db = P.pair == 2 ? P.tb : 0;
        d.first_state = (int)ds.size();
        d.first_act = (int)da.size();
        std::vector<KmHost> dm;                       // per K-block of this node
        d.first_wg = (int)dw.size();
        d.n_wg = (int)P.wgroups.size();
        const int rows = P.th + P.sep, box_tb = P.box_tb();
        if (P.k_total > 65535) return SR_ERR_UNSUPPORTED;
        // one 3-D view per run: (channels of a block, output channels, blocks of the run); a box of g blocks lands in
        // shared memory block after block, each an ordinary K-major swizzled tile
        std::map<std::pair<int, int>, int> run_map;   // (run, blocks in the box) -> tensor map
        for (const WGroup& wg : P.wgroups) {
            if (run_map.count({wg.run, wg.n})) continue;
            const WRun& R = P.runs[wg.run];
            CUtensorMap m;
            cuuint64_t dims[3] = {(cuuint64_t)R.bk, (cuuint64_t)P.rows_total(g), (cuuint64_t)R.n_blocks};
            cuuint64_t strides[2] = {(cuuint64_t)P.k_total * 2, (cuuint64_t)R.bk * 2};
            cuuint32_t box[3] = {(cuuint32_t)R.bk, (cuuint32_t)std::min(P.rows_total(g), 128), (cuuint32_t)wg.n};
            cuuint32_t es[3] = {1, 1, 1};
            if (encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, ws + P.wcat.offset + (size_t)R.first_col * 2, dims, strides, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(R.bk), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return SR_ERR_CUDA;
            maps.push_back(m);
            run_map[{wg.run, wg.n}] = (int)maps.size() - 1;
        }
        const size_t first_kw = dw.size();
        for (const WGroup& wg : P.wgroups) {
            TcKbWeight kw{};
            const size_t bytes = (size_t)wg.bytes;
            const int mi = run_map[{wg.run, wg.n}];
            if (wg.blk > 65535 || mi > 65535 || (bytes >> 4) > 65535) return SR_ERR_UNSUPPORTED;
            kw.blk = (uint16_t)wg.blk;
            kw.w_map = (uint16_t)mi;
            kw.w_bytes16 = (uint16_t)(bytes >> 4);
            dw.push_back(kw);
        }
        std::vector<int> group_of;                    // K-block -> weight group of the node
        for (size_t gi = 0; gi < P.wgroups.size(); ++gi)
            for (int j = 0; j < P.wgroups[gi].n; ++j) group_of.push_back((int)gi);
        for (size_t i = 0; i < P.kbs.size(); ++i) {
            const KbHost& kb = P.kbs[i];
            const SrHostEdge& he = g->edges[kb.edge];
            const SrHostNode& s = g->nodes[he.d.src];
            TcKbAct kl{};
            KmHost km;
            int map0 = -1, map1 = -1, qxv = 0, qyv = 0;
            kl.flags = (uint8_t)(he.R ? 1 : 0);
            km.x_load = kb.x_load;
            km.x_release = kb.x_release;
            km.w_step16 = (uint32_t)((std::min(P.rows_total(g), 128) * kb.bk * 2) >> 4);
            km.n_k16 = (uint32_t)(kb.bk / 16);
            km.desc_hi = desc_hi_of(kb.bk);
            const size_t x_bytes = (size_t)kb.bk * 2 * kb.x_width * rows * box_tb;
            const size_t l1_bytes = (size_t)lane1_shift_px(P, kb.x_width) * kb.bk * 2;
            const size_t sbo_bytes = (size_t)kb.x_width * 8 / P.tw * kb.bk * 2;
            if ((x_bytes >> 4) > 65535 || (l1_bytes >> 4) > 65535 || (sbo_bytes >> 4) > 0x3FFF) return SR_ERR_UNSUPPORTED;
            kl.x_bytes16 = (uint16_t)(x_bytes >> 4);
            km.x_sbo16 = (uint32_t)(sbo_bytes >> 4);
            km.x_l1off16 = (uint32_t)(l1_bytes >> 4);
            km.x_off16 = (uint32_t)((kb.x_shift * kb.bk * 2) >> 4);
            if (kb.stem) {
                const StemPlan& S = E->stems[kb.stem_index];
                for (int par = 0; par < 2; ++par)
                    (par ? map1 : map0) = act_map(ws + S.buf[par].offset, S.Kp, n.d.w, n.d.h, (size_t)S.Kp * 2,
                                                  (size_t)n.d.w * S.Kp * 2, (size_t)n.d.h * n.d.w * S.Kp * 2, kb.bk, kb.x_width, rows, box_tb);
                kl.c0_16 = (uint8_t)(kb.c0 / 16);
            } else if (!kb.x_load) {
                map0 = map1 = 0;                         // reuses the box the first tap of its class loaded
                kl.c0_16 = (uint8_t)(kb.c0 / 16);
            } else {
                // input pixel = stride * (output pixel + q) + r, q = floor((tap - pad) / stride), r the residue:
                // the residue-class view of the source makes the tap a dense box starting at (w0 + qx, h0 + qy)
                const int st = he.stride_eff;
                const int qy = kb.box_qy, ry = kb.box_ry, qx = kb.box_qx, rx = kb.box_rx;
                const int Hv = (s.d.h - ry + st - 1) / st, Wv = (s.d.w - rx + st - 1) / st;
                if (Hv <= 0 || Wv <= 0) return SR_ERR_UNSUPPORTED;
                for (int par = 0; par < 2; ++par) {
                    char* base = ws + s.state[par].offset + ((size_t)ry * s.d.w + rx) * s.d.c * 2;
                    (par ? map1 : map0) = act_map(base, s.d.c, Wv, Hv, (size_t)st * s.d.c * 2, (size_t)st * s.d.w * s.d.c * 2,
                                                  (size_t)s.d.h * s.d.w * s.d.c * 2, kb.bk, kb.x_width, rows, box_tb);
                }
                qxv = qx; qyv = qy; kl.c0_16 = (uint8_t)(kb.c0 / 16);
            }
            if (map0 < 0 || map1 < 0) return SR_ERR_CUDA;
            if (map0 > 65535 || map1 > 65535 || qxv < -128 || qxv > 127 || qyv < -128 || qyv > 127 || kb.c0 / 16 > 255) return SR_ERR_UNSUPPORTED;
            kl.x_map0 = (uint16_t)map0; kl.x_map1 = (uint16_t)map1;
            kl.qx = (int8_t)qxv; kl.qy = (int8_t)qyv;
            if (kb.in_wring) {
                // the box belongs to the block's weight group: the weight producer fetches it, no activation slot is used
                TcKbWeight& kw = dw[first_kw + group_of[i]];
                if (qxv != 0 || qyv != 0 || (kb.box_off & 1023) != 0 || (kb.box_off >> 4) > 65535) return SR_ERR_UNSUPPORTED;
                kw.x_off16 = (uint16_t)(kb.box_off >> 4);
                kw.x_map0 = kl.x_map0;
                kw.x_map1 = kl.x_map1;
                kw.c0_16 = kl.c0_16;
                kw.flags = kl.flags;
                km.x_load = km.x_release = false;
                km.x_off16 += (uint32_t)(kb.box_off >> 4);
                km.in_wring = true;
            } else if (kb.x_load) {
                da.push_back(kl);
            }
            dm.push_back(km);
        }
        d.n_act = (int)da.size() - d.first_act;
        // bursts: one per weight group; descriptor states: the distinct (weight, activation) upper words of the node
        size_t i0 = 0;
        for (const WGroup& wg : P.wgroups) {
            const KmHost& a = dm[i0];
            TcState st{};
            st.desc_hi = a.desc_hi;
            st.x_hi = (a.desc_hi & ~0x3FFFu) | a.x_sbo16;
            st.n_k16 = (uint16_t)a.n_k16;
            st.w_step16 = (uint16_t)a.w_step16;
            size_t si = (size_t)d.first_state;
            for (; si < ds.size(); ++si)
                if (std::memcmp(&ds[si], &st, sizeof(st)) == 0) break;
            if (si == ds.size()) ds.push_back(st);
            if (si - d.first_state > 255 || wg.n > 2 || (wg.n == 2 && P.pair != 0)) return SR_ERR_UNSUPPORTED;
            TcBurst b{};
            b.state = (uint8_t)(si - d.first_state);
            b.xa_off16 = (uint16_t)a.x_off16;
            b.flags = (uint8_t)((a.x_load ? 1 : 0) | (a.x_release ? 4 : 0) | (a.in_wring ? 32 : 0));
            if (a.in_wring && wg.n != 1) return SR_ERR_UNSUPPORTED;
            if (wg.n == 2) {
                const KmHost& c = dm[i0 + 1];
                if (c.desc_hi != a.desc_hi || c.x_sbo16 != a.x_sbo16) return SR_ERR_UNSUPPORTED;
                b.xb_off16 = (uint16_t)c.x_off16;
                b.flags |= (uint8_t)(16 | (c.x_load ? 2 : 0) | (c.x_release ? 8 : 0));
            } else {
                if (a.x_off16 + a.x_l1off16 > 65535) return SR_ERR_UNSUPPORTED;
                b.xb_off16 = (uint16_t)(a.x_off16 + a.x_l1off16);
            }
            db.push_back(b);
            i0 += (size_t)wg.n;
        }
        dn.push_back(d);
    }
    if (maps.size() * sizeof(CUtensorMap) > E->r_maps.bytes) return SR_ERR_UNSUPPORTED;
    E->n_maps = (int)maps.size();
    std::vector<TcTile> tiles;
    for (auto& v : E->group_tiles) tiles.insert(tiles.end(), v.begin(), v.end());
    std::vector<TcStem> stems;
    for (const StemPlan& S : E->stems) {
        const SrHostEdge& he = g->edges[S.edge];
        const SrHostNode& s = g->nodes[he.d.src];
        const SrHostNode& t = g->nodes[he.d.tgt];
        TcStem d{};
        for (int par = 0; par < 2; ++par) {
            d.src[par] = ws + s.state[par].offset;
            d.dst[par] = ws + S.buf[par].offset;
        }
        d.Hs = s.d.h; d.Ws = s.d.w; d.Cs = s.d.c; d.Ho = t.d.h; d.Wo = t.d.w;
        d.k = he.k_eff; d.stride = he.stride_eff; d.pad = he.pad_eff; d.Kp = S.Kp; d.K = he.K;
        stems.push_back(d);
    }
    auto up = [&](const SrRegion& r, const void* p, size_t bytes) {
        return bytes == 0 || cudaMemcpy(ws + r.offset, p, bytes, cudaMemcpyHostToDevice) == cudaSuccess;
    };
    if (!up(E->r_maps, maps.data(), maps.size() * sizeof(CUtensorMap)) || !up(E->r_nodes, dn.data(), dn.size() * sizeof(TcNode)) ||
        !up(E->r_kb_weight, dw.data(), dw.size() * sizeof(TcKbWeight)) || !up(E->r_kb_act, da.data(), da.size() * sizeof(TcKbAct)) ||
        !up(E->r_bursts, db.data(), db.size() * sizeof(TcBurst)) || !up(E->r_states, ds.data(), ds.size() * sizeof(TcState)) ||
        !up(E->r_tiles, tiles.data(), tiles.size() * sizeof(TcTile)) || !up(E->r_stems, stems.data(), stems.size() * sizeof(TcStem)))
        return SR_ERR_CUDA;
    return SR_OK;
}

sr_status sr_tc_set_weights(sr_graph* g, int edge, const float* w_eff)
{
    TcEngine* E = eng(g);
    if (!E) return SR_ERR_STATE;
    const SrHostEdge& he = g->edges[edge];
    const int ni = E->node_of[he.d.tgt];
    if (ni < 0) return SR_ERR_STATE;
    const NodePlan& P = E->nodes[ni];
    const SrHostNode& t = g->nodes[he.d.tgt];
    // the node's weight matrix keeps its columns in the order the K loop walks them: every K-block of this edge
    // takes its slice [C_out][block width] of the edge's own matrix (a staged edge: all of it, zero-padded)
    bool any = false;
    for (const KbHost& kb : P.kbs) {
        if (kb.edge != edge && kb.edge2 != edge) continue;
        const int row_off = kb.edge == edge ? kb.row_off : 64;
        any = true;
        const int n_src = kb.stem ? std::max(0, std::min(kb.bk, he.K - kb.src_col)) : kb.bk;
        std::vector<uint16_t> h((size_t)t.d.c * kb.bk, 0);
        for (int co = 0; co < t.d.c; ++co)
            for (int k = 0; k < n_src; ++k) {
                const __nv_bfloat16 b = __float2bfloat16_rn(w_eff[(size_t)co * he.K + kb.src_col + k]);
                std::memcpy(&h[(size_t)co * kb.bk + k], &b, 2);
            }
        char* dst = g->ws + P.wcat.offset + ((size_t)row_off * P.k_total + kb.k_off) * 2;
        if (cudaMemcpy2D(dst, (size_t)P.k_total * 2, h.data(), (size_t)kb.bk * 2, (size_t)kb.bk * 2, t.d.c,
                         cudaMemcpyHostToDevice) != cudaSuccess)
            return SR_ERR_CUDA;
    }
    if (!any) return SR_ERR_STATE;
    return SR_OK;
}

static int launch_stage(sr_graph* g, int t_off, int fixed_parity, cudaStream_t s)
{
    TcEngine* E = eng(g);
    if (!E || E->stems.empty()) return 0;
    size_t most = 0;
    for (const StemPlan& S : E->stems) {
        const SrHostNode& t = g->nodes[g->edges[S.edge].d.tgt];
        most = std::max(most, (size_t)g->batch * t.d.h * t.d.w);
    }
    const int blocks = (int)std::min<size_t>((size_t)E->sm_count * 8, (most + 255) / 256);
    sr_tc_stage_kernel<<<blocks, 256, 0, s>>>(reinterpret_cast<const TcStem*>(g->ws + E->r_stems.offset), (int)E->stems.size(),
                                              reinterpret_cast<const SrFrameCtl*>(g->ws + g->r_ctl.offset), t_off,
                                              fixed_parity, g->batch);
    return 1;
}

int sr_tc_stage_inputs(sr_graph* g, int t_off, cudaStream_t s) { return launch_stage(g, t_off, -1, s); }

int sr_tc_after_state_change(sr_graph* g, cudaStream_t s)
{
    // the shared work list's counters start from zero (every launch leaves them there; this covers a launch cut short)
    if (TcEngine* E = eng(g))
        if (g->ws) cudaMemsetAsync(g->ws + E->r_sched.offset, 0, 256, s);
    return launch_stage(g, 0, (int)(g->t & 1), s);
}

int sr_tc_launch_group(sr_graph* g, int group, int t_off, cudaStream_t s)
{
    TcEngine* E = eng(g);
    if (!E || E->group_tiles[group].empty()) return 0;
    const int n_a = E->group_n_a[group], a_slot = E->group_a_slot[group], n_w = E->group_n_w[group], w_slot = E->group_w_slot[group];
    const size_t smem = (size_t)n_a * a_slot + (size_t)n_w * w_slot + 1024;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    bool timed = g->opt_time_tc != 0 && cudaStreamIsCapturing(s, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone;
    if (timed) {
        if (E->ev_used + 2 > E->ev.size()) {
            if (E->ev.size() >= 4096) timed = false;
            else
                for (int i = 0; i < 2; ++i) {
                    cudaEvent_t e = nullptr;
                    if (cudaEventCreate(&e) != cudaSuccess) { timed = false; break; }
                    E->ev.push_back(e);
                }
        }
        if (timed && E->ev_used + 2 <= E->ev.size()) cudaEventRecord(E->ev[E->ev_used], s);
        else timed = false;
    }
    sr_tc_group_kernel<<<E->group_grid[group], kThreads, smem, s>>>(
        reinterpret_cast<const CUtensorMap*>(g->ws + E->r_maps.offset), reinterpret_cast<const TcNode*>(g->ws + E->r_nodes.offset),
        reinterpret_cast<const TcKbWeight*>(g->ws + E->r_kb_weight.offset), reinterpret_cast<const TcKbAct*>(g->ws + E->r_kb_act.offset),
        reinterpret_cast<const TcBurst*>(g->ws + E->r_bursts.offset), reinterpret_cast<const TcState*>(g->ws + E->r_states.offset),
        reinterpret_cast<const TcTile*>(g->ws + E->r_tiles.offset) + E->group_tile_offset[group],
        (int)E->group_tiles[group].size(), reinterpret_cast<SrFrameCtl*>(g->ws + g->r_ctl.offset), t_off, g->batch, n_a, a_slot,
        n_w, w_slot, E->group_ctas_per_sm[group] > 1 ? 256 : 512, (long long)g->opt_wait_ms * 2000000LL,
        g->opt_tc_lists == 0 ? reinterpret_cast<int*>(g->ws + E->r_sched.offset) : nullptr, E->group_n_own[group]);
    if (timed) {
        cudaEventRecord(E->ev[E->ev_used + 1], s);
        E->ev_used += 2;
    }
    return 1;
}

// Sum of the event-timed durations of the tensor-core group launches since the last call (synchronises).
sr_status sr_tc_timing(sr_graph* g, double* ms, long long* launches)
{
    TcEngine* E = eng(g);
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

bool sr_tc_group_has_work(const sr_graph* g, int group)
{
    TcEngine* E = eng(g);
    return E && !E->group_tiles[group].empty();
}

void sr_tc_destroy(sr_graph* g)
{
    if (g && g->tc) {
        for (cudaEvent_t e : eng(g)->ev) cudaEventDestroy(e);
        delete eng(g);
        g->tc = nullptr;
    }
}
