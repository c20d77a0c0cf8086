// Tensor-core engine: the node update  x_v = sigma(b_v + sum_e f_e(theta_e, x_src(e)))  (paper Sec. A1.2)
// for all convolutional nodes of one launch group as ONE grouped implicit GEMM on tcgen05 / TMEM.
//
// The sum over the incoming edges of a node is one convolution over the concatenated sources
// (paper Sec. A, "mathematically equivalent to concatenating all inputs"): the K loop of an output
// tile simply walks the K-blocks of every incoming edge, tap by tap, into one TMEM accumulator.
//
// GEMM shape.  D[c_out][pixel] = sum_k W[c_out][k] * X[pixel][k]: the weights are the M operand
// (128 rows per instruction, two halves for C_out > 128), up to 256 output pixels are the N operand.
// Measured on B200, one tcgen05.mma of M = 128 costs about 110 cycles however small N is and 128
// cycles at N = 256, and a tcgen05.commit is only free if about eight MMAs lie between commits; so
// every instruction is given N = 256 pixels and weight tiles are released in groups.
//
// Operands.  K-block = one filter tap x up to 64 input channels.  Activation tiles come straight from
// the NHWC state of the source node through 4-D TMA boxes (zero fill outside the image = zero
// padding); a stride-s edge reads one of s*s residue-class views of the source, so every tap is again
// a dense box.  Weight tiles come from the node's concatenated weight matrix [C_out][K] (K-major)
// through 2-D TMA boxes.  Few-channel input edges (C_in = 1 or 3) are staged per frame into an im2col
// tensor with K padded to 16/32/64 so that they are ordinary K-blocks.
//
// Pixel tile.  A tile is tb samples x th rows x tw columns (tw a multiple of 8, so an image row of
// the tile is a whole number of swizzle atoms).  Every activation box holds th + sep rows per sample
// (sep = k - 1 of the node's stride-1 k x k edges), and the N columns of the GEMM are the rows of
// that stacked box: column n = (b * (th + sep) + r) * tw + x.  Columns with r >= th are never stored.
// This makes the k taps of one filter column row-shifted windows of ONE box: the box is loaded once
// per filter column and the shared-memory descriptor of tap ky just starts ky * tw rows further down.
//
// Warp roles in a CTA of 192 threads: warp 0 = TMA producer, warp 1 = MMA issuer (owns TMEM),
// warps 2..5 = epilogue (TMEM lane = output channel; bias, ReLU, bf16, NHWC stores in which a warp
// writes 32 consecutive channels of one pixel).  Two accumulators in TMEM let the epilogue of a tile
// overlap the main loop of the next when they fit.  CTAs are persistent and walk a tile list sorted
// by decreasing work.  Every wait is bounded; on expiry the kernel records an error in the frame
// control block, drains its own copies, frees TMEM and returns.
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

constexpr int kMaxCols = 256;                         // pixels (N of the MMA) per tile
constexpr int kThreads = 224;
constexpr int kFifo = 16;                             // burst descriptors in flight between scout and issuer
constexpr int kMaxA = 4;                              // activation ring depth
constexpr int kWUnit = 4096, kMaxWUnits = 32;         // weight ring: units of 4 KiB
constexpr int kSmemBudget = 200 * 1024;
constexpr int kMaxNodeKb = 128;                       // K-blocks per node the shared-memory table holds

// One K-block of a node's reduction: 32 bytes, staged into shared memory per node so that the two
// single-thread roles never wait on global memory between barrier waits.
struct TcKBlock {
    uint32_t k_off;         // first K column in the node's weight matrix
    uint32_t desc_hi;       // upper word of the shared-memory matrix descriptors (swizzle, SBO, version)
    uint16_t x_map0, x_map1;// tensor map of the activation box for source frame parity 0 / 1
    uint16_t w_map;         // tensor map of the weight box
    int8_t qx, qy;          // box origin relative to the tile origin (columns, rows)
    uint16_t c0;            // first channel of the box
    uint16_t x_off16;       // (byte offset of this tap's window inside the activation slot) / 16
    uint16_t x_bytes16;     // (bytes of the activation box this block loads into a fresh slot) / 16; 0 = reuse the slot
    uint16_t w_bytes16;     // (bytes of the weight box) / 16
    uint8_t n_k16;          // MMA steps (K = 16 each) in this block
    uint8_t flags;          // 1: the edge reads frame t (R = 1), else frame t+1; 2: last reader of the activation
                            // slot; 4: first box of a weight group; 8: last box of a weight group
    uint8_t w_box;          // index of this block's weight box inside its group
    uint8_t x_sbo16;        // (bytes between 8-pixel groups of the activation operand) / 16: one image row of the box
    uint8_t pad_[4];
};
static_assert(sizeof(TcKBlock) == 32, "K-block table entries are copied as two 16-byte words");

struct TcNode {
    void* state[2];
    const float* bias;
    int32_t H, W, C, act;
    int32_t tw, th, tb, sep;        // tile geometry (see the file comment)
    int32_t n_cols;                 // N of the MMA: stacked rows of a tile, rounded up to 32
    int32_t n_mh;                   // halves of 128 output channels
    int32_t first_kb, n_kb;
    uint32_t idesc;
    int32_t w_box_units, w_group_units;
    int32_t pad_;
};

struct TcTile { int32_t node, b0, h0, w0, m0, pad_[3]; };   // m0: first output channel of the tile (0 or 128)

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
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* map, uint32_t bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
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
__global__ void __launch_bounds__(kThreads, 1)
sr_tc_group_kernel(const CUtensorMap* __restrict__ maps, const TcNode* __restrict__ nodes,
                   const TcKBlock* __restrict__ kbs, const TcTile* __restrict__ tiles, int n_tiles,
                   SrFrameCtl* __restrict__ ctl, int t_off, int B, int n_a, int a_slot, int n_wu, int w_slot_units, int tmem_cols,
                   long long wait_limit)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * kMaxA + 2 * kMaxWUnits + 4];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ uint4 kb_tab[2][2 * kMaxNodeKb];            // K-block tables of the producer's and the issuer's current node
    __shared__ __align__(16) uint16_t epi_buf[4][32 * 32]; // per epilogue warp: 32 pixels x 32 channels, bf16
    __shared__ int pix_off[kMaxCols];                      // element offset of every pixel of the current tile, -1 = not stored
    __shared__ __align__(16) uint4 fifo[kFifo][2];         // burst descriptors, scout -> issuer
    __shared__ volatile uint32_t fifo_read;                // descriptors the issuer has taken

    // weight ring first: an M = 128 instruction on a node with fewer than 128 output channels reads
    // rows past its weight box, which then still lie inside this allocation
    // A wait limit of zero (a host-side test hook) means "every wait has already expired": report it and return
    // before any barrier, tensor memory, copy or MMA is touched.
    if (wait_limit <= 0) {
        if (threadIdx.x == 0) atomicExch(&ctl->error, 1);
        return;
    }
    const uint32_t w_ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_ring = w_ring + (uint32_t)(n_wu * kWUnit);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t bar_afull = smem_u32(&bars[0]), bar_aempty = smem_u32(&bars[kMaxA]);
    const uint32_t bar_wfull = smem_u32(&bars[2 * kMaxA]), bar_wempty = smem_u32(&bars[2 * kMaxA + kMaxWUnits]);
    const uint32_t bar_tfull = smem_u32(&bars[2 * kMaxA + 2 * kMaxWUnits]), bar_tempty = bar_tfull + 16;

    if (threadIdx.x < kFifo) {
        fifo[threadIdx.x][0] = make_uint4(0, 0, 0, 0);
        fifo[threadIdx.x][1] = make_uint4(0, 0, 0, 0);
    }
    if (threadIdx.x == 0) {
        abort_flag = 0;
        fifo_read = 0;
        for (int s = 0; s < n_a; ++s) {
            mbar_init(bar_afull + 8 * s, 1);
            mbar_init(bar_aempty + 8 * s, 1);
        }
        for (int s = 0; s < n_wu; ++s) {
            mbar_init(bar_wfull + 8 * s, 1);
            mbar_init(bar_wempty + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tfull + 8 * a, 1);
            mbar_init(bar_tempty + 8 * a, 4);
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

    // Accumulator buffers: a tile whose n_mh * n_cols columns fit into 256 takes the less used of the
    // two 256-column buffers, a wider tile takes both.  uses[] counts the tiles a buffer has served;
    // the issuer and the epilogue warps walk the same tile list and make the same choice.
    uint32_t uses0 = 0, uses1 = 0;

    if (warp == 0 || warp == 6) {
        // The producer (warp 0) and the scout (warp 6) walk the same tile list.  At every change of node the whole warp
        // copies the node's K-block table into its own shared-memory buffer; lane 0 then runs the
        // block loop out of shared memory.
        uint4* my_tab = kb_tab[warp == 0 ? 0 : 1];
        uint32_t n_pub = 0;                                   // bursts published so far (scout)
        int cached_node = -1;
        // The weight ring is a ring of slots of w_slot_units 4 KiB units (the largest weight group of
        // the launch), handed back through one "empty" barrier per slot.  Box i of a group starts at
        // unit i * w_box_units of its slot and signals arrival on that unit's "full" barrier (a full
        // barrier per group would let the issuer wait for boxes whose activation slots it still
        // holds).  Which units lead a box depends on the node, and a unit's barrier flips phase only
        // when used, so both roles keep one phase bit per unit.
        const uint32_t n_ws = (uint32_t)(n_wu / w_slot_units);
        uint32_t ia = 0, wf_phase = 0, wf_used = 0, ws_cur = 0, a_cur = 0;
        uint32_t a_nxt = 0, a_ph = 0, w_nxt = 0, w_ph = 0;    // next slot of each ring and the phase of its barriers
        bool ok = true;
        for (int ti = blockIdx.x; ti < n_tiles; ti += gridDim.x) {
            const TcTile tl = tiles[ti];
            const int first_kb = nodes[tl.node].first_kb, n_kb = nodes[tl.node].n_kb;
            const uint32_t box_u = (uint32_t)nodes[tl.node].w_box_units;
            const uint32_t idesc = nodes[tl.node].idesc;
            if (tl.node != cached_node) {
                __syncwarp();
                const uint4* src = reinterpret_cast<const uint4*>(kbs + first_kb);
                for (int i = lane; i < 2 * n_kb; i += 32) my_tab[i] = src[i];
                cached_node = tl.node;
                __syncwarp();
            }
            if (lane == 0 && ok) {
                const TcKBlock* tab = reinterpret_cast<const TcKBlock*>(my_tab);
                if (warp == 0) {
                    // ------------------------------------------------------ TMA producer
                    for (int kb = 0; kb < n_kb; ++kb) {
                        const TcKBlock k = tab[kb];
                        if (k.x_bytes16) {
                            const uint32_t s = a_nxt;
                            if (!mbar_wait(bar_aempty + 8 * s, a_ph ^ 1, abortp, wait_limit)) { ok = false; break; }
                            if (++a_nxt == (uint32_t)n_a) { a_nxt = 0; a_ph ^= 1; }
                            mbar_expect_tx(bar_afull + 8 * s, (uint32_t)k.x_bytes16 << 4);
                            const int par = (k.flags & 1) ? prev : cur;
                            tma_load_4d(a_ring + s * a_slot, &maps[par ? k.x_map1 : k.x_map0], bar_afull + 8 * s, k.c0,
                                        tl.w0 + k.qx, tl.h0 + k.qy, tl.b0);
                            ++ia;
                        }
                        if (k.flags & 4) {
                            ws_cur = w_nxt;
                            if (!mbar_wait(bar_wempty + 8 * ws_cur, w_ph ^ 1, abortp, wait_limit)) { ok = false; break; }
                            if (++w_nxt == n_ws) { w_nxt = 0; w_ph ^= 1; }
                        }
                        const uint32_t unit = ws_cur * (uint32_t)w_slot_units + k.w_box * box_u;
                        mbar_expect_tx(bar_wfull + 8 * unit, (uint32_t)k.w_bytes16 << 4);
                        tma_load_2d(w_ring + unit * kWUnit, &maps[k.w_map], bar_wfull + 8 * unit, (int)k.k_off, tl.m0);
                        wf_phase ^= 1u << unit;
                        wf_used |= 1u << unit;
                    }
                } else {
                    // ------------------------------------------------------ scout
                    // Measured: whatever the issuing thread executes between two tcgen05.mma costs tensor-pipe
                    // time one for one (a probe of a ready barrier ~165 cycles, a shared-memory load ~110, a
                    // commit ~50), except for ~200 cycles per burst of >= 8 MMAs.  So this thread does all the
                    // waiting and address arithmetic and hands the issuer one 32-byte descriptor per weight
                    // group (up to 3 K-blocks = 12 MMAs): descriptor address words, flags, barriers to commit.
                    const uint32_t acc = (tmem_cols >= 512 && uses0 > uses1) ? 1u : 0u;   // 256 columns: one accumulator
                    if (!mbar_wait(bar_tempty + 8 * acc, ((acc ? uses1 : uses0) & 1) ^ 1, abortp, wait_limit)) ok = false;
                    int kb = 0;
                    while (kb < n_kb && ok) {
                        uint32_t lo[3] = {0u, 0u, 0u}, nt = 0, act_mask = 0, n_k16 = 0, desc_hi = 0, x_hi = 0, commit_w = 0, loads = 0;
                        const uint32_t first = kb == 0;
                        // a burst stays inside one weight group and never holds so many fresh activation slots
                        // that the producer could not load the next one (it would wait for this very burst)
                        const uint32_t max_loads = n_a > 2 ? (uint32_t)n_a - 1 : 1u;
                        while (nt < 3 && kb < n_kb) {
                            const TcKBlock k = tab[kb];
                            if (nt > 0 && k.x_bytes16 && loads >= max_loads) break;
                            if (k.x_bytes16) {
                                a_cur = a_nxt;
                                if (!mbar_wait(bar_afull + 8 * a_cur, a_ph, abortp, wait_limit)) { ok = false; break; }
                                if (++a_nxt == (uint32_t)n_a) { a_nxt = 0; a_ph ^= 1; }
                                ++loads;
                            }
                            if (k.flags & 4) {
                                ws_cur = w_nxt;
                                if (++w_nxt == n_ws) w_nxt = 0;
                            }
                            const uint32_t unit = ws_cur * (uint32_t)w_slot_units + k.w_box * box_u;
                            if (!mbar_wait(bar_wfull + 8 * unit, (wf_phase >> unit) & 1, abortp, wait_limit)) { ok = false; break; }
                            wf_phase ^= 1u << unit;
                            const uint32_t x_lo = (((a_ring + a_cur * a_slot) >> 4) + k.x_off16) & 0x3FFFu;
                            const uint32_t w_lo = ((w_ring + unit * kWUnit) >> 4) & 0x3FFFu;
                            lo[nt] = w_lo | (x_lo << 16);
                            if (k.flags & 2) act_mask |= 1u << a_cur;
                            n_k16 = k.n_k16;
                            desc_hi = k.desc_hi;
                            x_hi = (k.desc_hi & ~0x3FFFu) | k.x_sbo16;
                            ++nt;
                            ++kb;
                            if (k.flags & 8) { commit_w = 1; break; }
                        }
                        if (!ok) break;
                        ++n_pub;
                        if (n_pub - fifo_read >= (uint32_t)kFifo) {          // never overwrite a descriptor not yet taken
                            const long long t0 = clock64();
                            while (n_pub - fifo_read >= (uint32_t)kFifo)
                                if (abort_flag || clock64() - t0 > wait_limit) { abort_flag = 1; ok = false; break; }
                            if (!ok) break;
                        }
                        const uint32_t fl = nt | (n_k16 << 2) | (first << 5) | (acc << 6) | (commit_w << 7) | (ws_cur << 8) | (act_mask << 11) |
                                            ((kb == n_kb ? 1u : 0u) << 15);
                        const uint32_t e = smem_u32(&fifo[n_pub & (kFifo - 1)][0]);
                        st_shared_v4(e + 16, lo[0], lo[1], lo[2], x_hi);
                        __threadfence_block();
                        st_shared_v4(e, n_pub, desc_hi, idesc, fl);
                    }
                    if (acc == 0) ++uses0; else ++uses1;
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
        }
        if (warp == 6 && lane == 0) {
            ++n_pub;                                                                // tell the issuer to stop
            const uint32_t e = smem_u32(&fifo[n_pub & (kFifo - 1)][0]);
            st_shared_v4(e + 16, 0, 0, 0, n_pub);
            __threadfence_block();
            st_shared_v4(e, n_pub, 0, 0, 1u << 16);
        }
        if (warp == 0 && lane == 0) {
            // drain: every copy this thread started must have landed before the CTA may exit
            for (uint32_t j = 0; j < (uint32_t)n_a && j < ia; ++j) {
                const uint32_t i2 = ia - 1 - j;
                mbar_wait_drain(bar_afull + 8 * (i2 % n_a), (i2 / n_a) & 1, wait_limit);
            }
            for (uint32_t v = 0; v < (uint32_t)n_wu; ++v)
                if ((wf_used >> v) & 1) mbar_wait_drain(bar_wfull + 8 * v, ((wf_phase >> v) & 1) ^ 1, wait_limit);
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        // One thread; it reads burst descriptors and issues, nothing else (see the scout).
        if (lane == 0) {
            uint32_t n = 0;
            for (;;) {
                ++n;
                const uint32_t e = smem_u32(&fifo[n & (kFifo - 1)][0]);
                uint4 q0 = ld_shared_v4(e);
                if (q0.x != n) {
                    const long long t0 = clock64();
                    bool give_up = false;
                    while ((q0 = ld_shared_v4(e)).x != n) {
                        if (abort_flag || clock64() - t0 > wait_limit) { give_up = true; break; }
                    }
                    if (give_up) { abort_flag = 1; break; }
                }
                __threadfence_block();
                const uint4 q1 = ld_shared_v4(e + 16);
                fifo_read = n;
                const uint32_t fl = q0.w;
                if (fl & (1u << 16)) break;
                const uint32_t w_hi = q0.y, x_hi = q1.w, idesc = q0.z, nt = fl & 3u, nk = (fl >> 2) & 7u, acc = (fl >> 6) & 1u;
                const uint32_t d_tmem = tmem_base + acc * 256;
                if (fl & 32u) tc_fence_after();                          // first burst of a tile: the accumulator was just handed back
                uint32_t accum = (fl & 32u) ? 0u : 1u;
                const uint32_t los[3] = {q1.x, q1.y, q1.z};
#pragma unroll
                for (uint32_t t = 0; t < 3; ++t) {
                    if (t < nt) {
                        const uint32_t wl = (los[t] & 0x3FFFu) | 0x10000u, xl = (los[t] >> 16) | 0x10000u;
                        // a K = 16 step moves both operands 32 bytes along K: +2 in the descriptors' address field
                        for (uint32_t j = 0; j < nk; ++j) {
                            tc_mma_bf16_lohi(d_tmem, wl + 2 * j, w_hi, xl + 2 * j, x_hi, idesc, accum);
                            accum = 1u;
                        }
                    }
                }
                if (fl & 128u) tc_commit(bar_wempty + 8 * ((fl >> 8) & 7u));   // hands the weight slot back
                uint32_t m = (fl >> 11) & 15u;
                while (m) {                                              // activation slots this burst read last
                    const uint32_t sl = __ffs(m) - 1;
                    tc_commit(bar_aempty + 8 * sl);
                    m &= m - 1;
                }
                if (fl & (1u << 15)) tc_commit(bar_tfull + 8 * acc);     // accumulator complete
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (warps 2..5)
        // TMEM lane = output channel, TMEM column = pixel.  A warp turns 32 channels x 32 pixels into
        // NHWC order through a 2 KiB shared-memory buffer: every thread writes its channel of 32 pixels
        // (bias, ReLU, bf16), then reads back 8 consecutive channels of one pixel and stores them as one
        // 16-byte word, so a pixel's 32 channels leave the warp as one 64-byte run.  The element offset
        // of every pixel of the tile (or -1 for the separator rows and for pixels outside the image) is
        // tabulated once per tile.
        const int quarter = warp & 3;                       // TMEM lanes 32*quarter .. +31 belong to this warp
        const int et = threadIdx.x - 64;                    // 0..127 among the epilogue threads
        uint16_t* tbuf = &epi_buf[warp - 2][0];
        bool ok = true;
        for (int ti = blockIdx.x; ti < n_tiles && ok; ti += gridDim.x) {
            const TcTile tl = tiles[ti];
            const TcNode nd = nodes[tl.node];
            const int rows = nd.th + nd.sep;
            for (int n = et; n < nd.n_cols; n += 128) {
                const int x = n % nd.tw, q = n / nd.tw, r = q % rows, bi = q / rows;
                const int b = tl.b0 + bi, y = tl.h0 + r, xx = tl.w0 + x;
                const bool v = r < nd.th && bi < nd.tb && b < B && y < nd.H && xx < nd.W;
                pix_off[n] = v ? (int)((((size_t)b * nd.H + y) * nd.W + xx) * nd.C) : -1;
            }
            const bool wide = nd.n_mh * nd.n_cols > 256;
            const uint32_t acc = (!wide && tmem_cols >= 512 && uses0 > uses1) ? 1u : 0u;
            if (wide || acc == 0) {
                if (!mbar_wait(bar_tfull, uses0 & 1, abortp, wait_limit)) ok = false;
            }
            if (ok && (wide || acc == 1)) {
                if (!mbar_wait(bar_tfull + 8, uses1 & 1, abortp, wait_limit)) ok = false;
            }
            ok = __all_sync(0xffffffffu, ok);
            asm volatile("bar.sync 1, 128;" ::: "memory");           // the offset table is complete
            if (abort_flag) ok = false;
            if (!ok) break;
            tc_fence_after();
            __nv_bfloat16* out = static_cast<__nv_bfloat16*>(nd.state[cur]);
            for (int h = 0; h < nd.n_mh; ++h) {
                const int co_w = tl.m0 + h * 128 + quarter * 32;        // first channel of this warp
                const int co = co_w + lane;                             // TMEM lane = output channel
                const float bias = co < nd.C ? __ldg(nd.bias + co) : 0.f;
                const bool gvalid = co_w + (lane & 3) * 8 < nd.C;       // this thread's group of 8 channels exists
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * 256 + h * nd.n_cols;
                for (int c0 = 0; c0 < nd.n_cols; c0 += 32) {
                    uint32_t v[32];
                    tc_ld32(taddr + c0, v);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        float z = __uint_as_float(v[j]) + bias;
                        if (nd.act == 1) z = fmaxf(z, 0.f);
                        const __nv_bfloat16 hz = __float2bfloat16_rn(z);
                        tbuf[j * 32 + lane] = *reinterpret_cast<const uint16_t*>(&hz);
                    }
                    __syncwarp();
#pragma unroll
                    for (int pass = 0; pass < 4; ++pass) {
                        const int p = pass * 8 + (lane >> 2);
                        const int o = pix_off[c0 + p];
                        if (o >= 0 && gvalid) {
                            const uint4 w = *reinterpret_cast<const uint4*>(tbuf + p * 32 + (lane & 3) * 8);
                            *reinterpret_cast<uint4*>(out + (size_t)o + co_w + (lane & 3) * 8) = w;
                        }
                    }
                    __syncwarp();
                }
            }
            tc_fence_before();
            asm volatile("bar.sync 1, 128;" ::: "memory");           // everybody is done with the offset table
            if (lane == 0) {
                if (wide || acc == 0) mbar_arrive(bar_tempty);
                if (wide || acc == 1) mbar_arrive(bar_tempty + 8);
            }
            if (wide || acc == 0) ++uses0;
            if (wide || acc == 1) ++uses1;
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(&ctl->error, 1);
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
    __shared__ int tap_off[64];     // offset of element kk relative to the (unpadded) window origin, -1 = padding
    __shared__ short tap_dy[64], tap_dx[64];
    const int cur = fixed_parity >= 0 ? fixed_parity : (int)((ctl->t + t_off + 1) & 1);
    for (int si = 0; si < n_stems; ++si) {
        const TcStem st = stems[si];
        __syncthreads();
        if (threadIdx.x < 64) {
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
    int x_width;       // pixels per image row of the box (tile width, plus the pixel range of the taps it serves)
    bool x_release;
    int box_qy = 0, box_qx = 0, box_ry = 0, box_rx = 0;   // origin and residue class of the box (loading block)
};

struct NodePlan {
    int node;
    int tw, th, tb, sep, n_cols, n_mh;
    bool one_box;                   // tw == 8: one activation box per channel block serves all k x k taps
    int group;                      // weight boxes per group
    int k_total;                    // columns of the concatenated weight matrix
    std::vector<KbHost> kbs;
    SrRegion wcat;
    std::vector<int> edge_k_off;    // first column of each incoming edge (index parallel to in_edges)
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
    std::vector<int> group_tile_offset, group_a_slot, group_n_a, group_n_wu, group_w_slot, group_grid, group_ctas_per_sm;
    SrRegion r_maps, r_nodes, r_kbs, r_tiles, r_stems;
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
int stem_kp(int K) { return K <= 16 ? 16 : (K <= 32 ? 32 : 64); }
bool is_stem(const sr_graph* g, const SrHostEdge& e)
{
    const SrHostNode& s = g->nodes[e.d.src];
    return s.is_input && (s.d.c % 16) != 0 && e.K <= 64;
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

}  // namespace

// A node goes to the tensor cores if it sums convolutions only, has 16..256 output channels in
// multiples of 8, and every incoming edge either has C_in % 16 == 0 or is a few-channel input edge.
void sr_tc_select_nodes(sr_graph* g)
{
    for (size_t v = 0; v < g->nodes.size(); ++v) {
        SrHostNode& n = g->nodes[v];
        n.use_tc = false;
        if (n.is_input || n.dense_target || (int)v == g->info.output_node) continue;
        if (n.d.c % 8 != 0 || n.d.c < 16 || n.d.c > 256) continue;
        bool ok = true;
        int n_blocks = 0;
        for (int e : n.in_edges) {
            const SrHostEdge& he = g->edges[e];
            const SrHostNode& s = g->nodes[he.d.src];
            if (he.d.kind != SR_EDGE_CONV) ok = false;
            else if (s.d.c % 16 != 0 && !is_stem(g, he)) ok = false;
            else if (he.k_eff > 8) ok = false;
            else n_blocks += is_stem(g, he) ? 1 : he.k_eff * he.k_eff * (s.d.c / block_k(s.d.c));
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
    E->node_of.assign(g->nodes.size(), -1);
    E->stem_of_edge.assign(g->edges.size(), -1);
    auto take = [&](size_t bytes) {
        SrRegion r;
        r.offset = off;
        r.bytes = bytes;
        off = sr_align_up(off + bytes, 1024);
        return r;
    };
    for (size_t v = 0; v < g->nodes.size(); ++v) {
        const SrHostNode& n = g->nodes[v];
        if (!n.use_tc) continue;
        NodePlan P{};
        P.node = (int)v;
        // sep: how many image rows the taps that share one activation box are apart at most
        auto tap_q = [](int tap, int pad, int st, int& q, int& r) {
            const int a = tap - pad;
            q = (a >= 0) ? a / st : -((-a + st - 1) / st);
            r = a - q * st;
        };
        P.sep = 0;
        for (int e : n.in_edges) {
            const SrHostEdge& he = g->edges[e];
            if (is_stem(g, he)) continue;
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
        P.n_mh = 1;                                   // a node with more than 128 output channels is tiled in halves
        P.group = 3;
        int k_off = 0;
        for (int e : n.in_edges) {
            const SrHostEdge& he = g->edges[e];
            const SrHostNode& s = g->nodes[he.d.src];
            P.edge_k_off.push_back(k_off);
            if (is_stem(g, he)) {
                StemPlan S;
                S.edge = e;
                S.Kp = stem_kp(he.K);
                const size_t bytes = (size_t)g->batch * n.d.h * n.d.w * S.Kp * 2;
                S.buf[0] = take(bytes);
                S.buf[1] = take(bytes);
                E->stem_of_edge[e] = (int)E->stems.size();
                E->stems.push_back(S);
                P.kbs.push_back(KbHost{e, true, (int)E->stems.size() - 1, 0, 0, 0, S.Kp, k_off, true, 0, P.tw, true});
                k_off += S.Kp;
            } else {
                // Taps whose input pixels fall into the same residue class of the stride read the same view of the
                // source, shifted by whole pixels: they share ONE activation box and differ only in where their window
                // starts inside it (rows always; pixels too when the tile is 8 wide, because then the 8-pixel groups of
                // the operand are simply one box row apart, whatever the row length).
                const int bk = block_k(s.d.c), k = he.k_eff, st = he.stride_eff;
                const int edge_off = k_off;
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
                        int qy0 = 1 << 20, qx0 = 1 << 20, qx1 = -(1 << 20);
                        for (const Tap& t : taps) { qy0 = std::min(qy0, t.qy); qx0 = std::min(qx0, t.qx); qx1 = std::max(qx1, t.qx); }
                        const int bw = P.tw + (qx1 - qx0);
                        for (size_t i = 0; i < taps.size(); ++i) {
                            const Tap& t = taps[i];
                            // the first tap of the class carries the box origin (qy0, qx0) through its ky / kx fields
                            KbHost kb{e, false, -1, t.ky, t.kx, c0, bk, edge_off + (t.ky * k + t.kx) * s.d.c + c0,
                                      i == 0, (t.qy - qy0) * bw + (t.qx - qx0), bw, i + 1 == taps.size()};
                            kb.box_qy = qy0;
                            kb.box_qx = qx0;
                            kb.box_ry = std::get<0>(cl.first);
                            kb.box_rx = std::get<1>(cl.first);
                            P.kbs.push_back(kb);
                        }
                    }
                k_off += k * k * s.d.c;
            }
        }
        P.k_total = k_off;
        P.wcat = take((size_t)n.d.c * P.k_total * 2);
        E->node_of[v] = (int)E->nodes.size();
        E->nodes.push_back(P);
    }
    // tiles per group, largest reduction first
    E->group_tiles.assign(g->groups.size(), {});
    int n_tiles = 0, n_kbs = 0;
    for (size_t gi = 0; gi < g->groups.size(); ++gi) {
        std::vector<std::pair<long long, TcTile>> tl;
        int a_slot = 1024, w_slot = 1;
        for (int v : g->groups[gi]) {
            if (E->node_of[v] < 0) continue;
            const NodePlan& P = E->nodes[E->node_of[v]];
            const SrHostNode& n = g->nodes[v];
            for (int b0 = 0; b0 < g->batch; b0 += P.tb)
                for (int h0 = 0; h0 < n.d.h; h0 += P.th)
                    for (int w0 = 0; w0 < n.d.w; w0 += P.tw)
                        for (int m0 = 0; m0 < n.d.c; m0 += 128)
                            tl.push_back({(long long)P.kbs.size() * P.n_cols, TcTile{E->node_of[v], b0, h0, w0, m0, {0, 0, 0}}});
            w_slot = std::max(w_slot, std::max(1, (std::min(n.d.c, 128) * 128 + kWUnit - 1) / kWUnit) * P.group);
            // a window starts up to sep * tw rows into the box and the MMA reads n_cols rows from there
            for (const KbHost& kb : P.kbs) {
                const size_t box_px = (size_t)kb.x_width * (P.th + P.sep) * P.tb;
                // the last 8-pixel group a window reads: shift + (n_cols / 8 - 1) rows of the box + 8 pixels
                const size_t reach_px = (size_t)kb.x_shift + (size_t)(P.n_cols / 8 - 1) * (kb.x_width * 8 / P.tw) + 8;
                a_slot = std::max(a_slot, (int)sr_align_up(std::max(box_px, reach_px) * kb.bk * 2, 1024));
            }
        }
        std::stable_sort(tl.begin(), tl.end(), [](const auto& a, const auto& b) { return a.first > b.first; });
        for (auto& p : tl) E->group_tiles[gi].push_back(p.second);
        E->group_tile_offset.push_back(n_tiles);
        n_tiles += (int)tl.size();
        int n_wu = g->opt_b_units > 0 ? g->opt_b_units : 24;
        n_wu = std::max(2 * w_slot, std::min(kMaxWUnits, n_wu)) / w_slot * w_slot;
        int n_a = std::max(2, std::min(kMaxA, (kSmemBudget - n_wu * kWUnit) / a_slot));
        // Small launches (a few tiles per SM) are bound by the latency of one tile, not by throughput: give every
        // CTA the smallest rings and one accumulator, so that two CTAs share an SM and twice as many tiles are in flight.
        int per_sm = 1;
        if ((int)tl.size() <= 4 * 148 && 2 * w_slot * kWUnit + 2 * a_slot <= 88 * 1024) {
            per_sm = 2;
            n_wu = 2 * w_slot;
            n_a = 2;
        }
        E->group_ctas_per_sm.push_back(per_sm);
        E->group_a_slot.push_back(a_slot);
        E->group_n_a.push_back(n_a);
        E->group_n_wu.push_back(n_wu);
        E->group_w_slot.push_back(w_slot);
    }
    for (const NodePlan& P : E->nodes) n_kbs += (int)P.kbs.size();
    E->n_tiles = n_tiles;
    E->n_kbs = n_kbs;
    // upper bound on distinct tensor maps: two parities per K-block plus one weight map per (node, bk)
    E->r_maps = take(sizeof(CUtensorMap) * (size_t)(2 * n_kbs + 3 * E->nodes.size() + 1));
    E->r_nodes = take(sizeof(TcNode) * E->nodes.size());
    E->r_kbs = take(sizeof(TcKBlock) * (size_t)std::max(1, n_kbs));
    E->r_tiles = take(sizeof(TcTile) * (size_t)std::max(1, n_tiles));
    E->r_stems = take(sizeof(TcStem) * std::max<size_t>(1, E->stems.size()));
    return SR_OK;
}

sr_status sr_tc_bind(sr_graph* g)
{
    TcEngine* E = eng(g);
    if (!E) return SR_OK;
    EncodeTiledFn encode = encode_fn();
    if (!encode) return SR_ERR_CUDA;
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&E->sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (cudaFuncSetAttribute(sr_tc_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 1024) != cudaSuccess)
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
    std::vector<TcKBlock> dk;
    for (const NodePlan& P : E->nodes) {
        const SrHostNode& n = g->nodes[P.node];
        TcNode d{};
        d.state[0] = ws + n.state[0].offset;
        d.state[1] = ws + n.state[1].offset;
        d.bias = reinterpret_cast<const float*>(ws + n.bias.offset);
        d.H = n.d.h; d.W = n.d.w; d.C = n.d.c; d.act = n.d.act;
        d.tw = P.tw; d.th = P.th; d.tb = P.tb; d.sep = P.sep;
        d.n_cols = P.n_cols; d.n_mh = P.n_mh;
        d.first_kb = (int)dk.size();
        d.n_kb = (int)P.kbs.size();
        // instruction descriptor: D = f32, A = B = bf16, both K-major, M = 128 output channels, N = pixels
        d.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P.n_cols >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        d.w_box_units = std::max(1, (std::min(n.d.c, 128) * 128 + kWUnit - 1) / kWUnit);
        d.w_group_units = d.w_box_units * P.group;
        const int rows = P.th + P.sep;
        std::map<int, int> wmap;                      // bk -> weight tensor map
        for (const KbHost& kb : P.kbs) {
            if (wmap.count(kb.bk)) continue;
            CUtensorMap m;
            cuuint64_t dims[2] = {(cuuint64_t)P.k_total, (cuuint64_t)n.d.c};
            cuuint64_t strides[1] = {(cuuint64_t)P.k_total * 2};
            cuuint32_t box[2] = {(cuuint32_t)kb.bk, (cuuint32_t)std::min(n.d.c, 128)};
            cuuint32_t es[2] = {1, 1};
            if (encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ws + P.wcat.offset, dims, strides, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(kb.bk), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return SR_ERR_CUDA;
            maps.push_back(m);
            wmap[kb.bk] = (int)maps.size() - 1;
        }
        // weight groups: up to P.group consecutive K-blocks of equal channel-block width
        std::vector<int> box_of(P.kbs.size(), 0);
        std::vector<char> starts(P.kbs.size(), 0), ends(P.kbs.size(), 0);
        for (size_t i = 0, in_group = 0; i < P.kbs.size(); ++i) {
            if (in_group == 0 || (int)in_group == P.group || P.kbs[i].bk != P.kbs[i - 1].bk || P.kbs[i].x_width != P.kbs[i - 1].x_width) {
                starts[i] = 1;
                if (i > 0) ends[i - 1] = 1;
                in_group = 0;
            }
            box_of[i] = (int)in_group++;
        }
        if (!P.kbs.empty()) ends[P.kbs.size() - 1] = 1;
        for (size_t i = 0; i < P.kbs.size(); ++i) {
            const KbHost& kb = P.kbs[i];
            const SrHostEdge& he = g->edges[kb.edge];
            const SrHostNode& s = g->nodes[he.d.src];
            TcKBlock k{};
            int map0 = -1, map1 = -1, qxv = 0, qyv = 0;
            const bool g_start = starts[i] != 0, g_end = ends[i] != 0;
            k.flags = (uint8_t)((he.R ? 1 : 0) | (kb.x_release ? 2 : 0) | (g_start ? 4 : 0) | (g_end ? 8 : 0));
            k.w_box = (uint8_t)box_of[i];
            k.w_map = (uint16_t)wmap[kb.bk];
            k.k_off = (uint32_t)kb.k_off;
            k.n_k16 = (uint8_t)(kb.bk / 16);
            k.desc_hi = desc_hi_of(kb.bk);
            k.x_bytes16 = kb.x_load ? (uint16_t)((kb.bk * 2 * kb.x_width * rows * P.tb) >> 4) : 0;
            k.x_sbo16 = (uint8_t)((kb.x_width * 8 / P.tw * kb.bk * 2) >> 4);
            k.w_bytes16 = (uint16_t)((kb.bk * 2 * std::min(n.d.c, 128)) >> 4);
            k.x_off16 = (uint16_t)((kb.x_shift * kb.bk * 2) >> 4);
            if (kb.stem) {
                const StemPlan& S = E->stems[kb.stem_index];
                for (int par = 0; par < 2; ++par)
                    (par ? map1 : map0) = act_map(ws + S.buf[par].offset, S.Kp, n.d.w, n.d.h, (size_t)S.Kp * 2,
                                                  (size_t)n.d.w * S.Kp * 2, (size_t)n.d.h * n.d.w * S.Kp * 2, S.Kp, P.tw, rows, P.tb);
                k.c0 = 0;
            } else if (!kb.x_load) {
                map0 = map1 = 0;                         // reuses the box the first tap of this filter column loaded
                k.c0 = (uint16_t)kb.c0;
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
                                                  (size_t)s.d.h * s.d.w * s.d.c * 2, kb.bk, kb.x_width, rows, P.tb);
                }
                qxv = qx; qyv = qy; k.c0 = (uint16_t)kb.c0;
            }
            if (map0 < 0 || map1 < 0) return SR_ERR_CUDA;
            if (map0 > 65535 || map1 > 65535 || qxv < -128 || qxv > 127 || qyv < -128 || qyv > 127) return SR_ERR_UNSUPPORTED;
            k.x_map0 = (uint16_t)map0; k.x_map1 = (uint16_t)map1;
            k.qx = (int8_t)qxv; k.qy = (int8_t)qyv;
            dk.push_back(k);
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
        !up(E->r_kbs, dk.data(), dk.size() * sizeof(TcKBlock)) || !up(E->r_tiles, tiles.data(), tiles.size() * sizeof(TcTile)) ||
        !up(E->r_stems, stems.data(), stems.size() * sizeof(TcStem)))
        return SR_ERR_CUDA;
    E->group_grid.clear();
    for (size_t gi = 0; gi < E->group_tiles.size(); ++gi)
        E->group_grid.push_back((int)std::min<size_t>(E->group_tiles[gi].size(), (size_t)E->sm_count * E->group_ctas_per_sm[gi]));
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
    int k_off = -1, width = he.K;
    for (size_t i = 0; i < t.in_edges.size(); ++i)
        if (t.in_edges[i] == edge) k_off = P.edge_k_off[i];
    if (k_off < 0) return SR_ERR_STATE;
    if (E->stem_of_edge[edge] >= 0) width = E->stems[E->stem_of_edge[edge]].Kp;
    std::vector<uint16_t> h((size_t)t.d.c * width, 0);
    for (int co = 0; co < t.d.c; ++co)
        for (int k = 0; k < he.K; ++k) {
            const __nv_bfloat16 b = __float2bfloat16_rn(w_eff[(size_t)co * he.K + k]);
            std::memcpy(&h[(size_t)co * width + k], &b, 2);
        }
    char* dst = g->ws + P.wcat.offset + (size_t)k_off * 2;
    if (cudaMemcpy2D(dst, (size_t)P.k_total * 2, h.data(), (size_t)width * 2, (size_t)width * 2, t.d.c,
                     cudaMemcpyHostToDevice) != cudaSuccess)
        return SR_ERR_CUDA;
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

int sr_tc_after_state_change(sr_graph* g, cudaStream_t s) { return launch_stage(g, 0, (int)(g->t & 1), s); }

int sr_tc_launch_group(sr_graph* g, int group, int t_off, cudaStream_t s)
{
    TcEngine* E = eng(g);
    if (!E || E->group_tiles[group].empty()) return 0;
    const int n_a = E->group_n_a[group], a_slot = E->group_a_slot[group], n_wu = E->group_n_wu[group];
    const size_t smem = (size_t)n_a * a_slot + (size_t)n_wu * kWUnit + 1024;
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
        reinterpret_cast<const TcKBlock*>(g->ws + E->r_kbs.offset),
        reinterpret_cast<const TcTile*>(g->ws + E->r_tiles.offset) + E->group_tile_offset[group],
        (int)E->group_tiles[group].size(), reinterpret_cast<SrFrameCtl*>(g->ws + g->r_ctl.offset), t_off, g->batch, n_a, a_slot,
        n_wu, E->group_w_slot[group], E->group_ctas_per_sm[group] > 1 ? 256 : 512, (long long)g->opt_wait_ms * 2000000LL);
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
