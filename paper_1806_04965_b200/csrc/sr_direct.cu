// CUDA-core kernels of the frame update: the node update
//     x_v = sigma(b_v + sum_e f_e(theta_e, x_src(e)))          (paper Sec. A1.2)
// for every node of one launch group, in one launch.  They serve the fp32 mode, the dense heads and
// the few-channel nodes that are bound by memory traffic, and they are the reference engine the
// tensor-core kernel can be switched against.  Accumulation is fp32 in every mode.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "sr_internal.h"
#include "sr_kernels.h"

namespace {

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f(float* p, float v) { *p = v; }
__device__ __forceinline__ void from_f(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ void load4(const float* p, float (&v)[4])
{
    const float4 q = *reinterpret_cast<const float4*>(p);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&v)[4])
{
    const uint2 q = *reinterpret_cast<const uint2*>(p);
    v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xFFFF0000u);
    v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xFFFF0000u);
}

constexpr int kPix = 4;            // pixels per warp (conv nodes)
constexpr int kWarps = 4;          // warps per block
constexpr int kDenseB = 8;         // samples per warp (dense nodes)

// Conv node: a block covers kWarps*kPix consecutive pixels of one sample; lanes run over output
// channels, so weight reads ([K][C_out] rows) and state writes (NHWC) are coalesced and the input
// reads are warp-uniform broadcasts.
template <typename T>
__device__ void conv_item(const SrDevNode& nd, const SrDevEdge* edges, const SrDirectItem& it, int prev, int cur,
                          float* out_f32)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int HW = nd.H * nd.W;
    const int pbase = it.p0 + warp * kPix;
    int oy[kPix], ox[kPix];
    bool pv[kPix];
#pragma unroll
    for (int j = 0; j < kPix; ++j) {
        const int p = pbase + j;
        pv[j] = p < HW;
        oy[j] = pv[j] ? p / nd.W : 0;
        ox[j] = pv[j] ? p % nd.W : 0;
    }
    T* dst = static_cast<T*>(nd.state[cur]) + (size_t)it.b0 * HW * nd.C;
    for (int co0 = 0; co0 < nd.C; co0 += 32) {
        const int co = co0 + lane;
        const bool cv = co < nd.C;
        float acc[kPix];
#pragma unroll
        for (int j = 0; j < kPix; ++j) acc[j] = 0.f;
        for (int ei = 0; ei < nd.n_edges; ++ei) {
            const SrDevEdge& e = edges[nd.first_edge + ei];
            const T* src = static_cast<const T*>(e.src[e.R ? prev : cur]) + (size_t)it.b0 * e.Hs * e.Ws * e.Cs;
            const bool vec = (e.Cs & 3) == 0;
            for (int ky = 0; ky < e.k; ++ky)
                for (int kx = 0; kx < e.k; ++kx) {
                    const T* xp[kPix];
                    bool ok[kPix];
                    bool any = false;
#pragma unroll
                    for (int j = 0; j < kPix; ++j) {
                        const int iy = oy[j] * e.stride + ky - e.pad, ix = ox[j] * e.stride + kx - e.pad;
                        ok[j] = pv[j] && iy >= 0 && iy < e.Hs && ix >= 0 && ix < e.Ws;
                        xp[j] = src + ((size_t)(ok[j] ? iy : 0) * e.Ws + (ok[j] ? ix : 0)) * e.Cs;
                        any |= ok[j];
                    }
                    if (!any) continue;
                    const float* wp = e.w + (size_t)(ky * e.k + kx) * e.Cs * nd.C + co;
                    if (vec) {
                        for (int ci = 0; ci < e.Cs; ci += 4) {
                            float w[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) w[q] = cv ? wp[(size_t)(ci + q) * nd.C] : 0.f;
#pragma unroll
                            for (int j = 0; j < kPix; ++j) {
                                if (!ok[j]) continue;
                                float x[4];
                                load4(xp[j] + ci, x);
#pragma unroll
                                for (int q = 0; q < 4; ++q) acc[j] = fmaf(w[q], x[q], acc[j]);
                            }
                        }
                    } else {
                        for (int ci = 0; ci < e.Cs; ++ci) {
                            const float w = cv ? wp[(size_t)ci * nd.C] : 0.f;
#pragma unroll
                            for (int j = 0; j < kPix; ++j)
                                if (ok[j]) acc[j] = fmaf(w, to_f(xp[j][ci]), acc[j]);
                        }
                    }
                }
        }
        if (cv) {
            const float b = nd.bias[co];
#pragma unroll
            for (int j = 0; j < kPix; ++j) {
                if (!pv[j]) continue;
                float z = acc[j] + b;
                if (nd.act == 1) z = fmaxf(z, 0.f);
                from_f(dst + (size_t)(pbase + j) * nd.C + co, z);
                if (out_f32) out_f32[((size_t)it.b0 * HW + pbase + j) * nd.C + co] = z;
            }
        }
    }
}

// Dense node: one warp per output channel and chunk of kDenseB samples; lanes stride over the
// reduction index (coalesced weight and state reads), partial sums meet in a shuffle reduction.
// A mean-dense edge is the dense edge whose weight index is k mod C_in, scaled by 1/(H*W).
template <typename T>
__device__ void dense_item(const SrDevNode& nd, const SrDevEdge* edges, const SrDirectItem& it, int prev, int cur,
                           int B, float* out_f32)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int co = it.p0 + warp;
    if (co >= nd.C) return;
    const int nb = min(kDenseB, B - it.b0);
    float acc[kDenseB];
#pragma unroll
    for (int j = 0; j < kDenseB; ++j) acc[j] = 0.f;
    for (int ei = 0; ei < nd.n_edges; ++ei) {
        const SrDevEdge& e = edges[nd.first_edge + ei];
        const int Kx = e.Hs * e.Ws * e.Cs;                      // elements of one source sample
        const T* src = static_cast<const T*>(e.src[e.R ? prev : cur]) + (size_t)it.b0 * Kx;
        const float* wrow = e.w + (size_t)co * e.K;
        const float scale = (e.kind == SR_EDGE_MEAN_DENSE) ? 1.f / (float)(e.Hs * e.Ws) : 1.f;
        float part[kDenseB];
#pragma unroll
        for (int j = 0; j < kDenseB; ++j) part[j] = 0.f;
        for (int k = lane; k < Kx; k += 32) {
            const float w = wrow[(e.kind == SR_EDGE_MEAN_DENSE) ? (k % e.Cs) : k];
#pragma unroll
            for (int j = 0; j < kDenseB; ++j)
                if (j < nb) part[j] = fmaf(w, to_f(src[(size_t)j * Kx + k]), part[j]);
        }
#pragma unroll
        for (int j = 0; j < kDenseB; ++j) acc[j] += part[j] * scale;
    }
#pragma unroll
    for (int j = 0; j < kDenseB; ++j) {
        float v = acc[j];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        acc[j] = v;
    }
    if (lane == 0) {
        T* dst = static_cast<T*>(nd.state[cur]);
        const float b = nd.bias[co];
        for (int j = 0; j < nb; ++j) {
            float z = acc[j] + b;
            if (nd.act == 1) z = fmaxf(z, 0.f);
            from_f(dst + (size_t)(it.b0 + j) * nd.C + co, z);
            if (out_f32) out_f32[(size_t)(it.b0 + j) * nd.C + co] = z;
        }
    }
}


constexpr int kHeadCo = 16;        // outputs per block (dense nodes, one sample per block)
constexpr int kHeadMaxC = 1024;    // channels the mean buffer holds

// Dense node, one sample and kHeadCo outputs per block.  Every thread keeps a partial sum for each of
// the block's outputs over its own slice of the reduction index, so the weight loads of all outputs
// are independent and in flight together (the kernel is bound by load latency, not by arithmetic);
// a shuffle reduction and one pass through shared memory combine the slices.  A mean-dense edge first
// reduces the source over its pixels into shared memory (threads run over channels: coalesced NHWC
// reads).  Source and weight rows are read with 16-byte loads where the length allows it.
template <typename T>
__device__ void head_item(const SrDevNode& nd, const SrDevEdge* edges, const SrDirectItem& it, int prev, int cur,
                          float* out_f32)
{
    __shared__ float mean[kHeadMaxC];
    __shared__ float part[4 * kWarps * 32];
    __shared__ float red[kWarps][kHeadCo];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
    const int b = it.b0, co0 = it.p0;
    const int nco = min(it.pad_ >> 8, nd.C - co0);      // outputs of this block (at most kHeadCo)
    float acc[kHeadCo];
#pragma unroll
    for (int o = 0; o < kHeadCo; ++o) acc[o] = 0.f;
    for (int ei = 0; ei < nd.n_edges; ++ei) {
        const SrDevEdge& e = edges[nd.first_edge + ei];
        const int HW = e.Hs * e.Ws, Kx = HW * e.Cs;
        const T* src = static_cast<const T*>(e.src[e.R ? prev : cur]) + (size_t)b * Kx;
        const float* w0 = e.w + (size_t)co0 * e.K;
        if (e.kind == SR_EDGE_MEAN_DENSE) {
            // the sums run in a fixed order (no atomics), so a frame update is bit-reproducible
            __syncthreads();
            if ((e.Cs & 3) == 0 && e.Cs / 4 <= (int)blockDim.x) {
                // groups of Cs/4 threads share the pixels; a group's partial sums take one row of part[][Cs]
                // (groups * Cs <= 4 * blockDim.x floats), the rows are then added in group order
                const int vc = e.Cs / 4, groups = blockDim.x / vc;
                const int col = tid % vc, grp = tid / vc;
                if (grp < groups) {
                    float s4[4] = {0.f, 0.f, 0.f, 0.f};
                    for (int p = grp; p < HW; p += groups) {
                        float x[4];
                        load4(src + (size_t)p * e.Cs + 4 * col, x);
#pragma unroll
                        for (int q = 0; q < 4; ++q) s4[q] += x[q];
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) part[grp * e.Cs + 4 * col + q] = s4[q];
                }
                __syncthreads();
                for (int c = tid; c < e.Cs; c += blockDim.x) {
                    float m = 0.f;
                    for (int gq = 0; gq < groups; ++gq) m += part[gq * e.Cs + c];
                    mean[c] = m;
                }
            } else {
                for (int c = tid; c < e.Cs; c += blockDim.x) {
                    float m = 0.f;
                    for (int p = 0; p < HW; ++p) m += to_f(src[(size_t)p * e.Cs + c]);
                    mean[c] = m;
                }
            }
            __syncthreads();
            const float inv = 1.f / (float)HW;
            for (int c = tid; c < e.Cs; c += blockDim.x) {
                const float m = mean[c] * inv;
#pragma unroll
                for (int o = 0; o < kHeadCo; ++o)
                    if (o < nco) acc[o] = fmaf(w0[(size_t)o * e.K + c], m, acc[o]);
            }
        } else if ((Kx & 3) == 0) {
            // all blocks of a launch walk the same weight rows: every block starts at another step (its sample index),
            // so that they do not all ask the same L2 lines at the same moment
            const int stride = 4 * (int)blockDim.x, steps = (Kx + stride - 1) / stride;
            for (int s = 0; s < steps; ++s) {
                const int k = 4 * tid + ((s + b) % steps) * stride;
                if (k >= Kx) continue;
                float x[4];
                load4(src + k, x);
#pragma unroll
                for (int o = 0; o < kHeadCo; ++o) {
                    if (o < nco) {
                        const float4 w = *reinterpret_cast<const float4*>(w0 + (size_t)o * e.K + k);
                        acc[o] = fmaf(w.x, x[0], acc[o]); acc[o] = fmaf(w.y, x[1], acc[o]);
                        acc[o] = fmaf(w.z, x[2], acc[o]); acc[o] = fmaf(w.w, x[3], acc[o]);
                    }
                }
            }
        } else {
            for (int k = tid; k < Kx; k += blockDim.x) {
                const float x = to_f(src[k]);
#pragma unroll
                for (int o = 0; o < kHeadCo; ++o)
                    if (o < nco) acc[o] = fmaf(w0[(size_t)o * e.K + k], x, acc[o]);
            }
        }
    }
#pragma unroll
    for (int o = 0; o < kHeadCo; ++o) {
        float v = acc[o];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
        if (lane == 0) red[warp][o] = v;
    }
    __syncthreads();
    if (tid < nco) {
        float z = nd.bias[co0 + tid];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) z += red[w][tid];
        if (nd.act == 1) z = fmaxf(z, 0.f);
        from_f(static_cast<T*>(nd.state[cur]) + (size_t)b * nd.C + co0 + tid, z);
        if (out_f32) out_f32[(size_t)b * nd.C + co0 + tid] = z;
    }
}

template <typename T>
__global__ void __launch_bounds__(kWarps * 32)
sr_direct_group_kernel(const SrDevNode* __restrict__ nodes, const SrDevEdge* __restrict__ edges,
                       const SrDirectItem* __restrict__ items, const SrFrameCtl* __restrict__ ctl, int t_off, int B)
{
    const SrDirectItem it = items[blockIdx.x];
    const SrDevNode& nd = nodes[it.node];
    const long long t = ctl->t + t_off;                   // this launch computes frame t+1 from frame t
    const int prev = (int)(t & 1), cur = prev ^ 1;
    float* out = nullptr;
    if (nd.is_output && ctl->out_base) out = ctl->out_base + (ctl->run_t + t_off) * ctl->out_stride;
    if (nd.H == 1 && nd.W == 1 && edges[nd.first_edge].kind != SR_EDGE_CONV) {
        if ((it.pad_ & 0xFF) == 1) head_item<T>(nd, edges, it, prev, cur, out);
        else dense_item<T>(nd, edges, it, prev, cur, B, out);
    }
    else
        conv_item<T>(nd, edges, it, prev, cur, out);
}

// Frame input: the input nodes' frame-(t+1) state is the caller's frame.
__global__ void sr_input_kernel(const SrDevNode* __restrict__ nodes, const int* __restrict__ input_nodes, int n_inputs,
                                const SrFrameCtl* __restrict__ ctl, int t_off, size_t elem_bytes, int B)
{
    const long long t = ctl->t + t_off;
    const int cur = (int)((t + 1) & 1);
    for (int i = 0; i < n_inputs; ++i) {
        const SrDevNode& nd = nodes[input_nodes[i]];
        const size_t bytes = (size_t)B * nd.H * nd.W * nd.C * elem_bytes;
        const char* src = static_cast<const char*>(ctl->in_base[i]) + (ctl->run_t + t_off) * ctl->in_stride_bytes[i];
        char* dst = static_cast<char*>(nd.state[cur]);
        const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x, nth = (size_t)gridDim.x * blockDim.x;
        if (((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) == 0) {
            const size_t nv = bytes / 16;
            for (size_t j = tid; j < nv; j += nth)
                reinterpret_cast<uint4*>(dst)[j] = reinterpret_cast<const uint4*>(src)[j];
            for (size_t j = nv * 16 + tid; j < bytes; j += nth) dst[j] = src[j];
        } else {
            for (size_t j = tid; j < bytes; j += nth) dst[j] = src[j];
        }
    }
}

__global__ void sr_set_ctl_kernel(SrFrameCtl* ctl, SrFrameCtl v)
{
    const int err = ctl->error;
    *ctl = v;
    ctl->error = err;
}

__global__ void sr_advance_kernel(SrFrameCtl* ctl, int n)
{
    ctl->t += n;
    ctl->run_t += n;
}

}  // namespace

void sr_launch_direct_group(const sr_graph* g, int group, int t_off, cudaStream_t s)
{
    const int n = g->group_item_count[group];
    if (n == 0) return;
    const SrDevNode* nodes = reinterpret_cast<const SrDevNode*>(g->ws + g->r_nodes.offset);
    const SrDevEdge* edges = reinterpret_cast<const SrDevEdge*>(g->ws + g->r_edges.offset);
    const SrDirectItem* items = reinterpret_cast<const SrDirectItem*>(g->ws + g->r_items.offset) + g->group_item_offset[group];
    const SrFrameCtl* ctl = reinterpret_cast<const SrFrameCtl*>(g->ws + g->r_ctl.offset);
    if (g->dtype == SR_DTYPE_BF16)
        sr_direct_group_kernel<__nv_bfloat16><<<n, kWarps * 32, 0, s>>>(nodes, edges, items, ctl, t_off, g->batch);
    else
        sr_direct_group_kernel<float><<<n, kWarps * 32, 0, s>>>(nodes, edges, items, ctl, t_off, g->batch);
}

void sr_launch_input(const sr_graph* g, const int* input_nodes_dev, int t_off, cudaStream_t s)
{
    const SrDevNode* nodes = reinterpret_cast<const SrDevNode*>(g->ws + g->r_nodes.offset);
    const SrFrameCtl* ctl = reinterpret_cast<const SrFrameCtl*>(g->ws + g->r_ctl.offset);
    size_t most = 0;
    for (int v : g->input_nodes) {
        const sr_node_desc& d = g->nodes[v].d;
        most = std::max(most, (size_t)g->batch * d.h * d.w * d.c * g->elem);
    }
    int blocks = (int)std::min<size_t>(296, (most / 16 + 255) / 256 + 1);
    sr_input_kernel<<<blocks, 256, 0, s>>>(nodes, input_nodes_dev, (int)g->input_nodes.size(), ctl, t_off,
                                           (size_t)g->elem, g->batch);
}

void sr_launch_set_ctl(const sr_graph* g, const SrFrameCtl& v, cudaStream_t s)
{
    sr_set_ctl_kernel<<<1, 1, 0, s>>>(reinterpret_cast<SrFrameCtl*>(g->ws + g->r_ctl.offset), v);
}

void sr_launch_advance(const sr_graph* g, int n, cudaStream_t s)
{
    sr_advance_kernel<<<1, 1, 0, s>>>(reinterpret_cast<SrFrameCtl*>(g->ws + g->r_ctl.offset), n);
}

int sr_direct_conv_pixels_per_block() { return kWarps * kPix; }
int sr_direct_dense_outputs_per_block() { return kWarps; }
int sr_direct_dense_samples_per_block() { return kDenseB; }
int sr_direct_head_outputs_per_block() { return kHeadCo; }
int sr_direct_head_max_channels() { return kHeadMaxC; }
