/*
 * Oracle, numeric half: the frame update of a rolled-out network, written as the
 * paper defines it.  TEST INFRASTRUCTURE ONLY: plain loops, double precision,
 * no blocking, no fusion; nothing in the product path may link or call this.
 *
 * What it computes (paper Sec. A1.2 "Connecting the theory of networks with
 * deep neural networks" together with the frame index that Eq. (2) implies):
 *
 *     x_v^{t+1} = sigma_v( b_v + sum_{e=(u,v) in SRC_v} f_e(theta_e, x_u^{t+1-R(e)}) )
 *
 * for t = 0..T-1 and every non-input node v, nodes visited in increasing
 * tableau level inside a frame (the caller passes that order).  Input nodes
 * are given at all frames 0..T; every other state is zero at frame 0 (Sec. A,
 * "Training details": states of all but the input layers start at zero).
 * R(e) may exceed 1 (Sec. 6: an edge that bridges d > 1 frames stands for a chain of
 * d - 1 copy-nodes); where t + 1 - R(e) < 0 the edge contributes nothing, because
 * the copy-nodes it stands for start at zero like every other non-input node.
 * sigma is ReLU or the identity; b is a channel-wise bias; f_e is
 *   kind 0  a k x k cross-correlation with stride s and symmetric zero padding
 *           (k-1)/2, output size floor((n + 2p - k)/s) + 1; with pool = 2 it is
 *           followed by a 2x2 stride-2 average;
 *   kind 1  a dense map over the source flattened in (h, w, c) order;
 *   kind 2  the mean over h, w followed by a dense map over channels.
 *
 * Layouts: state [B][H][W][C]; conv weight [C_out][k][k][C_in]; dense weight
 * [C_out][H][W][C_in]; mean-dense weight [C_out][C_in].
 *
 * All states of all frames are kept and returned (the explicit rollout window).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct { int32_t h, w, c, act; } sro_node;
typedef struct { int32_t src, tgt, kind, k, stride, pool; } sro_edge;

static double round_bf16(double v)
{
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u) return (double)f;      /* inf / nan unchanged */
    u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* row oy of y_e for one sample, added into acc[h_t][w_t][c_t] (dense targets have the single row 0) */
static void edge_transform(const sro_node* s, const sro_node* t, const sro_edge* e,
                           const double* x, const double* w, double* acc, int oy)
{
    if (e->kind == 0) {
        const int k = e->k, st = e->stride, p = (k - 1) / 2;
        const int ch = (s->h + 2 * p - k) / st + 1;       /* conv output size before pooling */
        const int cw = (s->w + 2 * p - k) / st + 1;
        const int q = (e->pool == 2) ? 2 : 1;
        for (int ox = 0; ox < t->w; ++ox)
        for (int co = 0; co < t->c; ++co) {
            double sum = 0.0;
            for (int dy = 0; dy < q; ++dy)
            for (int dx = 0; dx < q; ++dx) {
                const int cy = oy * q + dy, cx = ox * q + dx;      /* conv output pixel */
                if (cy >= ch || cx >= cw) continue;
                for (int ky = 0; ky < k; ++ky)
                for (int kx = 0; kx < k; ++kx) {
                    const int iy = cy * st + ky - p, ix = cx * st + kx - p;
                    if (iy < 0 || iy >= s->h || ix < 0 || ix >= s->w) continue;
                    const double* xp = x + ((size_t)iy * s->w + ix) * s->c;
                    const double* wp = w + (((size_t)co * k + ky) * k + kx) * s->c;
                    double part = 0.0;
                    #pragma omp simd reduction(+:part)
                    for (int ci = 0; ci < s->c; ++ci) part += wp[ci] * xp[ci];
                    sum += part;
                }
            }
            acc[((size_t)oy * t->w + ox) * t->c + co] += sum / (double)(q * q);
        }
    } else if (e->kind == 1) {
        const size_t n = (size_t)s->h * s->w * s->c;
        for (int co = 0; co < t->c; ++co) {
            const double* wp = w + (size_t)co * n;
            double sum = 0.0;
            #pragma omp simd reduction(+:sum)
            for (size_t i = 0; i < n; ++i) sum += wp[i] * x[i];
            acc[co] += sum;
        }
    } else {
        const int hw = s->h * s->w;
        double* mean = (double*)calloc((size_t)s->c, sizeof(double));
        for (int i = 0; i < hw; ++i)
            for (int ci = 0; ci < s->c; ++ci) mean[ci] += x[(size_t)i * s->c + ci];
        for (int ci = 0; ci < s->c; ++ci) mean[ci] /= (double)hw;
        for (int co = 0; co < t->c; ++co) {
            double sum = 0.0;
            for (int ci = 0; ci < s->c; ++ci) sum += w[(size_t)co * s->c + ci] * mean[ci];
            acc[co] += sum;
        }
        free(mean);
    }
}

/*
 * states[v] : [T+1][B][h][w][c] doubles, caller-allocated.  For input nodes the
 * caller has filled all frames; for the others this routine fills frames 0..T.
 * order[]   : the non-input nodes sorted by increasing tableau level.
 * keep_frame0: 0 = frame 0 of every non-input node is set to zero (a rollout from the start);
 *              1 = frame 0 is taken as the caller filled it: the window continues an earlier one, whose last
 *                  frame becomes this window's frame 0 (Sec. 4, chaining of shallow rollout windows).
 * OpenMP spreads the independent (sample, output row) pairs of one node over the cores.
 * Returns 0, or -1 on a bad argument.
 */
int sro_rollout(int n_nodes, const sro_node* nodes, int n_edges, const sro_edge* edges, const uint8_t* R,
                const int32_t* order, int n_order, int B, int T,
                const double* const* weights, const double* const* bias, double* const* states,
                int round_states_bf16, int keep_frame0)
{
    if (n_nodes <= 0 || n_edges <= 0 || B <= 0 || T < 0) return -1;
    for (int i = 0; i < n_order && !keep_frame0; ++i) {         /* frame 0: zero */
        const sro_node* v = &nodes[order[i]];
        memset(states[order[i]], 0, sizeof(double) * (size_t)B * v->h * v->w * v->c);
    }
    for (int t = 0; t < T; ++t) {
        for (int i = 0; i < n_order; ++i) {
            const int vi = order[i];
            const sro_node* v = &nodes[vi];
            const size_t per = (size_t)v->h * v->w * v->c;
            double* xt1 = states[vi] + (size_t)(t + 1) * B * per;
            const size_t row = (size_t)v->w * v->c;
            #pragma omp parallel for collapse(2) schedule(dynamic, 1)
            for (int b = 0; b < B; ++b)
            for (int oy = 0; oy < v->h; ++oy) {
                double* acc = xt1 + (size_t)b * per;
                for (size_t j = oy * row; j < (oy + 1) * row; ++j) acc[j] = 0.0;
                for (int ei = 0; ei < n_edges; ++ei) {
                    const sro_edge* e = &edges[ei];
                    if (e->tgt != vi) continue;
                    const sro_node* s = &nodes[e->src];
                    const size_t sper = (size_t)s->h * s->w * s->c;
                    const int frame = t + 1 - (int)R[ei];
                    if (frame < 0) continue;                     /* before frame 0: the copy-nodes of a long edge hold zeros */
                    const double* x = states[e->src] + ((size_t)frame * B + b) * sper;
                    edge_transform(s, v, e, x, weights[ei], acc, oy);
                }
                for (size_t j = oy * row; j < (oy + 1) * row; ++j) {
                    double z = acc[j] + bias[vi][j % (size_t)v->c];
                    if (v->act == 1 && z < 0.0) z = 0.0;
                    acc[j] = round_states_bf16 ? round_bf16(z) : z;
                }
            }
        }
    }
    return 0;
}
