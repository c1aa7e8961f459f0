// TDES training objective, forward and backward in one kernel (Sec. 3.2 "Training", Eq. 7-12).
//
//   f(p,c,d)    = s (P[p] + u_d) . (C[c] + u_d) / sqrt(m)                                       (Eq. 6)
//   L_KL        = mean over groups of KL(softmax_c z_tgt || softmax_c (log q_d(c) + f(p,c,d)))   (Eq. 7-9)
//   L_pair      = mean over pairs of softplus(gamma - f(v+) + f(v-))                             (Eq. 10)
//   L_BCE       = mean over edges of w1 y softplus(-f) + (1 - y) softplus(f)                     (Eq. 11)
//   L           = lambda_KL L_KL + lambda_pair L_pair + lambda_BCE L_BCE                         (Eq. 12)
// and the gradient of L with respect to the table rows P[p], C[c], the depth embeddings u_d and the scale s.
//
// The work is a gather of table rows (m floats each) and a scatter-add of as many gradient rows: bound by memory
// and atomic traffic, not by arithmetic, so there is no tensor-core path here.  One warp per item (a group of K
// children, a pair, an edge): a lane holds four consecutive floats of every 128-float chunk of a row, dot products
// are warp reductions, gradient rows go out as 16-byte vector atomics (`red.global.add.v4.f32`), the few u rows are
// accumulated in shared memory per CTA and flushed once, losses and the scale's gradient are reduced per CTA.
// Token frequencies are heavy-tailed, and atomic additions to one row serialise in L2: every warp therefore keeps
// four gradient rows per table in shared memory (m <= 128), replaced by frequency (a hit raises a slot's credit, a
// miss lowers the lowest one and takes the slot over when it reaches zero), so the few hottest tokens' rows reach
// global memory once per warp instead of once per item.
// The order of the atomic additions is not fixed, so the gradients are reproducible only up to fp32 rounding.
#include <cuda_runtime.h>
#include <math.h>

#include "common.cuh"
#include "internal.h"

namespace graft {
namespace {

constexpr int kTrThreads = 256;
constexpr int kTrWarps = kTrThreads / 32;
constexpr int kTrMaxChunks = 4;  // m <= 512

struct TrainParams {
    const float* P;
    const float* C;
    const float* u;
    float k0;  // s / sqrt(m)
    float inv_sqrt_m;
    int V, L, m, K;
    int n_groups;
    const int32_t* g_parent;
    const int32_t* g_depth;
    const int32_t* g_child;
    const float* g_logq;
    const float* g_ztgt;
    int n_pairs;
    const int32_t* pairs;
    int n_edges;
    const int32_t* edges;
    float gamma, w1;
    float w_kl, w_pair, w_bce;      // lambda / number of items
    float lam_kl, lam_pair, lam_bce;
    double* loss;      // [4], zero at launch
    int32_t* skipped;  // [1] or NULL, zero at launch
    float* gP;
    float* gC;
    float* gu;
    float* gs;
};

template <int NCH>
struct Row {
    float4 v[NCH];
};

// row[tok] + u_d, four floats per lane per chunk (zeros past m)
template <int NCH>
__device__ __forceinline__ Row<NCH> load_row_plus_u(const float* table, const float* urow, int tok, int m, int lane) {
    Row<NCH> r;
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
        const int k4 = ch * 32 + lane;
        r.v[ch] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (k4 < m / 4) {
            const float4 t = __ldg((const float4*)(table + (size_t)tok * m) + k4);
            const float4 uu = __ldg((const float4*)urow + k4);
            r.v[ch] = make_float4(t.x + uu.x, t.y + uu.y, t.z + uu.z, t.w + uu.w);
        }
    }
    return r;
}
template <int NCH>
__device__ __forceinline__ float warp_dot(const Row<NCH>& a, const Row<NCH>& b) {
    float acc = 0.f;
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
        acc = fmaf(a.v[ch].x, b.v[ch].x, acc);
        acc = fmaf(a.v[ch].y, b.v[ch].y, acc);
        acc = fmaf(a.v[ch].z, b.v[ch].z, acc);
        acc = fmaf(a.v[ch].w, b.v[ch].w, acc);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, d);
    return acc;
}
// dst_row += coef * r  (global memory, vector atomics)
template <int NCH>
__device__ __forceinline__ void add_row_global(float* dst, int tok, int m, int lane, float coef, const Row<NCH>& r) {
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
        const int k4 = ch * 32 + lane;
        if (k4 < m / 4)
            atomicAdd((float4*)(dst + (size_t)tok * m) + k4,
                      make_float4(coef * r.v[ch].x, coef * r.v[ch].y, coef * r.v[ch].z, coef * r.v[ch].w));
    }
}
// A warp's four cached gradient rows of one table (m <= 128: one float4 per lane per row).
constexpr int kTrSlots = 4;
constexpr int kTrCreditMax = 64;
struct WarpCache {
    float* rows;  // [2][kTrSlots][128]
    int* tags;    // [2][kTrSlots] token id or -1
    int* credit;  // [2][kTrSlots]
};
// gradient row of token `tok` of table t (0: gP, 1: gC) += coef * r
// INSTALL = false: a token that is not cached goes straight to global memory without touching the slots' credits
// (the K children of a group: one hot token among them would otherwise be chased out by the other K - 1)
template <int NCH, bool INSTALL = true>
__device__ __forceinline__ void add_row(const TrainParams& p, const WarpCache& wc, int t, int tok, int lane, float coef,
                                        const Row<NCH>& r) {
    float* dst = t == 0 ? p.gP : p.gC;
    if (NCH != 1) {
        add_row_global<NCH>(dst, tok, p.m, lane, coef, r);
        return;
    }
    const int4 tg = *(const int4*)(wc.tags + kTrSlots * t);
    const int slot = tg.x == tok ? 0 : tg.y == tok ? 1 : tg.z == tok ? 2 : tg.w == tok ? 3 : -1;
    const float4 add = make_float4(coef * r.v[0].x, coef * r.v[0].y, coef * r.v[0].z, coef * r.v[0].w);
    if (slot >= 0) {  // hit
        float4* q = (float4*)(wc.rows + (size_t)(t * kTrSlots + slot) * 128) + lane;
        float4 v = *q;
        v.x += add.x;
        v.y += add.y;
        v.z += add.z;
        v.w += add.w;
        *q = v;
        if (lane == 0) {
            const int c = wc.credit[t * kTrSlots + slot];
            if (c < kTrCreditMax) wc.credit[t * kTrSlots + slot] = c + 1;
        }
        __syncwarp();
        return;
    }
    if (!INSTALL) {
        if (lane < p.m / 4) atomicAdd((float4*)(dst + (size_t)tok * p.m) + lane, add);
        return;
    }
    const int4 cr = *(const int4*)(wc.credit + kTrSlots * t);
    int victim = 0, cmin = cr.x;
    if (cr.y < cmin) victim = 1, cmin = cr.y;
    if (cr.z < cmin) victim = 2, cmin = cr.z;
    if (cr.w < cmin) victim = 3, cmin = cr.w;
    if (cmin > 0) {  // the slot keeps its row for now; this addition goes to global memory
        if (lane == 0) wc.credit[t * kTrSlots + victim] = cmin - 1;
        __syncwarp();
        if (lane < p.m / 4) atomicAdd((float4*)(dst + (size_t)tok * p.m) + lane, add);
        return;
    }
    // take the slot over: its row goes to global memory, the new token's starts with this addition
    const int old = wc.tags[t * kTrSlots + victim];
    float4* q = (float4*)(wc.rows + (size_t)(t * kTrSlots + victim) * 128) + lane;
    if (old >= 0 && lane < p.m / 4) atomicAdd((float4*)(dst + (size_t)old * p.m) + lane, *q);
    *q = add;
    __syncwarp();
    if (lane == 0) {
        wc.tags[t * kTrSlots + victim] = tok;
        wc.credit[t * kTrSlots + victim] = 1;
    }
    __syncwarp();
}
__device__ __forceinline__ void cache_flush(const TrainParams& p, const WarpCache& wc, int lane) {
    for (int t = 0; t < 2; ++t)
        for (int sl = 0; sl < kTrSlots; ++sl) {
            const int tok = wc.tags[t * kTrSlots + sl];
            if (tok >= 0 && lane < p.m / 4)
                atomicAdd((float4*)((t == 0 ? p.gP : p.gC) + (size_t)tok * p.m) + lane,
                          *((const float4*)(wc.rows + (size_t)(t * kTrSlots + sl) * 128) + lane));
        }
}
// the CTA's copy of gu: row d-1 += coef * (a + b)
template <int NCH>
__device__ __forceinline__ void add_u_shared(float* su, int d, int m, int lane, float coef, const Row<NCH>& a,
                                             const Row<NCH>& b) {
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
        const int k4 = ch * 32 + lane;
        if (k4 < m / 4) {
            float* q = su + (size_t)(d - 1) * m + 4 * k4;
            atomicAdd(q + 0, coef * (a.v[ch].x + b.v[ch].x));
            atomicAdd(q + 1, coef * (a.v[ch].y + b.v[ch].y));
            atomicAdd(q + 2, coef * (a.v[ch].z + b.v[ch].z));
            atomicAdd(q + 3, coef * (a.v[ch].w + b.v[ch].w));
        }
    }
}
__device__ __forceinline__ float softplus_f(float x) { return x > 0.f ? x + log1pf(expf(-x)) : log1pf(expf(x)); }
__device__ __forceinline__ float sigmoid_f(float x) {
    return x >= 0.f ? 1.f / (1.f + expf(-x)) : expf(x) / (1.f + expf(x));
}
__device__ __forceinline__ bool tok_ok(int t, int V) { return t >= 0 && t < V; }

// one edge (p, c, d): returns f; the rows stay in a and b for the backward step
template <int NCH>
__device__ __forceinline__ float edge_forward(const TrainParams& p, int tp, int tc, int d, int lane, Row<NCH>& a,
                                              Row<NCH>& b, float& dot) {
    const float* urow = p.u + (size_t)(d - 1) * p.m;
    a = load_row_plus_u<NCH>(p.P, urow, tp, p.m, lane);
    b = load_row_plus_u<NCH>(p.C, urow, tc, p.m, lane);
    dot = warp_dot<NCH>(a, b);
    return p.k0 * dot;
}
template <int NCH>
__device__ __forceinline__ void edge_backward(const TrainParams& p, const WarpCache& wc, float* su, int tp, int tc,
                                              int d, int lane, float gf, const Row<NCH>& a, const Row<NCH>& b,
                                              float dot, float& gs) {
    const float coef = gf * p.k0;
    add_row<NCH>(p, wc, 0, tp, lane, coef, b);
    add_row<NCH>(p, wc, 1, tc, lane, coef, a);
    add_u_shared<NCH>(su, d, p.m, lane, coef, a, b);
    gs += gf * dot * p.inv_sqrt_m;
}

template <int NCH>
__global__ void __launch_bounds__(kTrThreads) tdes_loss_kernel(const TrainParams p) {
    extern __shared__ __align__(16) float su[];  // [L][m] this CTA's share of gu
    __shared__ double s_loss[3];
    __shared__ float s_gs;
    __shared__ int s_skip;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool grad = p.gP != nullptr;
    WarpCache wc;  // behind su (NCH == 1 only): rows, then tags and credits, per warp
    {
        float* base = su + ((p.L * p.m + 3) & ~3);
        wc.rows = base + (size_t)warp * 2 * kTrSlots * 128;
        wc.tags = (int*)(base + (size_t)kTrWarps * 2 * kTrSlots * 128) + warp * 4 * kTrSlots;
        wc.credit = wc.tags + 2 * kTrSlots;
        if (NCH == 1 && lane < 2 * kTrSlots) {
            wc.tags[lane] = -1;
            wc.credit[lane] = 0;
        }
    }
    for (int i = threadIdx.x; i < p.L * p.m; i += kTrThreads) su[i] = 0.f;
    if (threadIdx.x < 3) s_loss[threadIdx.x] = 0.0;
    if (threadIdx.x == 0) {
        s_gs = 0.f;
        s_skip = 0;
    }
    __syncthreads();
    const int wid = blockIdx.x * kTrWarps + warp, nw = gridDim.x * kTrWarps;
    double l_kl = 0.0, l_pair = 0.0, l_bce = 0.0;  // this warp's sums (every lane holds the same value)
    float gs = 0.f;
    int skipped = 0;

    // ---- distribution level (Eq. 7-9): lane c owns child c
    for (int g = wid; g < p.n_groups; g += nw) {
        const int tp = p.g_parent[g], d = p.g_depth[g];
        const int tc = lane < p.K ? p.g_child[(size_t)g * p.K + lane] : 0;
        const bool ok = tok_ok(tp, p.V) && d >= 1 && d <= p.L && __all_sync(0xFFFFFFFFu, tok_ok(tc, p.V));
        if (!ok) {
            ++skipped;
            continue;
        }
        const float* urow = p.u + (size_t)(d - 1) * p.m;
        const Row<NCH> a = load_row_plus_u<NCH>(p.P, urow, tp, p.m, lane);
        float dot_c = 0.f;
#pragma unroll 4
        for (int c = 0; c < p.K; ++c) {
            const int t = __shfl_sync(0xFFFFFFFFu, tc, c);
            const Row<NCH> b = load_row_plus_u<NCH>(p.C, urow, t, p.m, lane);
            const float dt = warp_dot<NCH>(a, b);
            if (lane == c) dot_c = dt;
        }
        const float f_c = p.k0 * dot_c;
        const float z = lane < p.K ? p.g_ztgt[(size_t)g * p.K + lane] : -INFINITY;
        const float al = lane < p.K ? p.g_logq[(size_t)g * p.K + lane] + f_c : -INFINITY;
        float zmax = z, amax = al;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            zmax = fmaxf(zmax, __shfl_xor_sync(0xFFFFFFFFu, zmax, o));
            amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
        }
        float ez = lane < p.K ? expf(z - zmax) : 0.f, ea = lane < p.K ? expf(al - amax) : 0.f;
        float zsum = ez, asum = ea;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            zsum += __shfl_xor_sync(0xFFFFFFFFu, zsum, o);
            asum += __shfl_xor_sync(0xFFFFFFFFu, asum, o);
        }
        const float pt = ez / zsum, ph = ea / asum;
        float kl = 0.f;
        if (lane < p.K && pt > 0.f) kl = pt * ((z - zmax - logf(zsum)) - (al - amax - logf(asum)));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) kl += __shfl_xor_sync(0xFFFFFFFFu, kl, o);
        l_kl += (double)kl;
        if (grad) {
            const float gf_c = lane < p.K ? p.w_kl * (ph - pt) : 0.f;  // d L / d f_c
            Row<NCH> accP, accU;
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) accP.v[ch] = accU.v[ch] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
            for (int c = 0; c < p.K; ++c) {
                const int t = __shfl_sync(0xFFFFFFFFu, tc, c);
                const float coef = __shfl_sync(0xFFFFFFFFu, gf_c, c) * p.k0;
                const Row<NCH> b = load_row_plus_u<NCH>(p.C, urow, t, p.m, lane);
                add_row<NCH, false>(p, wc, 1, t, lane, coef, a);
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch) {
                    accP.v[ch].x = fmaf(coef, b.v[ch].x, accP.v[ch].x);
                    accP.v[ch].y = fmaf(coef, b.v[ch].y, accP.v[ch].y);
                    accP.v[ch].z = fmaf(coef, b.v[ch].z, accP.v[ch].z);
                    accP.v[ch].w = fmaf(coef, b.v[ch].w, accP.v[ch].w);
                    accU.v[ch].x = fmaf(coef, a.v[ch].x + b.v[ch].x, accU.v[ch].x);
                    accU.v[ch].y = fmaf(coef, a.v[ch].y + b.v[ch].y, accU.v[ch].y);
                    accU.v[ch].z = fmaf(coef, a.v[ch].z + b.v[ch].z, accU.v[ch].z);
                    accU.v[ch].w = fmaf(coef, a.v[ch].w + b.v[ch].w, accU.v[ch].w);
                }
            }
            add_row<NCH>(p, wc, 0, tp, lane, 1.f, accP);
            Row<NCH> zero;
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) zero.v[ch] = make_float4(0.f, 0.f, 0.f, 0.f);
            add_u_shared<NCH>(su, d, p.m, lane, 1.f, accU, zero);
            float gsc = gf_c * dot_c * p.inv_sqrt_m;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) gsc += __shfl_xor_sync(0xFFFFFFFFu, gsc, o);
            gs += gsc;
        }
    }
    // ---- pairwise level (Eq. 10)
    for (int i = wid; i < p.n_pairs; i += nw) {
        const int32_t* q = p.pairs + (size_t)i * 6;
        const int p1 = q[0], c1 = q[1], d1 = q[2], p2 = q[3], c2 = q[4], d2 = q[5];
        if (!(tok_ok(p1, p.V) && tok_ok(c1, p.V) && tok_ok(p2, p.V) && tok_ok(c2, p.V) && d1 >= 1 && d1 <= p.L &&
              d2 >= 1 && d2 <= p.L)) {
            ++skipped;
            continue;
        }
        Row<NCH> a1, b1, a2, b2;
        float dot1, dot2;
        const float f1 = edge_forward<NCH>(p, p1, c1, d1, lane, a1, b1, dot1);
        const float f2 = edge_forward<NCH>(p, p2, c2, d2, lane, a2, b2, dot2);
        const float x = p.gamma - f1 + f2;
        l_pair += (double)softplus_f(x);
        if (grad) {
            const float gx = p.w_pair * sigmoid_f(x);
            edge_backward<NCH>(p, wc, su, p1, c1, d1, lane, -gx, a1, b1, dot1, gs);
            edge_backward<NCH>(p, wc, su, p2, c2, d2, lane, gx, a2, b2, dot2, gs);
        }
    }
    // ---- edge level (Eq. 11)
    for (int i = wid; i < p.n_edges; i += nw) {
        const int32_t* e = p.edges + (size_t)i * 4;
        const int tp = e[0], tc = e[1], d = e[2];
        const float y = e[3] ? 1.f : 0.f;
        if (!(tok_ok(tp, p.V) && tok_ok(tc, p.V) && d >= 1 && d <= p.L)) {
            ++skipped;
            continue;
        }
        Row<NCH> a, b;
        float dot;
        const float f = edge_forward<NCH>(p, tp, tc, d, lane, a, b, dot);
        l_bce += (double)(p.w1 * y * softplus_f(-f) + (1.f - y) * softplus_f(f));
        if (grad) {
            const float gf = p.w_bce * (-p.w1 * y * sigmoid_f(-f) + (1.f - y) * sigmoid_f(f));
            edge_backward<NCH>(p, wc, su, tp, tc, d, lane, gf, a, b, dot, gs);
        }
    }
    if (NCH == 1 && grad) cache_flush(p, wc, lane);
    // ---- per-CTA reduction, then one round of global atomics
    if (lane == 0) {
        atomicAdd(&s_loss[0], l_kl);
        atomicAdd(&s_loss[1], l_pair);
        atomicAdd(&s_loss[2], l_bce);
        atomicAdd(&s_gs, gs);
        if (skipped) atomicAdd(&s_skip, skipped);
    }
    __syncthreads();
    if (grad)
        for (int i = threadIdx.x; i < p.L * p.m; i += kTrThreads)
            if (su[i] != 0.f) atomicAdd(p.gu + i, su[i]);
    if (threadIdx.x == 0) {
        const double kl = s_loss[0] / (double)(p.n_groups > 0 ? p.n_groups : 1);
        const double pr = s_loss[1] / (double)(p.n_pairs > 0 ? p.n_pairs : 1);
        const double bc = s_loss[2] / (double)(p.n_edges > 0 ? p.n_edges : 1);
        atomicAdd(p.loss + 0, kl);
        atomicAdd(p.loss + 1, pr);
        atomicAdd(p.loss + 2, bc);
        atomicAdd(p.loss + 3, (double)p.lam_kl * kl + (double)p.lam_pair * pr + (double)p.lam_bce * bc);
        if (grad && s_gs != 0.f) atomicAdd(p.gs, s_gs);
        if (p.skipped && s_skip) atomicAdd(p.skipped, s_skip);
    }
}

}  // namespace

static size_t tdes_loss_smem(const graft_config& cfg) {
    size_t b = (size_t)((cfg.L * cfg.m + 3) & ~3) * sizeof(float);  // gu
    if (cfg.m <= 128) b += (size_t)kTrWarps * (2 * kTrSlots * 128 * sizeof(float) + 4 * kTrSlots * sizeof(int));
    return b;
}

cudaError_t tdes_loss_launch(graft_ctx* ctx, const graft_tdes_traces* tr, const graft_tdes_loss_config* lc,
                             double* d_loss, int32_t* d_skipped, float* d_gP, float* d_gC, float* d_gu, float* d_gs,
                             cudaStream_t st) {
    const graft_config& cfg = ctx->cfg;
    TrainParams p;
    p.P = ctx->d_P;
    p.C = ctx->d_C;
    p.u = ctx->d_u;
    p.k0 = ctx->tdes_s / sqrtf((float)cfg.m);
    p.inv_sqrt_m = 1.0f / sqrtf((float)cfg.m);
    p.V = cfg.V;
    p.L = cfg.L;
    p.m = cfg.m;
    p.K = cfg.K;
    p.n_groups = tr->n_groups;
    p.g_parent = tr->d_g_parent;
    p.g_depth = tr->d_g_depth;
    p.g_child = tr->d_g_child;
    p.g_logq = tr->d_g_logq;
    p.g_ztgt = tr->d_g_ztgt;
    p.n_pairs = tr->n_pairs;
    p.pairs = tr->d_pairs;
    p.n_edges = tr->n_edges;
    p.edges = tr->d_edges;
    p.gamma = lc->gamma;
    p.w1 = lc->w1;
    p.lam_kl = lc->lambda_kl;
    p.lam_pair = lc->lambda_pair;
    p.lam_bce = lc->lambda_bce;
    p.w_kl = tr->n_groups > 0 ? lc->lambda_kl / (float)tr->n_groups : 0.f;
    p.w_pair = tr->n_pairs > 0 ? lc->lambda_pair / (float)tr->n_pairs : 0.f;
    p.w_bce = tr->n_edges > 0 ? lc->lambda_bce / (float)tr->n_edges : 0.f;
    p.loss = d_loss;
    p.skipped = d_skipped;
    p.gP = d_gP;
    p.gC = d_gC;
    p.gu = d_gu;
    p.gs = d_gs;
    cudaError_t e = cudaMemsetAsync(d_loss, 0, 4 * sizeof(double), st);
    if (e != cudaSuccess) return e;
    if (d_skipped) {
        e = cudaMemsetAsync(d_skipped, 0, sizeof(int32_t), st);
        if (e != cudaSuccess) return e;
    }
    const long long items = (long long)tr->n_groups + tr->n_pairs + tr->n_edges;
    if (items == 0) return cudaSuccess;
    long long grid = (items + kTrWarps - 1) / kTrWarps;
    const long long cap = (long long)ctx->num_sms * 4;
    if (grid > cap) grid = cap;
    const int nch = (cfg.m / 4 + 31) / 32;
    const size_t smem = tdes_loss_smem(cfg);
    if (nch <= 1)
        tdes_loss_kernel<1><<<(int)grid, kTrThreads, smem, st>>>(p);
    else if (nch == 2)
        tdes_loss_kernel<2><<<(int)grid, kTrThreads, smem, st>>>(p);
    else
        tdes_loss_kernel<kTrMaxChunks><<<(int)grid, kTrThreads, smem, st>>>(p);
    ctx->launches += 1;
    return cudaGetLastError();
}

cudaError_t tdes_loss_configure(const graft_config& cfg) {
    const int smem = (int)tdes_loss_smem(cfg);
    if (smem <= 48 * 1024) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(tdes_loss_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tdes_loss_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tdes_loss_kernel<kTrMaxChunks>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    return e;
}
bool tdes_loss_supported(const graft_config& cfg) { return cfg.m % 4 == 0 && cfg.m <= 128 * kTrMaxChunks; }

}  // namespace graft
