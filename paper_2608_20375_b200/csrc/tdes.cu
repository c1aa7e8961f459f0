// TDES (Sec. 3.2): the cached bi-tower projections and the per-round edge scores.
//
//   tdes_precompute_kernel   out[v] = W e_v + b            (text after Eq. 6: computed once per model)
//   tdes_edges_kernel        edge[d][i][c] = log q_d(c) + beta * (f - mean_c f),
//                            f = s (P[p_i] + u_d) . (C[c] + u_d) / sqrt(m)          (Eq. 4-6)
//                            for the first depths of every sequence (the arithmetic is in edge_score.cuh,
//                            which the tree kernel also uses for deeper depths)
//
// The per-round scorer is a gather of token-indexed table rows followed by K x K dot products of length
// m per depth -- not a dense contraction over hidden states -- so it runs as fp32 FMAs out of shared
// memory (tensor-core tf32/bf16 products would also break the 1e-5 score tolerance).
#include "common.cuh"
#include "internal.h"
#include "edge_score.cuh"
#include "saba.cuh"

namespace graft {
namespace {

// ---- table precompute: a plain shared-memory tiled fp32 GEMM (setup path, off the round) ---------------
constexpr int PT_V = 64, PT_M = 64, PT_E = 16;

template <bool BF16>
__global__ void __launch_bounds__(256) tdes_precompute_kernel(const void* __restrict__ emb, const float* __restrict__ W,
                                                              const float* __restrict__ bias, float* __restrict__ out,
                                                              int V, int E, int m) {
    __shared__ float sA[PT_E][PT_V + 1];  // emb tile, transposed
    __shared__ float sB[PT_E][PT_M + 1];  // W tile, transposed
    const int v0 = blockIdx.x * PT_V, k0 = blockIdx.y * PT_M;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;  // 16 x 16 threads, 4 x 4 outputs each
    float acc[4][4] = {};
    for (int e0 = 0; e0 < E; e0 += PT_E) {
        for (int i = threadIdx.x; i < PT_V * PT_E; i += 256) {
            int r = i / PT_E, c = i % PT_E;
            int v = v0 + r, e = e0 + c;
            float x = 0.f;
            if (v < V && e < E) {
                if (BF16)
                    x = __uint_as_float(((uint32_t)((const uint16_t*)emb)[(size_t)v * E + e]) << 16);
                else
                    x = ((const float*)emb)[(size_t)v * E + e];
            }
            sA[c][r] = x;
        }
        for (int i = threadIdx.x; i < PT_M * PT_E; i += 256) {
            int r = i / PT_E, c = i % PT_E;
            int k = k0 + r, e = e0 + c;
            sB[c][r] = (k < m && e < E) ? W[(size_t)k * E + e] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int e = 0; e < PT_E; ++e) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = sA[e][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = sB[e][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int v = v0 + ty * 4 + i;
        if (v >= V) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int k = k0 + tx * 4 + j;
            if (k < m) out[(size_t)v * m + k] = acc[i][j] + (bias ? bias[k] : 0.f);
        }
    }
}

// ---- edge scores: one CTA per (sequence, depth) --------------------------------------------------------
struct EdgeParams {
    const int32_t* topk_id;
    const float* topk_lp;
    const int32_t* root_token;
    const int32_t* row_status;
    const float* P;
    const float* C;
    const float* u;
    float* edge;      // [batch, L, K, K] by (parent rank, child rank)
    float* esort;     // same rows, each sorted by (edge descending, child rank ascending), stored rotated (es_col)
    uint8_t* eidx;    // child rank of every sorted entry
    int L, K, m, V;
    int rows;     // depths [0, rows) are scored for every sequence: one CTA each
    int rows_all; // CTAs per sequence: depths [rows, rows_all) are scored only for sequences whose trees will run deep
    float scale;  // s / sqrt(m)
    float beta;
    int root_edge;
    // the budget of every sequence (Sec. 3.3), worked out by its depth-0 CTA when saba_out is not NULL
    SabaResult* saba_out;         // [batch]
    const double* cos_pre;        // [batch, L] adjacent-position cosines from the vocab pass
    const int32_t* vp_err;
    const float* hist;            // [batch]
    const int32_t* prefix_len;    // [batch]
    const int32_t* fixed_budget;  // [batch], or NULL: SABA
    int bmin, bmax, bstep;
    SabaDev saba;
};

// WRITE_EDGE: also write the unsorted scores (the caller asked for the array); the tree kernel reads only the sorted rows
// KC, MC: K and m as compile-time constants (the configured workloads' 32 and 128), or 0: taken from the parameters
template <bool WRITE_EDGE, int KC, int MC>
__global__ void __launch_bounds__(256, 4) tdes_edges_kernel(const EdgeParams p) {
    extern __shared__ __align__(16) float smem[];
    pdl_launch_dependents();  // the tree kernel may move in as SMs free up; it waits for this grid before it reads
    pdl_wait();               // the candidates come from the vocab pass
    // the depths scored for every sequence come first in the grid, the depths that only deep trees need behind them: the
    // CTAs of the latter mostly exit at once and should not take the places of CTAs with work
    const int n_all = (int)gridDim.x / p.rows_all * p.rows;  // units that every sequence needs
    int b, j;
    if ((int)blockIdx.x < n_all) {
        b = (int)blockIdx.x / p.rows;
        j = (int)blockIdx.x - b * p.rows;
    } else {
        const int r = (int)blockIdx.x - n_all, nd = p.rows_all - p.rows;
        b = r / nd;
        j = p.rows + (r - b * nd);
    }
    if (j >= p.rows && !deep_tree_likely(p.topk_lp + (size_t)b * p.L * p.K, p.L, p.K)) return;  // (uniform)
    const int K = KC ? KC : p.K, m = MC ? MC : p.m, ld = m + 4;  // padded row: 16-byte aligned, conflict-free float4 reads
    float* sP = smem;                        // [K][ld]  parent rows + u_d
    float* sC = smem + (size_t)kMaxK * ld;   // [K][ld]  child rows + u_d
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_par = (j == 0) ? 1 : K;
    const size_t row = (size_t)b * p.L + j;
    if (j == 0 && p.saba_out != nullptr && warp == 7) {
        // the depth-0 unit has one parent, so this CTA has time to spare: its last warp works out the sequence's budget,
        // which the tree kernel would otherwise do in front of everything else
        const SabaResult r = saba_warp(p.saba, p.bmin, p.bmax, p.bstep, p.L, K, p.row_status + (size_t)b * p.L, p.vp_err,
                                       p.topk_lp + (size_t)b * p.L * K, p.cos_pre + (size_t)b * p.L, p.hist + b,
                                       p.prefix_len + b, p.fixed_budget ? p.fixed_budget + b : nullptr, lane);
        if (lane == 0) p.saba_out[b] = r;
    }
    float* outs = p.esort + row * K * K;
    uint8_t* outi = p.eidx + row * K * K;
    const int32_t* ids = p.topk_id + row * K;
    const float* lps = p.topk_lp + row * K;

    const bool bad = p.row_status != nullptr && (p.row_status[row] != 0 || (j > 0 && p.row_status[row - 1] != 0));
    const bool neutral = (p.beta == 0.0f) || (j == 0 && !p.root_edge) || bad;
    if (neutral) {
        // edge = log q exactly (the DDTree score of Eq. 3); bad rows get zeros
        // (log q is already ordered by rank, so the sorted rows are the rows themselves)
        for (int i = threadIdx.x; i < K * K; i += 256) {
            int par = i / K, c = i % K;
            const float v = (bad || par >= n_par) ? 0.f : lps[c];
            if (WRITE_EDGE) p.edge[row * K * K + i] = v;
            outs[par * K + es_col(c, par, K)] = v;
            outi[i] = (uint8_t)c;
        }
        return;
    }
    // gather: token ids first (one round trip), then every warp issues the loads of all its rows before it uses
    // any of them (a second round trip); one warp per table row, 16 bytes per lane
    __shared__ int toks[2 * kMaxK];
    if (threadIdx.x < n_par + K) {
        const int r = threadIdx.x;
        int32_t tok = r < n_par ? (j == 0 ? p.root_token[b] : p.topk_id[(row - 1) * K + r]) : ids[r - n_par];
        toks[r] = tok < 0 ? 0 : (tok >= p.V ? p.V - 1 : tok);
    }
    __syncthreads();
    const float* urow = p.u + (size_t)j * m;
    constexpr int RPW = 2 * kMaxK / 8;  // rows per warp at most
    const uint64_t keep = l2_policy_evict_last();
    for (int k40 = 0; k40 < m / 4; k40 += 32) {
        const int k4 = k40 + lane;
        float4 t[RPW];
#pragma unroll
        for (int q = 0; q < RPW; ++q) {
            const int r = warp + 8 * q;
            t[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < n_par + K && k4 < m / 4)
                t[q] = ldg_f4_keep((const float4*)((r < n_par ? p.P : p.C) + (size_t)toks[r] * m) + k4, keep);
        }
        if (k4 < m / 4) {
            const float4 uu = *(const float4*)(urow + k4 * 4);
#pragma unroll
            for (int q = 0; q < RPW; ++q) {
                const int r = warp + 8 * q;
                if (r < n_par + K) {
                    float* dst = (r < n_par ? sP + (size_t)r * ld : sC + (size_t)(r - n_par) * ld) + k4 * 4;
                    *(float4*)dst = make_float4(t[q].x + uu.x, t[q].y + uu.y, t[q].z + uu.z, t[q].w + uu.w);
                }
            }
        }
    }
    __syncthreads();
    // dot products into shared memory, then every warp finishes the rows of parents warp, warp+8, ...
    float* part = sC + (size_t)kMaxK * ld;  // [K][K]
    __shared__ uint32_t wsc[8][32];
    edge_dots<false>(sP, sC, nullptr, m, K, n_par, part, warp, lane);
    __syncthreads();
    const float inv_K = 1.0f / (float)K;
    for (int par = warp; par < K; par += 8) {
        float val;
        int rank;
        edge_row_finish(par < n_par ? part + (size_t)par * K : nullptr, lps, p.scale, p.beta, K, inv_K, wsc[warp], lane,
                        val, rank);
        if (lane < K) {
            if (WRITE_EDGE) p.edge[(row * K + par) * K + lane] = val;
            outs[(size_t)par * K + es_col(rank, par, K)] = val;
            outi[(size_t)par * K + rank] = (uint8_t)lane;
        }
    }
}

}  // namespace

cudaError_t tdes_precompute_launch(graft_ctx* ctx, const void* d_emb, graft_dtype dt, int E, const float* d_W,
                                   const float* d_b, float* d_out, cudaStream_t st) {
    const int V = ctx->cfg.V, m = ctx->cfg.m;
    dim3 grid((V + PT_V - 1) / PT_V, (m + PT_M - 1) / PT_M);
    if (dt == GRAFT_BF16)
        tdes_precompute_kernel<true><<<grid, 256, 0, st>>>(d_emb, d_W, d_b, d_out, V, E, m);
    else
        tdes_precompute_kernel<false><<<grid, 256, 0, st>>>(d_emb, d_W, d_b, d_out, V, E, m);
    ctx->launches += 1;
    return cudaGetLastError();
}

size_t tdes_edges_smem(const graft_config& cfg) {
    return ((size_t)2 * kMaxK * (cfg.m + 4) + (size_t)kMaxK * kMaxK) * sizeof(float);  // P rows, C rows, dot products
}

cudaError_t tdes_edges_configure(const graft_config& cfg) {
    const int bytes = (int)tdes_edges_smem(cfg);
    cudaError_t e = cudaFuncSetAttribute(tdes_edges_kernel<true, 0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tdes_edges_kernel<false, 0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tdes_edges_kernel<false, 32, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tdes_edges_kernel<false, 16, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tdes_edges_kernel<false, 8, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return e;
}

cudaError_t tdes_edges_launch(graft_ctx* ctx, int batch, const int32_t* d_topk_id, const float* d_topk_lp,
                              const int32_t* d_root_token, const int32_t* d_row_status, float* d_edge,
                              float* d_esort, uint8_t* d_eidx, int rows, SabaResult* d_saba_out, const float* d_hist,
                              const int32_t* d_prefix_len, const int32_t* d_fixed_budget, cudaStream_t st) {
    const graft_config& cfg = ctx->cfg;
    EdgeParams p;
    p.topk_id = d_topk_id;
    p.topk_lp = d_topk_lp;
    p.root_token = d_root_token;
    p.row_status = d_row_status;
    p.P = ctx->d_P;
    p.C = ctx->d_C;
    p.u = ctx->d_u;
    p.edge = d_edge;
    p.esort = d_esort;
    p.eidx = d_eidx;
    p.L = cfg.L;
    p.K = cfg.K;
    p.m = cfg.m;
    p.V = cfg.V;
    p.scale = ctx->tdes_s / sqrtf((float)cfg.m);
    p.beta = ctx->tdes_set ? cfg.beta : 0.0f;
    p.root_edge = cfg.root_edge;
    p.rows = rows;
    p.rows_all = d_edge || rows == cfg.L ? rows : cfg.L;  // (rows < L only when the tree kernel can score on demand)
    p.saba_out = d_row_status ? d_saba_out : nullptr;
    p.cos_pre = ctx->w_cos;
    p.vp_err = ctx->w_errflag;
    p.hist = d_hist;
    p.prefix_len = d_prefix_len;
    p.fixed_budget = d_fixed_budget;
    p.bmin = cfg.budget_min;
    p.bmax = cfg.budget_max;
    p.bstep = cfg.budget_step;
    p.saba = ctx->saba;
    void (*kern)(const EdgeParams) = d_edge ? tdes_edges_kernel<true, 0, 0> : tdes_edges_kernel<false, 0, 0>;
    if (!d_edge && cfg.m == 128) {  // K and m known at compile time
        if (cfg.K == 32) kern = tdes_edges_kernel<false, 32, 128>;
        if (cfg.K == 16) kern = tdes_edges_kernel<false, 16, 128>;
        if (cfg.K == 8) kern = tdes_edges_kernel<false, 8, 128>;
    }
    const cudaError_t e = launch_pdl(kern, dim3(batch * p.rows_all), dim3(256), tdes_edges_smem(cfg), st, p);
    ctx->launches += 1;
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace graft
