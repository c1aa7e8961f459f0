// Per-sequence tail of the round: SABA budget (Sec. 3.3, Eq. 14-17), best-first expansion by TDES path
// score until B_t nodes (Sec. 3.1; Eq. 13; the heap expansion described for DDTree), level-order emission
// with the packed ancestor mask, and the acceptance walk.
#include "common.cuh"
#include "internal.h"

namespace graft {
namespace {

// ---- adjacent-position cosines r_d = cos(h_d, h_{d+1}) (Eq. 15), one CTA per (sequence, d) ------------
template <bool BF16>
__global__ void __launch_bounds__(128) cosine_kernel(const void* __restrict__ hidden, double* __restrict__ cosv, int L,
                                                     int dh) {
    const int b = blockIdx.x / (L - 1), d = blockIdx.x % (L - 1);
    const size_t ra = ((size_t)b * L + d) * dh, rb = ra + dh;
    double ab = 0.0, aa = 0.0, bb = 0.0;
    for (int k = threadIdx.x; k < dh; k += 128) {
        float x, y;
        if (BF16) {
            x = __uint_as_float(((uint32_t)((const uint16_t*)hidden)[ra + k]) << 16);
            y = __uint_as_float(((uint32_t)((const uint16_t*)hidden)[rb + k]) << 16);
        } else {
            x = ((const float*)hidden)[ra + k];
            y = ((const float*)hidden)[rb + k];
        }
        ab += (double)x * (double)y;
        aa += (double)x * (double)x;
        bb += (double)y * (double)y;
    }
    __shared__ double red[3][4];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ab += __shfl_xor_sync(0xFFFFFFFFu, ab, o);
        aa += __shfl_xor_sync(0xFFFFFFFFu, aa, o);
        bb += __shfl_xor_sync(0xFFFFFFFFu, bb, o);
    }
    if ((threadIdx.x & 31) == 0) {
        red[0][threadIdx.x >> 5] = ab;
        red[1][threadIdx.x >> 5] = aa;
        red[2][threadIdx.x >> 5] = bb;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        ab = red[0][0] + red[0][1] + red[0][2] + red[0][3];
        aa = red[1][0] + red[1][1] + red[1][2] + red[1][3];
        bb = red[2][0] + red[2][1] + red[2][2] + red[2][3];
        cosv[(size_t)b * L + d] = (aa > 0.0 && bb > 0.0) ? ab / (sqrt(aa) * sqrt(bb)) : 0.0;
    }
}

// ---- tree kernel -------------------------------------------------------------------------------------------
struct TreeParams {
    const int32_t* topk_id;
    const float* topk_lp;
    const int32_t* row_status;
    const float* edge;
    const double* cosv;
    const int32_t* root_token;
    const float* hist;
    const int32_t* prefix_len;
    const int32_t* fixed_budget;
    graft_tree_out out;
    int L, K, nmax, W, bmin, bmax, bstep;
    int use_saba;
    SabaDev saba;
};

constexpr int TREE_THREADS = 256;

struct TreeSmem {
    float* edge;         // [L*K*K]
    float* S;            // [nmax]  path score, pop order
    uint32_t* taken;     // [nmax]  children already selected (bit per candidate rank)
    uint32_t* cur_key;   // [nmax]  ord(score) of the node's best unselected child, 0 = none
    uint32_t* sortkey;   // [nmax]
    int16_t* parent;     // [nmax]  pop-order index of the parent
    int16_t* canon;      // [nmax]  level-order index of pop-order node n
    int16_t* cparent;    // [nmax]  level-order parent, by level-order index
    int16_t* lvl_list;   // [nmax]
    uint8_t* cand;       // [nmax]
    uint8_t* depth;      // [nmax]
    uint8_t* cur_child;  // [nmax]
    int* lvl_count;      // [kMaxL + 2]
    int* lvl_start;      // [kMaxL + 2]
    int* lvl_fill;       // [kMaxL + 2]
    int* scal;           // [8]  0: budget, 1: n_nodes, 2: status
};

__host__ __device__ inline size_t tree_smem_layout(int L, int K, int nmax, TreeSmem* s, unsigned char* base) {
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += (bytes + 15) & ~(size_t)15;
        return o;
    };
    size_t o_edge = take((size_t)L * K * K * 4), o_S = take((size_t)nmax * 4), o_tk = take((size_t)nmax * 4),
           o_ck = take((size_t)nmax * 4), o_sk = take((size_t)nmax * 4), o_par = take((size_t)nmax * 2),
           o_can = take((size_t)nmax * 2), o_cp = take((size_t)nmax * 2), o_ll = take((size_t)nmax * 2),
           o_cand = take(nmax), o_dep = take(nmax), o_cc = take(nmax), o_lc = take((kMaxL + 2) * 4),
           o_ls = take((kMaxL + 2) * 4), o_lf = take((kMaxL + 2) * 4), o_sc = take(8 * 4);
    if (s) {
        s->edge = (float*)(base + o_edge);
        s->S = (float*)(base + o_S);
        s->taken = (uint32_t*)(base + o_tk);
        s->cur_key = (uint32_t*)(base + o_ck);
        s->sortkey = (uint32_t*)(base + o_sk);
        s->parent = (int16_t*)(base + o_par);
        s->canon = (int16_t*)(base + o_can);
        s->cparent = (int16_t*)(base + o_cp);
        s->lvl_list = (int16_t*)(base + o_ll);
        s->cand = base + o_cand;
        s->depth = base + o_dep;
        s->cur_child = base + o_cc;
        s->lvl_count = (int*)(base + o_lc);
        s->lvl_start = (int*)(base + o_ls);
        s->lvl_fill = (int*)(base + o_lf);
        s->scal = (int*)(base + o_sc);
    }
    return off;
}

__device__ __forceinline__ double saba_cost(const SabaDev& sp, double B, double prefix) {
    if (sp.cost_mode == 0) return sp.c0 + sp.c1 * B + sp.c2 * B * prefix;
    if (B <= sp.pts_n[0]) return sp.pts_t[0];
    for (int i = 1; i < sp.n_pts; ++i)
        if (B <= sp.pts_n[i]) {
            double w = (B - sp.pts_n[i - 1]) / (sp.pts_n[i] - sp.pts_n[i - 1]);
            return sp.pts_t[i - 1] + w * (sp.pts_t[i] - sp.pts_t[i - 1]);
        }
    return sp.pts_t[sp.n_pts - 1];
}

// The best unselected child of node n under (score descending, rank ascending); executed by a full warp.
__device__ __forceinline__ void compute_cursor(const TreeSmem& sm, int n, int L, int K, int lane) {
    const int d = sm.depth[n];
    uint32_t key = 0;
    if (d < L && lane < K && !((sm.taken[n] >> lane) & 1u)) {
        const float sc = sm.S[n] + sm.edge[((size_t)d * K + sm.cand[n]) * K + lane];
        key = ord_from_float(sc);
    }
    const uint32_t kmax = __reduce_max_sync(0xFFFFFFFFu, key);
    const uint32_t who = __ballot_sync(0xFFFFFFFFu, key == kmax && key != 0u);
    if (lane == 0) {
        sm.cur_key[n] = kmax;
        sm.cur_child[n] = (uint8_t)(who ? __ffs(who) - 1 : 0);
    }
}

// Among frontier entries with equal score: the shallower child first, then the lexicographically smaller
// prefix.  n1, n2 are the PARENTS of the competing children (distinct nodes).
__device__ __forceinline__ bool pops_before(const TreeSmem& sm, int n1, int n2) {
    const int d1 = sm.depth[n1], d2 = sm.depth[n2];
    if (d1 != d2) return d1 < d2;
    while (sm.parent[n1] != sm.parent[n2]) {
        n1 = sm.parent[n1];
        n2 = sm.parent[n2];
    }
    return sm.cand[n1] < sm.cand[n2];
}

__global__ void __launch_bounds__(TREE_THREADS) tree_kernel(const TreeParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TreeSmem sm;
    tree_smem_layout(p.L, p.K, p.nmax, &sm, smem_raw);
    const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int L = p.L, K = p.K, nmax = p.nmax, W = p.W;
    const graft_tree_out& o = p.out;

    // ---- status and budget ---------------------------------------------------------------------------
    for (int i = tid; i < L * K * K; i += TREE_THREADS) sm.edge[i] = p.edge[(size_t)b * L * K * K + i];
    if (warp == 0) {
        int st = 0;
        for (int j = lane; j < L; j += 32) st |= p.row_status[(size_t)b * L + j];
        st = __reduce_or_sync(0xFFFFFFFFu, st);
        int budget = 0;
        float state[4] = {0.f, 0.f, 0.f, 0.f};
        if (!(st & GRAFT_ST_BAD_LOGITS)) {
            if (!p.use_saba) {
                budget = p.fixed_budget[b];
                budget = budget < 0 ? 0 : (budget > p.bmax ? p.bmax : budget);
            } else {
                double conf = 0.0, rs = 0.0;
                for (int j = lane; j < L; j += 32) conf += exp((double)p.topk_lp[((size_t)b * L + j) * K]);
                for (int j = lane; j < L - 1; j += 32) rs += p.cosv[(size_t)b * L + j];
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) {
                    conf += __shfl_xor_sync(0xFFFFFFFFu, conf, d);
                    rs += __shfl_xor_sync(0xFFFFFFFFu, rs, d);
                }
                conf /= (double)L;
                double degen = 0.0;
                if (L >= 2) degen = rs / (double)(L - 1) + (p.cosv[(size_t)b * L + L - 2] - p.cosv[(size_t)b * L]);
                const double hist = (double)p.hist[b];
                double tau = p.saba.phi_conf * conf + p.saba.phi_degen * degen + p.saba.phi_hist * hist + p.saba.phi_bias;
                if (!(tau >= p.saba.tau_min)) {
                    tau = p.saba.tau_min;
                    st |= GRAFT_ST_TAU_CLAMPED;
                }
                const double prefix = (double)p.prefix_len[b];
                double ubest = -INFINITY;
                int bbest = p.bmin;
                for (int B = p.bmin + lane * p.bstep; B <= p.bmax; B += 32 * p.bstep) {
                    const double G = 1.0 - exp(-(double)B / tau);
                    const double u = G / saba_cost(p.saba, (double)B, prefix);
                    if (u > ubest) {
                        ubest = u;
                        bbest = B;
                    }
                }
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) {
                    const double u2 = __shfl_xor_sync(0xFFFFFFFFu, ubest, d);
                    const int b2 = __shfl_xor_sync(0xFFFFFFFFu, bbest, d);
                    if (u2 > ubest || (u2 == ubest && b2 < bbest)) {
                        ubest = u2;
                        bbest = b2;
                    }
                }
                budget = bbest;
                state[0] = (float)conf;
                state[1] = (float)degen;
                state[2] = (float)hist;
                state[3] = (float)tau;
            }
        }
        if (lane == 0) {
            sm.scal[0] = budget;
            sm.scal[2] = st;
            if (o.d_state) {
                for (int i = 0; i < 4; ++i) o.d_state[(size_t)b * 4 + i] = state[i];
            }
        }
    }
    __syncthreads();

    // ---- best-first expansion (warp 0) -----------------------------------------------------------------
    if (warp == 0) {
        const int budget = sm.scal[0];
        int st = sm.scal[2];
        if (lane == 0) {
            sm.parent[0] = -1;
            sm.cand[0] = 0;
            sm.depth[0] = 0;
            sm.S[0] = 0.0f;
            sm.taken[0] = 0u;
        }
        __syncwarp();
        int n_sel = 0;
        if (budget > 0) {
            compute_cursor(sm, 0, L, K, lane);
            __syncwarp();
        }
        while (n_sel < budget) {
            uint32_t best_key = 0;
            int best_n = -1;
            bool multi = false;
            for (int n = lane; n <= n_sel; n += 32) {
                const uint32_t k = sm.cur_key[n];
                if (k > best_key) {
                    best_key = k;
                    best_n = n;
                    multi = false;
                } else if (k == best_key && k != 0u) {
                    multi = true;
                }
            }
            const uint32_t gmax = __reduce_max_sync(0xFFFFFFFFu, best_key);
            if (gmax == 0u) {
                st |= GRAFT_ST_FRONTIER_EMPTY;
                break;
            }
            const uint32_t tied = __ballot_sync(0xFFFFFFFFu, best_key == gmax);
            const uint32_t anym = __ballot_sync(0xFFFFFFFFu, best_key == gmax && multi);
            int win;
            if (__popc(tied) == 1 && anym == 0u) {
                win = __shfl_sync(0xFFFFFFFFu, best_n, __ffs(tied) - 1);
            } else {
                // equal scores: order by (depth ascending, prefix lexicographic ascending)
                int mine = -1;
                for (int n = lane; n <= n_sel; n += 32)
                    if (sm.cur_key[n] == gmax && (mine < 0 || pops_before(sm, n, mine))) mine = n;
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) {
                    const int other = __shfl_xor_sync(0xFFFFFFFFu, mine, d);
                    if (other >= 0 && (mine < 0 || pops_before(sm, other, mine))) mine = other;
                }
                win = mine;
            }
            const int c = sm.cur_child[win];
            const int d = sm.depth[win] + 1;
            const float s_new = sm.S[win] + sm.edge[((size_t)(d - 1) * K + sm.cand[win]) * K + c];
            const int n_new = ++n_sel;
            __syncwarp();
            if (lane == 0) {
                sm.parent[n_new] = (int16_t)win;
                sm.cand[n_new] = (uint8_t)c;
                sm.depth[n_new] = (uint8_t)d;
                sm.S[n_new] = s_new;
                sm.taken[n_new] = 0u;
                sm.taken[win] |= (1u << c);
            }
            __syncwarp();
            compute_cursor(sm, win, L, K, lane);
            compute_cursor(sm, n_new, L, K, lane);
            __syncwarp();
        }
        if (lane == 0) {
            sm.scal[1] = n_sel + 1;
            sm.scal[2] = st;
        }
    }
    if (tid < kMaxL + 2) {
        sm.lvl_count[tid] = 0;
        sm.lvl_fill[tid] = 0;
    }
    __syncthreads();

    // ---- emission in level order -------------------------------------------------------------------------
    const int n_nodes = sm.scal[1];
    for (int n = tid; n < n_nodes; n += TREE_THREADS) atomicAdd(&sm.lvl_count[sm.depth[n]], 1);
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int d = 0; d <= L; ++d) {
            sm.lvl_start[d] = acc;
            acc += sm.lvl_count[d];
        }
        sm.canon[0] = 0;
    }
    __syncthreads();
    for (int n = tid; n < n_nodes; n += TREE_THREADS) {
        const int d = sm.depth[n];
        sm.lvl_list[sm.lvl_start[d] + atomicAdd(&sm.lvl_fill[d], 1)] = (int16_t)n;
    }
    __syncthreads();
    for (int d = 1; d <= L; ++d) {
        const int s0 = sm.lvl_start[d], cnt = sm.lvl_count[d];
        if (cnt == 0) break;  // uniform: deeper levels are empty too
        for (int i = tid; i < cnt; i += TREE_THREADS) {
            const int n = sm.lvl_list[s0 + i];
            sm.sortkey[n] = (uint32_t)sm.canon[sm.parent[n]] * 32u + sm.cand[n];
        }
        __syncthreads();
        for (int i = tid; i < cnt; i += TREE_THREADS) {
            const int n = sm.lvl_list[s0 + i];
            const uint32_t key = sm.sortkey[n];
            int rank = 0;
            for (int j = 0; j < cnt; ++j) rank += (sm.sortkey[sm.lvl_list[s0 + j]] < key) ? 1 : 0;
            sm.canon[n] = (int16_t)(s0 + rank);
        }
        __syncthreads();
    }
    const int prefix = p.prefix_len[b];
    const int root = p.root_token[b];
    const size_t ob = (size_t)b * nmax;
    for (int n = tid; n < n_nodes; n += TREE_THREADS) {
        const int i = sm.canon[n], d = sm.depth[n];
        const int par = n == 0 ? -1 : sm.canon[sm.parent[n]];
        sm.cparent[i] = (int16_t)par;
        o.d_token[ob + i] = n == 0 ? root : p.topk_id[((size_t)b * L + d - 1) * K + sm.cand[n]];
        o.d_parent[ob + i] = par;
        o.d_depth[ob + i] = d;
        o.d_position[ob + i] = prefix - 1 + d;
        o.d_path_score[ob + i] = sm.S[n];
    }
    for (int i = n_nodes + tid; i < nmax; i += TREE_THREADS) {
        o.d_token[ob + i] = -1;
        o.d_parent[ob + i] = -1;
        o.d_depth[ob + i] = -1;
        o.d_position[ob + i] = -1;
        o.d_path_score[ob + i] = 0.f;
    }
    __syncthreads();
    for (int idx = tid; idx < nmax * W; idx += TREE_THREADS) {
        const int i = idx / W, w = idx % W;
        uint32_t bits = 0u;
        if (i < n_nodes) {
            for (int a = i; a >= 0 && (a >> 5) >= w; a = sm.cparent[a])
                if ((a >> 5) == w) bits |= 1u << (a & 31);
        }
        o.d_mask[ob * W + idx] = bits;
    }
    if (tid == 0) {
        o.d_n_nodes[b] = n_nodes;
        o.d_budget[b] = sm.scal[0];
        o.d_status[b] = sm.scal[2];
    }
}

// ---- acceptance walk: one warp per sequence --------------------------------------------------------------
__global__ void __launch_bounds__(128) accept_kernel(const int32_t* __restrict__ n_nodes, const int32_t* __restrict__ token,
                                                     const int32_t* __restrict__ parent,
                                                     const int32_t* __restrict__ target_next, int batch, int nmax, int L,
                                                     int32_t* __restrict__ accept_len, int32_t* __restrict__ accept_path,
                                                     int32_t* __restrict__ bonus) {
    const int b = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (b >= batch) return;
    const size_t ob = (size_t)b * nmax;
    int nn = n_nodes[b];
    nn = nn < 1 ? 1 : (nn > nmax ? nmax : nn);
    int cur = 0, a = 0;
    while (a < L) {
        const int want = target_next[ob + cur];
        int found = -1;
        for (int i0 = cur + 1; i0 < nn && found < 0; i0 += 32) {  // children come after their parent
            const int i = i0 + lane;
            const bool hit = i < nn && parent[ob + i] == cur && token[ob + i] == want;
            const uint32_t m = __ballot_sync(0xFFFFFFFFu, hit);
            if (m) found = i0 + __ffs(m) - 1;
        }
        if (found < 0) break;
        if (lane == 0) accept_path[(size_t)b * L + a] = found;
        ++a;
        cur = found;
    }
    for (int i = a + lane; i < L; i += 32) accept_path[(size_t)b * L + i] = -1;
    if (lane == 0) {
        accept_len[b] = a;
        bonus[b] = target_next[ob + cur];
    }
}

}  // namespace

size_t tree_smem_bytes(const graft_config& cfg) {
    return tree_smem_layout(cfg.L, cfg.K, cfg.budget_max + 1, nullptr, nullptr);
}

cudaError_t tree_configure(const graft_config& cfg) {
    return cudaFuncSetAttribute(tree_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tree_smem_bytes(cfg));
}

cudaError_t cosine_launch(graft_ctx* ctx, int batch, const void* d_hidden, double* d_cos, cudaStream_t st) {
    const graft_config& cfg = ctx->cfg;
    if (cfg.L < 2) return cudaSuccess;
    if (cfg.hidden_dtype == GRAFT_BF16)
        cosine_kernel<true><<<batch * (cfg.L - 1), 128, 0, st>>>(d_hidden, d_cos, cfg.L, cfg.hidden_dim);
    else
        cosine_kernel<false><<<batch * (cfg.L - 1), 128, 0, st>>>(d_hidden, d_cos, cfg.L, cfg.hidden_dim);
    ctx->launches += 1;
    return cudaGetLastError();
}

cudaError_t tree_launch(graft_ctx* ctx, int batch, const int32_t* d_topk_id, const float* d_topk_lp,
                        const int32_t* d_row_status, const float* d_edge, const double* d_cos,
                        const int32_t* d_root_token, const float* d_hist, const int32_t* d_prefix_len,
                        const int32_t* d_fixed_budget, const graft_tree_out* out, cudaStream_t st) {
    const graft_config& cfg = ctx->cfg;
    TreeParams p;
    p.topk_id = d_topk_id;
    p.topk_lp = d_topk_lp;
    p.row_status = d_row_status;
    p.edge = d_edge;
    p.cosv = d_cos;
    p.root_token = d_root_token;
    p.hist = d_hist;
    p.prefix_len = d_prefix_len;
    p.fixed_budget = d_fixed_budget;
    p.out = *out;
    p.L = cfg.L;
    p.K = cfg.K;
    p.nmax = ctx->nmax;
    p.W = ctx->mask_words;
    p.bmin = cfg.budget_min;
    p.bmax = cfg.budget_max;
    p.bstep = cfg.budget_step;
    p.use_saba = d_fixed_budget == nullptr;
    p.saba = ctx->saba;
    tree_kernel<<<batch, TREE_THREADS, tree_smem_bytes(cfg), st>>>(p);
    ctx->launches += 1;
    return cudaGetLastError();
}

cudaError_t accept_launch(graft_ctx* ctx, int batch, const graft_tree_out* trees, const int32_t* d_target_next,
                          int32_t* d_accept_len, int32_t* d_accept_path, int32_t* d_bonus, cudaStream_t st) {
    accept_kernel<<<(batch + 3) / 4, 128, 0, st>>>(trees->d_n_nodes, trees->d_token, trees->d_parent, d_target_next,
                                                   batch, ctx->nmax, ctx->cfg.L, d_accept_len, d_accept_path, d_bonus);
    ctx->launches += 1;
    return cudaGetLastError();
}

}  // namespace graft
