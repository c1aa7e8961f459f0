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
    const float* esort;   // [batch, L, K, K] edge rows sorted by (edge desc, child rank asc)
    const uint8_t* eidx;  // child rank of each sorted entry
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
    float* es;           // [L*K*K]  sorted edge rows
    uint8_t* ei;         // [L*K*K]  child rank of each sorted entry
    uint64_t* ent;       // [32*33]  frontier entry of node n at [(n & 31) * 33 + (n >> 5)], 0 = none
    uint64_t* poplog;    // [nmax]   the entry that was selected as node n (node 0: the root's pseudo entry)
    uint32_t* chmask;    // [nmax]   candidate ranks of the node's selected children, one bit each
    int* cc;             // [nmax]   per-level scratch: child counts in level order, then their exclusive scan
    uint32_t* stage;     // [8 warps * 32 rows * W] mask rows staged for coalesced stores
    float* S;            // [nmax]   path score, selection order
    uint32_t* sortkey;   // [nmax]
    int16_t* parent;     // [nmax]   selection-order index of the parent
    int16_t* canon;      // [nmax]   level-order index of selection-order node n
    int16_t* cparent;    // [nmax]   level-order parent, by level-order index
    int16_t* lvl_list;   // [nmax]
    uint8_t* cand;       // [nmax]
    uint8_t* depth;      // [nmax]
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
    size_t o_es = take((size_t)L * K * K * 4), o_ei = take((size_t)L * K * K), o_ent = take((size_t)32 * 33 * 8), o_log = take((size_t)nmax * 8), o_chm = take((size_t)nmax * 4), o_cc = take((size_t)nmax * 4), o_stage = take((size_t)8 * 32 * ((nmax + 31) / 32) * 4),
           o_S = take((size_t)nmax * 4), o_sk = take((size_t)nmax * 4), o_par = take((size_t)nmax * 2),
           o_can = take((size_t)nmax * 2), o_cp = take((size_t)nmax * 2), o_ll = take((size_t)nmax * 2),
           o_cand = take(nmax), o_dep = take(nmax), o_lc = take((kMaxL + 2) * 4), o_ls = take((kMaxL + 2) * 4),
           o_lf = take((kMaxL + 2) * 4), o_sc = take(8 * 4);
    if (s) {
        s->es = (float*)(base + o_es);
        s->ei = base + o_ei;
        s->ent = (uint64_t*)(base + o_ent);
        s->poplog = (uint64_t*)(base + o_log);
        s->chmask = (uint32_t*)(base + o_chm);
        s->cc = (int*)(base + o_cc);
        s->stage = (uint32_t*)(base + o_stage);
        s->S = (float*)(base + o_S);
        s->sortkey = (uint32_t*)(base + o_sk);
        s->parent = (int16_t*)(base + o_par);
        s->canon = (int16_t*)(base + o_can);
        s->cparent = (int16_t*)(base + o_cp);
        s->lvl_list = (int16_t*)(base + o_ll);
        s->cand = base + o_cand;
        s->depth = base + o_dep;
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

// Frontier entry: one per selected node, naming that node's best child not yet selected.  A plain 64-bit
// maximum over the entries is the next node to select:
//   bits 63..32  ord(path score of the child)                      -> score descending
//   bits 30..25  32 - depth of the child                           -> then the shallower child
//   bits 24..15  1023 - selection index of the parent              -> then the parent selected earlier
//   bits 14..10  position of the child in the parent's sorted row  (under one parent the sorted row gives
//   bits  9..5   candidate rank of the parent                       edge descending, rank ascending)
//   bits  4..0   candidate rank of the child
__device__ __forceinline__ uint64_t pack_entry(float score, int child_depth, int parent_sel, int pos, int parent_cand,
                                               int child_cand) {
    const uint32_t lo = ((uint32_t)(32 - child_depth) << 25) | ((uint32_t)(1023 - parent_sel) << 15) |
                        ((uint32_t)pos << 10) | ((uint32_t)parent_cand << 5) | (uint32_t)child_cand;
    return ((uint64_t)ord_from_float(score) << 32) | lo;
}

// Warp-wide maximum of a 64-bit key: one redux on the high word, then the low word of the (usually single)
// lane that holds it.
__device__ __forceinline__ uint64_t warp_max64(uint64_t x) {
    const uint32_t hi = (uint32_t)(x >> 32), lo = (uint32_t)x;
    const uint32_t hm = __reduce_max_sync(0xFFFFFFFFu, hi);
    const uint32_t tie = __ballot_sync(0xFFFFFFFFu, hi == hm);
    uint32_t lm;
    if ((tie & (tie - 1)) == 0u)
        lm = __shfl_sync(0xFFFFFFFFu, lo, __ffs(tie) - 1);
    else
        lm = __reduce_max_sync(0xFFFFFFFFu, hi == hm ? lo : 0u);
    return ((uint64_t)hm << 32) | lm;
}

__global__ void __launch_bounds__(TREE_THREADS) tree_kernel(const TreeParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TreeSmem sm;
    tree_smem_layout(p.L, p.K, p.nmax, &sm, smem_raw);
    const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int L = p.L, K = p.K, nmax = p.nmax, W = p.W;
    const graft_tree_out& o = p.out;

    // ---- status and budget ---------------------------------------------------------------------------
#ifdef GRAFT_TREE_PROF
    long long t_prof0 = clock64(), t_prof1 = 0, t_prof2 = 0;
#endif
    {
        const int ne = L * K * K;
        if ((ne & 3) == 0) {
            const float4* src = (const float4*)(p.esort + (size_t)b * ne);
            for (int i = tid; i < ne / 4; i += TREE_THREADS) ((float4*)sm.es)[i] = src[i];
        } else {
            for (int i = tid; i < ne; i += TREE_THREADS) sm.es[i] = p.esort[(size_t)b * ne + i];
        }
        for (int i = tid; i < L * K * K; i += TREE_THREADS) sm.ei[i] = p.eidx[(size_t)b * L * K * K + i];
    }
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

#ifdef GRAFT_TREE_PROF
    t_prof1 = clock64();
#endif
    // ---- best-first expansion (warp 0) -----------------------------------------------------------------
    if (warp == 0) {
        // Column `lane` of the entry table (nodes n with n & 31 == lane) belongs to this lane, which keeps the
        // column's maximum in a register.  One step selects `cur`, the maximum entry: the parent's entry moves
        // to its next sorted child and the new node gets an entry.  Only the parent's column changes, so the
        // next maximum is the largest of (a) that column re-reduced by the 32 lanes together, (b) the new
        // node's entry and (c) the maximum over all other columns, which does not depend on this step's
        // updates and is reduced in the shadow of the loads.
        constexpr int NSP = 33;
        const int budget = sm.scal[0];
        int st = sm.scal[2];
        for (int i = lane; i < 32 * NSP; i += 32) sm.ent[i] = 0ull;
        uint64_t best = 0ull;
        if (lane == 0) {
            best = pack_entry(0.0f + sm.es[0], 1, 0, 0, 0, sm.ei[0]);
            sm.ent[0] = best;
            sm.poplog[0] = (uint64_t)ord_from_float(0.0f) << 32;
        }
        __syncwarp();
        uint64_t cur = warp_max64(best);
        int n_sel = 0;
        // Inside the loop a path score is never -0 (sums that start from +0), so the order-preserving map
        // needs no zero canonicalisation here.
        while (n_sel < budget) {
            const uint32_t hmax = (uint32_t)(cur >> 32), lmax = (uint32_t)cur;
            if (hmax == 0u) {
                st |= GRAFT_ST_FRONTIER_EMPTY;
                break;
            }
            const int n_new = ++n_sel;
            const uint32_t dm = (lmax >> 25) & 63u;  // 32 - depth of the selected child
            const int d = 32 - (int)dm;
            const int n_par = 1023 - (int)((lmax >> 15) & 1023u);
            const int pos = (int)((lmax >> 10) & 31u);
            const int cpar = (int)((lmax >> 5) & 31u);
            const int c = (int)(lmax & 31u);
            const int colA = n_par & 31, slotA = n_par >> 5, colB = n_new & 31, slotB = n_new >> 5;
            const uint64_t others = warp_max64(lane == colA ? 0ull : best);
            // every lane reads the same few words (broadcasts) and its own entry of the parent's column
            const bool adv = pos + 1 < K, deeper = d < L;
            const int at1 = adv ? ((d - 1) * K + cpar) * K + pos + 1 : 0;
            const int at2 = deeper ? (d * K + c) * K : 0;
            const uint32_t sp_o = ((const uint32_t*)sm.poplog)[2 * n_par + 1];  // ord(path score of the parent)
            const float e1 = sm.es[at1], e2 = sm.es[at2];
            const uint32_t i1 = sm.ei[at1], i2 = sm.ei[at2];
            uint64_t col = sm.ent[colA * NSP + lane];
            const float sp = __uint_as_float(sp_o ^ (~(uint32_t)((int32_t)sp_o >> 31) | 0x80000000u));
            const float s_new = __uint_as_float(hmax ^ (~(uint32_t)((int32_t)hmax >> 31) | 0x80000000u));
            const uint32_t u1 = __float_as_uint(sp + e1), u2 = __float_as_uint(s_new + e2);
            const uint32_t h1 = u1 ^ ((uint32_t)((int32_t)u1 >> 31) | 0x80000000u);
            const uint32_t h2 = u2 ^ ((uint32_t)((int32_t)u2 >> 31) | 0x80000000u);
            const uint32_t l1 = ((lmax & ~31u) + (1u << 10)) | i1;
            const uint32_t l2 = ((dm - 1u) << 25) | ((uint32_t)(1023 - n_new) << 15) | ((uint32_t)c << 5) | i2;
            const uint64_t e_adv = adv ? (((uint64_t)h1 << 32) | l1) : 0ull;
            const uint64_t e_new = deeper ? (((uint64_t)h2 << 32) | l2) : 0ull;
            if (lane == 0) {
                sm.ent[colA * NSP + slotA] = e_adv;
                sm.ent[colB * NSP + slotB] = e_new;
                sm.poplog[n_new] = cur;
            }
            if (lane == slotA) col = e_adv;
            if (colB == colA && lane == slotB) col = e_new;
            const uint64_t colbest = warp_max64(col);
            if (lane == colA) best = colbest;
            if (lane == colB) best = e_new > best ? e_new : best;
            cur = others > colbest ? others : colbest;
            cur = e_new > cur ? e_new : cur;
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

#ifdef GRAFT_TREE_PROF
    t_prof2 = clock64();
#endif
    // ---- emission in level order -------------------------------------------------------------------------
    // Level order = depth ascending, then the parent's level-order index, then candidate rank.  Level by level:
    // the child counts of level d-1, laid out in level order, are scanned; a node of level d lands at
    // (start of level d) + (children of earlier parents) + (selected siblings of lower rank).
    const int n_nodes = sm.scal[1];
    for (int n = tid; n < nmax; n += TREE_THREADS) sm.chmask[n] = 0u;
    __syncthreads();
    for (int n = tid; n < n_nodes; n += TREE_THREADS) {  // unpack the selection log
        const uint64_t e = sm.poplog[n];
        const uint32_t lo = (uint32_t)e;
        const int d = n == 0 ? 0 : 32 - (int)((lo >> 25) & 63u);
        const int par = n == 0 ? -1 : 1023 - (int)((lo >> 15) & 1023u);
        sm.parent[n] = (int16_t)par;
        sm.cand[n] = (uint8_t)(lo & 31u);
        sm.depth[n] = (uint8_t)d;
        sm.S[n] = __uint_as_float(bits_from_ord((uint32_t)(e >> 32)));
        if (n > 0) atomicOr(&sm.chmask[par], 1u << (lo & 31u));
        atomicAdd(&sm.lvl_count[d], 1);
    }
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
        const int s_prev = sm.lvl_start[d - 1], n_prev = sm.lvl_count[d - 1];
        const int s_cur = sm.lvl_start[d], n_cur = sm.lvl_count[d];
        if (n_cur == 0) break;  // uniform: deeper levels are empty too
        for (int i = tid; i < n_prev; i += TREE_THREADS) {
            const int y = sm.lvl_list[s_prev + i];
            sm.cc[sm.canon[y] - s_prev] = __popc(sm.chmask[y]);
        }
        __syncthreads();
        if (warp == 0) {  // exclusive scan of cc[0..n_prev): a contiguous chunk per lane, then a warp scan
            const int ch = (n_prev + 31) / 32;
            const int lo_i = lane * ch, hi_i = min(n_prev, lo_i + ch);
            int sum = 0;
            for (int i = lo_i; i < hi_i; ++i) sum += sm.cc[i];
            int incl = sum;
#pragma unroll
            for (int o2 = 1; o2 < 32; o2 <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o2);
                if (lane >= o2) incl += t;
            }
            int run = incl - sum;
            for (int i = lo_i; i < hi_i; ++i) {
                const int v = sm.cc[i];
                sm.cc[i] = run;
                run += v;
            }
        }
        __syncthreads();
        for (int i = tid; i < n_cur; i += TREE_THREADS) {
            const int x = sm.lvl_list[s_cur + i];
            const int y = sm.parent[x];
            sm.canon[x] = (int16_t)(s_cur + sm.cc[sm.canon[y] - s_prev] +
                                    __popc(sm.chmask[y] & ((1u << sm.cand[x]) - 1u)));
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
    // ancestor masks: each thread builds one row in its warp's staging tile (walking up, level-order indices
    // only decrease, so the row is produced from its highest word down); the warp then stores its 32 rows,
    // which are contiguous in the output, with coalesced writes
    {
        uint32_t* tile = sm.stage + (size_t)warp * 32 * W;
        for (int i0 = warp * 32; i0 < nmax; i0 += TREE_THREADS) {
            const int i = i0 + lane;
            uint32_t* row = tile + lane * W;
            if (i < n_nodes) {
                int w = W - 1;
                uint32_t bits = 0u;
                for (int a = i; a >= 0; a = sm.cparent[a]) {
                    const int wa = a >> 5;
                    while (w > wa) {
                        row[w] = bits;
                        bits = 0u;
                        --w;
                    }
                    bits |= 1u << (a & 31);
                }
                row[w] = bits;
                for (--w; w >= 0; --w) row[w] = 0u;
            } else {
                for (int w = 0; w < W; ++w) row[w] = 0u;
            }
            __syncwarp();
            const int rows = min(32, nmax - i0);
            uint32_t* dst = o.d_mask + (ob + i0) * W;
            for (int k = lane; k < rows * W; k += 32) dst[k] = tile[k];
            __syncwarp();
        }
    }
#ifdef GRAFT_TREE_PROF
    __syncthreads();
    if (tid == 0 && o.d_state) {
        o.d_state[(size_t)b * 4 + 0] = (float)(t_prof1 - t_prof0);
        o.d_state[(size_t)b * 4 + 1] = (float)(t_prof2 - t_prof1);
        o.d_state[(size_t)b * 4 + 2] = (float)(clock64() - t_prof2);
    }
#endif
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
                        const int32_t* d_row_status, const float* d_esort, const uint8_t* d_eidx, const double* d_cos,
                        const int32_t* d_root_token, const float* d_hist, const int32_t* d_prefix_len,
                        const int32_t* d_fixed_budget, const graft_tree_out* out, cudaStream_t st) {
    const graft_config& cfg = ctx->cfg;
    TreeParams p;
    p.topk_id = d_topk_id;
    p.topk_lp = d_topk_lp;
    p.row_status = d_row_status;
    p.esort = d_esort;
    p.eidx = d_eidx;
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
