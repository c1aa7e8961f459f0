// Per-sequence tail of the round: SABA budget (Sec. 3.3, Eq. 14-17), best-first expansion by TDES path
// score until B_t nodes (Sec. 3.1; Eq. 13; the heap expansion described for DDTree), level-order emission
// with the packed ancestor mask, and the acceptance walk (which also keeps the acceptance history of Eq. 15).
// Edge scores of depths that the edge-score kernel did not cover are worked out here when an expansion reaches them.
#include "common.cuh"
#include "internal.h"
#include "edge_score.cuh"
#include "saba.cuh"

namespace graft {
namespace {

// ---- tree kernel -------------------------------------------------------------------------------------------
struct TreeParams {
    const int32_t* topk_id;
    const float* topk_lp;
    const int32_t* row_status;
    const double* cos_pre;  // [batch, L] adjacent-position cosines (Eq. 15), written by the vocab pass
    const int32_t* vp_err;  // word 0: a bounded wait of the vocab pass ran out (sticky)
    const float* esort;   // [batch, L, K, K] edge rows sorted by (edge desc, child rank asc), each rotated by its parent rank (es_col)
    const uint8_t* eidx;  // child rank of each sorted entry
    const int32_t* root_token;
    const float* hist;
    const int32_t* prefix_len;
    const int32_t* fixed_budget;
    graft_tree_out out;
    int L, K, nmax, W, bmin, bmax, bstep;
    int ncap;  // capacity of the node table of the parallel phase
    // Edge scores (Eq. 4-6): the rows of depths [0, rows_pre) come from the edge-score kernel through esort / eidx;
    // deeper rows are scored inside this kernel (lazy = 1), level by level, only if the expansion gets there.
    int rows_pre;
    int rows_adaptive;  // the edge-score kernel also scored the deeper rows of sequences whose trees will run deep
    int lazy;
    int lazy_m;  // m when the shared-memory layout holds the buffers of the on-demand scorer, else 0
    const float* P;
    const float* C;
    const float* u;
    float scale, beta;
    int root_edge, m, V;
    int use_saba;
    SabaDev saba;
    const SabaResult* saba_pre;  // [batch] budget, status and state worked out by the edge-score kernel, or NULL
};

constexpr int TREE_THREADS = 1024;  // one CTA per SM (shared memory bound): all warps serve the parallel phases

struct TreeSmem {
    float* es;           // [L*K*K]  sorted edge rows
    uint8_t* ei;         // [L*K*K]  child rank of each sorted entry
    // node table of the parallel phase (append-only; node 0 = root).  Levels follow one another, and within a level
    // the nodes stand in the order of their prefixes (the parent's place in its level, then the candidate rank), which
    // is the level order of the emitted tree: a subset taken in table order is already in level order
    uint32_t* nkey;      // [ncap]   bottleneck key = min over the path of ord(path score); later: compact index
    float* nS;           // [ncap]   path score
    uint32_t* ninfo;     // [ncap]   parent's table index | candidate rank << 13 | depth << 18 | place in the parent's sorted row << 24
    // compact arrays by selection index n (0 = root; a parent's index is smaller than its children's)
    uint64_t* ent;       // [nmax]   frontier entry of node n: its best unselected child, 0 = none
    float* S;            // [nmax]   path score
    uint32_t* chmask;    // [nmax]   candidate ranks of the node's selected children, one bit each
    int16_t* parent;     // [nmax]
    int16_t* canon;      // [nmax]   level-order index of node n
    int16_t* cparent;    // [nmax]   level-order parent, by level-order index
    uint8_t* cand;       // [nmax]
    uint8_t* depth;      // [nmax]
    // emission scratch, laid over the node table (dead by then)
    int16_t* lvl_list;   // [nmax]
    int16_t* cc;         // [2][nmax] per-level child counts in level order, then their exclusive scan (two levels)
    uint32_t* stage;     // [8 warps * 32 rows * W] mask rows staged for coalesced stores
    uint32_t* hist;      // [2208] histograms of the threshold searches; scan and child-mask scratch of the level expansion
    int* lvl_count;      // [kMaxL + 2]
    int* lvl_start;      // [kMaxL + 2]
    int* lvl_fill;       // [kMaxL + 2]
    double* cosv;        // [kMaxL]  adjacent-position cosines r_d (Eq. 15)
    // on-demand edge scoring only:
    float* gP;           // [K][m+4]  gathered parent rows P[token]
    float* gC;           // [K][m+4]  gathered child rows C[token]
    float* gU;           // [m]       u_d
    int32_t* tokid;      // [L*K]     candidate tokens
    float* lpv;          // [L*K]     their log q
    int* scal;           // [16] 0 budget, 1 n_nodes, 2 status, 3 table size, 4 overflow, 6/7 radix-select hand-over
};

__host__ __device__ inline size_t tree_smem_layout(int L, int K, int nmax, int ncap, int lazy_m, TreeSmem* s,
                                                   unsigned char* base) {
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += (bytes + 15) & ~(size_t)15;
        return o;
    };
    const int W = (nmax + 31) / 32;
    size_t o_es = take((size_t)L * K * K * 4), o_ei = take((size_t)L * K * K);
    size_t emis = (((size_t)nmax * 2 + 15) & ~(size_t)15) + (((size_t)nmax * 4 + 15) & ~(size_t)15) + (size_t)8 * 32 * W * 4;
    size_t table = (size_t)ncap * 12;
    size_t o_tab = take(table > emis ? table : emis);
    size_t o_ent = take((size_t)nmax * 8), o_S = take((size_t)nmax * 4), o_chm = take((size_t)nmax * 4),
           o_par = take((size_t)nmax * 2), o_can = take((size_t)nmax * 2), o_cp = take((size_t)nmax * 2),
           o_cand = take(nmax), o_dep = take(nmax), o_hist = take(2208 * 4), o_lc = take((kMaxL + 2) * 4),
           o_ls = take((kMaxL + 2) * 4), o_lf = take((kMaxL + 2) * 4), o_sc = take(16 * 4), o_cos = take(kMaxL * 8);
    size_t o_gp = 0, o_gc = 0, o_gu = 0, o_tk = 0, o_lp = 0;
    if (lazy_m > 0) {
        o_gp = take((size_t)K * (lazy_m + 4) * 4);
        o_gc = take((size_t)K * (lazy_m + 4) * 4);
        o_gu = take((size_t)lazy_m * 4);
        o_tk = take((size_t)L * K * 4);
        o_lp = take((size_t)L * K * 4);
    }
    if (s) {
        s->es = (float*)(base + o_es);
        s->ei = base + o_ei;
        s->nkey = (uint32_t*)(base + o_tab);
        s->nS = (float*)(base + o_tab + (size_t)ncap * 4);
        s->ninfo = (uint32_t*)(base + o_tab + (size_t)ncap * 8);
        s->lvl_list = (int16_t*)(base + o_tab);
        s->cc = (int16_t*)(base + o_tab + (((size_t)nmax * 2 + 15) & ~(size_t)15));
        s->stage = (uint32_t*)(base + o_tab + (((size_t)nmax * 2 + 15) & ~(size_t)15) + (((size_t)nmax * 4 + 15) & ~(size_t)15));
        s->ent = (uint64_t*)(base + o_ent);
        s->S = (float*)(base + o_S);
        s->chmask = (uint32_t*)(base + o_chm);
        s->parent = (int16_t*)(base + o_par);
        s->canon = (int16_t*)(base + o_can);
        s->cparent = (int16_t*)(base + o_cp);
        s->cand = base + o_cand;
        s->depth = base + o_dep;
        s->hist = (uint32_t*)(base + o_hist);
        s->lvl_count = (int*)(base + o_lc);
        s->lvl_start = (int*)(base + o_ls);
        s->lvl_fill = (int*)(base + o_lf);
        s->scal = (int*)(base + o_sc);
        s->cosv = (double*)(base + o_cos);
        s->gP = (float*)(base + o_gp);
        s->gC = (float*)(base + o_gc);
        s->gU = (float*)(base + o_gu);
        s->tokid = (int32_t*)(base + o_tk);
        s->lpv = (float*)(base + o_lp);
    }
    return off;
}

// capacity of the node table: what fits beside the edge rows in ~200 KB of shared memory, at most 6144 nodes
// (parent indices are 13 bits) and at least enough for a full budget's worth of nodes
__host__ __device__ inline int tree_node_cap(int L, int K, int nmax, int lazy_m) {
    const int W = (nmax + 31) / 32;
    const size_t emis = (((size_t)nmax * 2 + 15) & ~(size_t)15) + (((size_t)nmax * 4 + 15) & ~(size_t)15) +
                        (size_t)8 * 32 * W * 4;
    const size_t fixed = tree_smem_layout(L, K, nmax, 0, lazy_m, nullptr, nullptr);  // counts `emis` for the table
    const size_t room = fixed < (size_t)222 * 1024 ? (size_t)222 * 1024 - fixed : 0;
    long long cap = (long long)((emis + room) / 12);
    if (cap > 6144) cap = 6144;
    if (cap < 2 * nmax) cap = 2 * nmax;
    return (int)cap;
}

// Frontier entry of a selected node: its best child that is not selected yet.
//   bits 63..32  ord(path score of the child)
//   bits 30..25  32 - depth of the child (larger = shallower)
//   bits 14..10  position of the child in the parent's sorted row
//   bits  9..5   candidate rank of the parent
//   bits  4..0   candidate rank of the child
__device__ __forceinline__ uint64_t pack_entry(float score, int child_depth, int pos, int parent_cand, int child_cand) {
    const uint32_t lo = ((uint32_t)(32 - child_depth) << 25) | ((uint32_t)pos << 10) | ((uint32_t)parent_cand << 5) |
                        (uint32_t)child_cand;
    return ((uint64_t)ord_from_float(score) << 32) | lo;
}

// Does the prefix of node n1 come before the prefix of node n2 in lexicographic order of candidate ranks?
// Both at the same depth, n1 != n2.
__device__ __forceinline__ bool path_less(const TreeSmem& sm, int n1, int n2) {
    for (int step = 0; step < kMaxL && sm.parent[n1] != sm.parent[n2]; ++step) {  // (depth <= L: the bound is never hit)
        n1 = sm.parent[n1];
        n2 = sm.parent[n2];
        if (n1 < 0 || n2 < 0) return n1 < n2;
    }
    return sm.cand[n1] < sm.cand[n2];
}

// Order of two frontier entries (owned by nodes n1, n2): path score descending, then the shallower child,
// then the parent whose prefix is lexicographically smaller.  n < 0 = no entry.
__device__ __forceinline__ bool entry_before(const TreeSmem& sm, uint64_t e1, int n1, uint64_t e2, int n2) {
    if (n2 < 0) return n1 >= 0;
    if (n1 < 0) return false;
    const uint32_t h1 = (uint32_t)(e1 >> 32), h2 = (uint32_t)(e2 >> 32);
    if (h1 != h2) return h1 > h2;
    const uint32_t d1 = ((uint32_t)e1 >> 25) & 63u, d2 = ((uint32_t)e2 >> 25) & 63u;
    if (d1 != d2) return d1 > d2;
    return path_less(sm, n1, n2);
}

// B-th largest of keys[lo..hi) (hi - lo >= kth >= 1) by an 8-bit radix select; every thread of the CTA calls it.
// Passes [pass0, pass1) of four are run: with pass1 < 4 only the top 8 * pass1 bits are resolved and the rest is
// returned as zero, a lower bound of the B-th largest key; a later call on the same keys can take up the search
// where this one stopped (pass0 = the earlier pass1, prefix and remaining as returned).  The 256 bins exist in four
// copies (neighbouring warps use different ones) and in two generations, so that the next pass's bins are cleared
// while this pass's are scanned.
__device__ uint32_t cta_kth_largest(const TreeSmem& sm, const uint32_t* keys, int lo, int hi, int kth, int pass0,
                                    int pass1, uint32_t prefix, int& remaining, int tid) {
    const int warp = tid >> 5, lane = tid & 31;
    uint32_t mask = pass0 == 0 ? 0u : 0xFFFFFFFFu << (32 - 8 * pass0);
    if (pass0 == 0) {
        prefix = 0u;
        remaining = kth;
    }
    sm.hist[(pass0 & 1) * 1024 + tid] = 0u;
    __syncthreads();
    for (int pass = pass0; pass < pass1; ++pass) {
        const int shift = 24 - 8 * pass;
        uint32_t* h = sm.hist + (pass & 1) * 1024 + (warp & 3) * 256;
        for (int i = lo + tid; i < hi; i += TREE_THREADS) {
            const uint32_t k = keys[i];
            if ((k & mask) == prefix) atomicAdd(&h[(k >> shift) & 255u], 1u);
        }
        sm.hist[((pass + 1) & 1) * 1024 + tid] = 0u;  // the other generation, for the next pass
        __syncthreads();
        if (warp == 0) {  // lane l owns bins 255-8l .. 248-8l, from the top down
            const uint32_t* hh = sm.hist + (pass & 1) * 1024;
            int c[8], sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int bin = 255 - 8 * lane - j;
                c[j] = (int)(hh[bin] + hh[256 + bin] + hh[512 + bin] + hh[768 + bin]);
                sum += c[j];
            }
            int incl = sum;
#pragma unroll
            for (int o2 = 1; o2 < 32; o2 <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o2);
                if (lane >= o2) incl += t;
            }
            const int excl = incl - sum;
            if (excl < remaining && remaining <= incl) {
                int acc = excl, digit = 255 - 8 * lane, rem = remaining - excl;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (acc < remaining && remaining <= acc + c[j]) {
                        digit = 255 - 8 * lane - j;
                        rem = remaining - acc;
                    }
                    acc += c[j];
                }
                sm.scal[6] = digit;
                sm.scal[7] = rem;
            }
        }
        __syncthreads();
        prefix |= (uint32_t)sm.scal[6] << shift;
        mask |= 255u << shift;
        remaining = sm.scal[7];
    }
    return prefix;
}

// The same search over keys that are not stored anywhere: the keys of the children that the threads' nodes are
// about to append (this thread's node: `cnt` children, key of child r = min(kx, ord(sx + es[row + r]))).  Two passes:
// the leading 16 bits of the kth largest of them, the rest zero -- a lower bound of it.  At most kth nodes of one
// level can end up in the tree, so this bound may replace a lower threshold before a level is appended; it keeps
// a level from flooding the node table while few keys are known (sharply peaked rows: every deviation from the
// best chain costs tens of units, and the B-th largest key of the table stays far down for several levels).
// Every thread of the CTA calls it; the children number at least kth in all.
__device__ uint32_t cta_kth_largest_of_children_radix(const TreeSmem& sm, int cnt, uint32_t kx, float sx, int row,
                                                      int cx, int K, int kth, int tid) {
    const int warp = tid >> 5, lane = tid & 31;
    uint32_t prefix = 0u, mask = 0u;
    int remaining = kth;
    sm.hist[tid] = 0u;
    __syncthreads();
    for (int pass = 0; pass < 2; ++pass) {
        const int shift = 24 - 8 * pass;
        uint32_t* h = sm.hist + (pass & 1) * 1024 + (warp & 3) * 256;
        for (int r = 0; r < cnt; ++r) {
            const uint32_t oc = ord_from_float(sx + sm.es[row + es_col(r, cx, K)]);
            const uint32_t k = oc < kx ? oc : kx;
            if ((k & mask) == prefix) atomicAdd(&h[(k >> shift) & 255u], 1u);
        }
        sm.hist[((pass + 1) & 1) * 1024 + tid] = 0u;  // the other generation, for the next pass
        __syncthreads();
        if (warp == 0) {  // lane l owns bins 255-8l .. 248-8l, from the top down
            const uint32_t* hh = sm.hist + (pass & 1) * 1024;
            int c[8], sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int bin = 255 - 8 * lane - j;
                c[j] = (int)(hh[bin] + hh[256 + bin] + hh[512 + bin] + hh[768 + bin]);
                sum += c[j];
            }
            int incl = sum;
#pragma unroll
            for (int o2 = 1; o2 < 32; o2 <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o2);
                if (lane >= o2) incl += t;
            }
            const int excl = incl - sum;
            if (excl < remaining && remaining <= incl) {
                int acc = excl, digit = 255 - 8 * lane, rem = remaining - excl;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (acc < remaining && remaining <= acc + c[j]) {
                        digit = 255 - 8 * lane - j;
                        rem = remaining - acc;
                    }
                    acc += c[j];
                }
                sm.scal[6] = digit;
                sm.scal[7] = rem;
            }
        }
        __syncthreads();
        prefix |= (uint32_t)sm.scal[6] << shift;
        mask |= 255u << shift;
        remaining = sm.scal[7];
    }
    __syncthreads();
    return prefix;
}

// Threshold searches work on 1024 bins of equal width in SCORE below the best score (the root's best child): bin b
// holds the keys whose score lies in (top - (b + 1) w, top - b w], w = 1/32, so the bins reach 32 below the top; what
// lies further down (or is -inf) shares the last bin.  The same expression gives a key's bin wherever it is needed.
constexpr float kSelBinsPerUnit = 32.0f;
__device__ __forceinline__ int select_bin(uint32_t key, float top) {
    const float d = (top - __uint_as_float(bits_from_ord(key))) * kSelBinsPerUnit;
    if (!(d < 1023.0f)) return 1023;  // (also NaN)
    return d > 0.0f ? (int)d : 0;
}

// A lower bound of the kth largest key among the children that the threads' nodes are about to append (see
// cta_kth_largest_of_children_radix): one pass over 1024 bins of equal width in score between the current threshold
// (every child counted reaches it) and the best child, whose lower edge is the bound; the radix passes only if that
// range is not finite (their top bits crowd into a few counters, which thousands of atomics then queue on; bins in
// score spread them).
__device__ uint32_t cta_kth_largest_of_children(const TreeSmem& sm, int cnt, uint32_t kx, float sx, int row, int cx,
                                                int K, int kth, uint32_t theta, int tid) {
    const int warp = tid >> 5, lane = tid & 31;
    uint32_t* h = sm.hist;  // [1024 + 32], then [1] the best child key
    h[tid] = 0u;
    if (tid < 33) h[1024 + tid] = 0u;
    __syncthreads();
    {
        uint32_t best = 0u;  // a node's first child has its largest key
        if (cnt > 0) {
            const uint32_t oc = ord_from_float(sx + sm.es[row + cx]);  // (entry 0 stands at column cx)
            best = oc < kx ? oc : kx;
        }
        best = __reduce_max_sync(0xFFFFFFFFu, best);
        if (lane == 0 && best) atomicMax(&h[1056], best);
    }
    __syncthreads();
    const float top = __uint_as_float(bits_from_ord(h[1056])), low = __uint_as_float(bits_from_ord(theta));
    const float scale = 1023.0f / (top - low);
    if (!(scale > 0.0f) || !(scale < 1e30f)) {  // (uniform) no finite range: -inf scores, or all children equal
        __syncthreads();
        return cta_kth_largest_of_children_radix(sm, cnt, kx, sx, row, cx, K, kth, tid);
    }
    for (int r = 0; r < cnt; ++r) {
        const uint32_t oc = ord_from_float(sx + sm.es[row + es_col(r, cx, K)]);
        const float sc = __uint_as_float(bits_from_ord(oc < kx ? oc : kx));
        const float df = (top - sc) * scale;
        const int d = df > 0.0f ? (df < 1023.0f ? (int)df : 1023) : 0;
        atomicAdd(&h[d + (d >> 5)], 1u);
    }
    __syncthreads();
    if (warp == 0) {  // lane l owns bins 32 l .. 32 l + 31 (bin 0 holds the largest keys)
        const uint32_t* mine = h + 33 * lane;
        int sum = 0;
#pragma unroll 8
        for (int q = 0; q < 32; ++q) sum += (int)mine[q];
        int incl = sum;
#pragma unroll
        for (int o2 = 1; o2 < 32; o2 <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o2);
            if (lane >= o2) incl += t;
        }
        const int excl = incl - sum;
        if (excl < kth && kth <= incl) {
            int acc = excl, bin = 32 * lane;
            for (int q = 0; q < 32; ++q) {
                const int c = (int)mine[q];
                if (acc < kth && kth <= acc + c) bin = 32 * lane + q;
                acc += c;
            }
            sm.scal[6] = bin;
        }
    }
    __syncthreads();
    const int bin = sm.scal[6];
    __syncthreads();
    // the lower edge of the bin, less a hundredth of a bin for the rounding of the bin index; never below theta
    const uint32_t bound = ord_from_float(top - ((float)(bin + 1) + 0.01f) / scale);
    return bound > theta ? bound : theta;
}

// Where the B-th largest key lies and the rank wanted there.
struct SelBucket {
    int bin;          // the bin of select_bin, or -1: the closed key range [lo, hi] instead
    uint32_t lo, hi;
    int rem;          // the B-th largest of all is the rem-th largest of the keys in the bucket
    bool valid;
};
__device__ __forceinline__ bool select_in_bucket(const SelBucket& st, uint32_t key, float top) {
    return st.bin >= 0 ? select_bin(key, top) == st.bin : (key >= st.lo && key <= st.hi);
}

// One histogram pass over keys[lo_i..hi_i) finds the bin that holds the B-th largest key, and a lower bound of that
// key (the bin's lower edge less a hundredth of a bin: the rounding of select_bin is below 1e-4 of a bin).  A bin
// spans about as much as a key's top 16 bits do at the scores met here, so the bound prunes as well as two 8-bit
// radix passes would, for one pass.  If the B-th largest falls into the shared last bin, two radix passes find its
// 16-bit bucket instead.  Bins are padded by one word per 32 (the flood search's lanes own 32 consecutive bins each
// and read them without bank conflicts).  Every thread of the CTA calls this; hi_i - lo_i >= kth >= 1.
__device__ uint32_t cta_select_bucket(const TreeSmem& sm, const uint32_t* keys, int lo_i, int hi_i, int kth, float top,
                                      SelBucket& st, int tid) {
    const int warp = tid >> 5, lane = tid & 31;
    uint32_t* h = sm.hist;  // [1024 + 32] bins, [1060 + 32] sums of 32 bins
    h[tid] = 0u;
    if (tid < 32) h[1024 + tid] = 0u;
    __syncthreads();
    for (int i = lo_i + tid; i < hi_i; i += TREE_THREADS) {
        const int d = select_bin(keys[i], top);
        atomicAdd(&h[d + (d >> 5)], 1u);
    }
    __syncthreads();
    // warp w adds up bins 32 w .. 32 w + 31 (bin 0 holds the largest keys); warp 0 then finds the group of 32 bins that
    // holds the kth largest key in a scan of the 32 sums, and the bin in a scan of that group: two short steps
    {
        const uint32_t wsum = __reduce_add_sync(0xFFFFFFFFu, h[33 * warp + lane]);
        if (lane == 0) h[1060 + warp] = wsum;
    }
    __syncthreads();
    if (warp == 0) {
        const int ws = (int)h[1060 + lane];
        int incl = ws;
#pragma unroll
        for (int o2 = 1; o2 < 32; o2 <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o2);
            if (lane >= o2) incl += t;
        }
        const uint32_t gm = __ballot_sync(0xFFFFFFFFu, incl - ws < kth && kth <= incl);  // (one lane: kth <= keys in all)
        const int g = gm ? __ffs(gm) - 1 : 31;
        const int base = __shfl_sync(0xFFFFFFFFu, incl - ws, g);
        const int c = (int)h[33 * g + lane];
        int inc2 = c;
#pragma unroll
        for (int o2 = 1; o2 < 32; o2 <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, inc2, o2);
            if (lane >= o2) inc2 += t;
        }
        if (base + inc2 - c < kth && kth <= base + inc2) {
            sm.scal[6] = 32 * g + lane;
            sm.scal[7] = kth - (base + inc2 - c);
        }
    }
    __syncthreads();
    const int bin = sm.scal[6];
    st.rem = sm.scal[7];
    st.valid = true;
    if (bin >= 1023) {  // (uniform) below the range the bins resolve
        __syncthreads();
        int rem = 0;
        const uint32_t prefix = cta_kth_largest(sm, keys, lo_i, hi_i, kth, 0, 2, 0u, rem, tid);
        st.bin = -1;
        st.lo = prefix;
        st.hi = prefix | 0xFFFFu;
        st.rem = rem;
        return st.lo;
    }
    st.bin = bin;
    st.lo = st.hi = 0u;
    return ord_from_float(top - ((float)(bin + 1) + 0.01f) / kSelBinsPerUnit);
}

// The exact B-th largest key once its bucket is known: the keys inside it are few (path scores are spread over
// many more values than there are buckets), so they are collected and ranked against each other directly; if there
// are more than the list holds (heavy ties), a full radix select runs instead.
// *n_reach: how many of all the keys reach the value returned (kth if no other key ties with it), or -1 if unknown.
__device__ uint32_t cta_finish_select(const TreeSmem& sm, const uint32_t* keys, int lo_i, int hi_i, int kth, float top,
                                      const SelBucket& st, int tid, int* n_reach) {
    constexpr int kCap = 512;
    uint32_t* list = sm.hist;           // [kCap] (the histogram space is idle between selects)
    int* cnt = (int*)(sm.hist + 1100);  // [1]
    if (tid == 0) *cnt = 0;
    __syncthreads();
    for (int i = lo_i + tid; i < hi_i; i += TREE_THREADS) {
        const uint32_t k = keys[i];
        if (select_in_bucket(st, k, top)) {
            const int pos = atomicAdd(cnt, 1);
            if (pos < kCap) list[pos] = k;
        }
    }
    __syncthreads();
    const int n = *cnt;
    if (n > kCap) {  // (uniform)
        __syncthreads();
        int rem = 0;
        *n_reach = -1;
        return cta_kth_largest(sm, keys, lo_i, hi_i, kth, 0, 4, 0u, rem, tid);
    }
    const int remaining = st.rem;
    for (int i = tid; i < n; i += TREE_THREADS) {
        const uint32_t k = list[i];
        int gt = 0, ge = 0;
        for (int j = 0; j < n; ++j) {
            const uint32_t o = list[j];
            gt += o > k ? 1 : 0;
            ge += o >= k ? 1 : 0;
        }
        if (gt < remaining && remaining <= ge) {  // (every writer writes the same values)
            sm.scal[6] = (int)k;
            sm.scal[7] = kth - remaining + ge;  // the keys above the bucket, and those of the bucket that reach k
        }
    }
    __syncthreads();
    const uint32_t v = (uint32_t)sm.scal[6];
    *n_reach = sm.scal[7];
    __syncthreads();  // the list and the result word are free again
    return v;
}

// The smallest of keys[lo_i..hi_i) that reaches the bound `theta` of the B-th largest key: a bound of it as well (the
// B-th largest is one of those keys), reached by the same keys, and an actual key -- where hundreds of keys tie just
// above a bucket's edge, their value.  The whole CTA; word: one word of scratch.
__device__ __forceinline__ uint32_t cta_snap_to_key(const uint32_t* keys, int lo_i, int hi_i, uint32_t theta, uint32_t* word,
                                                    int tid) {
    if (tid == 0) *word = 0xFFFFFFFFu;
    __syncthreads();
    uint32_t mn = 0xFFFFFFFFu;
    for (int i = lo_i + tid; i < hi_i; i += TREE_THREADS) {
        const uint32_t k = keys[i];
        mn = (k >= theta && k < mn) ? k : mn;
    }
    mn = __reduce_min_sync(0xFFFFFFFFu, mn);
    if ((tid & 31) == 0 && mn != 0xFFFFFFFFu) atomicMin(word, mn);
    __syncthreads();
    const uint32_t v = *word;
    __syncthreads();
    return v == 0xFFFFFFFFu ? theta : v;
}

// The order in which best-first takes prefixes of equal key, as one number (larger = earlier): path score, then
// shallower, then the parent's place in the table, then the place in the parent's sorted row.
__device__ __forceinline__ uint64_t tie_order(float S, uint32_t info) {
    return ((uint64_t)ord_from_float(S) << 24) |
           (uint64_t)(((63u - ((info >> 18) & 63u)) << 18) | ((8191u - (info & 8191u)) << 5) | (31u - ((info >> 24) & 31u)));
}

// ---- edge scores on demand --------------------------------------------------------------------------------------
// Row j of the edge scores (children at depth j+1), Eq. 4-6: the table rows P[parent token], C[child token] and
// u_j are copied into shared memory asynchronously (16-byte cp.async chunks spread over the CTA, issued while the
// level above is expanded); K x K dot products of (P + u_j) and (C + u_j) in fp32, centred over the children, plus
// log q; each parent's row is then ordered by (edge descending, child rank ascending).
__device__ __forceinline__ bool lazy_neutral(const TreeParams& p, int j) {
    return p.beta == 0.0f || (j == 0 && !p.root_edge);
}
// (the table rows of frequent tokens are read round after round: L2 is asked to keep them, as in the edge-score kernel)
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src) {
    const uint64_t keep = l2_policy_evict_last();
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "l"(keep)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Every thread calls this; the copies of one row form one group per thread.
__device__ __forceinline__ void lazy_issue_gather(const TreeParams& p, const TreeSmem& sm, int j, int root_token, int tid,
                                                  const int K, const int m) {
    if (j >= p.L || lazy_neutral(p, j)) return;
    const int ld = m + 4, q4 = m / 4, n_par = j == 0 ? 1 : K;
    const int warp = tid >> 5, lane = tid & 31;
    for (int r = warp; r <= n_par + K; r += TREE_THREADS / 32) {  // a warp per table row, a lane per 16 bytes
        const float* src;
        float* dst;
        if (r == n_par + K) {
            src = p.u + (size_t)j * m;
            dst = sm.gU;
        } else {
            int tok = r < n_par ? (j == 0 ? root_token : sm.tokid[(j - 1) * K + r]) : sm.tokid[j * K + r - n_par];
            tok = tok < 0 ? 0 : (tok >= p.V ? p.V - 1 : tok);
            src = (r < n_par ? p.P : p.C) + (size_t)tok * m;
            dst = r < n_par ? sm.gP + (size_t)r * ld : sm.gC + (size_t)(r - n_par) * ld;
        }
        for (int k4 = lane; k4 < q4; k4 += 32) cp_async16(smem_u32(dst + 4 * k4), src + 4 * k4);
    }
    cp_async_commit();
}
// Every thread of the CTA calls this.
// `inflight` is the depth whose table rows are on their way (or -1).
__device__ __forceinline__ void lazy_score_row(const TreeParams& p, const TreeSmem& sm, int j, int root_token, int tid,
                                               int& inflight, const int K, const int m) {
    const int n_par = j == 0 ? 1 : K;
    const int warp = tid >> 5, lane = tid & 31;
    float* es = sm.es + (size_t)j * K * K;
    uint8_t* ei = sm.ei + (size_t)j * K * K;
    const float* lps = sm.lpv + j * K;
    if (lazy_neutral(p, j)) {
        // edge = log q exactly (the DDTree score of Eq. 3); log q is already ordered by rank
        for (int i = tid; i < K * K; i += TREE_THREADS) {
            es[(i / K) * K + es_col(i % K, i / K, K)] = (i / K) < n_par ? lps[i % K] : 0.f;
            ei[i] = (uint8_t)(i % K);
        }
        __syncthreads();
        return;
    }
    if (inflight != j) lazy_issue_gather(p, sm, j, root_token, tid, K, m);
    cp_async_wait_all();
    __syncthreads();
    float* part = (float*)sm.hist;                // [K][K] dot products (the histogram space is idle here)
    uint32_t* wsc = sm.hist + 1024 + warp * 32;   // [32] per warp
    if (warp < 8) edge_dots<true>(sm.gP, sm.gC, sm.gU, m, K, n_par, part, warp, lane);
    __syncthreads();
    lazy_issue_gather(p, sm, j + 1, root_token, tid, K, m);  // the table rows of this depth are no longer read
    inflight = j + 1;
    const float inv_K = 1.0f / (float)K;
    for (int par = warp; par < K; par += TREE_THREADS / 32) {  // one warp per parent
        float val;
        int rank;
        edge_row_finish(par < n_par ? part + (size_t)par * K : nullptr, lps, p.scale, p.beta, K, inv_K, wsc, lane, val,
                        rank);
        if (lane < K) {
            es[(size_t)par * K + es_col(rank, par, K)] = val;
            ei[(size_t)par * K + rank] = (uint8_t)lane;
        }
    }
    __syncthreads();
}

// KC, MC: the number of candidates per position and the width of the TDES tables as compile-time constants (the
// configured workloads' K = 32, m = 128: every index computation with K becomes a shift), or 0: taken from the parameters
// FAST: the usual round is known at compile time as well -- the budget comes from the edge-score kernel (no SABA
// arithmetic in this instance) and deeper rows are scored on demand
// TIES: the instance for rounds without edge scores (beta = 0), where exactly equal probabilities make hundreds of
// prefixes tie with the B-th largest key: it resolves them in parallel (the other instances leave more than 32 tied
// keys to the sequential expansion; with edge scores in the keys such ties do not occur in tens, and the code's mere
// presence costs this register-bound kernel 0.4 us a round)
template <int KC, int MC, bool FAST, int NMAXC = 0, bool TIES = false>
__global__ void __launch_bounds__(TREE_THREADS) tree_kernel(const TreeParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int K = KC ? KC : p.K, p_m = MC ? MC : p.m;
    const bool p_lazy = FAST ? true : p.lazy != 0;
    TreeSmem sm;
    const int ncap = NMAXC ? 6144 : p.ncap;  // (the instance with the outputs' size known is used at full capacity only)
    tree_smem_layout(p.L, K, NMAXC ? NMAXC : p.nmax, ncap, p.lazy_m, &sm, smem_raw);
    const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int L = p.L, nmax = NMAXC ? NMAXC : p.nmax, W = NMAXC ? (NMAXC + 31) / 32 : p.W;
    const graft_tree_out& o = p.out;
    pdl_launch_dependents();  // an acceptance walk queued behind this kernel may move in; it waits for this grid
    pdl_wait();  // candidates, cosines and edge rows come from the kernels ahead in the stream

    // ---- status and budget ---------------------------------------------------------------------------
    // the sorted edge rows of this sequence: bulk copies through the TMA unit when the 16-byte rules allow it
    // (they land while warp 0 works out the budget), plain loads otherwise
    __shared__ __align__(8) uint64_t rows_bar;
    __shared__ int rows_abort;
    const int rows_pre = p.rows_pre;
    const int ne = rows_pre * K * K;  // entries that come from the edge-score kernel for every sequence
    const bool bulk = ne > 0 && (ne % 16) == 0;
    // the prologue's loads from global memory are all issued before the first of them is used: one round trip
    const int root = p.root_token[b];
    const float lp_top = p.rows_adaptive ? deep_tree_load(p.topk_lp + (size_t)b * L * K, L, K) : 0.f;
    SabaResult pre_r;
    pre_r.budget = 0;
    pre_r.status = 0;
    pre_r.state[0] = pre_r.state[1] = pre_r.state[2] = pre_r.state[3] = 0.f;
    if ((FAST || p.saba_pre) && tid == 0) pre_r = p.saba_pre[b];
    int32_t lz_tok = 0;
    float lz_lp = 0.f;
    if (p_lazy && tid < L * K) {  // (L K <= 1024: a thread per candidate)
        lz_tok = p.topk_id[(size_t)b * L * K + tid];
        lz_lp = p.topk_lp[(size_t)b * L * K + tid];
    }
    int rows_done = rows_pre;  // rows [0, rows_done) are in shared memory
    int inflight = -1;           // on-demand scoring: depth whose table rows are being fetched
    if (tid == 0) {
        rows_abort = 0;
        mbar_init(smem_u32(&rows_bar), 1);
        mbar_fence_init();
    }
    const size_t seq_e = (size_t)b * L * K * K;  // this sequence's rows in esort / eidx
    if (bulk) {
        if (tid == 0) {
            mbar_arrive_expect_tx(smem_u32(&rows_bar), (uint32_t)ne * 5u);
            const char* g_es = (const char*)(p.esort + seq_e);
            const char* g_ei = (const char*)(p.eidx + seq_e);
            for (uint32_t off = 0; off < (uint32_t)ne * 4u; off += 16384u) {
                const uint32_t bytes = (uint32_t)ne * 4u - off < 16384u ? (uint32_t)ne * 4u - off : 16384u;
                tma_load_1d(smem_u32((char*)sm.es + off), g_es + off, bytes, smem_u32(&rows_bar));
            }
            for (uint32_t off = 0; off < (uint32_t)ne; off += 16384u) {
                const uint32_t bytes = (uint32_t)ne - off < 16384u ? (uint32_t)ne - off : 16384u;
                tma_load_1d(smem_u32((char*)sm.ei + off), g_ei + off, bytes, smem_u32(&rows_bar));
            }
        }
    } else {
        for (int i = tid; i < ne; i += TREE_THREADS) {
            sm.es[i] = p.esort[seq_e + i];
            sm.ei[i] = p.eidx[seq_e + i];
        }
    }
    if (p_lazy) {  // the candidates of every depth, for the rows that may have to be scored here
        if (tid < L * K) {
            sm.tokid[tid] = lz_tok;
            sm.lpv[tid] = lz_lp;
        }
        if (rows_pre == 0) {  // the table rows of depth 0 arrive while the budget is worked out
            __syncthreads();
            lazy_issue_gather(p, sm, 0, root, tid, K, p_m);
            inflight = 0;
        }
    }
    // a sequence whose tree will run deep had its deeper rows scored by the edge-score kernel as well (they are needed
    // several levels from here: plain loads, consumed after many barriers)
    if (p.rows_adaptive && deep_tree_decide(lp_top, L)) {  // (uniform)
        for (int i = ne + tid; i < L * K * K; i += TREE_THREADS) {
            sm.es[i] = p.esort[seq_e + i];
            sm.ei[i] = p.eidx[seq_e + i];
        }
        rows_done = L;
    }
    // adjacent-position cosines r_d = cos(h_d, h_{d+1}) (Eq. 15): written by the vocab pass
    if (!FAST && p.use_saba && !p.saba_pre && tid < L - 1) sm.cosv[tid] = p.cos_pre[(size_t)b * L + tid];
    __syncthreads();
    // While warp 0 works out the budget, the other warps expand levels 0 and 1 in full (1 + K + K^2 nodes), which
    // needs no budget: with fewer than B nodes in the table every child is appended anyway, and if B is smaller
    // than that the extra nodes only fall below the threshold found afterwards.
    const bool spec = bulk && rows_pre >= 2 && L >= 2 && 1 + K + K * K <= ncap;
    if (spec && warp >= 1) {
        mbar_wait_bounded(smem_u32(&rows_bar), 0, &rows_abort);
        const int t1 = tid - 32, nth = TREE_THREADS - 32;
        if (t1 == 0) {
            sm.nkey[0] = 0xFFFFFFFFu;
            sm.nS[0] = 0.0f;
            sm.ninfo[0] = 0u;
        }
        if (t1 < K) {  // level 0: the root's children, row (depth 0, parent rank 0); a child's slot is its rank
            const float sc = 0.0f + sm.es[t1];
            const int c = sm.ei[t1];
            sm.nkey[1 + c] = ord_from_float(sc);
            sm.nS[1 + c] = sc;
            sm.ninfo[1 + c] = 0u | ((uint32_t)c << 13) | (1u << 18) | ((uint32_t)t1 << 24);
        }
        named_bar_sync(1, nth);
        for (int j = t1; j < K * K; j += nth) {  // level 1
            const int xi = j / K, r = j - xi * K, x = 1 + xi;
            const uint32_t kx = sm.nkey[x];
            const int cx = (int)((sm.ninfo[x] >> 13) & 31u), row = (K + cx) * K;
            const float sc = sm.nS[x] + sm.es[row + es_col(r, cx, K)];
            const uint32_t oc = ord_from_float(sc);
            const int c = sm.ei[row + r], at = 1 + K + xi * K + c;
            sm.nkey[at] = oc < kx ? oc : kx;
            sm.nS[at] = sc;
            sm.ninfo[at] = (uint32_t)x | ((uint32_t)c << 13) | (2u << 18) | ((uint32_t)r << 24);
        }
    }
    if (warp == 0) {  // status and budget: from the edge-score kernel if it ran ahead, else worked out here
        SabaResult r;
        if (FAST || p.saba_pre)
            r = pre_r;  // (lane 0's copy is the one used below)
        else
            r = saba_warp(p.saba, p.bmin, p.bmax, p.bstep, L, K, p.row_status + (size_t)b * L, p.vp_err,
                          p.topk_lp + (size_t)b * L * K, sm.cosv, p.hist + b, p.prefix_len + b,
                          p.use_saba ? nullptr : p.fixed_budget + b, lane);
        if (lane == 0) {
            sm.scal[0] = r.budget;
            sm.scal[2] = r.status;
            if (o.d_state) {
                for (int i = 0; i < 4; ++i) o.d_state[(size_t)b * 4 + i] = r.state[i];
            }
        }
    }
    __syncthreads();
    if (bulk) {
        // bounded wait for the bulk copies; on a timeout the sequence is reported through its status word
        if (!mbar_wait_bounded(smem_u32(&rows_bar), 0, &rows_abort) && tid == 0) sm.scal[2] |= GRAFT_ST_INTERNAL;
        __syncthreads();
    }

    // ---- best-first expansion ------------------------------------------------------------------------------
    // Best-first expansion selects prefixes in non-increasing order of their bottleneck key (the minimum path
    // score along the prefix), so after B selections the tree is the set of prefixes with key above the B-th
    // largest key theta, plus some of those with key == theta.  Phase 1 (whole CTA) finds theta and the set
    // {key > theta} level by level: the alive nodes of depth d append their children that can still matter
    // (key >= current theta; a prefix of the parent's sorted row), then theta becomes the B-th largest key seen
    // so far (radix select).  Phase 2 (one warp) continues the exact sequential expansion from that state for
    // the few remaining selections among equal keys.  If the node table overflows, phase 2 does everything.
    const int budget = sm.scal[0];
    int n_gt = 0;  // selected so far (root excluded)
    if (tid == 0) {
        sm.nkey[0] = 0xFFFFFFFFu;
        sm.nS[0] = 0.0f;
        sm.ninfo[0] = 0u;
        sm.parent[0] = -1;
        sm.cand[0] = 0;
        sm.depth[0] = 0;
        sm.S[0] = 0.0f;
    }
    __syncthreads();
    bool table_ok = budget > 0;
    // ordered: the parallel phase selected the whole tree, and its nodes stand in level order already (no sequential
    // tail, no placement): true unless several keys tie with the B-th largest or the node table overflowed
    bool ordered = false;
    int n_reach = -1;  // keys that reach the final theta, if the search that found it counted them
    uint32_t theta = 0u;
    // (TIES instances) th_depth: the depth of the deepest node whose key theta counts -- at least B keys of nodes that
    // deep or shallower reach theta.  A child deeper than that whose own path score equals theta exactly stands behind
    // all of them in best-first's order of equal keys (its score is no higher than any of theirs and it is deeper; each
    // of them becomes available before it could be taken, since their ancestors stand before it too): it can never be
    // selected and is not appended.  theta is moved up to an actual key after every search so that the equality is met
    // where it matters: when hundreds of prefixes tie at theta and their best children (probability 1) tie there as
    // well, level after level, until the table overflows.
    int th_depth = 99;
    if (budget > 0) {
        int ntot = 1, n_at_select = 1;
        SelBucket sel;
        sel.valid = false;
        float sel_top = 0.0f;  // the best score (the root's best child): where the bins of the threshold searches start
        if (spec) {  // levels 0 and 1 are in the table already: the threshold they give, then on from level 2
            ntot = 1 + K + K * K;
            if (ntot - 1 >= budget) {
                sel_top = 0.0f + sm.es[0];  // the root's best child
                // The threshold of levels 0 and 1 alone is loose: the best child of every level-1 node is a prefix too, and
                // its key costs one look at the node's sorted row.  Those K^2 keys stand behind the table for the search
                // (the level's real children overwrite them), which then gives a bound closer to the final one and a
                // level 2 that appends a third of what it would.
                int nsel = ntot;
                if (L > 2 && rows_done > 2 && ntot + K * K <= ncap) {  // (uniform)
                    for (int j = tid; j < K * K; j += TREE_THREADS) {
                        const int x = 1 + K + j;
                        const uint32_t kx = sm.nkey[x];
                        const int cx = (int)((sm.ninfo[x] >> 13) & 31u);
                        const uint32_t oc = ord_from_float(sm.nS[x] + sm.es[(2 * K + cx) * K + cx]);  // (entry 0: column cx)
                        sm.nkey[ntot + j] = oc < kx ? oc : kx;
                    }
                    nsel = ntot + K * K;
                    __syncthreads();
                }
                theta = cta_select_bucket(sm, sm.nkey, 1, nsel, budget, sel_top, sel, tid);
                if (TIES) {
                    __syncthreads();
                    theta = cta_snap_to_key(sm.nkey, 1, nsel, theta, sm.hist + 1100, tid);
                    th_depth = nsel != ntot ? 3 : 2;
                }
                if (nsel != ntot) sel.valid = false;  // (the bucket counts keys that are not in the table)
                n_at_select = ntot;
            }
            __syncthreads();
        }
        // (the bounds of the level being expanded and the end of the table are the same in every thread: no thread has to
        // publish them, and a level costs three barriers -- two in the scan, one at its end)
        int lv0 = spec ? 1 + K : 0, lv1 = spec ? 1 + K + K * K : 1;
        for (int d = spec ? 2 : 0; d < L; ++d) {
            const int b0 = lv0, b1 = lv1;
            if (b1 == b0) break;
            int lvl_end = ntot;
            bool over = false;  // the node table is full
            if (d >= rows_done) {  // the edge rows of this depth: scored now, never if the expansion stops above it
                int alive = 0;  // (nor if no node of the level can still have a selected child)
                for (int x = b0 + tid; x < b1; x += TREE_THREADS) alive |= sm.nkey[x] >= theta ? 1 : 0;
                if (!__syncthreads_or(alive)) break;
                lazy_score_row(p, sm, d, root, tid, inflight, K, p_m);
                rows_done = d + 1;
            }
            // grow: can a node appended here have a child that reaches theta?  (Its best child stands first in its sorted
            // row.)  If none can, the next level would append nothing: the loop ends here instead of finding that out
            // with a whole pass.  theta only rises, so "cannot now" stays true.
            int grow = 0;
            if (theta == 0u) {
                grow = d + 1 < L ? 1 : 0;
                // no threshold yet (fewer than B nodes so far): every child of every node of the level is appended,
                // one thread per (node, child), at a position that needs no atomic
                const int total = (b1 - b0) * K;
                if (ntot + total > ncap) {
                    over = true;
                } else {
                    for (int j = tid; j < total; j += TREE_THREADS) {
                        const int xi = j / K, r = j - xi * K, x = b0 + xi;
                        const uint32_t kx = sm.nkey[x];
                        const int cx = (int)((sm.ninfo[x] >> 13) & 31u), row = (d * K + cx) * K;
                        const float sc = sm.nS[x] + sm.es[row + es_col(r, cx, K)];
                        const uint32_t oc = ord_from_float(sc);
                        const int c = sm.ei[row + r], at = ntot + xi * K + c;  // (a full row: a child's slot is its rank)
                        sm.nkey[at] = oc < kx ? oc : kx;
                        sm.nS[at] = sc;
                        sm.ninfo[at] = (uint32_t)x | ((uint32_t)c << 13) | ((uint32_t)(d + 1) << 18) | ((uint32_t)r << 24);
                    }
                    lvl_end = ntot + total;
                }
            } else {
                // The children that can still matter are a prefix of a node's sorted row (scores only fall along the
                // row); its length comes from a binary search.  The level is taken in chunks of 1024 nodes: one thread
                // per node finds the length and the set of candidate ranks in that prefix, a scan of the lengths places
                // the chunk's children in the table in the order of the nodes, then one thread per child (its node found
                // in the scan by binary search) writes it, behind its siblings of lower rank.  No shared counter, a node
                // with many children holds nobody up, and the table stays in level order.
                int cur = ntot;
                int* pre = (int*)sm.hist;            // [1024] inclusive scan of the chunk, then [32] warp totals
                uint32_t* cmask = sm.hist + 1100;    // [1024] candidate ranks of the children a node appends
                // At most B nodes of a level end up in the tree: a chunk that would append many times more children than
                // that (or more than the table has room for) first raises theta to (a lower bound of) the B-th largest
                // key among those children.  (The search costs about as much as two ordinary levels: ordinary rounds,
                // whose levels stay within a few times B, never run it.)
                const int flood = 8 * budget > 1024 ? 8 * budget : 1024;
                for (int c0 = b0; c0 < b1; c0 += TREE_THREADS) {  // (uniform)
                  const int x = c0 + tid;
                  int total = 0;
                  for (int attempt = 0;; ++attempt) {  // (uniform: at most two rounds)
                    const uint32_t th_in = theta + ((TIES && d + 1 > th_depth) ? 1u : 0u);  // what a child's score must reach
                    int cnt = 0;
                    uint32_t mask = 0u, kx = 0u;
                    float sx = 0.0f;
                    int row = 0, cx = 0;
                    if (x < b1) {
                        kx = sm.nkey[x];
                        if (kx >= theta) {  // (else dead: none of its descendants can be selected)
                            cx = (int)((sm.ninfo[x] >> 13) & 31u);
                            row = (d * K + cx) * K;
                            sx = sm.nS[x];
                            int lo_r = 0, hi_r = K;  // first r in [0, K] whose key falls below theta
                            while (lo_r < hi_r) {
                                const int mid = (lo_r + hi_r) >> 1;
                                const uint32_t oc = ord_from_float(sx + sm.es[row + es_col(mid, cx, K)]);
                                if (oc >= th_in)  // (kx >= theta already: the child's key min(kx, oc) reaches theta iff oc does)
                                    lo_r = mid + 1;
                                else
                                    hi_r = mid;
                            }
                            cnt = lo_r;
                            // the candidate ranks of the first cnt entries, four at a time where the rows are whole words;
                            // a long prefix is taken as all ranks less those of the entries behind it
                            const bool tail = 2 * cnt > K;
                            const int r_lo = tail ? cnt : 0, r_hi = tail ? K : cnt;
                            if ((K & 3) == 0) {
                                const uint32_t* eiw = (const uint32_t*)(sm.ei + row);
                                for (int r0 = r_lo & ~3; r0 < r_hi; r0 += 4) {
                                    const uint32_t q = eiw[r0 >> 2];
                                    if (r0 >= r_lo) mask |= 1u << (q & 31u);
                                    if (r0 + 1 >= r_lo && r0 + 1 < r_hi) mask |= 1u << ((q >> 8) & 31u);
                                    if (r0 + 2 >= r_lo && r0 + 2 < r_hi) mask |= 1u << ((q >> 16) & 31u);
                                    if (r0 + 3 >= r_lo && r0 + 3 < r_hi) mask |= 1u << ((q >> 24) & 31u);
                                }
                            } else {
                                for (int r = r_lo; r < r_hi; ++r) mask |= 1u << sm.ei[row + r];
                            }
                            if (tail) mask = (K == 32 ? 0xFFFFFFFFu : (1u << K) - 1u) & ~mask;
                        }
                    }
                    cmask[tid] = mask;
                    int incl = cnt;
#pragma unroll
                    for (int o2 = 1; o2 < 32; o2 <<= 1) {
                        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o2);
                        if (lane >= o2) incl += t;
                    }
                    if (lane == 31) pre[TREE_THREADS + warp] = incl;
                    __syncthreads();
                    const int wt = pre[TREE_THREADS + lane];
                    int wincl = wt;
#pragma unroll
                    for (int o2 = 1; o2 < 32; o2 <<= 1) {
                        const int t = __shfl_up_sync(0xFFFFFFFFu, wincl, o2);
                        if (lane >= o2) wincl += t;
                    }
                    total = __shfl_sync(0xFFFFFFFFu, wincl, 31);
                    pre[tid] = __shfl_sync(0xFFFFFFFFu, wincl - wt, warp) + incl;
                    __syncthreads();
                    if (attempt == 0 && total >= budget && (total > flood || cur + total > ncap)) {  // (uniform) the search below uses the scan's space: count again
                        const uint32_t tl = cta_kth_largest_of_children(sm, cnt, kx, sx, row, cx, K, budget, theta, tid);
                        theta = tl > theta ? tl : theta;
                        if (TIES) th_depth = d + 1;
                        continue;
                    }
                    break;
                  }
                    if (cur + total > ncap) {  // (uniform)
                        over = true;
                        break;
                    }
                    for (int i = tid; i < total; i += TREE_THREADS) {
                        int lo_t = 0, hi_t = TREE_THREADS - 1;  // owner: the first thread whose scan exceeds i
                        while (lo_t < hi_t) {
                            const int mid = (lo_t + hi_t) >> 1;
                            if (pre[mid] > i)
                                hi_t = mid;
                            else
                                lo_t = mid + 1;
                        }
                        const int first = lo_t ? pre[lo_t - 1] : 0;
                        const int r = i - first, xo = c0 + lo_t;
                        const uint32_t kx = sm.nkey[xo];
                        const int co = (int)((sm.ninfo[xo] >> 13) & 31u), row = (d * K + co) * K;
                        const float sc = sm.nS[xo] + sm.es[row + es_col(r, co, K)];
                        const uint32_t oc = ord_from_float(sc);
                        const int c = sm.ei[row + r];
                        const int at = cur + first + __popc(cmask[lo_t] & ((1u << c) - 1u));
                        if (d + 1 < L) {
                            if (d + 1 < rows_done) {
                                const uint32_t ob = ord_from_float(sc + sm.es[((d + 1) * K + c) * K + c]);  // (entry 0: column c)
                                grow |= (ob >= theta && oc >= theta) ? 1 : 0;
                            } else {
                                grow = 1;  // (that row is not scored yet)
                            }
                        }
                        sm.nkey[at] = oc < kx ? oc : kx;
                        sm.nS[at] = sc;
                        sm.ninfo[at] = (uint32_t)xo | ((uint32_t)c << 13) | ((uint32_t)(d + 1) << 18) | ((uint32_t)r << 24);
                    }
                    cur += total;
                    if (c0 + TREE_THREADS < b1) __syncthreads();  // the scan space is reused by the next chunk
                }
                lvl_end = cur;
            }
            const int any_grow = __syncthreads_or(grow);  // (the level's nodes are in the table for every thread)
            const int nt = lvl_end;
            if (over) {
                table_ok = false;
                break;
            }
            if (nt == ntot) break;  // nothing appended: no deeper level
            lv0 = ntot;
            lv1 = nt;
            ntot = nt;
            if (!any_grow) break;  // no node of the new level can have a child in the tree
            // theta only has to be a lower bound of its final value while the levels are built (it prunes), so
            // the exact B-th largest key is recomputed only when the table has grown noticeably
            if (ntot - 1 >= budget && (theta == 0u || ntot - n_at_select >= ntot / 8)) {
                sel_top = 0.0f + sm.es[0];  // the root's best child
                theta = cta_select_bucket(sm, sm.nkey, 1, ntot, budget, sel_top, sel, tid);  // a lower bound
                if (TIES) {
                    __syncthreads();
                    theta = cta_snap_to_key(sm.nkey, 1, ntot, theta, sm.hist + 1100, tid);
                    th_depth = d + 1;
                }
                n_at_select = ntot;
                __syncthreads();  // (its bins share the space of the next level's scan)
            }
        }
        __syncthreads();
        if (table_ok && ntot - 1 >= budget) {
            // the exact value: the last 16-bit search still holds if nothing was appended after it
            if (!(n_at_select == ntot && sel.valid)) {
                sel_top = 0.0f + sm.es[0];  // the root's best child
                cta_select_bucket(sm, sm.nkey, 1, ntot, budget, sel_top, sel, tid);
            }
            theta = cta_finish_select(sm, sm.nkey, 1, ntot, budget, sel_top, sel, tid, &n_reach);
        }
        __syncthreads();
        if (table_ok) {
            const int per = (ntot + TREE_THREADS - 1) / TREE_THREADS;
            const int i0 = tid * per < ntot ? tid * per : ntot, i1 = i0 + per < ntot ? i0 + per : ntot;
            // The tree is {key > theta} plus some of the keys equal to theta.  If exactly B keys reach theta (no other
            // key ties with the B-th largest: the usual case), {key >= theta} is the whole tree; so is the table itself
            // when it holds fewer than B nodes (theta = 0: every prefix there is has been appended).
            uint32_t cut = theta;  // nodes with key > cut are taken here
            if (theta != 0u) {
                if (n_reach < 0) {  // (uniform) the radix search does not count them: one pass over the table
                    int ge = 0;
                    for (int i = i0 > 1 ? i0 : 1; i < i1; ++i) ge += sm.nkey[i] >= theta ? 1 : 0;
                    ge = __reduce_add_sync(0xFFFFFFFFu, ge);
                    if (tid == 0) sm.scal[8] = 0;
                    __syncthreads();
                    if (lane == 0 && ge) atomicAdd(&sm.scal[8], ge);
                    __syncthreads();
                    n_reach = sm.scal[8];
                }
                if (n_reach == budget) {  // (uniform)
                    cut = theta - 1u;
                    ordered = true;
                } else if (n_reach > budget) {  // (uniform)
                    // A few keys tie with the B-th largest.  Best-first takes prefixes of equal path score in the order
                    // (shallower first, then the parent's place in its level, then the place in the parent's sorted row),
                    // and a prefix only after its parent; among the tied nodes -- all in the table -- that is a short
                    // simulation by one warp, a lane per tied node (up to 32 of them; more go to the sequential
                    // expansion below).  The nodes it takes get a key above theta, and the tree is again a subset of the
                    // table in table order.
                    int* tlist = (int*)sm.hist;  // [32] table indices of the tied nodes, [32]: their number
                    if (tid == 0) tlist[32] = 0;
                    __syncthreads();
                    for (int i = i0 > 1 ? i0 : 1; i < i1; ++i) {
                        if (sm.nkey[i] == theta) {
                            const int pos = atomicAdd(&tlist[32], 1);
                            if (pos < 32) tlist[pos] = i;
                        }
                    }
                    __syncthreads();
                    const int nt = tlist[32];
                    if (nt <= 32) {  // (uniform)
                        if (warp == 0) {
                            const int want = budget - (n_reach - nt);  // how many of the tied nodes belong to the tree
                            const int me = lane < nt ? tlist[lane] : 0;
                            const uint32_t info = lane < nt ? sm.ninfo[me] : 0u;
                            const int par = (int)(info & 8191u);
                            const uint32_t hi = lane < nt ? ord_from_float(sm.nS[me]) : 0u;
                            const uint32_t lo = ((63u - ((info >> 18) & 63u)) << 18) | ((8191u - (uint32_t)par) << 5) |
                                                (31u - ((info >> 24) & 31u));
                            bool avail = lane < nt && sm.nkey[par] > theta;  // (else the parent is a tied node itself)
                            bool picked = false;
                            for (int step = 0; step < want; ++step) {
                                const uint32_t bh = __reduce_max_sync(0xFFFFFFFFu, avail && !picked ? hi : 0u);
                                const uint32_t bl = __reduce_max_sync(0xFFFFFFFFu, avail && !picked && hi == bh ? lo + 1u : 0u);
                                if (bl == 0u) break;  // (nothing to take: cannot happen while want <= nt)
                                const bool mine = avail && !picked && hi == bh && lo + 1u == bl;
                                const int taken = __shfl_sync(0xFFFFFFFFu, me, __ffs(__ballot_sync(0xFFFFFFFFu, mine)) - 1);
                                if (mine) picked = true;
                                if (lane < nt && par == taken) avail = true;
                            }
                            if (picked) sm.nkey[me] = theta + 1u;
                        }
                        __syncthreads();
                        ordered = true;
                    } else if (TIES) {
                        // Many keys tie with the B-th largest: exactly equal probabilities (flat or one-hot rows) and no
                        // edge scores to tell them apart.  Where every tied node whose parent is tied too stands behind
                        // that parent in the order of equal keys -- path scores that do not rise along a path: always so
                        // without edge scores -- the best available tied node is always the best remaining one, so
                        // best-first takes the tied nodes in that order outright: the `want` first of them are found by
                        // a search over the bits of the order (path score, then shallower, parent's place, place in the
                        // parent's row: 56 bits, two a step with three counts each).  Otherwise: the sequential
                        // expansion below.
                        const int want = budget - (n_reach - nt);
                        int mono = 1, same = 1;  // same: every tied node's own path score is theta (the usual tie)
                        for (int i = i0 > 1 ? i0 : 1; i < i1; ++i) {
                            if (sm.nkey[i] != theta) continue;
                            same &= ord_from_float(sm.nS[i]) == theta ? 1 : 0;
                            const int par = (int)(sm.ninfo[i] & 8191u);
                            if (sm.nkey[par] == theta && !(tie_order(sm.nS[par], sm.ninfo[par]) > tie_order(sm.nS[i], sm.ninfo[i])))
                                mono = 0;
                        }
                        uint32_t* cnt = sm.hist + 64;  // [3 * 28] the counts of the steps
                        if (tid < 84) cnt[tid] = 0u;
                        same = __syncthreads_and(same);
                        if (__syncthreads_and(mono)) {  // (uniform)
                            // (equal path scores: the upper 32 bits of the order are known, twelve steps remain)
                            uint64_t kth = same ? (uint64_t)theta << 24 : 0ull;
#pragma unroll 1
                            for (int step = same ? 16 : 0; step < 28; ++step) {
                                const int bit = 54 - 2 * step;
                                const uint64_t t1 = kth | (1ull << bit), t2 = kth | (2ull << bit), t3 = kth | (3ull << bit);
                                int c1 = 0, c2 = 0, c3 = 0;
                                for (int i = i0 > 1 ? i0 : 1; i < i1; ++i) {
                                    if (sm.nkey[i] != theta) continue;
                                    const uint64_t o = tie_order(sm.nS[i], sm.ninfo[i]);
                                    c1 += (o >= t1) ? 1 : 0;
                                    c2 += (o >= t2) ? 1 : 0;
                                    c3 += (o >= t3) ? 1 : 0;
                                }
                                c1 = __reduce_add_sync(0xFFFFFFFFu, c1);
                                c2 = __reduce_add_sync(0xFFFFFFFFu, c2);
                                c3 = __reduce_add_sync(0xFFFFFFFFu, c3);
                                if (lane == 0 && c1) {
                                    atomicAdd(&cnt[3 * step], (uint32_t)c1);
                                    atomicAdd(&cnt[3 * step + 1], (uint32_t)c2);
                                    atomicAdd(&cnt[3 * step + 2], (uint32_t)c3);
                                }
                                __syncthreads();
                                const int n1 = (int)cnt[3 * step], n2 = (int)cnt[3 * step + 1], n3 = (int)cnt[3 * step + 2];
                                kth = n3 >= want ? t3 : (n2 >= want ? t2 : (n1 >= want ? t1 : kth));
                            }
                            for (int i = i0 > 1 ? i0 : 1; i < i1; ++i)
                                if (sm.nkey[i] == theta && tie_order(sm.nS[i], sm.ninfo[i]) >= kth) sm.nkey[i] = theta + 1u;
                            __syncthreads();
                            ordered = true;
                        }
                    }
                }
            } else if (ntot - 1 < budget) {
                ordered = true;  // fewer prefixes than the budget: all of them
            }
            int cnt = 0;
            for (int i = i0; i < i1; ++i) cnt += (i == 0 || sm.nkey[i] > cut) ? 1 : 0;
            int incl = cnt;
#pragma unroll
            for (int o2 = 1; o2 < 32; o2 <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o2);
                if (lane >= o2) incl += t;
            }
            if (lane == 31) sm.hist[warp] = (uint32_t)incl;
            __syncthreads();
            const int wt = (int)sm.hist[lane];  // (32 warps: a lane per warp total)
            int wincl = wt;
#pragma unroll
            for (int o2 = 1; o2 < 32; o2 <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, wincl, o2);
                if (lane >= o2) wincl += t;
            }
            const int woff = __shfl_sync(0xFFFFFFFFu, wincl - wt, warp);
            const int total = __shfl_sync(0xFFFFFFFFu, wincl, 31);
            int run = woff + incl - cnt;
            __syncthreads();
            for (int i = i0; i < i1; ++i) {
                const bool sel = (i == 0 || sm.nkey[i] > cut);
                sm.nkey[i] = sel ? (uint32_t)run : 0xFFFFFFFFu;  // the key is no longer needed: keep the compact index
                run += sel ? 1 : 0;
            }
            __syncthreads();
            for (int i = i0; i < i1; ++i) {
                const uint32_t n = sm.nkey[i];
                if (n == 0xFFFFFFFFu || i == 0) continue;
                const uint32_t info = sm.ninfo[i];
                sm.parent[n] = (int16_t)sm.nkey[info & 8191u];
                sm.cand[n] = (uint8_t)((info >> 13) & 31u);
                sm.depth[n] = (uint8_t)((info >> 18) & 63u);
                sm.S[n] = sm.nS[i];
            }
            n_gt = total - 1;
            __syncthreads();
            // (for the sequential tail only) frontier entries of the selected nodes: the first child of the sorted row
            // that is not selected, i.e. the first with ord(score) <= theta
            for (int n = tid; n <= n_gt && !ordered; n += TREE_THREADS) {
                const int d = sm.depth[n];
                uint64_t e = 0ull;
                if (d < L) {
                    const int row = (d * K + sm.cand[n]) * K;
                    const float sn = sm.S[n];
                    int pos = 0, hi_p = K;  // first entry of the (ordered) row whose key is not above theta
                    while (pos < hi_p) {
                        const int mid = (pos + hi_p) >> 1;
                        if (ord_from_float(sn + sm.es[row + es_col(mid, sm.cand[n], K)]) > theta)
                            pos = mid + 1;
                        else
                            hi_p = mid;
                    }
                    if (pos < K) e = pack_entry(sn + sm.es[row + es_col(pos, sm.cand[n], K)], d + 1, pos, sm.cand[n], sm.ei[row + pos]);
                }
                sm.ent[n] = e;
            }
        }
    }
    if (p_lazy && !table_ok && budget > 0) {  // the sequential fall-back may reach any depth
        for (; rows_done < L; ++rows_done) lazy_score_row(p, sm, rows_done, root, tid, inflight, K, p_m);
    }
    if (!table_ok && tid == 0) sm.ent[0] = budget > 0 ? pack_entry(0.0f + sm.es[0], 1, 0, 0, sm.ei[0]) : 0ull;
    if (ordered) {  // (uniform) the tree is complete and in level order
        if (tid == 0) {
            sm.scal[1] = n_gt + 1;
            if (n_gt < budget) sm.scal[2] |= GRAFT_ST_FRONTIER_EMPTY;
        }
    } else {
    // emission needs every node's child mask and the node count of every level: cleared here, filled for the nodes
    // selected so far by warps 1..31 while warp 0 runs the sequential tail, and for the tail's nodes by warp 0
    if (tid < kMaxL + 2) {
        sm.lvl_count[tid] = 0;
        sm.lvl_fill[tid] = 0;
    }
    for (int n = tid; n < nmax; n += TREE_THREADS) sm.chmask[n] = 0u;
    __syncthreads();
    const int n_pre = table_ok ? n_gt : 0;  // nodes 0..n_pre are final before the tail starts
    if (warp >= 1) {
        for (int n = tid - 32; n <= n_pre; n += TREE_THREADS - 32) {
            if (n > 0) atomicOr(&sm.chmask[sm.parent[n]], 1u << sm.cand[n]);
            atomicAdd(&sm.lvl_count[sm.depth[n]], 1);
        }
    }
    if (warp == 0) {
        // Phase 2: exact sequential expansion.  Every step scans all frontier entries (one per selected node)
        // for the best under the full order, including the lexicographic rule for equal scores.
        int st = sm.scal[2];
        int n_sel = table_ok ? n_gt : 0;
        while (n_sel < budget) {
            uint64_t be = 0ull;
            int bn = -1;
            for (int n = lane; n <= n_sel; n += 32) {
                const uint64_t e = sm.ent[n];
                if (e != 0ull && entry_before(sm, e, n, be, bn)) {
                    be = e;
                    bn = n;
                }
            }
#pragma unroll
            for (int o2 = 16; o2 > 0; o2 >>= 1) {
                const uint64_t oe = __shfl_xor_sync(0xFFFFFFFFu, be, o2);
                const int on = __shfl_xor_sync(0xFFFFFFFFu, bn, o2);
                if (entry_before(sm, oe, on, be, bn)) {
                    be = oe;
                    bn = on;
                }
            }
            if (bn < 0) {
                st |= GRAFT_ST_FRONTIER_EMPTY;
                break;
            }
            const uint32_t lo = (uint32_t)be;
            const int d = 32 - (int)((lo >> 25) & 63u), pos = (int)((lo >> 10) & 31u);
            const int cpar = (int)((lo >> 5) & 31u), c = (int)(lo & 31u);
            const float s_new = __uint_as_float(bits_from_ord((uint32_t)(be >> 32)));
            const int n_new = ++n_sel;
            if (lane == 0) {
                sm.parent[n_new] = (int16_t)bn;
                sm.cand[n_new] = (uint8_t)c;
                sm.depth[n_new] = (uint8_t)d;
                sm.S[n_new] = s_new;
                uint64_t e_adv = 0ull, e_new = 0ull;
                if (pos + 1 < K) {
                    const int at = ((d - 1) * K + cpar) * K;
                    e_adv = pack_entry(sm.S[bn] + sm.es[at + es_col(pos + 1, cpar, K)], d, pos + 1, cpar, sm.ei[at + pos + 1]);
                }
                if (d < L && n_sel < budget) {  // (after the last selection the entry is never read)
                    // a node selected here has a key >= theta, so it sits in the table and the row of its depth
                    // was scored when its level was expanded
                    if (d >= rows_done) {
                        st |= GRAFT_ST_INTERNAL;
                    } else {
                        const int at = (d * K + c) * K;
                        e_new = pack_entry(s_new + sm.es[at + c], d + 1, 0, c, sm.ei[at]);  // (entry 0 stands at column c)
                    }
                }
                sm.ent[bn] = e_adv;
                sm.ent[n_new] = e_new;
            }
            __syncwarp();
        }
        for (int n = n_pre + 1 + lane; n <= n_sel; n += 32) {  // the tail's nodes
            atomicOr(&sm.chmask[sm.parent[n]], 1u << sm.cand[n]);
            atomicAdd(&sm.lvl_count[sm.depth[n]], 1);
        }
        if (lane == 0) {
            sm.scal[1] = n_sel + 1;
            sm.scal[2] = st;
        }
    }
    }  // !ordered
    if (!ordered) __syncthreads();  // (uniform; an ordered tree needs nothing from the block above)

    // ---- emission in level order -------------------------------------------------------------------------
    // Level order = depth ascending, then the parent's level-order index, then candidate rank.  Level by level:
    // the child counts of level d-1, laid out in level order, are scanned; a node of level d lands at
    // (start of level d) + (children of earlier parents) + (selected siblings of lower rank).
    // The placement is a chain of short steps over at most nmax nodes: one warp runs it with warp-level
    // synchronisation only (a barrier of the whole CTA per step cost more than the steps), while the other warps
    // write the padding of the outputs, which depends on the node count alone.
    const int n_nodes = ordered ? n_gt + 1 : sm.scal[1];
    const int prefix = p.prefix_len[b];
    const size_t ob = (size_t)b * nmax;
    if (warp == 0 && !ordered) {
        // starts of the levels 0..L: an exclusive scan of the counts (L <= 32: lane = level, and one more)
        {
            const int c0 = lane <= L ? sm.lvl_count[lane] : 0;
            int incl = c0;
#pragma unroll
            for (int o2 = 1; o2 < 32; o2 <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o2);
                if (lane >= o2) incl += t;
            }
            if (lane <= L) sm.lvl_start[lane] = incl - c0;
            const int below32 = __shfl_sync(0xFFFFFFFFu, incl, 31);
            if (lane == 0 && L == 32) sm.lvl_start[32] = below32;
            if (lane == 0) {
                sm.canon[0] = 0;
                // cc holds the child counts of the previous level in level order; it is double-buffered (two halves
                // of nmax entries) so that a level's nodes leave their own counts for the next level as they are placed
                sm.cc[0] = (int16_t)__popc(sm.chmask[0]);
            }
        }
        __syncwarp();
        for (int n = lane; n < n_nodes; n += 32) {  // the nodes of every level, in no particular order
            const int d = sm.depth[n];
            sm.lvl_list[sm.lvl_start[d] + atomicAdd(&sm.lvl_fill[d], 1)] = (int16_t)n;
        }
        __syncwarp();
        for (int d = 1; d <= L; ++d) {
            const int s_prev = sm.lvl_start[d - 1], n_prev = sm.lvl_count[d - 1];
            const int s_cur = sm.lvl_start[d], n_cur = sm.lvl_count[d];
            if (n_cur == 0) break;  // deeper levels are empty too
            int16_t* ccp = sm.cc + ((d - 1) & 1) * nmax;
            int16_t* ccn = sm.cc + (d & 1) * nmax;
            int carry = 0;  // exclusive scan of ccp[0..n_prev), 32 entries at a time
            for (int base = 0; base < n_prev; base += 32) {
                const int i = base + lane;
                const int v = i < n_prev ? ccp[i] : 0;
                int incl = v;
#pragma unroll
                for (int o2 = 1; o2 < 32; o2 <<= 1) {
                    const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o2);
                    if (lane >= o2) incl += t;
                }
                if (i < n_prev) ccp[i] = (int16_t)(carry + incl - v);
                carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
            }
            __syncwarp();
            for (int i = lane; i < n_cur; i += 32) {
                const int x = sm.lvl_list[s_cur + i];
                const int y = sm.parent[x];
                const int at = s_cur + ccp[sm.canon[y] - s_prev] + __popc(sm.chmask[y] & ((1u << sm.cand[x]) - 1u));
                sm.canon[x] = (int16_t)at;
                ccn[at - s_cur] = (int16_t)__popc(sm.chmask[x]);
            }
            __syncwarp();
        }
    } else if (warp != 0) {
        for (int i = n_nodes + tid - 32; i < nmax; i += TREE_THREADS - 32) {
            o.d_token[ob + i] = -1;
            o.d_parent[ob + i] = -1;
            o.d_depth[ob + i] = -1;
            o.d_position[ob + i] = -1;
            o.d_path_score[ob + i] = 0.f;
        }
        // mask rows from the first multiple of 32 at or above n_nodes on are all padding
        const int z0 = ((n_nodes + 31) / 32) * 32;
        for (size_t k = (size_t)z0 * W + tid - 32; k < (size_t)nmax * W; k += TREE_THREADS - 32) o.d_mask[ob * W + k] = 0u;
    }
    if (!ordered) __syncthreads();  // (the placement above; the padding is nobody's input)
    for (int n = tid; n < n_nodes; n += TREE_THREADS) {
        const int i = ordered ? n : sm.canon[n], d = sm.depth[n];
        const int par = n == 0 ? -1 : (ordered ? sm.parent[n] : sm.canon[sm.parent[n]]);
        sm.cparent[i] = (int16_t)par;
        o.d_token[ob + i] = n == 0 ? root
                                   : (p_lazy ? sm.tokid[(d - 1) * K + sm.cand[n]]  // (staged in the prologue)
                                             : p.topk_id[((size_t)b * L + d - 1) * K + sm.cand[n]]);
        o.d_parent[ob + i] = par;
        o.d_depth[ob + i] = d;
        o.d_position[ob + i] = prefix - 1 + d;
        o.d_path_score[ob + i] = sm.S[n];
    }
    __syncthreads();
    // ancestor masks: each thread builds one row in its warp's staging tile; the warp then stores its 32 rows,
    // which are contiguous in the output, with coalesced writes.  Padding rows are zero-filled directly.
    {
        const size_t stage_off = (((size_t)nmax * 2 + 15) & ~(size_t)15) + (((size_t)nmax * 4 + 15) & ~(size_t)15);
        const size_t region = (size_t)ncap * 12 > stage_off + (size_t)8 * 32 * W * 4 ? (size_t)ncap * 12
                                                                                         : stage_off + (size_t)8 * 32 * W * 4;
        int mw = (int)((region - stage_off) / ((size_t)32 * W * 4));
        mw = mw > TREE_THREADS / 32 ? TREE_THREADS / 32 : mw;
        uint32_t* tile = sm.stage + (size_t)warp * 32 * W;
        for (int i0 = warp * 32; i0 < n_nodes && warp < mw; i0 += mw * 32) {
            const int i = i0 + lane;
            uint32_t* row = tile + lane * W;
            // the tile is cleared by the warp together, then a lane sets the bits of its node's ancestors (itself included)
            for (int k = lane; k < 32 * W; k += 32) tile[k] = 0u;
            __syncwarp();
            if (i < n_nodes) {
                int steps = 0;  // a node has at most L ancestors: the bound keeps the walk finite whatever the arrays hold
                for (int a = i; a >= 0 && a < nmax && steps <= L; a = sm.cparent[a], ++steps) row[a >> 5] |= 1u << (a & 31);
            }
            __syncwarp();
            const int rows = min(32, nmax - i0);
            uint32_t* dst = o.d_mask + (ob + i0) * W;
            for (int k = lane; k < rows * W; k += 32) dst[k] = tile[k];
            __syncwarp();
        }
    }
    if (p_lazy) cp_async_wait_all();  // table rows fetched ahead for a depth that was never scored
    if (tid == 0) {
        o.d_n_nodes[b] = n_nodes;
        o.d_budget[b] = sm.scal[0];
        o.d_status[b] = sm.scal[2] | (rows_abort ? GRAFT_ST_INTERNAL : 0);
    }
}

// ---- acceptance walk: one CTA per sequence ---------------------------------------------------------------------
// The tree (parents, tokens) and the target's next tokens are staged in shared memory by 128 threads with all
// loads in flight together; warp 0 then walks out of shared memory.  In level order the parent indices never
// decrease, so the children of the current node are found by a binary search for the first node whose parent
// is >= it.
struct AcceptParams {
    const int32_t* n_nodes;
    const int32_t* token;
    const int32_t* parent;
    const int32_t* target_next;
    int batch, nmax, L;
    int32_t* accept_len;
    int32_t* accept_path;
    int32_t* bonus;
    // acceptance history (Eq. 15), updated here when hist_w > 0
    int hist_w;
    int32_t* hist_window;
    int32_t* hist_count;
    float* hist_out;
};

__global__ void __launch_bounds__(128) accept_kernel(const AcceptParams ap) {
    const int32_t* __restrict__ n_nodes = ap.n_nodes;
    const int32_t* __restrict__ token = ap.token;
    const int32_t* __restrict__ parent = ap.parent;
    const int32_t* __restrict__ target_next = ap.target_next;
    const int nmax = ap.nmax, L = ap.L;
    int32_t* __restrict__ accept_len = ap.accept_len;
    int32_t* __restrict__ accept_path = ap.accept_path;
    int32_t* __restrict__ bonus = ap.bonus;
    pdl_launch_dependents();  // the next round's vocab pass may set up its CTAs; it waits for this grid before it reads
    pdl_wait();  // the tree may come from a tree kernel that is still running ahead in the stream
    extern __shared__ __align__(16) int32_t acc_smem[];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    int32_t* par = acc_smem;
    int32_t* tok = par + nmax;
    int32_t* tn = tok + nmax;
    const size_t ob = (size_t)b * nmax;
    // every slot of the three arrays is staged, padding included, so that these loads do not wait for the node count
    // (one round trip to global memory instead of two); the walk below never looks beyond the count
    int nn = n_nodes[b];
    {
        constexpr int U = 8;  // 128 threads x 8 covers the largest tree (1024 nodes) in one round
        int32_t vp[U], vt[U], vn[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = tid + 128 * u;
            vp[u] = i < nmax ? parent[ob + i] : 0;
            vt[u] = i < nmax ? token[ob + i] : 0;
            vn[u] = i < nmax ? target_next[ob + i] : 0;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = tid + 128 * u;
            if (i < nmax) {
                par[i] = vp[u];
                tok[i] = vt[u];
                tn[i] = vn[u];
            }
        }
    }
    nn = nn < 1 ? 1 : (nn > nmax ? nmax : nn);
    __syncthreads();
    if (tid >= 32) return;
    int cur = 0, a = 0;
    while (a < L) {
        const int want = tn[cur];
        int lo = cur + 1, hi = nn;  // first index in (cur, nn) whose parent is >= cur
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (par[mid] >= cur)
                hi = mid;
            else
                lo = mid + 1;
        }
        int found = -1;
        for (int i0 = lo; i0 < nn && found < 0; i0 += 32) {  // the children of cur are contiguous from lo on
            const int i = i0 + lane;
            const bool child = i < nn && par[i] == cur;
            const uint32_t hit = __ballot_sync(0xFFFFFFFFu, child && tok[i] == want);
            const uint32_t more = __ballot_sync(0xFFFFFFFFu, child);
            if (hit) found = i0 + __ffs(hit) - 1;
            if (more != 0xFFFFFFFFu) break;  // ran past the last child
        }
        if (found < 0) break;
        if (lane == 0) accept_path[(size_t)b * L + a] = found;
        ++a;
        cur = found;
    }
    for (int i = a + lane; i < L; i += 32) accept_path[(size_t)b * L + i] = -1;
    if (lane == 0) {
        accept_len[b] = a;
        bonus[b] = tn[cur];
        if (ap.hist_w > 0) {  // hist for the next round: mean of the last min(rounds, w) accepted lengths
            const int w = ap.hist_w;
            int n = ap.hist_count[b];
            int32_t* ring = ap.hist_window + (size_t)b * w;
            ring[n % w] = a;
            n += 1;
            ap.hist_count[b] = n;
            const int cnt = n < w ? n : w;
            int sum = 0;
            for (int i = 0; i < cnt; ++i) sum += ring[i];
            ap.hist_out[b] = (float)((double)sum / (double)cnt);
        }
    }
}

}  // namespace

// Edge scores are computed inside the tree kernel when its gather buffers fit in shared memory beside the rest.
bool tree_lazy_fits(const graft_config& cfg) {
    const int nmax = cfg.budget_max + 1;
    return tree_smem_layout(cfg.L, cfg.K, nmax, 2 * nmax, cfg.m, nullptr, nullptr) <= (size_t)222 * 1024;
}

size_t tree_smem_bytes(const graft_config& cfg) {
    const int nmax = cfg.budget_max + 1;
    const int lazy_m = tree_lazy_fits(cfg) ? cfg.m : 0;
    return tree_smem_layout(cfg.L, cfg.K, nmax, tree_node_cap(cfg.L, cfg.K, nmax, lazy_m), lazy_m, nullptr, nullptr);
}

cudaError_t tree_configure(const graft_config& cfg) {
    const int bytes = (int)tree_smem_bytes(cfg);
    cudaError_t e = cudaFuncSetAttribute(tree_kernel<0, 0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<32, 128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<32, 128, true, 513>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<16, 128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<8, 128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<0, 0, false, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<32, 128, true, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return e;
}

cudaError_t tree_launch(graft_ctx* ctx, int batch, const int32_t* d_topk_id, const float* d_topk_lp,
                        const int32_t* d_row_status, const float* d_esort, const uint8_t* d_eidx, const void* d_hidden,
                        const int32_t* d_root_token, const float* d_hist, const int32_t* d_prefix_len,
                        const int32_t* d_fixed_budget, const double* d_cos, const SabaResult* d_saba_pre,
                        const graft_tree_out* out, cudaStream_t st) {
    const graft_config& cfg = ctx->cfg;
    TreeParams p;
    p.topk_id = d_topk_id;
    p.topk_lp = d_topk_lp;
    p.row_status = d_row_status;
    p.vp_err = ctx->w_errflag;
    p.cos_pre = d_cos;
    p.esort = d_esort;
    p.eidx = d_eidx;
    (void)d_hidden;  // read by the vocab pass, which leaves the cosines in d_cos
    p.root_token = d_root_token;
    p.hist = d_hist;
    p.prefix_len = d_prefix_len;
    p.fixed_budget = d_fixed_budget;
    p.out = *out;
    p.L = cfg.L;
    p.K = cfg.K;
    p.nmax = ctx->nmax;
    p.W = ctx->mask_words;
    p.rows_pre = ctx->edge_rows;
    p.lazy = p.rows_pre < cfg.L ? 1 : 0;  // (only possible when tree_lazy_fits)
    p.rows_adaptive = (p.lazy && p.rows_pre > 0 && d_saba_pre != nullptr) ? 1 : 0;
    p.lazy_m = tree_lazy_fits(cfg) ? cfg.m : 0;
    p.ncap = tree_node_cap(cfg.L, cfg.K, ctx->nmax, p.lazy_m);
    p.P = ctx->d_P;
    p.C = ctx->d_C;
    p.u = ctx->d_u;
    p.scale = ctx->tdes_s / sqrtf((float)cfg.m);
    p.beta = ctx->tdes_set ? cfg.beta : 0.0f;
    p.root_edge = cfg.root_edge;
    p.m = cfg.m;
    p.V = cfg.V;
    p.bmin = cfg.budget_min;
    p.bmax = cfg.budget_max;
    p.bstep = cfg.budget_step;
    p.use_saba = d_fixed_budget == nullptr;
    p.saba = ctx->saba;
    p.saba_pre = d_saba_pre;
    // the instances with K and m known at compile time serve the usual round (the budget from the edge-score kernel,
    // deeper rows on demand)
    const bool usual = cfg.m == 128 && p.lazy && p.saba_pre != nullptr;
    void (*kern)(const TreeParams) = tree_kernel<0, 0, false>;
    if (usual && cfg.K == 32) kern = (ctx->nmax == 513 && p.ncap == 6144) ? tree_kernel<32, 128, true, 513> : tree_kernel<32, 128, true>;
    if (usual && cfg.K == 16) kern = tree_kernel<16, 128, true>;
    if (usual && cfg.K == 8) kern = tree_kernel<8, 128, true>;
    if (p.beta == 0.0f) kern = (usual && cfg.K == 32) ? tree_kernel<32, 128, true, 0, true> : tree_kernel<0, 0, false, 0, true>;
    const cudaError_t e = launch_pdl(kern, dim3(batch), dim3(TREE_THREADS), tree_smem_bytes(cfg), st, p);
    ctx->launches += 1;
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t accept_launch(graft_ctx* ctx, int batch, const graft_tree_out* trees, const int32_t* d_target_next,
                          int32_t* d_accept_len, int32_t* d_accept_path, int32_t* d_bonus, cudaStream_t st) {
    AcceptParams ap;
    ap.n_nodes = trees->d_n_nodes;
    ap.token = trees->d_token;
    ap.parent = trees->d_parent;
    ap.target_next = d_target_next;
    ap.batch = batch;
    ap.nmax = ctx->nmax;
    ap.L = ctx->cfg.L;
    ap.accept_len = d_accept_len;
    ap.accept_path = d_accept_path;
    ap.bonus = d_bonus;
    ap.hist_w = ctx->hist_w;
    ap.hist_window = ctx->hist_window;
    ap.hist_count = ctx->hist_count;
    ap.hist_out = ctx->hist_out;
    const cudaError_t e = launch_pdl(accept_kernel, dim3(batch), dim3(128), (size_t)3 * ctx->nmax * sizeof(int32_t), st, ap);
    ctx->launches += 1;
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace graft
