/*
 * GRAFT draft-tree construction -- CPU ORACLE (test infrastructure, not product code).
 *
 * A plain, slow, obviously-correct restatement of what the GRAFT paper defines for one
 * decoding round, in the paper's order and notation.  It shares no code with the CUDA
 * library, is never called by it, and may only be used by tests, the smoke check and the
 * benchmark's CPU-baseline leg.  Floating point is fp64 unless a value is *defined* as an
 * fp32 quantity (candidate log-probabilities, edge scores and path scores are fp32 values;
 * path scores are accumulated root-to-leaf with fp32 additions so that ranking decisions are
 * taken in the same precision as the library takes them).
 *
 * Steps (all pointers are host pointers; arrays are row-major and contiguous):
 *   O0  oracle_tdes_tables    cached projections g_p(e_v), g_c(e_v)        (Sec. 3.2, text after Eq. 6)
 *   O1  oracle_vocab_pass     log q_{t,d} and the K top-ranked tokens      (Preliminaries, "DFlash one-pass marginals"; Eq. 3)
 *   O2  oracle_saba           decoding state, gain, cost, budget           (Sec. 3.3, Eq. 14-17)
 *   O3  oracle_tdes_edges     centred bi-tower edge scores                 (Sec. 3.2, Eq. 4-6)
 *   O4  oracle_select         best-first expansion until B_t nodes         (Preliminaries "DDTree"; Sec. 3.1; Eq. 13)
 *   O5  oracle_emit           level-order tree, positions, ancestor mask   (Preliminaries "Tree-based speculative decoding")
 *   O6  oracle_accept         longest accepted path                        (Preliminaries, a_t)
 *   O7  oracle_hist_update    hist_t over the last w accepted lengths      (Sec. 3.3, Eq. 15)
 *   --  oracle_replay_check   is a given node set a valid best-first outcome up to eps?
 *
 * Pins: every function here is pinned by tests that do not call it to produce their own
 * expectation (closed forms, invariants, brute-force enumeration, library routines).  The
 * paper prints no numeric worked example, so end-to-end values beyond those pins are
 * "parity unpinned"; each function below states its pins.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_F32 0
#define ORC_BF16 1
#define ORC_MAX_L 32

/* status bits, per sequence */
#define ORC_ST_BAD_LOGITS 1      /* NaN, +inf, or a row with no finite entry */
#define ORC_ST_TAU_CLAMPED 2     /* phi . s fell below tau_min */
#define ORC_ST_FRONTIER_EMPTY 4  /* fewer reachable prefixes than the budget */

static float orc_load(const void *base, int dtype, size_t i) {
    if (dtype == ORC_F32) return ((const float *)base)[i];
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[i]) << 16; /* bf16 -> fp32 is exact */
    float f;
    memcpy(&f, &bits, 4);
    return f;
}

/* ------------------------------------------------------------------------------------------
 * O0.  P[v] = W_p e_v + b_p,  C[v] = W_c e_v + b_c   (the two linear projections g_p and g_c
 * of Sec. 3.2; a function of the token id alone, hence tabulated once per model).  fp64 accumulate,
 * rounded once to fp32.  bias may be NULL.
 * Pins: identity weights reproduce the embedding; agreement with a library matmul.
 * ------------------------------------------------------------------------------------------ */
int oracle_tdes_tables(const void *emb, int emb_dtype, int V, int E, int m, const float *W,
                       const float *bias, float *out /* [V,m] */) {
    for (int v = 0; v < V; ++v)
        for (int k = 0; k < m; ++k) {
            double acc = bias ? (double)bias[k] : 0.0;
            for (int e = 0; e < E; ++e)
                acc += (double)W[(size_t)k * E + e] * (double)orc_load(emb, emb_dtype, (size_t)v * E + e);
            out[(size_t)v * m + k] = (float)acc;
        }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * O1.  For every row (one future position d of one sequence): q_{t,d} = softmax over the
 * whole vocabulary; the K top-ranked tokens c^{(1)}..c^{(K)} ranked by (logit descending,
 * token id ascending); lp[r] = log q_{t,d}(c^{(r)}) as an fp32 value.
 * Pins: sum_v exp(lp_v) = 1; uniform row -> -ln V and ids 0..K-1; library log_softmax/topk;
 * shift invariance.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    float z;
    int32_t id;
} orc_zi;

static int orc_cmp_zi(const void *a, const void *b) {
    const orc_zi *x = (const orc_zi *)a, *y = (const orc_zi *)b;
    if (x->z > y->z) return -1;
    if (x->z < y->z) return 1;
    return (x->id > y->id) - (x->id < y->id);
}

int oracle_vocab_pass(const void *logits, int dtype, int64_t rows, int V, int K, int32_t *topk_id /* [rows,K] */,
                      float *topk_lp /* [rows,K] */, double *lse /* [rows] */, int32_t *row_status /* [rows] */) {
    orc_zi *buf = (orc_zi *)malloc(sizeof(orc_zi) * (size_t)V);
    if (!buf) return -1;
    for (int64_t r = 0; r < rows; ++r) {
        int bad = 0;
        float M = -INFINITY;
        for (int v = 0; v < V; ++v) {
            float z = orc_load(logits, dtype, (size_t)r * V + v);
            if (isnan(z) || z == INFINITY) bad = 1;
            if (z > M) M = z;
            buf[v].z = z;
            buf[v].id = v;
        }
        if (M == -INFINITY) bad = 1;
        row_status[r] = bad ? ORC_ST_BAD_LOGITS : 0;
        if (bad) {
            lse[r] = NAN;
            for (int k = 0; k < K; ++k) {
                topk_id[r * K + k] = -1;
                topk_lp[r * K + k] = 0.0f;
            }
            continue;
        }
        double Z = 0.0;
        for (int v = 0; v < V; ++v) Z += exp((double)buf[v].z - (double)M);
        double l = (double)M + log(Z);
        lse[r] = l;
        qsort(buf, (size_t)V, sizeof(orc_zi), orc_cmp_zi);
        for (int k = 0; k < K; ++k) {
            topk_id[r * K + k] = buf[k].id;
            topk_lp[r * K + k] = (float)((double)buf[k].z - l);
        }
    }
    free(buf);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * O2.  SABA (Sec. 3.3).  conf_t = (1/D) sum_d q_{t,d}(c^{(1)})  (a probability, Eq. 15);
 * r_d = cos(h_d, h_{d+1}); degen_t = mean_d r_d + (r_{D-1} - r_1); hist_t is supplied;
 * tau = phi . [conf, degen, hist] + phi_bias, clamped below by tau_min;
 * G(B) = 1 - exp(-B / tau) (Eq. 16);  C(B) = c0 + c1 B + c2 B prefix (Eq. 17) or a linear
 * interpolation of a supplied (n_i, t_i) table clamped at its ends;  U = G / C (Eq. 14);
 * B_t = argmax over the grid {bmin, bmin+step, ... <= bmax}, smallest B on ties.
 * Outputs: state[4] = conf, degen, hist, tau (fp64); budget; U over the grid (for the
 * near-tie rule of the parity tests).
 * Pins: identical / orthogonal hidden rows; constant cost -> bmax; tau -> tau_min;
 * brute-force grid max; quasi-concavity against a bisection root.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    double phi_conf, phi_degen, phi_hist, phi_bias, tau_min;
    int32_t cost_mode; /* 0 affine, 1 table */
    double c0, c1, c2;
    int32_t n_pts;
    const double *pts_n, *pts_t;
} orc_saba_params;

static double orc_cost(const orc_saba_params *p, double B, double prefix) {
    if (p->cost_mode == 0) return p->c0 + p->c1 * B + p->c2 * B * prefix;
    if (B <= p->pts_n[0]) return p->pts_t[0];
    for (int i = 1; i < p->n_pts; ++i)
        if (B <= p->pts_n[i]) {
            double w = (B - p->pts_n[i - 1]) / (p->pts_n[i] - p->pts_n[i - 1]);
            return p->pts_t[i - 1] + w * (p->pts_t[i] - p->pts_t[i - 1]);
        }
    return p->pts_t[p->n_pts - 1];
}

int oracle_saba(const float *lp0 /* [L] log q of the top-1 token per depth */, const void *hidden /* [L,dh] */,
                int hidden_dtype, int L, int dh, double hist, int32_t prefix_len, const orc_saba_params *p, int bmin,
                int bmax, int bstep, double *state /* [4] */, int32_t *budget, double *U /* [grid] */,
                int32_t *status) {
    double conf = 0.0;
    for (int d = 0; d < L; ++d) conf += exp((double)lp0[d]);
    conf /= (double)L;
    double degen = 0.0;
    if (L >= 2) {
        double r_first = 0.0, r_last = 0.0, r_sum = 0.0;
        for (int d = 0; d + 1 < L; ++d) {
            double ab = 0.0, aa = 0.0, bb = 0.0;
            for (int k = 0; k < dh; ++k) {
                double a = (double)orc_load(hidden, hidden_dtype, (size_t)d * dh + k);
                double b = (double)orc_load(hidden, hidden_dtype, (size_t)(d + 1) * dh + k);
                ab += a * b;
                aa += a * a;
                bb += b * b;
            }
            double r = (aa > 0.0 && bb > 0.0) ? ab / (sqrt(aa) * sqrt(bb)) : 0.0;
            if (d == 0) r_first = r;
            if (d == L - 2) r_last = r;
            r_sum += r;
        }
        degen = r_sum / (double)(L - 1) + (r_last - r_first);
    }
    double tau = p->phi_conf * conf + p->phi_degen * degen + p->phi_hist * hist + p->phi_bias;
    *status = 0;
    if (!(tau >= p->tau_min)) {
        tau = p->tau_min;
        *status |= ORC_ST_TAU_CLAMPED;
    }
    state[0] = conf;
    state[1] = degen;
    state[2] = hist;
    state[3] = tau;
    int best = bmin;
    double Ubest = -INFINITY;
    int g = 0;
    for (int B = bmin; B <= bmax; B += bstep, ++g) {
        double G = 1.0 - exp(-(double)B / tau);
        double u = G / orc_cost(p, (double)B, (double)prefix_len);
        if (U) U[g] = u;
        if (u > Ubest) {
            Ubest = u;
            best = B;
        }
    }
    *budget = best;
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * O3.  TDES edge scores (Eq. 4-6).  For depth d = 1..L (row j = d-1), parents are the depth
 * d-1 candidates (the single root token at d = 1), children are the K depth-d candidates
 * (the set C_{p,d} is the same K candidates for every parent):
 *    f(p,c,d)  = s (P[p] + u_d)^T (C[c] + u_d) / sqrt(m)                     (Eq. 6)
 *    f~(p,c,d) = f(p,c,d) - (1/K) sum_c' f(p,c',d)                            (Eq. 5)
 *    edge      = log q_{t,d}(c) + beta f~(p,c,d)                              (Eq. 4)
 * edge is [L,K,K] (depth, parent index, child index); depth 1 fills parent row 0 only
 * (other rows are written as 0).  root_edge = 0 sets f~ = 0 at depth 1.
 * Pins: rows of f~ sum to zero; beta = 0 gives lp exactly; K = 1 gives f~ = 0; W_c = 0 gives
 * f~ = 0; the algebraic restatement with centred child vectors.
 * ------------------------------------------------------------------------------------------ */
int oracle_tdes_edges(const int32_t *topk_id /* [L,K] */, const float *topk_lp /* [L,K] */, int32_t root_token,
                      const float *P, const float *C /* [V,m] */, const float *u /* [L,m] */, double s, double beta,
                      int root_edge, int L, int K, int m, float *edge /* [L,K,K] */) {
    double *f = (double *)malloc(sizeof(double) * (size_t)K);
    if (!f) return -1;
    for (int j = 0; j < L; ++j) {
        int n_par = (j == 0) ? 1 : K;
        for (int i = 0; i < K; ++i) {
            float *row = edge + ((size_t)j * K + i) * K;
            if (i >= n_par) {
                for (int c = 0; c < K; ++c) row[c] = 0.0f;
                continue;
            }
            int32_t p = (j == 0) ? root_token : topk_id[(j - 1) * K + i];
            double mean = 0.0;
            for (int c = 0; c < K; ++c) {
                int32_t ct = topk_id[j * K + c];
                double acc = 0.0;
                for (int k = 0; k < m; ++k)
                    acc += ((double)P[(size_t)p * m + k] + (double)u[j * m + k]) *
                           ((double)C[(size_t)ct * m + k] + (double)u[j * m + k]);
                f[c] = s * acc / sqrt((double)m);
                mean += f[c];
            }
            mean /= (double)K;
            for (int c = 0; c < K; ++c) {
                double ft = (j == 0 && !root_edge) ? 0.0 : f[c] - mean;
                row[c] = (float)((double)topk_lp[j * K + c] + beta * ft);
            }
        }
    }
    free(f);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * O4.  Best-first expansion (the "max-heap of candidate prefixes" of the DDTree paragraph,
 * ranked by the TDES path score of Eq. 13, stopped at B_t nodes, Sec. 3.1).  A prefix is a
 * tuple of candidate indices (c_1..c_l).  S(()) = 0; S(u) = fp32(S(parent) + edge).  The
 * frontier starts with the K depth-1 prefixes; each step removes the frontier maximum, adds it
 * to the tree and inserts its K extensions.  The frontier is an explicit array scanned
 * linearly; no heap.
 *
 * The paper does not say how equal scores are ordered.  The total order used here depends only
 * on the prefixes themselves (not on the history of the expansion):  path score descending;
 * then length ascending; then the parent prefix in lexicographic order of its candidate ranks;
 * then, under one parent, edge score descending and candidate rank ascending (a parent's
 * children are taken in the order of their edge scores).
 *
 * Output: sel_tuple [n_sel, L] (unused slots -1), sel_len, sel_S in pop order.
 * Pins: exhaustive enumeration for L,K <= 4 (a top-B set by path score when edges <= 0; a
 * top-B set by bottleneck key always); an independently written from-scratch frontier
 * recomputation; chain of top-1 tokens; complete tree when B >= number of prefixes.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    float S;
    float e;        /* the last edge's score */
    int32_t len;
    int8_t t[ORC_MAX_L];
} orc_prefix;

static int orc_before(const orc_prefix *a, const orc_prefix *b) { /* does a pop before b? */
    if (a->S > b->S) return 1;
    if (a->S < b->S) return 0;
    if (a->len != b->len) return a->len < b->len;
    for (int i = 0; i + 1 < a->len; ++i) /* the parents, lexicographically */
        if (a->t[i] != b->t[i]) return a->t[i] < b->t[i];
    if (a->e > b->e) return 1;
    if (a->e < b->e) return 0;
    return a->t[a->len - 1] < b->t[b->len - 1];
}

int oracle_select(const float *edge /* [L,K,K] */, int L, int K, int budget, int32_t *sel_tuple /* [budget,L] */,
                  int32_t *sel_len /* [budget] */, float *sel_S /* [budget] */, int32_t *n_sel) {
    if (L > ORC_MAX_L || K > 127) return -2;
    size_t cap = (size_t)K + (size_t)budget * (size_t)K + 1;
    orc_prefix *fr = (orc_prefix *)malloc(sizeof(orc_prefix) * cap);
    if (!fr) return -1;
    size_t nf = 0;
    for (int c = 0; c < K; ++c) {
        orc_prefix x;
        memset(&x, 0, sizeof x);
        x.e = edge[c]; /* depth 1, parent row 0 */
        x.S = (float)(0.0f + x.e);
        x.len = 1;
        x.t[0] = (int8_t)c;
        fr[nf++] = x;
    }
    int n = 0;
    while (n < budget && nf > 0) {
        size_t best = 0;
        for (size_t i = 1; i < nf; ++i)
            if (orc_before(&fr[i], &fr[best])) best = i;
        orc_prefix x = fr[best];
        fr[best] = fr[nf - 1];
        --nf;
        for (int i = 0; i < L; ++i) sel_tuple[(size_t)n * L + i] = (i < x.len) ? x.t[i] : -1;
        sel_len[n] = x.len;
        sel_S[n] = x.S;
        ++n;
        if (x.len < L) {
            int j = x.len; /* row of the child depth */
            int par = x.t[x.len - 1];
            for (int c = 0; c < K; ++c) {
                orc_prefix y = x;
                y.e = edge[((size_t)j * K + par) * K + c];
                volatile float sum = x.S + y.e; /* one fp32 rounding */
                y.S = sum;
                y.t[y.len] = (int8_t)c;
                y.len = x.len + 1;
                fr[nf++] = y;
            }
        }
    }
    *n_sel = n;
    free(fr);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * O5.  Emission.  The selected prefixes are laid out in canonical level order (length
 * ascending, tuple lexicographic ascending); node 0 is the root (the last committed token).
 * token / parent / depth / position id = prefix_len - 1 + depth / path score / packed
 * ancestor-or-self bitmask (bit j of row i set iff j = i or j is an ancestor of i; this is
 * the tree-attention mask restricted to the tree).  Rows n_nodes..Nmax-1 are padding:
 * token, parent, depth, position = -1, score 0, mask 0.
 * Pins: structural invariants (prefix-closed, parent < child, popcount = depth + 1, ...).
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t len;
    int32_t t[ORC_MAX_L];
    float S;
} orc_node;

static int orc_cmp_node(const void *a, const void *b) {
    const orc_node *x = (const orc_node *)a, *y = (const orc_node *)b;
    if (x->len != y->len) return x->len < y->len ? -1 : 1;
    for (int i = 0; i < x->len; ++i)
        if (x->t[i] != y->t[i]) return x->t[i] < y->t[i] ? -1 : 1;
    return 0;
}

int oracle_emit(const int32_t *sel_tuple, const int32_t *sel_len, const float *sel_S, int n_sel, int L, int K,
                const int32_t *topk_id /* [L,K] */, int32_t root_token, int32_t prefix_len, int Nmax, int W,
                int32_t *n_nodes, int32_t *token, int32_t *parent, int32_t *depth, int32_t *position,
                float *path_score, uint32_t *mask /* [Nmax,W] */, int32_t *cand /* [Nmax] may be NULL */) {
    (void)K;
    orc_node *nd = (orc_node *)malloc(sizeof(orc_node) * (size_t)(n_sel + 1));
    if (!nd) return -1;
    nd[0].len = 0;
    nd[0].S = 0.0f;
    for (int i = 0; i < n_sel; ++i) {
        nd[i + 1].len = sel_len[i];
        nd[i + 1].S = sel_S[i];
        for (int k = 0; k < L; ++k) nd[i + 1].t[k] = sel_tuple[(size_t)i * L + k];
    }
    int n = n_sel + 1;
    qsort(nd, (size_t)n, sizeof(orc_node), orc_cmp_node);
    for (int i = 0; i < Nmax; ++i) {
        token[i] = parent[i] = depth[i] = position[i] = -1;
        path_score[i] = 0.0f;
        if (cand) cand[i] = -1;
        for (int w = 0; w < W; ++w) mask[(size_t)i * W + w] = 0u;
    }
    *n_nodes = n;
    for (int i = 0; i < n; ++i) {
        int len = nd[i].len;
        depth[i] = len;
        position[i] = prefix_len - 1 + len;
        path_score[i] = nd[i].S;
        if (len == 0) {
            token[i] = root_token;
            parent[i] = -1;
        } else {
            token[i] = topk_id[(len - 1) * K + nd[i].t[len - 1]];
            if (cand) cand[i] = nd[i].t[len - 1];
            int par = -1; /* the node whose tuple is this tuple minus its last entry */
            for (int q = 0; q < i; ++q) {
                if (nd[q].len != len - 1) continue;
                int same = 1;
                for (int k = 0; k < len - 1; ++k)
                    if (nd[q].t[k] != nd[i].t[k]) same = 0;
                if (same) par = q;
            }
            parent[i] = par; /* -1 here would mean the set is not prefix-closed */
        }
        for (int a = i; a >= 0; a = parent[a]) mask[(size_t)i * W + (a >> 5)] |= (1u << (a & 31));
    }
    free(nd);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * O6.  Acceptance walk: starting at the root, follow the child whose token equals the
 * target's next token after the current node; a_t counts the accepted draft tokens; the
 * bonus token is the target's next token after the last accepted node.
 * Pins: a hand-built tree with three target scripts; chain tree; path invariants.
 * ------------------------------------------------------------------------------------------ */
int oracle_accept(int n_nodes, const int32_t *token, const int32_t *parent, const int32_t *target_next /* [Nmax] */,
                  int L, int32_t *accept_len, int32_t *accept_path /* [L] */, int32_t *bonus) {
    for (int i = 0; i < L; ++i) accept_path[i] = -1;
    int cur = 0, a = 0;
    for (;;) {
        int32_t want = target_next[cur];
        int nxt = -1;
        for (int i = 1; i < n_nodes; ++i)
            if (parent[i] == cur && token[i] == want) {
                nxt = i;
                break;
            }
        if (nxt < 0 || a >= L) break;
        accept_path[a++] = nxt;
        cur = nxt;
    }
    *accept_len = a;
    *bonus = target_next[cur];
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * O7.  Acceptance history (Eq. 15): hist_t = (1/w) sum_{i=1..w} a_{t-i}.  `a_hist` holds every
 * accepted length so far, oldest first (n_rounds of them); the result is hist for the next round.
 * Reading for the first rounds, where fewer than w lengths exist (the paper does not say): the
 * mean of those that exist, and 0 before the first round.
 * Pins: a constant history gives that constant; a step change crosses over in exactly w rounds;
 * the definition recomputed with a library mean over the last w entries.
 * ------------------------------------------------------------------------------------------ */
double oracle_hist_update(const int32_t *a_hist, int n_rounds, int w) {
    if (n_rounds <= 0 || w <= 0) return 0.0;
    const int m = n_rounds < w ? n_rounds : w;
    double s = 0.0;
    for (int i = 1; i <= m; ++i) s += (double)a_hist[n_rounds - i];
    return s / (double)m;
}

/* ------------------------------------------------------------------------------------------
 * Replay check used by the parity tests when a library tree differs from the oracle's: is
 * the node set G (given as a tree over candidate indices: parent[], cand[], depth[], node 0
 * the root) a valid outcome of best-first expansion on THIS oracle's edge scores if every
 * score comparison may be off by eps?  Replays |G|-1 steps; at each step the best frontier
 * member that belongs to G is taken, and its score must be within 2 eps of the best score
 * in the whole frontier (all unselected children of selected nodes).
 * Returns 0 if valid, 1 if not; *worst receives the largest shortfall seen.
 * ------------------------------------------------------------------------------------------ */
int oracle_replay_check(const float *edge, int L, int K, int n_nodes, const int32_t *parent, const int32_t *cand,
                        const int32_t *depth, double eps, double *worst) {
    float *S = (float *)calloc((size_t)n_nodes, sizeof(float));
    char *sel = (char *)calloc((size_t)n_nodes, 1);
    int32_t *childof = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_nodes * (size_t)K);
    if (!S || !sel || !childof) return -1;
    for (size_t i = 0; i < (size_t)n_nodes * (size_t)K; ++i) childof[i] = -1;
    int rc = 0;
    *worst = 0.0;
    for (int i = 1; i < n_nodes; ++i) {
        if (parent[i] < 0 || parent[i] >= i || cand[i] < 0 || cand[i] >= K || depth[i] != depth[parent[i]] + 1 ||
            depth[i] > L || childof[(size_t)parent[i] * K + cand[i]] >= 0) {
            rc = 1;
            goto done;
        }
        childof[(size_t)parent[i] * K + cand[i]] = i;
    }
    sel[0] = 1;
    S[0] = 0.0f;
    for (int step = 1; step < n_nodes; ++step) {
        double best_all = -INFINITY, best_g = -INFINITY;
        int best_node = -1;
        for (int q = 0; q < n_nodes; ++q) {
            if (!sel[q] || depth[q] >= L) continue;
            int j = depth[q];
            int par = (q == 0) ? 0 : cand[q];
            for (int c = 0; c < K; ++c) {
                int child = childof[(size_t)q * K + c];
                if (child >= 0 && sel[child]) continue;
                volatile float sc = S[q] + edge[((size_t)j * K + par) * K + c];
                if ((double)sc > best_all) best_all = (double)sc;
                if (child >= 0 && (double)sc > best_g) {
                    best_g = (double)sc;
                    best_node = child;
                }
            }
        }
        if (best_node < 0) {
            rc = 1;
            goto done;
        }
        double short_by = best_all - best_g;
        if (short_by > *worst) *worst = short_by;
        if (short_by > 2.0 * eps) {
            rc = 1;
            goto done;
        }
        sel[best_node] = 1;
        S[best_node] = (float)best_g;
    }
done:
    free(S);
    free(sel);
    free(childof);
    return rc;
}

/* ------------------------------------------------------------------------------------------
 * One whole round for a batch of sequences, the steps above in the paper's order
 * (candidates -> SABA -> TDES -> best-first -> emission).  fixed_budget may be NULL (SABA).
 * Optional outputs may be NULL.
 * ------------------------------------------------------------------------------------------ */
int oracle_build_trees(int batch, int L, int V, int K, int m, int dh, const void *logits, int logits_dtype,
                       const void *hidden, int hidden_dtype, const int32_t *root_token, const double *hist,
                       const int32_t *prefix_len, const int32_t *fixed_budget, const orc_saba_params *saba, int bmin,
                       int bmax, int bstep, const float *P, const float *C, const float *u, double s, double beta,
                       int root_edge, int Nmax, int W,
                       /* outputs */ int32_t *n_nodes, int32_t *budget, int32_t *token, int32_t *parent,
                       int32_t *depth, int32_t *position, float *path_score, uint32_t *mask, int32_t *status,
                       int32_t *cand, int32_t *topk_id, float *topk_lp, double *lse, float *edge, double *state,
                       double *Ugrid /* [batch, grid] */) {
    int grid = (bmax - bmin) / bstep + 1;
    size_t esz = (logits_dtype == ORC_F32) ? 4 : 2, hsz = (hidden_dtype == ORC_F32) ? 4 : 2;
    int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)L * K);
    float *lps = (float *)malloc(sizeof(float) * (size_t)L * K);
    double *ls = (double *)malloc(sizeof(double) * (size_t)L);
    int32_t *rst = (int32_t *)malloc(sizeof(int32_t) * (size_t)L);
    float *ed = (float *)malloc(sizeof(float) * (size_t)L * K * K);
    int32_t *stup = (int32_t *)malloc(sizeof(int32_t) * (size_t)(bmax + 1) * L);
    int32_t *slen = (int32_t *)malloc(sizeof(int32_t) * (size_t)(bmax + 1));
    float *sS = (float *)malloc(sizeof(float) * (size_t)(bmax + 1));
    float *lp0 = (float *)malloc(sizeof(float) * (size_t)L);
    if (!ids || !lps || !ls || !rst || !ed || !stup || !slen || !sS || !lp0) return -1;
    for (int b = 0; b < batch; ++b) {
        int st = 0;
        oracle_vocab_pass((const char *)logits + (size_t)b * L * V * esz, logits_dtype, L, V, K, ids, lps, ls, rst);
        for (int j = 0; j < L; ++j) st |= rst[j];
        int B = 0, nsel = 0;
        double stt[4] = {0, 0, 0, 0};
        if (!(st & ORC_ST_BAD_LOGITS)) {
            if (fixed_budget) {
                B = fixed_budget[b];
                if (B > bmax) B = bmax;
                if (B < 0) B = 0;
            } else {
                int sst = 0;
                for (int j = 0; j < L; ++j) lp0[j] = lps[j * K];
                oracle_saba(lp0, (const char *)hidden + (size_t)b * L * dh * hsz, hidden_dtype, L, dh, hist[b],
                            prefix_len[b], saba, bmin, bmax, bstep, stt, &B, Ugrid ? Ugrid + (size_t)b * grid : NULL,
                            &sst);
                st |= sst;
            }
            oracle_tdes_edges(ids, lps, root_token[b], P, C, u, s, beta, root_edge, L, K, m, ed);
            oracle_select(ed, L, K, B, stup, slen, sS, &nsel);
            if (nsel < B) st |= ORC_ST_FRONTIER_EMPTY;
        } else {
            memset(ed, 0, sizeof(float) * (size_t)L * K * K);
        }
        oracle_emit(stup, slen, sS, nsel, L, K, ids, root_token[b], prefix_len[b], Nmax, W, n_nodes + b,
                    token + (size_t)b * Nmax, parent + (size_t)b * Nmax, depth + (size_t)b * Nmax,
                    position + (size_t)b * Nmax, path_score + (size_t)b * Nmax, mask + (size_t)b * Nmax * W,
                    cand ? cand + (size_t)b * Nmax : NULL);
        budget[b] = B;
        status[b] = st;
        if (topk_id) memcpy(topk_id + (size_t)b * L * K, ids, sizeof(int32_t) * (size_t)L * K);
        if (topk_lp) memcpy(topk_lp + (size_t)b * L * K, lps, sizeof(float) * (size_t)L * K);
        if (lse) memcpy(lse + (size_t)b * L, ls, sizeof(double) * (size_t)L);
        if (edge) memcpy(edge + (size_t)b * L * K * K, ed, sizeof(float) * (size_t)L * K * K);
        if (state) memcpy(state + (size_t)b * 4, stt, sizeof stt);
    }
    free(ids); free(lps); free(ls); free(rst); free(ed); free(stup); free(slen); free(sS); free(lp0);
    return 0;
}
