/*
 * graft.h -- C ABI of the B200 (sm_100a) GRAFT draft-tree builder.
 *
 * One decoding round of GRAFT (Sec. 3 "Method", overview in Sec. 3.1): given a diffusion
 * drafter's one-pass block output -- logits q_{t,d}(.) over the vocabulary for d = 1..L and the
 * hidden states h_{t,d} -- and the decoding state, build for every sequence of a batch the
 * prefix-closed draft tree that the target model will verify, and afterwards walk the tree
 * against the target's next tokens.
 *
 * Conventions
 *   - Pointers named d_* are DEVICE pointers; all others are HOST pointers.  The caller owns
 *     every buffer it passes in; the library never frees or reallocates them.  A context owns
 *     only its own scratch (sized from max_batch at creation) and copies of the parameters.
 *   - All tensors are dense, row-major, contiguous.  Logits rows may start at any address that
 *     is a multiple of the element size (rows need not be 16-byte aligned).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only
 *     enqueue work on it and return; results are valid once the stream has reached that point.
 *   - The return value reports host-side argument / launch errors, synchronously.  Data errors
 *     are reported per sequence in d_status (bit flags below); nothing ever traps on the device.
 *   - One context must not be used from two streams at the same time (the scratch is shared).
 *   - There is no CPU fallback: without a CUDA device every entry point except
 *     graft_status_str / graft_version returns GRAFT_ERR_CUDA.
 *
 * Limits (else GRAFT_ERR_UNSUPPORTED): 1 <= K <= 32, K <= V, 1 <= L <= 32, V < 2^31 - 64,
 *   m a multiple of 4 with 4 <= m <= 512, budget_max <= 1023, budget_step >= 1,
 *   L*K*K*4 bytes <= 128 KiB (edge scores live in shared memory), hidden_dim >= 1.
 */
#ifndef GRAFT_H_
#define GRAFT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct graft_ctx graft_ctx; /* opaque */

typedef enum {
    GRAFT_OK = 0,
    GRAFT_ERR_INVALID_ARG = 1, /* NULL where a pointer is required, batch out of range, ... */
    GRAFT_ERR_UNSUPPORTED = 2, /* a size outside the limits above */
    GRAFT_ERR_CUDA = 3,        /* a CUDA runtime call failed (no device, launch error, ...) */
    GRAFT_ERR_WORKSPACE = 4,   /* scratch allocation failed */
    GRAFT_ERR_STATE = 5        /* call order: TDES tables or SABA parameters not set */
} graft_status;

typedef enum { GRAFT_F32 = 0, GRAFT_BF16 = 1 } graft_dtype;

/* per-sequence bits written to d_status */
#define GRAFT_ST_BAD_LOGITS 1     /* a logits row holds NaN or +inf, or no finite entry: root-only tree */
#define GRAFT_ST_TAU_CLAMPED 2    /* SABA: phi . s_t fell below tau_min and was clamped */
#define GRAFT_ST_FRONTIER_EMPTY 4 /* fewer reachable prefixes than the budget */
#define GRAFT_ST_INTERNAL 8       /* a bounded device-side wait ran out (should never happen) */

typedef struct {
    int32_t V;          /* vocabulary size */
    int32_t L;          /* block length: future positions d = 1..L (the paper's D) */
    int32_t K;          /* candidates kept per position */
    int32_t m;          /* width of the TDES scoring space (Eq. 6) */
    int32_t hidden_dim; /* width of h_{t,d} */
    int32_t max_batch;
    int32_t budget_min, budget_max, budget_step; /* SABA grid {min, min+step, .. <= max} (Sec. 3.3: 32..512 step 16) */
    float beta;         /* residual strength of Eq. 4; 0 gives the DDTree score of Eq. 3 */
    int32_t root_edge;  /* 1: depth-1 edges are scored against the root token; 0: f~ = 0 at depth 1 */
    graft_dtype logits_dtype, hidden_dtype;
} graft_config;

/* SABA parameters (Sec. 3.3).  tau = phi . [conf, degen, hist] + phi_bias, clamped below by tau_min
 * (Eq. 16's saturation scale).  Cost C_t(B): mode 0 = c0 + c1 B + c2 B prefix_t (Eq. 17); mode 1 = linear
 * interpolation of the n_pts points (pts_n[i], pts_t[i]) (pts_n strictly increasing, n_pts <= 16), held
 * constant outside them.  pts_* are host arrays and are copied. */
typedef struct {
    float phi_conf, phi_degen, phi_hist, phi_bias;
    float tau_min;
    int32_t cost_mode;
    float c0, c1, c2;
    int32_t n_pts;
    const float* pts_n;
    const float* pts_t;
} graft_saba_params;

/* Outputs of graft_build_trees.  Nmax = budget_max + 1 rows per sequence (node 0 is the root, i.e. the
 * last committed token); W = ceil(Nmax / 32) mask words per row.  Nodes are in level order (depth
 * ascending, then by the parent's index, then by candidate rank).  Rows n_nodes.. are padding: token,
 * parent, depth, position = -1, path_score = 0, mask = 0. */
typedef struct {
    int32_t* d_n_nodes;    /* [batch] 1 + number of draft nodes */
    int32_t* d_budget;     /* [batch] B_t */
    int32_t* d_token;      /* [batch, Nmax] */
    int32_t* d_parent;     /* [batch, Nmax] root: -1 */
    int32_t* d_depth;      /* [batch, Nmax] root: 0 */
    int32_t* d_position;   /* [batch, Nmax] prefix_len - 1 + depth */
    float* d_path_score;   /* [batch, Nmax] S_TDES(u) of Eq. 13, accumulated root to leaf in fp32 */
    uint32_t* d_mask;      /* [batch, Nmax, W] bit j of row i set iff j == i or j is an ancestor of i */
    int32_t* d_status;     /* [batch] GRAFT_ST_* bits */
    /* optional intermediate outputs, each may be NULL: */
    int32_t* d_topk_id;    /* [batch, L, K] c^{(r)}_{t,d}, ranked by (logit descending, token id ascending) */
    float* d_topk_lp;      /* [batch, L, K] log q_{t,d}(c^{(r)}) */
    float* d_lse;          /* [batch, L] log sum_v exp(logit) */
    float* d_edge;         /* [batch, L, K, K] S_TDES(v) indexed (depth, parent rank, child rank); depth 1 uses
                              parent row 0 only, its other rows are 0 */
    float* d_state;        /* [batch, 4] conf_t, degen_t, hist_t, tau (zeros when the budget is fixed) */
} graft_tree_out;

/* Create / destroy a context.  Allocates the scratch for max_batch sequences.  Sets *out = NULL on error. */
graft_status graft_create(const graft_config* cfg, graft_ctx** out);
graft_status graft_destroy(graft_ctx* ctx);
size_t graft_nmax(const graft_ctx* ctx);       /* budget_max + 1 */
size_t graft_mask_words(const graft_ctx* ctx); /* ceil(Nmax / 32) */

/* SABA parameters (Sec. 3.3, Eq. 14-17).  Required before graft_build_trees is called without a
 * fixed budget. */
graft_status graft_set_saba(graft_ctx* ctx, const graft_saba_params* p);

/* TDES tables (Sec. 3.2, text after Eq. 6: the projected embeddings depend only on the token id and are
 * computed once).  d_P, d_C: [V, m] fp32, 16-byte aligned, P[v] = g_p(e_v), C[v] = g_c(e_v); d_u: [L, m]
 * fp32 depth embeddings u_d; s: the scale of Eq. 6.  The tables are borrowed until the context is
 * destroyed or the tables are set again.  u is copied on `stream`. */
graft_status graft_set_tdes_tables(graft_ctx* ctx, const float* d_P, const float* d_C, const float* d_u, float s,
                                   void* stream);

/* How many depths the edge-score kernel covers ahead of the expansion.  The scores of Eq. 4-6 are needed only for
 * depths that the best-first expansion reaches, which is not known in advance: depths [0, rows) are scored for every
 * sequence by a kernel of their own, deeper ones inside the tree kernel when an expansion gets there.  The trees do
 * not depend on the split at all: both scorers run the same arithmetic in the same order, so a score has the same
 * bits whichever kernel produced it.
 * rows in [0, L]; the default is min(L, 8), or L when the on-demand scorer's buffers do not fit in shared memory
 * (then any other value is GRAFT_ERR_INVALID_ARG).  Host-only call; takes effect from the next round.
 * (A tuning knob of this implementation; the paper scores all edges.) */
graft_status graft_set_edge_rows(graft_ctx* ctx, int32_t rows);
int32_t graft_edge_rows(const graft_ctx* ctx);

/* Table precompute (same passage): d_out[v] = W e_v + b for one tower.  d_emb [V, E] (dtype as given),
 * d_W [m, E] fp32, d_b [m] fp32 or NULL, d_out [V, m] fp32.  fp32 accumulation.  Call once per tower.
 * With bf16 embeddings (16-byte aligned, E a multiple of 8) the products run on the tensor cores: the embeddings are
 * exact operands and W enters as three bf16 parts, so the result differs from the fp32 one only by the order of
 * the additions; the first such call allocates scratch in the context (3 m E bf16 values and the GEMM's
 * workspace; GRAFT_ERR_WORKSPACE if that fails).  This is the once-per-model setup step, not the round. */
graft_status graft_tdes_precompute(graft_ctx* ctx, const void* d_emb, graft_dtype emb_dtype, int32_t E,
                                   const float* d_W, const float* d_b, float* d_out, void* stream);

/* The round (Sec. 3.1): candidates (Preliminaries, "DFlash one-pass marginals") -> SABA budget (Sec. 3.3)
 * -> TDES edge scores (Eq. 4-6) -> best-first expansion by path score (Eq. 13) until B_t nodes -> emission.
 *   d_logits       [batch, L, V]  drafter logits, dtype cfg.logits_dtype
 *   d_hidden       [batch, L, hidden_dim], dtype cfg.hidden_dtype; may be NULL iff d_fixed_budget != NULL
 *   d_root_token   [batch] last committed token (parent of the depth-1 edges)
 *   d_hist         [batch] hist_t = mean of the last w accepted lengths (Eq. 15); may be NULL iff fixed budget
 *   d_prefix_len   [batch] tokens in the prefix x^(t), the root included
 *   d_fixed_budget [batch] or NULL.  NULL: B_t from SABA.  Else B_t = clamp(value, 0, budget_max).
 * Requires graft_set_tdes_tables unless beta == 0 (then edge = log q and no table is read). */
graft_status graft_build_trees(graft_ctx* ctx, int32_t batch, const void* d_logits, const void* d_hidden,
                               const int32_t* d_root_token, const float* d_hist, const int32_t* d_prefix_len,
                               const int32_t* d_fixed_budget, const graft_tree_out* out, void* stream);

/* The steps of the round on their own (the same kernels graft_build_trees runs), for per-step timing
 * and parity checks. */
/* Vocab pass: per (sequence, position) log-sum-exp over V and the K top-ranked tokens with their log q.
 * d_row_status [batch*L] (may be NULL) receives per row 0, GRAFT_ST_BAD_LOGITS, and / or GRAFT_ST_INTERNAL when a
 * bounded device-side wait ran out in a thread block that worked on the row (its outputs are then not valid; the
 * call itself still returns GRAFT_OK and the context stays usable).  The same holds for graft_vocab_pass_static
 * and, through the shards' pieces, for graft_vocab_pass_partial / graft_vocab_merge. */
graft_status graft_vocab_pass(graft_ctx* ctx, int32_t batch, const void* d_logits, int32_t* d_topk_id,
                              float* d_topk_lp, float* d_lse, int32_t* d_row_status, void* stream);
/* TDES edge scores (Eq. 4-6) from candidates: d_edge [batch, L, K, K]. */
graft_status graft_tdes_edges(graft_ctx* ctx, int32_t batch, const int32_t* d_topk_id, const float* d_topk_lp,
                              const int32_t* d_root_token, float* d_edge, void* stream);

/* Allocation-free vocab pass (the paper has no counterpart: this entry point exists for the host side only).
 * Same computation and outputs as graft_vocab_pass, but it needs no context and calls no cudaMalloc, cudaFree
 * or other allocating routine: the kernel's scratch (records of rows shared between CTAs, per-row arrival
 * counters) lives in a static device array inside the library (about 0.4 MB, held by every GPU that loads the
 * library until the process exits).  It is meant for callers that cannot let a library allocate -- a serving
 * process that gave all device memory to its own pool at start-up, or code that has to stay off the driver's
 * allocation lock on its latency path.
 *   Limits: batch * L <= 16384 rows and at most 512 CTAs (the kernel launches one per SM); beyond them
 *   GRAFT_ERR_UNSUPPORTED.
 *   d_row_status [batch * L] is required here.
 *   The first call on each device looks up the array's device address and sets the kernel's shared-memory
 *   attribute; make that first call before any stream capture begins.
 *   All calls on a device share the one array: two calls whose kernels overlap on the GPU (different streams
 *   without ordering) race on it.  Calls ordered on one stream are fine; each clears what must start at zero. */
graft_status graft_vocab_pass_static(int32_t batch, int32_t L, int32_t V, int32_t K, graft_dtype logits_dtype,
                                     const void* d_logits, int32_t* d_topk_id, float* d_topk_lp, float* d_lse,
                                     int32_t* d_row_status, void* stream);

/* Vocabulary-parallel vocab pass (the logits of a tensor-parallel LM head are split over V across GPUs).  Each GPU runs
 * graft_vocab_pass_partial on its shard: per row it leaves the log-sum-exp pieces and the K best keys of the shard
 * (token ids local to the shard).  The partials of all shards, gathered into one buffer in shard order (one NCCL
 * all-gather of 280 bytes per row and shard; they land in local memory first), are merged by graft_vocab_merge into
 * the outputs graft_vocab_pass gives for the full row: the same candidates (value descending, global id
 * ascending), log q over the whole vocabulary.  The context of graft_vocab_pass_partial is one created with V =
 * the shard's width (and K = min(K, width) when a shard is narrower than K); graft_vocab_merge uses only K and L
 * of its context.
 *   d_out     [batch*L] partials of this shard
 *   d_parts   [n_shards, batch*L] partials of all shards;  h_v_offset [n_shards] first global id of each shard
 * (The paper has one drafter on one GPU; this is the one-exchange sharding of its dominant step.) */
typedef struct {
    double c;          /* reference exponent (log2 domain) */
    double s;          /* sum_v 2^(z_v log2(e) - c) over the shard */
    uint32_t vmax_ord; /* largest logit of the shard, as an order-preserving integer */
    uint32_t nkeys;    /* valid keys (min(K, shard width)); bit 31: a bounded device-side wait ran out while this
                          shard was scanned (graft_vocab_merge reports it as GRAFT_ST_INTERNAL) */
    uint64_t keys[32]; /* (order-preserving value << 32) | (0xFFFFFFFF - local id), descending */
} graft_vocab_partial;
graft_status graft_vocab_pass_partial(graft_ctx* ctx, int32_t batch, const void* d_logits_shard,
                                      graft_vocab_partial* d_out, void* stream);
graft_status graft_vocab_merge(graft_ctx* ctx, int32_t batch, int32_t n_shards, const graft_vocab_partial* d_parts,
                               const int32_t* h_v_offset, int32_t* d_topk_id, float* d_topk_lp, float* d_lse,
                               int32_t* d_row_status, void* stream);

/* Acceptance walk (Preliminaries, "Speculative decoding": a_t; "Tree-based speculative decoding": the longest
 * accepted path is committed).  d_target_next [batch, Nmax]: d_target_next[b, i] is the target model's next token
 * after node i (all Nmax entries of a sequence are read; those at or beyond its node count may hold anything).  The tree
 * must be in the level order graft_build_trees emits (parent indices never decrease along the node index).
 * Starting at the root, follow the child whose token equals target_next of the current node.
 *   d_accept_len  [batch]     number of accepted draft tokens a_t (bonus token not counted)
 *   d_accept_path [batch, L]  node indices of the accepted path, -1 padded
 *   d_bonus_token [batch]     target_next of the last accepted node */
graft_status graft_accept(graft_ctx* ctx, int32_t batch, const graft_tree_out* trees, const int32_t* d_target_next,
                          int32_t* d_accept_len, int32_t* d_accept_path, int32_t* d_bonus_token, void* stream);

/* Acceptance history on the device (Eq. 15: hist_t = mean of the last w accepted lengths), so that a decoding loop
 * needs no host round trip between graft_accept and the next graft_build_trees.  After this call every
 * graft_accept also appends a_t of sequence b to d_window[b] (a ring of w int32, caller-owned, start it zeroed),
 * advances d_count[b] (int32 rounds seen, start at 0) and writes d_hist[b] = mean of the last min(count, w)
 * lengths (the paper does not say what hist is before w rounds exist; 0 before the first).  Pass d_hist as the
 * d_hist argument of the next graft_build_trees.  w in [1, 64]; w = 0 (pointers ignored) switches it off.
 * Host-only call; the buffers are borrowed until it is called again or the context is destroyed. */
graft_status graft_set_hist_window(graft_ctx* ctx, int32_t w, int32_t* d_window, int32_t* d_count, float* d_hist);

/* TDES training objective, forward and backward (Sec. 3.2 "Training", Eq. 7-12), on traces resident on the device.
 * Every pointer of graft_tdes_traces is a DEVICE pointer (borrowed for the call); a list with n = 0 may be NULL.
 *   groups (distribution level, Eq. 7-9): d_g_parent [n_groups] parent token, d_g_depth [n_groups] depth d in 1..L,
 *     d_g_child [n_groups, K] the K children C_{p,d} (K = cfg.K), d_g_logq [n_groups, K] draft log q_d(c),
 *     d_g_ztgt [n_groups, K] target-model logits z_tgt[p, c];
 *   pairs (Eq. 10): d_pairs [n_pairs, 6] = (p+, c+, d+, p-, c-, d-), a target-compatible edge and an alternative;
 *   edges (Eq. 11): d_edges [n_edges, 4] = (p, c, d, y), y = 1 when c is the target's next token under p. */
typedef struct graft_tdes_traces {
    int32_t n_groups;
    const int32_t* d_g_parent;
    const int32_t* d_g_depth;
    const int32_t* d_g_child;
    const float* d_g_logq;
    const float* d_g_ztgt;
    int32_t n_pairs;
    const int32_t* d_pairs;
    int32_t n_edges;
    const int32_t* d_edges;
} graft_tdes_traces;

typedef struct graft_tdes_loss_config {
    float gamma;       /* margin of Eq. 10 */
    float w1;          /* weight of the positive edges in Eq. 11 */
    float lambda_kl;   /* Eq. 12 */
    float lambda_pair;
    float lambda_bce;
} graft_tdes_loss_config;

/* With the scorer of Eq. 6 taken from the context (graft_set_tdes_tables: P, C, u, s):
 *   d_loss [4] (fp64, overwritten) = L_KL, L_pair, L_BCE (each the mean over its items, 0 for an empty list) and
 *     L = lambda_KL L_KL + lambda_pair L_pair + lambda_BCE L_BCE;
 *   d_gP, d_gC [V, m], d_gu [L, m], d_gs [1] (fp32, 16-byte aligned): the gradient of L with respect to the table
 *     rows P[v] = g_p(e_v), C[v] = g_c(e_v), the depth embeddings and the scale is ADDED to them (the caller zeroes
 *     them; the additions are atomic and their order is not fixed, so results repeat only up to fp32 rounding).
 *     All four NULL: losses only.  (The gradient for the weights of g_p is then gP^T E, one matrix product with
 *     the frozen embeddings, left to the caller.)
 *   d_skipped [1] or NULL (overwritten): items left out because a token id is outside [0, V) or a depth outside
 *     [1, L]; they still count in the means' denominators.
 * fp32 arithmetic, fp64 loss sums.  GRAFT_ERR_STATE before graft_set_tdes_tables; GRAFT_ERR_UNSUPPORTED for m > 512;
 * GRAFT_ERR_INVALID_ARG for a NULL list with n > 0, a negative n, or only some of the gradient pointers NULL. */
graft_status graft_tdes_loss(graft_ctx* ctx, const graft_tdes_traces* traces, const graft_tdes_loss_config* cfg,
                             double* d_loss, int32_t* d_skipped, float* d_gP, float* d_gC, float* d_gu, float* d_gs,
                             void* stream);

/* Least-squares fit of the SABA gain and cost models (Eq. 16, 17) to replay logs resident on the device.  The paper
 * fits them on held-out prompts by same-prefix budget replay without giving the procedure; this is ordinary least
 * squares on n logged rounds:
 *   d_state [n, 3] fp32 (conf, degen, hist of Eq. 15), d_budget [n] int32 B, d_gain [n] fp32 (the share of the
 *   attainable accepted length that budget B reached, in [0, 1]), d_prefix_len [n] int32, d_latency [n] fp32 (the
 *   round's cost in the unit C_t is wanted in).
 *   Gain: a logged 0 < g < 1 gives tau = -B / ln(1 - g); (phi, bias) minimise sum (tau - phi . s - bias)^2 (rounds
 *   with g <= 0 or g >= 1 are left out).  Cost: (c0, c1, c2) minimise sum (T - c0 - c1 B - c2 B prefix)^2.
 *   d_out [10] fp64 (overwritten): phi_conf, phi_degen, phi_hist, phi_bias, c0, c1, c2, rounds used for the gain
 *   fit, rounds used for the cost fit, status (bit 0: gain system singular or fewer than 4 rounds, bit 1: cost
 *   system singular or fewer than 3; the parameters of a failed fit are 0).  The values go into graft_saba_params
 *   on the host (graft_set_saba).  fp64 arithmetic. */
graft_status graft_saba_fit(graft_ctx* ctx, int64_t n, const float* d_state, const int32_t* d_budget,
                            const float* d_gain, const int32_t* d_prefix_len, const float* d_latency, double* d_out,
                            void* stream);

/* Host-buffer form of graft_build_trees for end-to-end use: every pointer here is a HOST pointer (pinned
 * memory makes the copies asynchronous).  Copies the inputs host->device into context-owned staging buffers
 * (allocated on first use, sized for max_batch), runs the same kernels as graft_build_trees, copies
 * n_nodes, budget, status, token, parent, depth, position, path_score and mask device->host into h_out's
 * arrays, and synchronises `stream` before returning.  h_out's optional fields must be NULL. */
graft_status graft_build_trees_host(graft_ctx* ctx, int32_t batch, const void* h_logits, const void* h_hidden,
                                    const int32_t* h_root_token, const float* h_hist, const int32_t* h_prefix_len,
                                    const int32_t* h_fixed_budget, const graft_tree_out* h_out, void* stream);

/* Number of kernels the library has launched through this context since creation. */
uint64_t graft_launch_count(const graft_ctx* ctx);

/* Per-kernel device timing of graft_build_trees.  graft_set_timing(ctx, 1) makes every later call record
 * CUDA events on its stream around the vocab-pass kernel, the edge-score kernel and the tree kernel (a ring
 * of the last 64 calls) and resets the call count; graft_set_timing(ctx, 2) does the same without the reset
 * (to sample some calls of a longer run), 0 stops recording.  graft_read_timing waits for the newest recorded
 * call and returns the number of calls summed (at most 64) and the summed milliseconds of each kernel. */
graft_status graft_set_timing(graft_ctx* ctx, int32_t enable);
graft_status graft_read_timing(graft_ctx* ctx, int32_t* n_calls, float* vocab_ms, float* tdes_ms, float* tree_ms);

const char* graft_status_str(graft_status s);
const char* graft_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GRAFT_H_ */
