// C ABI of libgraft: context, argument validation, kernel sequencing.  See include/graft.h.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "internal.h"

namespace graft {
cudaError_t tdes_edges_configure(const graft_config& cfg);
cudaError_t tree_configure(const graft_config& cfg);
size_t tdes_edges_smem(const graft_config& cfg);
}  // namespace graft

using namespace graft;

namespace {

constexpr int kTimingRing = 64;

struct Timing {
    cudaEvent_t ev[kTimingRing][4];
    bool created = false;
    uint64_t calls = 0;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

graft_status validate_config(const graft_config* c) {
    if (!c) return GRAFT_ERR_INVALID_ARG;
    if (c->max_batch < 1 || c->budget_min < 0 || c->budget_max < c->budget_min) return GRAFT_ERR_INVALID_ARG;
    if (c->logits_dtype != GRAFT_F32 && c->logits_dtype != GRAFT_BF16) return GRAFT_ERR_INVALID_ARG;
    if (c->hidden_dtype != GRAFT_F32 && c->hidden_dtype != GRAFT_BF16) return GRAFT_ERR_INVALID_ARG;
    if (!(c->beta == c->beta)) return GRAFT_ERR_INVALID_ARG;
    if (c->K < 1 || c->K > kMaxK || c->K > c->V) return GRAFT_ERR_UNSUPPORTED;
    if (c->L < 1 || c->L > kMaxL) return GRAFT_ERR_UNSUPPORTED;
    if (c->V < 1 || (long long)c->V > 2147483647LL - 64) return GRAFT_ERR_UNSUPPORTED;
    if (c->m < 4 || c->m > 512 || (c->m % 4) != 0) return GRAFT_ERR_UNSUPPORTED;
    if (c->budget_max > 1023 || c->budget_step < 1) return GRAFT_ERR_UNSUPPORTED;
    if ((size_t)c->L * c->K * c->K * 4 > 128 * 1024) return GRAFT_ERR_UNSUPPORTED;
    if (c->hidden_dim < 1) return GRAFT_ERR_UNSUPPORTED;
    if ((long long)c->max_batch * c->L > (1 << 24)) return GRAFT_ERR_UNSUPPORTED;
    return GRAFT_OK;
}

struct CtxExtra {
    Timing timing;
    // host staging for graft_build_trees_host
    char* d_in = nullptr;
    char* d_out = nullptr;
    size_t in_bytes = 0, out_bytes = 0;
};

CtxExtra* extra_of(graft_ctx* ctx) { return (CtxExtra*)ctx->stage; }

}  // namespace

extern "C" {

const char* graft_status_str(graft_status s) {
    switch (s) {
        case GRAFT_OK: return "ok";
        case GRAFT_ERR_INVALID_ARG: return "invalid argument";
        case GRAFT_ERR_UNSUPPORTED: return "size outside the supported limits";
        case GRAFT_ERR_CUDA: return "CUDA runtime error";
        case GRAFT_ERR_WORKSPACE: return "scratch allocation failed";
        case GRAFT_ERR_STATE: return "parameters not set (TDES tables or SABA)";
    }
    return "unknown status";
}



const char* graft_version(void) { return "graft-b200 0.1 (sm_100a)"; }

graft_status graft_create(const graft_config* cfg, graft_ctx** out) {
    if (!out) return GRAFT_ERR_INVALID_ARG;
    *out = nullptr;
    graft_status vs = validate_config(cfg);
    if (vs != GRAFT_OK) return vs;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return GRAFT_ERR_CUDA;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        cudaGetLastError();
        return GRAFT_ERR_CUDA;
    }
    graft_ctx* ctx = new (std::nothrow) graft_ctx();
    if (!ctx) return GRAFT_ERR_WORKSPACE;
    memset(ctx, 0, sizeof(*ctx));
    ctx->cfg = *cfg;
    ctx->device = dev;
    ctx->num_sms = prop.multiProcessorCount;
    ctx->nmax = cfg->budget_max + 1;
    ctx->mask_words = (ctx->nmax + 31) / 32;
    ctx->grid_pts = (cfg->budget_max - cfg->budget_min) / cfg->budget_step + 1;
    ctx->tdes_s = 1.0f;
    ctx->stage = new (std::nothrow) CtxExtra();
    if (!ctx->stage) {
        delete ctx;
        return GRAFT_ERR_WORKSPACE;
    }

    size_t vp_smem = 0;
    if (vp_configure(*cfg, ctx->num_sms, &vp_smem) != cudaSuccess || tdes_edges_configure(*cfg) != cudaSuccess ||
        (tdes_loss_supported(*cfg) && tdes_loss_configure(*cfg) != cudaSuccess) ||
        tree_configure(*cfg) != cudaSuccess) {
        cudaGetLastError();
        delete extra_of(ctx);
        delete ctx;
        return GRAFT_ERR_UNSUPPORTED;
    }

    const size_t B = cfg->max_batch, L = cfg->L, K = cfg->K;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off = align_up(off + bytes, 256);
        return o;
    };
    const size_t o_rec = take((size_t)ctx->num_sms * 2 * 2 * sizeof(VpRecord));
    const size_t o_cnt = take(B * L * sizeof(int));
    const size_t o_id = take(B * L * K * 4), o_lp = take(B * L * K * 4), o_lse = take(B * L * 4);
    const size_t o_rs = take(B * L * 4), o_edge = take(B * L * K * K * 4);
    const size_t o_es = take(B * L * K * K * 4), o_ei = take(B * L * K * K);
    const size_t o_u = take(L * (size_t)cfg->m * 4), o_err = take(256), o_cos = take(B * L * 8), o_saba = take(B * sizeof(SabaResult)), o_fit = take(32 * 8);
    ctx->ws_bytes = off;
    if (cudaMalloc(&ctx->ws, ctx->ws_bytes) != cudaSuccess) {
        cudaGetLastError();
        delete extra_of(ctx);
        delete ctx;
        return GRAFT_ERR_WORKSPACE;
    }
    if (cudaMemset(ctx->ws, 0, ctx->ws_bytes) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(ctx->ws);
        delete extra_of(ctx);
        delete ctx;
        return GRAFT_ERR_CUDA;
    }
    char* base = (char*)ctx->ws;
    ctx->vp_records = (VpRecord*)(base + o_rec);
    ctx->vp_row_counter = (int*)(base + o_cnt);
    ctx->w_topk_id = (int32_t*)(base + o_id);
    ctx->w_topk_lp = (float*)(base + o_lp);
    ctx->w_lse = (float*)(base + o_lse);
    ctx->w_row_status = (int32_t*)(base + o_rs);
    ctx->w_edge = (float*)(base + o_edge);
    ctx->w_esort = (float*)(base + o_es);
    ctx->w_eidx = (uint8_t*)(base + o_ei);
    ctx->d_u = (float*)(base + o_u);
    ctx->tables_scratch = nullptr;
    ctx->tables_scratch_bytes = 0;
    ctx->hist_w = 0;
    ctx->hist_window = nullptr;
    ctx->hist_count = nullptr;
    ctx->hist_out = nullptr;
    ctx->edge_rows = tree_lazy_fits(*cfg) ? (cfg->L < 8 ? cfg->L : 8) : cfg->L;
    ctx->w_errflag = (int32_t*)(base + o_err);
    ctx->w_cos = (double*)(base + o_cos);
    ctx->w_saba = (SabaResult*)(base + o_saba);
    ctx->w_fit = (double*)(base + o_fit);
    *out = ctx;
    return GRAFT_OK;
}

graft_status graft_destroy(graft_ctx* ctx) {
    if (!ctx) return GRAFT_ERR_INVALID_ARG;
    CtxExtra* ex = extra_of(ctx);
    if (ex) {
        if (ex->timing.created)
            for (int i = 0; i < kTimingRing; ++i)
                for (int j = 0; j < 4; ++j) cudaEventDestroy(ex->timing.ev[i][j]);
        if (ex->d_in) cudaFree(ex->d_in);
        if (ex->d_out) cudaFree(ex->d_out);
        delete ex;
    }
    if (ctx->tables_scratch) cudaFree(ctx->tables_scratch);
    if (ctx->ws) cudaFree(ctx->ws);
    delete ctx;
    return GRAFT_OK;
}

size_t graft_nmax(const graft_ctx* ctx) { return ctx ? (size_t)ctx->nmax : 0; }
size_t graft_mask_words(const graft_ctx* ctx) { return ctx ? (size_t)ctx->mask_words : 0; }
uint64_t graft_launch_count(const graft_ctx* ctx) { return ctx ? ctx->launches : 0; }

graft_status graft_set_saba(graft_ctx* ctx, const graft_saba_params* p) {
    if (!ctx || !p) return GRAFT_ERR_INVALID_ARG;
    if (p->cost_mode != 0 && p->cost_mode != 1) return GRAFT_ERR_INVALID_ARG;
    SabaDev s;
    memset(&s, 0, sizeof s);
    s.phi_conf = p->phi_conf;
    s.phi_degen = p->phi_degen;
    s.phi_hist = p->phi_hist;
    s.phi_bias = p->phi_bias;
    s.tau_min = p->tau_min;
    s.cost_mode = p->cost_mode;
    s.c0 = p->c0;
    s.c1 = p->c1;
    s.c2 = p->c2;
    if (!(p->tau_min > 0.0f)) return GRAFT_ERR_INVALID_ARG;
    if (p->cost_mode == 1) {
        if (p->n_pts < 1 || p->n_pts > kMaxCostPts || !p->pts_n || !p->pts_t) return GRAFT_ERR_INVALID_ARG;
        for (int i = 0; i < p->n_pts; ++i) {
            if (i > 0 && !(p->pts_n[i] > p->pts_n[i - 1])) return GRAFT_ERR_INVALID_ARG;
            s.pts_n[i] = p->pts_n[i];
            s.pts_t[i] = p->pts_t[i];
        }
        s.n_pts = p->n_pts;
    }
    ctx->saba = s;
    ctx->saba_set = true;
    return GRAFT_OK;
}

graft_status graft_set_tdes_tables(graft_ctx* ctx, const float* d_P, const float* d_C, const float* d_u, float s,
                                   void* stream) {
    if (!ctx || !d_P || !d_C || !d_u) return GRAFT_ERR_INVALID_ARG;
    if (((uintptr_t)d_P & 15) || ((uintptr_t)d_C & 15)) return GRAFT_ERR_INVALID_ARG;
    if (!(s > 0.0f)) return GRAFT_ERR_INVALID_ARG;
    if (cudaMemcpyAsync(ctx->d_u, d_u, (size_t)ctx->cfg.L * ctx->cfg.m * 4, cudaMemcpyDeviceToDevice,
                        (cudaStream_t)stream) != cudaSuccess) {
        cudaGetLastError();
        return GRAFT_ERR_CUDA;
    }
    ctx->d_P = d_P;
    ctx->d_C = d_C;
    ctx->tdes_s = s;
    ctx->tdes_set = true;
    return GRAFT_OK;
}

graft_status graft_set_edge_rows(graft_ctx* ctx, int32_t rows) {
    if (!ctx || rows < 0 || rows > ctx->cfg.L) return GRAFT_ERR_INVALID_ARG;
    if (rows < ctx->cfg.L && !tree_lazy_fits(ctx->cfg)) return GRAFT_ERR_INVALID_ARG;
    ctx->edge_rows = rows;
    return GRAFT_OK;
}

int32_t graft_edge_rows(const graft_ctx* ctx) { return ctx ? ctx->edge_rows : -1; }

graft_status graft_tdes_precompute(graft_ctx* ctx, const void* d_emb, graft_dtype emb_dtype, int32_t E,
                                   const float* d_W, const float* d_b, float* d_out, void* stream) {
    if (!ctx || !d_emb || !d_W || !d_out || E < 1) return GRAFT_ERR_INVALID_ARG;
    if (emb_dtype != GRAFT_F32 && emb_dtype != GRAFT_BF16) return GRAFT_ERR_INVALID_ARG;
    // bf16 embeddings: the tensor cores (the embeddings are exact operands, W goes in as three bf16 parts); its
    // scratch is allocated on the first such call (this is the once-per-model setup step, not the round)
    if (emb_dtype == GRAFT_BF16) {
        const size_t need = tables_tc_scratch_bytes(ctx->cfg.V, E, ctx->cfg.m);
        if (need > 0) {
            if (ctx->tables_scratch_bytes < need) {
                if (ctx->tables_scratch) cudaFree(ctx->tables_scratch);
                ctx->tables_scratch = nullptr;
                ctx->tables_scratch_bytes = 0;
                if (cudaMalloc(&ctx->tables_scratch, need) != cudaSuccess) {
                    cudaGetLastError();
                    return GRAFT_ERR_WORKSPACE;
                }
                ctx->tables_scratch_bytes = need;
            }
            int n = 0;
            const cudaError_t e = tables_tc_launch(d_emb, ctx->cfg.V, E, ctx->cfg.m, d_W, d_b, d_out, ctx->tables_scratch, &n,
                                               (cudaStream_t)stream);
            ctx->launches += (uint64_t)n;
            if (e == cudaSuccess) return GRAFT_OK;
            if (e != cudaErrorNotSupported) {
                cudaGetLastError();
                return GRAFT_ERR_CUDA;
            }
        }
    }
    if (tdes_precompute_launch(ctx, d_emb, emb_dtype, E, d_W, d_b, d_out, (cudaStream_t)stream) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    return GRAFT_OK;
}

graft_status graft_vocab_pass(graft_ctx* ctx, int32_t batch, const void* d_logits, int32_t* d_topk_id,
                              float* d_topk_lp, float* d_lse, int32_t* d_row_status, void* stream) {
    if (!ctx || !d_logits || !d_topk_id || !d_topk_lp || !d_lse) return GRAFT_ERR_INVALID_ARG;
    if (batch < 1 || batch > ctx->cfg.max_batch) return GRAFT_ERR_INVALID_ARG;
    const int esz = ctx->cfg.logits_dtype == GRAFT_BF16 ? 2 : 4;
    if ((uintptr_t)d_logits % esz) return GRAFT_ERR_INVALID_ARG;
    if (vp_launch(ctx, batch, d_logits, d_topk_id, d_topk_lp, d_lse, d_row_status ? d_row_status : ctx->w_row_status,
                  nullptr, nullptr, nullptr, (cudaStream_t)stream) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    return GRAFT_OK;
}

graft_status graft_saba_fit(graft_ctx* ctx, int64_t n, const float* d_state, const int32_t* d_budget,
                            const float* d_gain, const int32_t* d_prefix_len, const float* d_latency, double* d_out,
                            void* stream) {
    if (!ctx || n < 1 || !d_state || !d_budget || !d_gain || !d_prefix_len || !d_latency || !d_out)
        return GRAFT_ERR_INVALID_ARG;
    if (saba_fit_launch(ctx, (long long)n, d_state, d_budget, d_gain, d_prefix_len, d_latency, d_out,
                        (cudaStream_t)stream) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    return GRAFT_OK;
}

graft_status graft_tdes_loss(graft_ctx* ctx, const graft_tdes_traces* tr, const graft_tdes_loss_config* lc,
                             double* d_loss, int32_t* d_skipped, float* d_gP, float* d_gC, float* d_gu, float* d_gs,
                             void* stream) {
    if (!ctx || !tr || !lc || !d_loss) return GRAFT_ERR_INVALID_ARG;
    if (!ctx->tdes_set) return GRAFT_ERR_STATE;
    if (!tdes_loss_supported(ctx->cfg)) return GRAFT_ERR_UNSUPPORTED;
    if (tr->n_groups < 0 || tr->n_pairs < 0 || tr->n_edges < 0) return GRAFT_ERR_INVALID_ARG;
    if (tr->n_groups > 0 && (!tr->d_g_parent || !tr->d_g_depth || !tr->d_g_child || !tr->d_g_logq || !tr->d_g_ztgt))
        return GRAFT_ERR_INVALID_ARG;
    if ((tr->n_pairs > 0 && !tr->d_pairs) || (tr->n_edges > 0 && !tr->d_edges)) return GRAFT_ERR_INVALID_ARG;
    const int n_grad = (d_gP != nullptr) + (d_gC != nullptr) + (d_gu != nullptr) + (d_gs != nullptr);
    if (n_grad != 0 && n_grad != 4) return GRAFT_ERR_INVALID_ARG;
    if (((uintptr_t)d_gP | (uintptr_t)d_gC | (uintptr_t)d_gu) & 15) return GRAFT_ERR_INVALID_ARG;
    if (tdes_loss_launch(ctx, tr, lc, d_loss, d_skipped, d_gP, d_gC, d_gu, d_gs, (cudaStream_t)stream) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    return GRAFT_OK;
}

graft_status graft_tdes_edges(graft_ctx* ctx, int32_t batch, const int32_t* d_topk_id, const float* d_topk_lp,
                              const int32_t* d_root_token, float* d_edge, void* stream) {
    if (!ctx || !d_topk_id || !d_topk_lp || !d_root_token || !d_edge) return GRAFT_ERR_INVALID_ARG;
    if (batch < 1 || batch > ctx->cfg.max_batch) return GRAFT_ERR_INVALID_ARG;
    if (ctx->cfg.beta != 0.0f && !ctx->tdes_set) return GRAFT_ERR_STATE;
    if (tdes_edges_launch(ctx, batch, d_topk_id, d_topk_lp, d_root_token, nullptr, d_edge, ctx->w_esort, ctx->w_eidx,
                          ctx->cfg.L, nullptr, nullptr, nullptr, nullptr, (cudaStream_t)stream) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    return GRAFT_OK;
}


graft_status graft_set_timing(graft_ctx* ctx, int32_t enable) {
    if (!ctx) return GRAFT_ERR_INVALID_ARG;
    CtxExtra* ex = extra_of(ctx);
    if (enable && !ex->timing.created) {
        for (int i = 0; i < kTimingRing; ++i)
            for (int j = 0; j < 4; ++j)
                if (cudaEventCreate(&ex->timing.ev[i][j]) != cudaSuccess) return GRAFT_ERR_CUDA;
        ex->timing.created = true;
    }
    if (enable == 1) ex->timing.calls = 0;
    ctx->timing = enable ? 1 : 0;
    return GRAFT_OK;
}

graft_status graft_read_timing(graft_ctx* ctx, int32_t* n_calls, float* vocab_ms, float* tdes_ms, float* tree_ms) {
    if (!ctx || !n_calls || !vocab_ms || !tdes_ms || !tree_ms) return GRAFT_ERR_INVALID_ARG;
    CtxExtra* ex = extra_of(ctx);
    *n_calls = 0;
    *vocab_ms = *tdes_ms = *tree_ms = 0.f;
    if (!ex->timing.created) return GRAFT_ERR_STATE;
    const uint64_t n = ex->timing.calls < (uint64_t)kTimingRing ? ex->timing.calls : (uint64_t)kTimingRing;
    for (uint64_t k = 0; k < n; ++k) {
        const int slot = (int)((ex->timing.calls - 1 - k) % kTimingRing);
        if (cudaEventSynchronize(ex->timing.ev[slot][3]) != cudaSuccess) return GRAFT_ERR_CUDA;
        float a = 0, b = 0, c = 0;
        if (cudaEventElapsedTime(&a, ex->timing.ev[slot][0], ex->timing.ev[slot][1]) != cudaSuccess ||
            cudaEventElapsedTime(&b, ex->timing.ev[slot][1], ex->timing.ev[slot][2]) != cudaSuccess ||
            cudaEventElapsedTime(&c, ex->timing.ev[slot][2], ex->timing.ev[slot][3]) != cudaSuccess)
            return GRAFT_ERR_CUDA;
        *vocab_ms += a;
        *tdes_ms += b;
        *tree_ms += c;
    }
    *n_calls = (int32_t)n;
    return GRAFT_OK;
}

graft_status graft_build_trees(graft_ctx* ctx, int32_t batch, const void* d_logits, const void* d_hidden,
                               const int32_t* d_root_token, const float* d_hist, const int32_t* d_prefix_len,
                               const int32_t* d_fixed_budget, const graft_tree_out* out, void* stream) {
    if (!ctx || !out || !d_logits || !d_root_token || !d_prefix_len) return GRAFT_ERR_INVALID_ARG;
    if (batch < 1 || batch > ctx->cfg.max_batch) return GRAFT_ERR_INVALID_ARG;
    if (!out->d_n_nodes || !out->d_budget || !out->d_token || !out->d_parent || !out->d_depth || !out->d_position ||
        !out->d_path_score || !out->d_mask || !out->d_status)
        return GRAFT_ERR_INVALID_ARG;
    const bool use_saba = d_fixed_budget == nullptr;
    if (use_saba && (!d_hidden || !d_hist)) return GRAFT_ERR_INVALID_ARG;
    if (use_saba && !ctx->saba_set) return GRAFT_ERR_STATE;
    if (ctx->cfg.beta != 0.0f && !ctx->tdes_set) return GRAFT_ERR_STATE;
    const int esz = ctx->cfg.logits_dtype == GRAFT_BF16 ? 2 : 4;
    if ((uintptr_t)d_logits % esz) return GRAFT_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    CtxExtra* ex = extra_of(ctx);
    cudaEvent_t* ev = nullptr;
    if (ctx->timing && ex->timing.created) ev = ex->timing.ev[ex->timing.calls % kTimingRing];

    int32_t* ids = out->d_topk_id ? out->d_topk_id : ctx->w_topk_id;
    float* lps = out->d_topk_lp ? out->d_topk_lp : ctx->w_topk_lp;
    float* lse = out->d_lse ? out->d_lse : ctx->w_lse;
    float* edge = out->d_edge;  // NULL: the edge kernel writes only the sorted rows the tree kernel reads

    if (ev) cudaEventRecord(ev[0], st);
    if (vp_launch(ctx, batch, d_logits, ids, lps, lse, ctx->w_row_status, use_saba ? d_hidden : nullptr, ctx->w_cos,
                  nullptr, st) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    if (ev) cudaEventRecord(ev[1], st);
    // Edge scores of Eq. 4-6: the kernel scores the depths [0, edge_rows) for every sequence (all depths when the
    // caller asks for the score array); the tree kernel scores deeper rows itself if an expansion gets that far.
    // The depth-0 CTA of each sequence in that kernel also works out the sequence's budget (Sec. 3.3), which the tree
    // kernel then only reads; without an edge-score kernel the tree kernel does it itself.
    const int rows = out->d_edge ? ctx->cfg.L : ctx->edge_rows;
    if (rows > 0 && tdes_edges_launch(ctx, batch, ids, lps, d_root_token, ctx->w_row_status, edge, ctx->w_esort,
                                      ctx->w_eidx, rows, ctx->w_saba, d_hist, d_prefix_len, d_fixed_budget,
                                      st) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    if (ev) cudaEventRecord(ev[2], st);
    if (tree_launch(ctx, batch, ids, lps, ctx->w_row_status, ctx->w_esort, ctx->w_eidx, d_hidden, d_root_token, d_hist,
                    d_prefix_len, d_fixed_budget, ctx->w_cos, rows > 0 ? ctx->w_saba : nullptr, out, st) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    if (ev) {
        cudaEventRecord(ev[3], st);
        ex->timing.calls += 1;
    }
    return GRAFT_OK;
}

graft_status graft_accept(graft_ctx* ctx, int32_t batch, const graft_tree_out* trees, const int32_t* d_target_next,
                          int32_t* d_accept_len, int32_t* d_accept_path, int32_t* d_bonus_token, void* stream) {
    if (!ctx || !trees || !d_target_next || !d_accept_len || !d_accept_path || !d_bonus_token)
        return GRAFT_ERR_INVALID_ARG;
    if (!trees->d_n_nodes || !trees->d_token || !trees->d_parent) return GRAFT_ERR_INVALID_ARG;
    if (batch < 1 || batch > ctx->cfg.max_batch) return GRAFT_ERR_INVALID_ARG;
    if (accept_launch(ctx, batch, trees, d_target_next, d_accept_len, d_accept_path, d_bonus_token,
                      (cudaStream_t)stream) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    return GRAFT_OK;
}

static_assert(sizeof(graft_vocab_partial) == 280, "the Python binding gathers partials as 280-byte records");

graft_status graft_vocab_pass_partial(graft_ctx* ctx, int32_t batch, const void* d_logits_shard,
                                      graft_vocab_partial* d_out, void* stream) {
    if (!ctx || !d_logits_shard || !d_out) return GRAFT_ERR_INVALID_ARG;
    if (batch < 1 || batch > ctx->cfg.max_batch) return GRAFT_ERR_INVALID_ARG;
    const int esz = ctx->cfg.logits_dtype == GRAFT_BF16 ? 2 : 4;
    if ((uintptr_t)d_logits_shard % esz || (uintptr_t)d_out % 8) return GRAFT_ERR_INVALID_ARG;
    if (vp_launch(ctx, batch, d_logits_shard, ctx->w_topk_id, ctx->w_topk_lp, ctx->w_lse, ctx->w_row_status, nullptr,
                  nullptr, d_out, (cudaStream_t)stream) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    return GRAFT_OK;
}

graft_status graft_vocab_merge(graft_ctx* ctx, int32_t batch, int32_t n_shards, const graft_vocab_partial* d_parts,
                               const int32_t* h_v_offset, int32_t* d_topk_id, float* d_topk_lp, float* d_lse,
                               int32_t* d_row_status, void* stream) {
    if (!ctx || !d_parts || !h_v_offset || !d_topk_id || !d_topk_lp || !d_lse || !d_row_status)
        return GRAFT_ERR_INVALID_ARG;
    if (batch < 1 || n_shards < 1 || n_shards > vp_merge_max_shards()) return GRAFT_ERR_INVALID_ARG;
    for (int i = 0; i < n_shards; ++i)
        if (h_v_offset[i] < 0 || (i > 0 && h_v_offset[i] <= h_v_offset[i - 1])) return GRAFT_ERR_INVALID_ARG;
    if (vp_merge_launch(ctx, batch, n_shards, d_parts, h_v_offset, d_topk_id, d_topk_lp, d_lse, d_row_status,
                        (cudaStream_t)stream) != cudaSuccess)
        return GRAFT_ERR_CUDA;
    return GRAFT_OK;
}

graft_status graft_set_hist_window(graft_ctx* ctx, int32_t w, int32_t* d_window, int32_t* d_count, float* d_hist) {
    if (!ctx || w < 0 || w > 64) return GRAFT_ERR_INVALID_ARG;
    if (w > 0 && (!d_window || !d_count || !d_hist)) return GRAFT_ERR_INVALID_ARG;
    ctx->hist_w = w;
    ctx->hist_window = w ? d_window : nullptr;
    ctx->hist_count = w ? d_count : nullptr;
    ctx->hist_out = w ? d_hist : nullptr;
    return GRAFT_OK;
}

graft_status graft_build_trees_host(graft_ctx* ctx, int32_t batch, const void* h_logits, const void* h_hidden,
                                    const int32_t* h_root_token, const float* h_hist, const int32_t* h_prefix_len,
                                    const int32_t* h_fixed_budget, const graft_tree_out* h_out, void* stream) {
    if (!ctx || !h_out || !h_logits || !h_root_token || !h_prefix_len) return GRAFT_ERR_INVALID_ARG;
    if (batch < 1 || batch > ctx->cfg.max_batch) return GRAFT_ERR_INVALID_ARG;
    if (h_out->d_topk_id || h_out->d_topk_lp || h_out->d_lse || h_out->d_edge || h_out->d_state)
        return GRAFT_ERR_INVALID_ARG;
    const bool use_saba = h_fixed_budget == nullptr;
    if (use_saba && (!h_hidden || !h_hist)) return GRAFT_ERR_INVALID_ARG;
    const graft_config& c = ctx->cfg;
    CtxExtra* ex = extra_of(ctx);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t MB = c.max_batch, L = c.L, N = ctx->nmax, W = ctx->mask_words;
    const size_t lsz = (c.logits_dtype == GRAFT_BF16 ? 2 : 4), hsz = (c.hidden_dtype == GRAFT_BF16 ? 2 : 4);
    // input staging layout
    const size_t i_logits = 0, i_hidden = align_up(i_logits + MB * L * c.V * lsz, 256),
                 i_root = align_up(i_hidden + MB * L * c.hidden_dim * hsz, 256), i_hist = align_up(i_root + MB * 4, 256),
                 i_prefix = align_up(i_hist + MB * 4, 256), i_fixed = align_up(i_prefix + MB * 4, 256),
                 i_end = align_up(i_fixed + MB * 4, 256);
    // output staging layout
    const size_t o_nn = 0, o_bud = align_up(o_nn + MB * 4, 256), o_st = align_up(o_bud + MB * 4, 256),
                 o_tok = align_up(o_st + MB * 4, 256), o_par = align_up(o_tok + MB * N * 4, 256),
                 o_dep = align_up(o_par + MB * N * 4, 256), o_pos = align_up(o_dep + MB * N * 4, 256),
                 o_sc = align_up(o_pos + MB * N * 4, 256), o_mask = align_up(o_sc + MB * N * 4, 256),
                 o_end = align_up(o_mask + MB * N * W * 4, 256);
    if (!ex->d_in) {
        if (cudaMalloc((void**)&ex->d_in, i_end) != cudaSuccess || cudaMalloc((void**)&ex->d_out, o_end) != cudaSuccess) {
            cudaGetLastError();
            if (ex->d_in) cudaFree(ex->d_in);
            ex->d_in = nullptr;
            return GRAFT_ERR_WORKSPACE;
        }
        ex->in_bytes = i_end;
        ex->out_bytes = o_end;
    }
    const size_t nb = batch;
    cudaError_t e = cudaMemcpyAsync(ex->d_in + i_logits, h_logits, nb * L * c.V * lsz, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && use_saba) {
        e = cudaMemcpyAsync(ex->d_in + i_hidden, h_hidden, nb * L * c.hidden_dim * hsz, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(ex->d_in + i_hist, h_hist, nb * 4, cudaMemcpyHostToDevice, st);
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(ex->d_in + i_root, h_root_token, nb * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ex->d_in + i_prefix, h_prefix_len, nb * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && !use_saba)
        e = cudaMemcpyAsync(ex->d_in + i_fixed, h_fixed_budget, nb * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return GRAFT_ERR_CUDA;
    }
    graft_tree_out d;
    memset(&d, 0, sizeof d);
    d.d_n_nodes = (int32_t*)(ex->d_out + o_nn);
    d.d_budget = (int32_t*)(ex->d_out + o_bud);
    d.d_status = (int32_t*)(ex->d_out + o_st);
    d.d_token = (int32_t*)(ex->d_out + o_tok);
    d.d_parent = (int32_t*)(ex->d_out + o_par);
    d.d_depth = (int32_t*)(ex->d_out + o_dep);
    d.d_position = (int32_t*)(ex->d_out + o_pos);
    d.d_path_score = (float*)(ex->d_out + o_sc);
    d.d_mask = (uint32_t*)(ex->d_out + o_mask);
    graft_status gs = graft_build_trees(
        ctx, batch, ex->d_in + i_logits, use_saba ? ex->d_in + i_hidden : nullptr, (const int32_t*)(ex->d_in + i_root),
        use_saba ? (const float*)(ex->d_in + i_hist) : nullptr, (const int32_t*)(ex->d_in + i_prefix),
        use_saba ? nullptr : (const int32_t*)(ex->d_in + i_fixed), &d, stream);
    if (gs != GRAFT_OK) return gs;
    struct {
        void* h;
        const void* dsrc;
        size_t bytes;
    } cp[] = {
        {h_out->d_n_nodes, d.d_n_nodes, nb * 4},          {h_out->d_budget, d.d_budget, nb * 4},
        {h_out->d_status, d.d_status, nb * 4},            {h_out->d_token, d.d_token, nb * N * 4},
        {h_out->d_parent, d.d_parent, nb * N * 4},        {h_out->d_depth, d.d_depth, nb * N * 4},
        {h_out->d_position, d.d_position, nb * N * 4},    {h_out->d_path_score, d.d_path_score, nb * N * 4},
        {h_out->d_mask, d.d_mask, nb * N * W * 4},
    };
    for (auto& x : cp) {
        if (!x.h) return GRAFT_ERR_INVALID_ARG;
        if (cudaMemcpyAsync(x.h, x.dsrc, x.bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
            cudaGetLastError();
            return GRAFT_ERR_CUDA;
        }
    }
    if (cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return GRAFT_ERR_CUDA;
    }
    return GRAFT_OK;
}

}  // extern "C"
