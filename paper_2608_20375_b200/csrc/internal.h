// Internal declarations shared by the translation units of libgraft (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/graft.h"

namespace graft {

constexpr int kMaxK = 32;
constexpr int kMaxL = 32;
constexpr int kMaxCostPts = 16;

// ---- vocab pass -----------------------------------------------------------------------------
constexpr int kVpConsumerWarps = 16;                 // streaming warps (one CTA per SM)
constexpr int kVpConsumers = kVpConsumerWarps * 32;  // 512
constexpr int kVpEpiThreads = 128;                   // four warps per epilogue group
constexpr int kVpEpiGroups = 2;                      // the groups take alternate segments
constexpr int kVpBufs = 4;                           // hand-over buffers between streaming and epilogue warps
constexpr int kVpGroups = 64;   // groups of streaming threads whose maxima bound the K-th largest element (>= kMaxK)
constexpr int kVpThreads = kVpConsumers + kVpEpiGroups * kVpEpiThreads + 64;  // + one producer warp + one cosine warp
constexpr int kVpTileBytes = 32768;                  // one ring stage (2 KiB per streaming warp)
constexpr int kVpQuantum = 2048;                     // elements; granularity of the work partition
constexpr int kVpCandCap = 1280;                     // candidate keys held in shared memory (K chunks of 32 elements and their ties)
constexpr int kVpHitCap = 512;                       // chunk hits held in shared memory
constexpr int kVpRankCap = 256;                      // candidates ranked against each other at most

// What one CTA leaves behind for a row that it shares with other CTAs.
struct VpRecord {
    float c;      // reference exponent (log2 domain)
    float s;      // sum_v 2^(z_v log2e - c) over the segment
    float vmax;   // largest logit of the segment
    uint32_t nkeys;
    uint64_t keys[kMaxK];  // the segment's best keys, descending
};

struct VpPlan {
    int grid;            // CTAs launched
    int stages;          // ring depth
    int max_seg_tiles;   // tiles in the longest segment a CTA can get
    size_t smem_bytes;
};

struct SabaDev {
    double phi_conf, phi_degen, phi_hist, phi_bias, tau_min;
    int cost_mode;
    double c0, c1, c2;
    int n_pts;
    double pts_n[kMaxCostPts], pts_t[kMaxCostPts];
};

// Budget, status and decoding state of one sequence (Sec. 3.3), handed from the edge-score kernel to the tree kernel.
struct SabaResult {
    int32_t budget;
    int32_t status;  // OR of the rows' status words, the vocab pass's error flag, GRAFT_ST_TAU_CLAMPED
    float state[4];  // conf, degen, hist, tau
};

}  // namespace graft

struct graft_ctx {
    graft_config cfg;
    int device;
    int num_sms;
    int nmax, mask_words, grid_pts;
    bool saba_set, tdes_set;
    graft::SabaDev saba;
    const float* d_P;
    const float* d_C;
    float* d_u;  // owned copy [L, m]
    float tdes_s;
    int hist_w;            // acceptance-history window (0 = off) and the caller's buffers for it
    int32_t* hist_window;  // [max_batch, hist_w]
    int32_t* hist_count;   // [max_batch]
    float* hist_out;       // [max_batch]
    int edge_rows;  // depths [0, edge_rows) are scored by the edge-score kernel, deeper ones on demand in the tree kernel
    // scratch (one allocation)
    void* ws;
    size_t ws_bytes;
    graft::VpRecord* vp_records;  // [grid, 2]
    int* vp_row_counter;          // [max_batch * L], zero between launches
    int32_t* w_topk_id;           // [max_batch, L, K]
    float* w_topk_lp;             // [max_batch, L, K]
    float* w_lse;                 // [max_batch, L]
    int32_t* w_row_status;        // [max_batch, L]
    float* w_edge;                // [max_batch, L, K, K]
    float* w_esort;               // [max_batch, L, K, K] rows sorted by edge score
    uint8_t* w_eidx;              // [max_batch, L, K, K] child rank of each sorted entry
    double* w_cos;                // [max_batch, L] adjacent-position cosines (Eq. 15)
    graft::SabaResult* w_saba;    // [max_batch] budgets worked out by the edge-score kernel
    double* w_fit;                // [32] normal equations of graft_saba_fit and its arrival counter, zero between calls
    int32_t* w_errflag;           // [1] device-side internal error flag
    graft::VpPlan vp_plan;
    // scratch of the tensor-core table precompute (allocated on its first use: three bf16 copies of W, GEMM workspace)
    void* tables_scratch;
    size_t tables_scratch_bytes;
    // host-buffer staging (allocated on first use of graft_build_trees_host)
    void* stage;
    size_t stage_bytes;
    // bookkeeping
    uint64_t launches;
    int timing;
    cudaEvent_t ev[6];
};

namespace graft {

// Launch `kernel` so that it may overlap the tail of the kernel ahead of it in the stream (programmatic dependent
// launch).  The kernel must call pdl_wait() before it reads what that kernel wrote.
template <typename P>
inline cudaError_t launch_pdl(void (*kernel)(P), dim3 grid, dim3 block, size_t smem, cudaStream_t st, const P& params) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute at;
    at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at.val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = &at;
    lc.numAttrs = 1;
    return cudaLaunchKernelEx(&lc, kernel, params);
}

VpPlan vp_make_plan(const graft_config& cfg, int num_sms, int batch);
cudaError_t vp_configure(const graft_config& cfg, int num_sms, size_t* max_smem);
cudaError_t vp_launch(graft_ctx* ctx, int batch, const void* d_logits, int32_t* d_topk_id, float* d_topk_lp,
                      float* d_lse, int32_t* d_row_status, const void* d_hidden, double* d_cos,
                      graft_vocab_partial* d_partial, cudaStream_t st);
// d_hidden != NULL: one more warp per CTA also writes the adjacent-position cosines of the SABA state (Eq. 15)
// to d_cos [batch, L]; d_partial != NULL: the rows' pieces go there instead of the outputs (vocabulary-parallel use)
cudaError_t vp_merge_launch(graft_ctx* ctx, int batch, int n_shards, const graft_vocab_partial* d_parts,
                            const int32_t* h_v_offset, int32_t* d_topk_id, float* d_topk_lp, float* d_lse,
                            int32_t* d_row_status, cudaStream_t st);
int vp_merge_max_shards();

cudaError_t tdes_precompute_launch(graft_ctx* ctx, const void* d_emb, graft_dtype dt, int E, const float* d_W,
                                   const float* d_b, float* d_out, cudaStream_t st);
// table precompute on the tensor cores (bf16 embeddings): bf16 GEMMs with fp32 accumulation (csrc/tables_gemm.cu;
// csrc/tables_gemm_stub.cu when the library is built without a CUTLASS tree: the scratch size is then 0 and
// the FMA kernel runs instead)
size_t tables_tc_scratch_bytes(int V, int E, int m);
cudaError_t tables_tc_launch(const void* d_emb, int V, int E, int m, const float* d_W, const float* d_b, float* d_out,
                         void* d_scratch, int* launches, cudaStream_t st);
cudaError_t tdes_edges_launch(graft_ctx* ctx, int batch, const int32_t* d_topk_id, const float* d_topk_lp,
                              const int32_t* d_root_token, const int32_t* d_row_status, float* d_edge,
                              float* d_esort, uint8_t* d_eidx, int rows, SabaResult* d_saba_out, const float* d_hist,
                              const int32_t* d_prefix_len, const int32_t* d_fixed_budget, cudaStream_t st);
// depths [0, rows); d_saba_out != NULL: the depth-0 CTA of every sequence also works out its budget (Sec. 3.3) from
// the context's cosines, d_hist and d_prefix_len (or takes it from d_fixed_budget when that is not NULL)
cudaError_t tree_launch(graft_ctx* ctx, int batch, const int32_t* d_topk_id, const float* d_topk_lp,
                        const int32_t* d_row_status, const float* d_esort, const uint8_t* d_eidx, const void* d_hidden,
                        const int32_t* d_root_token, const float* d_hist, const int32_t* d_prefix_len,
                        const int32_t* d_fixed_budget, const double* d_cos, const SabaResult* d_saba_pre,
                        const graft_tree_out* out, cudaStream_t st);
cudaError_t accept_launch(graft_ctx* ctx, int batch, const graft_tree_out* trees, const int32_t* d_target_next,
                          int32_t* d_accept_len, int32_t* d_accept_path, int32_t* d_bonus, cudaStream_t st);
// TDES training objective, forward + backward (csrc/tdes_train.cu)
cudaError_t tdes_loss_launch(graft_ctx* ctx, const graft_tdes_traces* tr, const graft_tdes_loss_config* lc,
                             double* d_loss, int32_t* d_skipped, float* d_gP, float* d_gC, float* d_gu, float* d_gs,
                             cudaStream_t st);
cudaError_t tdes_loss_configure(const graft_config& cfg);
bool tdes_loss_supported(const graft_config& cfg);
cudaError_t saba_fit_launch(graft_ctx* ctx, long long n, const float* d_state, const int32_t* d_budget,
                            const float* d_gain, const int32_t* d_prefix, const float* d_latency, double* d_out,
                            cudaStream_t st);
size_t tree_smem_bytes(const graft_config& cfg);
bool tree_lazy_fits(const graft_config& cfg);  // edge scores are computed inside the tree kernel

}  // namespace graft
