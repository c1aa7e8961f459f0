// SABA: the budget of one sequence from its decoding state (Sec. 3.3, Eq. 14-17), by one warp in fp64.
//
//   conf  = (1/L) sum_d q_d(c_d^(1)),  degen = mean_d r_d + (r_{L-1} - r_1),  hist: the caller's            (Eq. 15)
//   tau   = phi . (conf, degen, hist) + bias, clamped below at tau_min
//   G(B)  = 1 - exp(-B / tau)                                                                                 (Eq. 16)
//   C(B)  = c0 + c1 B + c2 B prefix, or a piecewise-linear table                                              (Eq. 17)
//   B_t   = argmax over the budget grid of G / C, the smaller budget on a tie                                 (Eq. 14)
// Shared by the edge-score kernel (whose depth-0 CTA of a sequence has little else to do) and the tree kernel (when
// no edge-score kernel runs ahead of it), so that the budget has the same bits wherever it was computed.
#pragma once
#include "common.cuh"
#include "internal.h"

namespace graft {

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

// Every lane of one warp calls this; every lane returns the same result.
//   row_status, topk_lp, cosv: this sequence's [L], [L, K], [L-1] (cosv in shared or global memory)
//   fixed_budget: NULL selects SABA, else the sequence's budget is *fixed_budget clamped to [0, bmax]
__device__ __forceinline__ SabaResult saba_warp(const SabaDev& saba, int bmin, int bmax, int bstep, int L, int K,
                                                const int32_t* row_status, const int32_t* vp_err,
                                                const float* topk_lp, const double* cosv, const float* hist_p,
                                                const int32_t* prefix_p, const int32_t* fixed_budget, int lane) {
    SabaResult r;
    // everything that comes from global memory is asked for first
    int st = 0;
    for (int j = lane; j < L; j += 32) st |= row_status[j];
    const int err = vp_err[0];
    const bool use_saba = fixed_budget == nullptr;
    double conf = 0.0, rs = 0.0, c_first = 0.0, c_last = 0.0;
    float hist_f = 0.f;
    int prefix_i = 0, fixed = 0;
    if (use_saba) {
        for (int j = lane; j < L; j += 32) conf += exp((double)topk_lp[(size_t)j * K]);
        for (int j = lane; j < L - 1; j += 32) rs += cosv[j];
        if (L >= 2) {
            c_first = cosv[0];
            c_last = cosv[L - 2];
        }
        hist_f = hist_p[0];
        prefix_i = prefix_p[0];
    } else {
        fixed = fixed_budget[0];
    }
    st = __reduce_or_sync(0xFFFFFFFFu, st);
    if (err & 1) st |= GRAFT_ST_INTERNAL;
    r.budget = 0;
    r.state[0] = r.state[1] = r.state[2] = r.state[3] = 0.f;
    if (!(st & GRAFT_ST_BAD_LOGITS)) {
        if (!use_saba) {
            r.budget = fixed < 0 ? 0 : (fixed > bmax ? bmax : fixed);
        } else {
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                conf += __shfl_xor_sync(0xFFFFFFFFu, conf, d);
                rs += __shfl_xor_sync(0xFFFFFFFFu, rs, d);
            }
            conf /= (double)L;
            double degen = 0.0;
            if (L >= 2) degen = rs / (double)(L - 1) + (c_last - c_first);
            const double hist = (double)hist_f;
            double tau = saba.phi_conf * conf + saba.phi_degen * degen + saba.phi_hist * hist + saba.phi_bias;
            if (!(tau >= saba.tau_min)) {
                tau = saba.tau_min;
                st |= GRAFT_ST_TAU_CLAMPED;
            }
            const double prefix = (double)prefix_i;
            double ubest = -INFINITY;
            int bbest = bmin;
            for (int B = bmin + lane * bstep; B <= bmax; B += 32 * bstep) {
                const double G = 1.0 - exp(-(double)B / tau);
                const double u = G / saba_cost(saba, (double)B, prefix);
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
            r.budget = bbest;
            r.state[0] = (float)conf;
            r.state[1] = (float)degen;
            r.state[2] = (float)hist;
            r.state[3] = (float)tau;
        }
    }
    r.status = st;
    return r;
}

}  // namespace graft
