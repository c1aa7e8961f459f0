/*
 * GRAFT TDES training objective -- CPU ORACLE (test infrastructure, not product code).
 *
 * O8  oracle_tdes_loss: the three supervision signals of the TDES scorer and their weighted sum
 * (Sec. 3.2 "Training", Eq. 7-12), with the gradients with respect to everything the scorer of
 * Eq. 6 is made of: the cached projections P[v] = g_p(e_v) and C[v] = g_c(e_v), the depth
 * embeddings u_d and the scale s.  (The gradient with respect to the weights of g_p is then
 * gP^T E, a plain matrix product with the frozen embeddings, and is not part of this function.)
 * Plain loops in fp64, in the paper's order and notation; shares no code with the CUDA library.
 *
 *   f(p,c,d)      = s (P[p] + u_d)^T (C[c] + u_d) / sqrt(m)                                  (Eq. 6)
 *   pi_tgt(c)     = softmax_c z_tgt[p,c]                                                      (Eq. 7)
 *   pi_theta(c)   = softmax_c (log q_d(c) + f(p,c,d))                                         (Eq. 8)
 *   L_KL          = mean over groups (p,d) of KL(pi_tgt || pi_theta)                          (Eq. 9)
 *   L_pair        = mean over pairs of softplus(gamma - f(v+) + f(v-))                        (Eq. 10)
 *   L_BCE         = - mean over edges of [w1 y log sigma(f) + (1 - y) log(1 - sigma(f))]      (Eq. 11)
 *   L             = lambda_KL L_KL + lambda_pair L_pair + lambda_BCE L_BCE                    (Eq. 12)
 *
 * The expectations are sample means over the items given (an empty list contributes 0).  Depths
 * are d = 1..L and use row d-1 of u.  The gradients are those of L and are ADDED to gP, gC, gu,
 * gs (the caller zeroes them).
 *
 * Pins (tests/test_oracle_tdes_loss.py): each loss against the library routine it reduces to
 * (torch kl_div, softplus, binary_cross_entropy_with_logits with pos_weight) on scores computed
 * by a matrix product; hand-computed values of a two-child, m = 1 example; KL = 0 when the draft
 * already equals the target and f is constant over the children; every gradient array against
 * central finite differences of the loss; the whole gradient against reverse-mode automatic
 * differentiation of the plain definition in fp64.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

typedef struct {
    double gamma, w1, lambda_kl, lambda_pair, lambda_bce;
} orc_tdes_loss_cfg;

static double orc_f(const float *P, const float *C, const float *u, double s, int m, int32_t p, int32_t c, int d) {
    double acc = 0.0;
    for (int k = 0; k < m; ++k)
        acc += ((double)P[(size_t)p * m + k] + (double)u[(size_t)(d - 1) * m + k]) *
               ((double)C[(size_t)c * m + k] + (double)u[(size_t)(d - 1) * m + k]);
    return s * acc / sqrt((double)m);
}

/* add gf * df/d(.) of one edge (p, c, d) to the gradient arrays */
static void orc_f_backward(const float *P, const float *C, const float *u, double s, int m, int32_t p, int32_t c,
                           int d, double gf, double *gP, double *gC, double *gu, double *gs) {
    const double k0 = s / sqrt((double)m);
    double dot = 0.0;
    for (int k = 0; k < m; ++k) {
        const double a = (double)P[(size_t)p * m + k] + (double)u[(size_t)(d - 1) * m + k];
        const double b = (double)C[(size_t)c * m + k] + (double)u[(size_t)(d - 1) * m + k];
        gP[(size_t)p * m + k] += gf * k0 * b;
        gC[(size_t)c * m + k] += gf * k0 * a;
        gu[(size_t)(d - 1) * m + k] += gf * k0 * (a + b);
        dot += a * b;
    }
    *gs += gf * dot / sqrt((double)m);
}

static double orc_softplus(double x) { return x > 0.0 ? x + log1p(exp(-x)) : log1p(exp(x)); }
static double orc_sigmoid(double x) { return x >= 0.0 ? 1.0 / (1.0 + exp(-x)) : exp(x) / (1.0 + exp(x)); }

/*
 * groups: n_groups x (parent token, depth, K child tokens, K draft log-probabilities, K target logits)
 * pairs:  n_pairs  x (p+, c+, d+, p-, c-, d-)
 * edges:  n_edges  x (p, c, d, y)
 * loss[4] = L_KL, L_pair, L_BCE, L.  gP, gC [V,m], gu [L,m], gs [1] in fp64 (may all be NULL: loss only).
 */
int oracle_tdes_loss(const float *P, const float *C, const float *u, double s, int V, int L, int m, int K,
                     int n_groups, const int32_t *g_parent, const int32_t *g_depth, const int32_t *g_child,
                     const float *g_logq, const float *g_ztgt, int n_pairs, const int32_t *pairs, int n_edges,
                     const int32_t *edges, const orc_tdes_loss_cfg *cfg, double *loss, double *gP, double *gC,
                     double *gu, double *gs) {
    const int grad = gP && gC && gu && gs;
    double l_kl = 0.0, l_pair = 0.0, l_bce = 0.0;
    double *f = (double *)malloc(sizeof(double) * (size_t)(3 * (K > 0 ? K : 1)));
    if (!f) return -1;
    double *pt = f + K, *ph = f + 2 * K;
    (void)V;
    /* distribution level (Eq. 7-9) */
    for (int g = 0; g < n_groups; ++g) {
        const int32_t p = g_parent[g];
        const int d = g_depth[g];
        if (d < 1 || d > L) { free(f); return -2; }
        double zmax = -INFINITY, amax = -INFINITY;
        for (int c = 0; c < K; ++c) {
            f[c] = orc_f(P, C, u, s, m, p, g_child[(size_t)g * K + c], d);
            const double a = (double)g_logq[(size_t)g * K + c] + f[c];
            if (a > amax) amax = a;
            if ((double)g_ztgt[(size_t)g * K + c] > zmax) zmax = (double)g_ztgt[(size_t)g * K + c];
        }
        double zsum = 0.0, asum = 0.0;
        for (int c = 0; c < K; ++c) {
            zsum += exp((double)g_ztgt[(size_t)g * K + c] - zmax);
            asum += exp((double)g_logq[(size_t)g * K + c] + f[c] - amax);
        }
        double kl = 0.0;
        for (int c = 0; c < K; ++c) {
            const double log_pt = (double)g_ztgt[(size_t)g * K + c] - zmax - log(zsum);
            const double log_ph = (double)g_logq[(size_t)g * K + c] + f[c] - amax - log(asum);
            pt[c] = exp(log_pt);
            ph[c] = exp(log_ph);
            if (pt[c] > 0.0) kl += pt[c] * (log_pt - log_ph);
        }
        l_kl += kl / (double)n_groups;
        if (grad)
            for (int c = 0; c < K; ++c) /* d KL / d f_c = pi_theta(c) - pi_tgt(c) */
                orc_f_backward(P, C, u, s, m, p, g_child[(size_t)g * K + c], d,
                               cfg->lambda_kl * (ph[c] - pt[c]) / (double)n_groups, gP, gC, gu, gs);
    }
    /* pairwise level (Eq. 10) */
    for (int i = 0; i < n_pairs; ++i) {
        const int32_t *q = pairs + (size_t)i * 6;
        if (q[2] < 1 || q[2] > L || q[5] < 1 || q[5] > L) { free(f); return -2; }
        const double fp = orc_f(P, C, u, s, m, q[0], q[1], q[2]);
        const double fn = orc_f(P, C, u, s, m, q[3], q[4], q[5]);
        const double x = cfg->gamma - fp + fn;
        l_pair += orc_softplus(x) / (double)n_pairs;
        if (grad) {
            const double gx = cfg->lambda_pair * orc_sigmoid(x) / (double)n_pairs;
            orc_f_backward(P, C, u, s, m, q[0], q[1], q[2], -gx, gP, gC, gu, gs);
            orc_f_backward(P, C, u, s, m, q[3], q[4], q[5], gx, gP, gC, gu, gs);
        }
    }
    /* edge level (Eq. 11): -log sigma(f) = softplus(-f), -log(1 - sigma(f)) = softplus(f) */
    for (int i = 0; i < n_edges; ++i) {
        const int32_t *e = edges + (size_t)i * 4;
        if (e[2] < 1 || e[2] > L) { free(f); return -2; }
        const double fe = orc_f(P, C, u, s, m, e[0], e[1], e[2]);
        const double y = e[3] ? 1.0 : 0.0;
        l_bce += (cfg->w1 * y * orc_softplus(-fe) + (1.0 - y) * orc_softplus(fe)) / (double)n_edges;
        if (grad) {
            const double gfe = -cfg->w1 * y * orc_sigmoid(-fe) + (1.0 - y) * orc_sigmoid(fe);
            orc_f_backward(P, C, u, s, m, e[0], e[1], e[2], cfg->lambda_bce * gfe / (double)n_edges, gP, gC, gu, gs);
        }
    }
    loss[0] = l_kl;
    loss[1] = l_pair;
    loss[2] = l_bce;
    loss[3] = cfg->lambda_kl * l_kl + cfg->lambda_pair * l_pair + cfg->lambda_bce * l_bce; /* Eq. 12 */
    free(f);
    return 0;
}
