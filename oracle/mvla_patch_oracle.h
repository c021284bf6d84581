/*
 * mvla_patch_oracle.h -- plain fp64 CPU statement of Alg. 1 taken literally, patch by patch.
 *
 * TEST INFRASTRUCTURE ONLY (as mvla_oracle.h): called by the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg, never by the product path; it shares no code with the CUDA path.
 *
 * Paper: "2D or 3D: Who Governs Salience in VLA Models?"  Here a "patch" p owns one 2D image token
 * and one 3D point token (visual token p and visual token P + p of a sample with n_2d = n_3d = P),
 * and the four indicators of Alg. 1 exist PER PATCH:
 *   M^S1_{2D,3D},p : share of the L1 feature norm of the patch's 2D / 3D token (Eq. 3-1 before "avg");
 *   M^S2_2D,p      : share of the L1 norm of the 2D token's attention vector (Eq. P2D);
 *   M^S2_3D,p      : the same share for the part of the 3D token's attention vector that is
 *                    orthogonal to the 2D token's (Eq. 3-4, Eq. P3D).
 * Then, in the order of Alg. 1: temporal predictor per patch and indicator (Eqs. 8, 9), dual
 * threshold per patch (Sec. 4.1), 1-D K-Means (K = 3) on the patches' total attention with the
 * rules for background / robot / target-object patches (Sec. 4.2), candidate fusion and masks
 * (Sec. 4.4, Eq. 10).
 *
 * Parity status.  The decomposition, the indicator ratios, the K-Means step, the rule table and the
 * fusion are pinned by the CPU tests (hand-worked vectors, invariants, scikit-learn's Lloyd
 * iteration from the same start, a truth table written out from Alg. 1).  Choices the paper leaves
 * open and that therefore have no outside pin ("parity unpinned" against the paper): the K-Means
 * start (min, mean, max) and stop rule, "comprehensive attention score" = the patch's attention
 * mass, the baselines mu as means of the SMOOTHED shares, and the quantified target-object rule.
 *
 * The random numbers of the background rule (rand() < 0.9) are an INPUT: one uniform number in
 * [0, 1) per patch.
 */
#ifndef MVLA_PATCH_ORACLE_H
#define MVLA_PATCH_ORACLE_H

#include <stdint.h>

#include "mvla_oracle.h"

#ifdef __cplusplus
extern "C" {
#endif

enum { ORACLE_LABEL_BG = 0, ORACLE_LABEL_ROB = 1, ORACLE_LABEL_OBJ = 2 };

typedef struct oracle_patch_params {
    double tau_2d, tau_3d;        /* Sec. 4.1 */
    double beta;                  /* Eq. 9 */
    int32_t window_k;             /* Eq. 8 -> Eq. 9 */
    double eps_3d;                /* target-object rule: "3D response -> 0" means M^S2_3D,p < eps_3d */
    double obj_2d_min;            /* target-object rule: "2D reliance >> 0" means M^S2_2D,p > obj_2d_min */
    double bg_prune_prob;         /* background rule: pruned when u_p < bg_prune_prob (0.9) */
    int32_t kmeans_max_iter;
    int32_t cold_start_full_keep;
} oracle_patch_params;

/* Smoothed state of one (prune point, sample): steps absorbed and X^ for every patch,
 * xhat[p][0..3] = [M^S1_2D, M^S1_3D, M^S2_2D, M^S2_3D]. */
typedef struct oracle_patch_state {
    int32_t t;
    double *xhat;                 /* [P][4] */
} oracle_patch_state;

typedef struct oracle_patch_diag {
    int32_t t;
    int32_t iters;                /* K-Means assignment rounds run */
    int32_t n_label[3];           /* patches per label (bg, rob, obj) */
    int32_t k_2d, k_3d;           /* kept tokens per modality */
    double centre[3];             /* ascending */
    double mu_2d, mu_3d;          /* baselines (Sec. 4.2) */
    double kmeans_margin;         /* smallest gap between a point's two nearest centre distances seen in any round */
} oracle_patch_diag;

/* Sec. 3.2.1: the attention matrix itself.  alpha[(h * n_txt + i) * n_vis + j] = softmax over all
 * visual keys j of <q_hi, k_hj> / sqrt(d); visual tokens numbered 2D first. */
void oracle_attention(const float *q, const float *k, int32_t n_heads, int32_t head_dim,
                      const oracle_sample *s, double *alpha);

/* Eq. 3-4 for one pair of vectors of length n: a3 = para + ortho with para parallel to a2 and
 * <ortho, a2> = 0.  a2 = 0 leaves ortho = a3. */
void oracle_ortho_decompose(const double *a2, const double *a3, int32_t n, double *para, double *ortho);

/* Per-patch indicators.  alpha as above ([rows_a = H n_txt][n_vis = 2P]); l1 [2P] feature norms.
 * x[p][0..3] = [M^S1_2D, M^S1_3D, M^S2_2D, M^S2_3D] (Eq. 3-1, P2D, P3D per patch). */
void oracle_patch_indicators(const double *alpha, int32_t rows_a, int32_t n_patch, const double *l1,
                             double *x);

/* Lloyd's iteration in one dimension, K = 3.  Start: centres (min, mean, max).  Each round assigns
 * every point to its nearest centre (ties to the lower centre); if no label changed since the round
 * before, stop; otherwise every non-empty cluster's centre becomes the mean of its points.  At most
 * max_iter rounds.  labels[p] in {0,1,2} by ascending centre.  Returns the rounds run. */
int32_t oracle_kmeans1d(const double *v, int32_t n, int32_t max_iter, int32_t *labels,
                        double centre[3], double *margin);

/* Sec. 4.1 for one patch. */
int32_t oracle_patch_c_s1(double mhat_s1_3d, double tau_2d, double tau_3d);

/* Sec. 4.2 / Alg. 1 stage 3 for one patch: label, its smoothed shares, the baselines, its uniform number. */
int32_t oracle_patch_c_s2(int32_t label, double m2, double m3, double mu_2d, double mu_3d, double u,
                          const oracle_patch_params *p);

/* Sec. 4.4 for one patch: C_final (0 = the patch is discarded). */
int32_t oracle_patch_fuse(int32_t c_s1, int32_t c_s2);

/* Alg. 1 stages 1-4 given this step's observations.  a: per-token attention scores [2P] (their sum
 * over a patch's two tokens is what K-Means clusters); x: [P][4]; u: [P].  Updates st.  Outputs
 * (nullable): labels [P], cand [P][3] = (C_S1, C_S2, C_final), kept_idx ascending positions relative
 * to seq_off merged with all text positions.  Returns the number of kept positions. */
int32_t oracle_patch_select(const double *a, const double *x, const double *u, const oracle_sample *s,
                            const oracle_patch_params *p, oracle_patch_state *st, int32_t *labels,
                            int32_t *cand, int32_t *kept_idx, oracle_patch_diag *diag);

/* The whole step for one sample (n_2d must equal n_3d).  attn_out [2P], x_out [P][4] nullable. */
int32_t oracle_patch_step(const float *q, const float *k, const float *hidden, int32_t n_heads,
                          int32_t head_dim, int32_t d_model, const oracle_sample *s, const double *u,
                          const oracle_patch_params *p, oracle_patch_state *st, int32_t *labels,
                          int32_t *cand, int32_t *kept_idx, oracle_patch_diag *diag, double *attn_out,
                          double *x_out);

#ifdef __cplusplus
}
#endif
#endif
