/*
 * mvla_oracle.h -- plain fp64 CPU statement of the MVLA prune step.
 *
 * TEST INFRASTRUCTURE ONLY.  This is the slow, obviously-correct reference
 * against which the CUDA library is judged; only the test-suite, the smoke
 * check and the benchmark's CPU-baseline leg may call it.  It shares no code
 * with the CUDA path.
 *
 * What it computes follows the paper "2D or 3D: Who Governs Salience in VLA
 * Models? -- Tri-Stage Token Pruning Framework with Modality Salience
 * Awareness": attention scores of the instruction tokens over the visual
 * tokens (Sec. 3.2.1), the feature-norm share (Eq. 3-1), the attention share
 * (Eq. P2D / P3D), the temporal predictor (Alg. 1 step 1; Eqs. 8, 9), the
 * dual-threshold gate (Sec. 4.1), the target-object rule (Sec. 4.2), the
 * candidate fusion (Sec. 4.4), and the retention masks (Eq. 10) realised as
 * kept-index lists under a keep budget.
 *
 * Parity status: salience, norms, state update, gates, select and compaction
 * are pinned by the CPU tests (closed forms, brute force, invariants).  The
 * budget-split formula (oracle_budget_adaptive) and the modality-level reading
 * of Eq. 3-1 / Eq. P3D are "parity unpinned" against the paper: it prints no
 * worked example; only the invariants (sum equals the budget, floors, the
 * uniform-attention case) are pinned.
 *
 * All inputs are float arrays holding the exact bf16 / fp32 input values; all
 * arithmetic is double.
 */
#ifndef MVLA_ORACLE_H
#define MVLA_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORACLE_SET_2D = 1, ORACLE_SET_3D = 2 };   /* candidate sets as bit sets */
enum { ORACLE_MODE_FIXED = 0, ORACLE_MODE_ADAPTIVE = 1 };

/* One batch element: three contiguous segments of a packed token-major
 * sequence; offsets are rows relative to seq_off. */
typedef struct oracle_sample {
    int32_t seq_off;
    int32_t off_txt, n_txt;
    int32_t off_2d, n_2d;
    int32_t off_3d, n_3d;
    double keep_2d, keep_3d;   /* FIXED: fraction kept per modality */
    double keep_total;         /* ADAPTIVE: fraction of all visual tokens kept */
} oracle_sample;

typedef struct oracle_params {
    double tau_2d, tau_3d;     /* Sec. 4.1 thresholds */
    double beta;               /* Eq. 9 momentum */
    int32_t window_k;          /* Eq. 8 -> Eq. 9 switch */
    double eps_3d;             /* Sec. 4.2 "3D response near zero" */
    double floor_ratio;        /* weak global perception floor (Sec. 4.2, 10 %) */
    int32_t cold_start_full_keep; /* Alg. 1: t == 1 returns all tokens */
} oracle_params;

/* Smoothed state of one (prune point, sample): step counter, per-token
 * smoothed score, and the four smoothed indicators
 * [M^S1_2D, M^S1_3D, M^S2_2D, M^S2_3D]. */
typedef struct oracle_state {
    int32_t t;                 /* number of steps already absorbed */
    double *ahat;              /* [n_2d + n_3d] */
    double mhat[4];
} oracle_state;

/* Per-step record of everything decided. */
typedef struct oracle_diag {
    int32_t t;                 /* 1-based step this call was */
    double x[4];               /* instantaneous indicators */
    double mhat[4];            /* smoothed indicators */
    int32_t c_s1, c_s2, c_final;
    int32_t budget, k_2d, k_3d;
    int32_t near_half;         /* budget split within tolerance of a .5 rounding boundary */
    int32_t near_gate;         /* a gate operand within tolerance of its threshold */
} oracle_diag;

/* Sec. 3.2.1: scaled dot-product logits of every text query against every
 * visual key, softmax over all visual keys jointly, mean over heads and
 * queries.  q, k: [rows, H, d].  a_out: [n_2d + n_3d], 2D tokens first. */
void oracle_salience(const float *q, const float *k, int32_t n_heads, int32_t head_dim,
                     const oracle_sample *s, double *a_out);

/* The same for grouped-query attention: k is [rows, n_kv_heads, d], n_heads a multiple of
 * n_kv_heads, query head h attends through key head h / (n_heads / n_kv_heads). */
void oracle_salience_gqa(const float *q, const float *k, int32_t n_heads, int32_t n_kv_heads,
                         int32_t head_dim, const oracle_sample *s, double *a_out);

/* Sec. 4.3 / 5.2 (consecutive frames share content): oracle_salience that reuses the previous action
 * step's logits for visual keys whose rows did not change.  logits: [H][n_txt][n_vis] doubles owned by the
 * caller across steps (read when cache_valid, always left holding this step's logits); changed: one byte per
 * row of the packed tensors, non-zero = rewritten since the previous step (NULL: everything); a changed
 * text row recomputes everything.  n_recomputed (nullable): visual keys whose logits were recomputed. */
void oracle_salience_cached(const float *q, const float *k, int32_t n_heads, int32_t head_dim,
                            const oracle_sample *s, const uint8_t *changed, int32_t cache_valid,
                            double *logits, double *a_out, int32_t *n_recomputed);

/* Sec. 3.1.2: L1 norm of each visual token's feature row.  hidden: [rows, D]. */
void oracle_l1norm(const float *hidden, int32_t d_model, const oracle_sample *s, double *n_out);

/* Eq. 3-1 and Eq. P2D/P3D at modality granularity.  l1 may be NULL (then the
 * S1 pair is left at 0.5 / 0.5). x = [M^S1_2D, M^S1_3D, M^S2_2D, M^S2_3D]. */
void oracle_indicators(const double *a, const double *l1, int32_t n_2d, int32_t n_3d, double x[4]);

/* Alg. 1 step 1 / Eqs. 8, 9: t is the 1-based step being absorbed. */
void oracle_state_update(int32_t t, int32_t window_k, double beta, int32_t n,
                         const double *x, double *xhat);

/* Per-modality normalisation to mean 1. */
void oracle_normalise(const double *ahat, int32_t n_2d, int32_t n_3d, double *z);

/* Sec. 4.1 dual threshold, Sec. 4.2 target-object rule, Sec. 4.4 fusion. */
void oracle_gates(const double mhat[4], const oracle_params *p,
                  int32_t *c_s1, int32_t *c_s2, int32_t *c_final, int32_t *near_gate);

int32_t oracle_round_half_up(double x);
void oracle_budget_fixed(const oracle_sample *s, int32_t *k_2d, int32_t *k_3d);
int32_t oracle_budget_total(const oracle_sample *s);
void oracle_budget_adaptive(const oracle_sample *s, const oracle_params *p, double mhat_s2_3d,
                            int32_t c_final, int32_t *k_2d, int32_t *k_3d, int32_t *near_half);

/* Eq. 10 under a budget: per modality the k_m largest scores, ties to the
 * lower index; output positions (relative to seq_off), ascending, merged with
 * all text positions.  Returns the number of indices written. */
int32_t oracle_select(const double *z, const oracle_sample *s, int32_t k_2d, int32_t k_3d,
                      int32_t *kept_idx);

/* Sec. 4.4 last step: surviving rows proceed.  Byte copy of rows. */
void oracle_compact(const void *src, int64_t row_bytes, int32_t seq_off,
                    const int32_t *kept_idx, int32_t n_kept, void *dst);

/* Alg. 1 from the scores on (stages 1-4 and the selection): takes the attention scores a
 * [n_2d + n_3d] and the feature norms l1 (NULL: the S1 pair stays 0.5 / 0.5) as they come out of
 * oracle_salience / oracle_l1norm, advances the state, decides, and writes the kept positions.
 * ahat_out / z_out / diag may be NULL.  Returns the kept count. */
int32_t oracle_decide_step(const double *a, const double *l1, const oracle_sample *s,
                           const oracle_params *p, int32_t mode, oracle_state *st,
                           int32_t *kept_idx, oracle_diag *diag, double *ahat_out, double *z_out);

/* The whole step for one sample: oracle_salience (+ oracle_l1norm in ADAPTIVE mode), then
 * oracle_decide_step.  hidden may be NULL in FIXED mode.
 * attn_out / l1_out / ahat_out / z_out may be NULL.  Returns kept count. */
int32_t oracle_prune_step(const float *q, const float *k, const float *hidden,
                          int32_t n_heads, int32_t head_dim, int32_t d_model,
                          const oracle_sample *s, const oracle_params *p, int32_t mode,
                          oracle_state *st, int32_t *kept_idx, oracle_diag *diag,
                          double *attn_out, double *l1_out, double *ahat_out, double *z_out);

/* Threads the head loop of oracle_salience may use (reporting only). */
int32_t oracle_num_threads(void);
/* Threads for the head loops from now on (timing on one core and on all; the arithmetic does not change). */
void oracle_set_num_threads(int32_t n);

#ifdef __cplusplus
}
#endif
#endif
