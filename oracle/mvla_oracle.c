/*
 * mvla_oracle.c -- plain fp64 CPU statement of the MVLA prune step.
 *
 * TEST INFRASTRUCTURE ONLY (see mvla_oracle.h).  Plain loops, no blocking, no
 * fusion; the only parallelism is an OpenMP loop over attention heads whose
 * per-head results are summed afterwards in head order, so the arithmetic is
 * the same with any thread count.
 */
#include "mvla_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* Used only to FLAG decisions that sit on a boundary: the modality shares are ratios of sums of
 * several hundred scores, which an fp32 implementation reproduces to about 1e-6; 1e-4 relative is
 * a generous bound on that error. */
#define IND_TOL 1e-4

/* Row (relative to seq_off) of visual token j, with 2D tokens numbered first. */
static int32_t vis_row(const oracle_sample *s, int32_t j)
{
    return j < s->n_2d ? s->off_2d + j : s->off_3d + (j - s->n_2d);
}

/* ---- Sec. 3.2.1: attention scores alpha of text queries over visual keys ---- */
void oracle_salience(const float *q, const float *k, int32_t n_heads, int32_t head_dim,
                     const oracle_sample *s, double *a_out)
{
    oracle_salience_gqa(q, k, n_heads, n_heads, head_dim, s, a_out);
}

/* The same with grouped key heads: K is [rows, n_kv_heads, d] and query head h reads key head
 * h / (n_heads / n_kv_heads) (the usual grouped-query layout of the host models). */
void oracle_salience_gqa(const float *q, const float *k, int32_t n_heads, int32_t n_kv_heads,
                         int32_t head_dim, const oracle_sample *s, double *a_out)
{
    const int32_t H = n_heads, d = head_dim, nt = s->n_txt, nv = s->n_2d + s->n_3d;
    const int64_t row = (int64_t)H * d;                  /* elements of a Q row */
    const int64_t krow = (int64_t)n_kv_heads * d;        /* elements of a K row */
    const int32_t group = H / n_kv_heads;                /* query heads per key head */
    double *per_head = (double *)calloc((size_t)H * nv, sizeof(double));

#pragma omp parallel for schedule(static)
    for (int32_t h = 0; h < H; ++h) {
        double *logit = (double *)malloc((size_t)nv * sizeof(double));
        for (int32_t i = 0; i < nt; ++i) {
            const float *qi = q + ((int64_t)s->seq_off + s->off_txt + i) * row + (int64_t)h * d;
            /* logits l[h,i,j] = <q_hi, k_hj> / sqrt(d) */
            double mx = -INFINITY;
            for (int32_t j = 0; j < nv; ++j) {
                const float *kj = k + ((int64_t)s->seq_off + vis_row(s, j)) * krow + (int64_t)(h / group) * d;
                double acc = 0.0;
                for (int32_t c = 0; c < d; ++c) acc += (double)qi[c] * (double)kj[c];
                logit[j] = acc / sqrt((double)d);
                if (logit[j] > mx) mx = logit[j];
            }
            /* softmax over all visual keys (2D and 3D jointly) */
            double den = 0.0;
            for (int32_t j = 0; j < nv; ++j) den += exp(logit[j] - mx);
            for (int32_t j = 0; j < nv; ++j)
                per_head[(size_t)h * nv + j] += exp(logit[j] - mx) / den;
        }
        free(logit);
    }
    /* mean over heads and queries: the L1 norm of token j's attention vector
     * (Eq. 3-3 uses that norm) up to the constant 1/(H n_t) */
    for (int32_t j = 0; j < nv; ++j) {
        double acc = 0.0;
        for (int32_t h = 0; h < H; ++h) acc += per_head[(size_t)h * nv + j];
        a_out[j] = acc / ((double)H * (double)nt);
    }
    free(per_head);
}

/* ---- Sec. 4.3 / 5.2: consecutive frames share most of their content, so the logits of rows that did not
 * change since the previous action step need not be recomputed.  `logits` ([H][n_txt][n_vis], kept by the
 * caller between steps) holds the previous step's logits when `cache_valid`; `changed` has one byte per
 * row of the packed tensors (non-zero: the row was rewritten since the previous step).  A changed text
 * row invalidates everything (every logit has that query in it or is renormalised with it); otherwise
 * only the columns of changed visual keys are recomputed.  With a truthful mask the result equals
 * oracle_salience on the current inputs. ---- */
void oracle_salience_cached(const float *q, const float *k, int32_t n_heads, int32_t head_dim,
                            const oracle_sample *s, const uint8_t *changed, int32_t cache_valid,
                            double *logits, double *a_out, int32_t *n_recomputed)
{
    const int32_t H = n_heads, d = head_dim, nt = s->n_txt, nv = s->n_2d + s->n_3d;
    const int64_t row = (int64_t)H * d;
    int32_t all = !cache_valid || changed == NULL;
    for (int32_t i = 0; i < nt && !all; ++i)
        if (changed[(int64_t)s->seq_off + s->off_txt + i]) all = 1;
    int32_t redone = 0;
    for (int32_t j = 0; j < nv; ++j) {
        const int64_t krow = (int64_t)s->seq_off + vis_row(s, j);
        if (!all && !changed[krow]) continue;                 /* the previous step's logits of key j stand */
        ++redone;
        for (int32_t h = 0; h < H; ++h)
            for (int32_t ti = 0; ti < nt; ++ti) {
                const float *qrow = q + ((int64_t)s->seq_off + s->off_txt + ti) * row;
                const float *krw = k + krow * row;
                double dot = 0.0;
                for (int32_t c = 0; c < d; ++c) dot += (double)qrow[(int64_t)h * d + c] * (double)krw[(int64_t)h * d + c];
                logits[((size_t)h * nt + ti) * nv + j] = dot / sqrt((double)d);
            }
    }
    /* softmax over all visual keys, then the mean over heads and queries, in the order of oracle_salience */
    double *head_sum = (double *)calloc((size_t)H * nv, sizeof(double));
    for (int32_t h = 0; h < H; ++h)
        for (int32_t ti = 0; ti < nt; ++ti) {
            const double *l = logits + ((size_t)h * nt + ti) * nv;
            double top = -INFINITY, z = 0.0;
            for (int32_t j = 0; j < nv; ++j) if (l[j] > top) top = l[j];
            for (int32_t j = 0; j < nv; ++j) z += exp(l[j] - top);
            for (int32_t j = 0; j < nv; ++j) head_sum[(size_t)h * nv + j] += exp(l[j] - top) / z;
        }
    const double pairs = (double)H * (double)nt;
    for (int32_t j = 0; j < nv; ++j) {
        double total = 0.0;
        for (int32_t h = 0; h < H; ++h) total += head_sum[(size_t)h * nv + j];
        a_out[j] = total / pairs;
    }
    free(head_sum);
    if (n_recomputed) *n_recomputed = redone;
}

/* ---- Sec. 3.1.2: L1 feature norm per visual token ---- */
void oracle_l1norm(const float *hidden, int32_t d_model, const oracle_sample *s, double *n_out)
{
    const int32_t nv = s->n_2d + s->n_3d;
    for (int32_t j = 0; j < nv; ++j) {
        const float *r = hidden + ((int64_t)s->seq_off + vis_row(s, j)) * d_model;
        double acc = 0.0;
        for (int32_t c = 0; c < d_model; ++c) acc += fabs((double)r[c]);
        n_out[j] = acc;
    }
}

/* ---- Eq. 3-1 and Eqs. P2D / P3D, read at modality granularity ----
 * S1: share of the mean L1 feature norm per modality.
 * S2: share of the attention mass per modality. */
void oracle_indicators(const double *a, const double *l1, int32_t n_2d, int32_t n_3d, double x[4])
{
    const int32_t nv = n_2d + n_3d;
    double a2 = 0.0, a3 = 0.0;
    for (int32_t j = 0; j < n_2d; ++j) a2 += a[j];
    for (int32_t j = n_2d; j < nv; ++j) a3 += a[j];
    x[3] = a3 / (a2 + a3);
    x[2] = 1.0 - x[3];
    if (l1) {
        double s2 = 0.0, s3 = 0.0;
        for (int32_t j = 0; j < n_2d; ++j) s2 += l1[j];
        for (int32_t j = n_2d; j < nv; ++j) s3 += l1[j];
        const double m2 = n_2d > 0 ? s2 / n_2d : 0.0;
        const double m3 = n_3d > 0 ? s3 / n_3d : 0.0;
        x[1] = m3 / (m2 + m3);
        x[0] = 1.0 - x[1];
    } else {
        x[0] = 0.5;
        x[1] = 0.5;
    }
}

/* ---- Alg. 1 step 1; Eq. 8 (1 < t < k) and Eq. 9 (t >= k); t = 1 copies ---- */
void oracle_state_update(int32_t t, int32_t window_k, double beta, int32_t n,
                         const double *x, double *xhat)
{
    for (int32_t j = 0; j < n; ++j) {
        if (t <= 1)
            xhat[j] = x[j];
        else if (t < window_k)
            xhat[j] = ((double)(t - 1) / (double)t) * xhat[j] + (1.0 / (double)t) * x[j];
        else
            xhat[j] = beta * xhat[j] + (1.0 - beta) * x[j];
    }
}

/* ---- per-modality normalisation: mean 1 inside each modality ---- */
void oracle_normalise(const double *ahat, int32_t n_2d, int32_t n_3d, double *z)
{
    const int32_t nv = n_2d + n_3d;
    double s2 = 0.0, s3 = 0.0;
    for (int32_t j = 0; j < n_2d; ++j) s2 += ahat[j];
    for (int32_t j = n_2d; j < nv; ++j) s3 += ahat[j];
    for (int32_t j = 0; j < n_2d; ++j) z[j] = ahat[j] * (double)n_2d / s2;
    for (int32_t j = n_2d; j < nv; ++j) z[j] = ahat[j] * (double)n_3d / s3;
}

static int near(double v, double thr)
{
    return fabs(v - thr) <= IND_TOL * fabs(thr);
}

/* ---- Sec. 4.1 (dual threshold), Sec. 4.2 (target-object rule), Sec. 4.4 (fusion) ---- */
void oracle_gates(const double mhat[4], const oracle_params *p,
                  int32_t *c_s1, int32_t *c_s2, int32_t *c_final, int32_t *near_gate)
{
    const double s1_3d = mhat[1], s2_3d = mhat[3];
    int32_t c1, c2, cf;
    if (s1_3d < p->tau_2d) c1 = ORACLE_SET_2D;            /* 2D dominates */
    else if (s1_3d > p->tau_3d) c1 = ORACLE_SET_3D;       /* 3D dominates */
    else c1 = ORACLE_SET_2D | ORACLE_SET_3D;              /* balanced: tau_2d <= M <= tau_3d */
    /* dual protection unless the 3D response is near zero (then 2D only) */
    c2 = (s2_3d < p->eps_3d) ? ORACLE_SET_2D : (ORACLE_SET_2D | ORACLE_SET_3D);
    cf = c2 & c1;
    if (cf == 0) cf = c2;                                 /* conflict resolution */
    *c_s1 = c1; *c_s2 = c2; *c_final = cf;
    if (near_gate)
        *near_gate = near(s1_3d, p->tau_2d) || near(s1_3d, p->tau_3d) || near(s2_3d, p->eps_3d);
}

int32_t oracle_round_half_up(double x)
{
    return (int32_t)floor(x + 0.5);
}

static int32_t imin(int32_t a, int32_t b) { return a < b ? a : b; }
static int32_t imax(int32_t a, int32_t b) { return a > b ? a : b; }

void oracle_budget_fixed(const oracle_sample *s, int32_t *k_2d, int32_t *k_3d)
{
    *k_2d = imin(s->n_2d, oracle_round_half_up(s->keep_2d * (double)s->n_2d));
    *k_3d = imin(s->n_3d, oracle_round_half_up(s->keep_3d * (double)s->n_3d));
}

int32_t oracle_budget_total(const oracle_sample *s)
{
    const int32_t nv = s->n_2d + s->n_3d;
    return imin(nv, oracle_round_half_up(s->keep_total * (double)nv));
}

/* Split a total budget B between the modalities: the 3D share follows the
 * smoothed 3D attention share when both modalities are candidates, and goes
 * to one modality when the fused candidate set names only that one; each
 * modality keeps a floor (the "weak global perception" 10 %). */
void oracle_budget_adaptive(const oracle_sample *s, const oracle_params *p, double mhat_s2_3d,
                            int32_t c_final, int32_t *k_2d, int32_t *k_3d, int32_t *near_half)
{
    const int32_t n2 = s->n_2d, n3 = s->n_3d, nv = n2 + n3;
    const int32_t B = oracle_budget_total(s);
    const int32_t kmin2 = imin((int32_t)ceil(p->floor_ratio * (double)n2),
                               (int32_t)floor((double)B * (double)n2 / (double)nv));
    const int32_t kmin3 = imin((int32_t)ceil(p->floor_ratio * (double)n3),
                               (int32_t)floor((double)B * (double)n3 / (double)nv));
    double w3;
    if (c_final == (ORACLE_SET_2D | ORACLE_SET_3D)) w3 = mhat_s2_3d;
    else if (c_final == ORACLE_SET_2D) w3 = 0.0;
    else w3 = 1.0;
    const int32_t lo = imax(kmin3, B - n2);
    const int32_t hi = imin(n3, B - kmin2);
    const double target = (double)B * w3;
    int32_t k3 = oracle_round_half_up(target);
    if (k3 < lo) k3 = lo;
    if (k3 > hi) k3 = hi;
    *k_3d = k3;
    *k_2d = B - k3;
    if (near_half) {
        const double frac = target - floor(target);
        *near_half = fabs(frac - 0.5) <= IND_TOL * target;
    }
}

/* ---- Eq. 10 under a budget: stable full sort per modality ---- */
typedef struct { double z; int32_t j; } scored;

static int cmp_scored(const void *pa, const void *pb)
{
    const scored *a = (const scored *)pa, *b = (const scored *)pb;
    if (a->z > b->z) return -1;          /* larger score first */
    if (a->z < b->z) return 1;
    /* equal or unordered scores: lower index first; NaN after every number */
    const int an = isnan(a->z), bn = isnan(b->z);
    if (an != bn) return an ? 1 : -1;
    return (a->j > b->j) - (a->j < b->j);
}

static int cmp_i32(const void *pa, const void *pb)
{
    const int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

int32_t oracle_select(const double *z, const oracle_sample *s, int32_t k_2d, int32_t k_3d,
                      int32_t *kept_idx)
{
    int32_t n = 0;
    const int32_t seg_off[2] = { s->off_2d, s->off_3d };
    const int32_t seg_n[2] = { s->n_2d, s->n_3d };
    const int32_t seg_k[2] = { k_2d, k_3d };
    const int32_t base[2] = { 0, s->n_2d };
    for (int m = 0; m < 2; ++m) {
        scored *v = (scored *)malloc((size_t)(seg_n[m] > 0 ? seg_n[m] : 1) * sizeof(scored));
        for (int32_t j = 0; j < seg_n[m]; ++j) { v[j].z = z[base[m] + j]; v[j].j = j; }
        qsort(v, (size_t)seg_n[m], sizeof(scored), cmp_scored);   /* total order => unique result */
        for (int32_t r = 0; r < seg_k[m]; ++r) kept_idx[n++] = seg_off[m] + v[r].j;
        free(v);
    }
    for (int32_t i = 0; i < s->n_txt; ++i) kept_idx[n++] = s->off_txt + i;  /* text always proceeds */
    qsort(kept_idx, (size_t)n, sizeof(int32_t), cmp_i32);
    return n;
}

/* ---- Sec. 4.4: tokens with mask 1 proceed; the rest are dropped ---- */
void oracle_compact(const void *src, int64_t row_bytes, int32_t seq_off,
                    const int32_t *kept_idx, int32_t n_kept, void *dst)
{
    for (int32_t r = 0; r < n_kept; ++r)
        memcpy((char *)dst + (int64_t)r * row_bytes,
               (const char *)src + ((int64_t)seq_off + kept_idx[r]) * row_bytes, (size_t)row_bytes);
}

/* ---- Alg. 1 from the scores on: everything that follows the attention and the feature norms ---- */
int32_t oracle_decide_step(const double *a, const double *l1, const oracle_sample *s,
                           const oracle_params *p, int32_t mode, oracle_state *st,
                           int32_t *kept_idx, oracle_diag *diag, double *ahat_out, double *z_out)
{
    const int32_t n2 = s->n_2d, n3 = s->n_3d, nv = n2 + n3;
    double *z = (double *)malloc((size_t)nv * sizeof(double));
    double x[4];
    oracle_diag dg;
    memset(&dg, 0, sizeof dg);

    oracle_indicators(a, l1, n2, n3, x);

    /* action-iteration stage first (Alg. 1): smooth the per-token scores and the indicators */
    const int32_t t = st->t + 1;
    oracle_state_update(t, p->window_k, p->beta, nv, a, st->ahat);
    oracle_state_update(t, p->window_k, p->beta, 4, x, st->mhat);
    st->t = t;

    /* the later stages are written on the predicted (hatted) quantities */
    oracle_normalise(st->ahat, n2, n3, z);
    oracle_gates(st->mhat, p, &dg.c_s1, &dg.c_s2, &dg.c_final, &dg.near_gate);

    int32_t k2, k3;
    if (t == 1 && p->cold_start_full_keep) {
        k2 = n2; k3 = n3;                                  /* cold start: all tokens proceed */
    } else if (mode == ORACLE_MODE_FIXED) {
        oracle_budget_fixed(s, &k2, &k3);
    } else {
        oracle_budget_adaptive(s, p, st->mhat[3], dg.c_final, &k2, &k3, &dg.near_half);
    }
    const int32_t n_kept = oracle_select(z, s, k2, k3, kept_idx);

    dg.t = t; dg.k_2d = k2; dg.k_3d = k3; dg.budget = k2 + k3;
    memcpy(dg.x, x, sizeof x);
    memcpy(dg.mhat, st->mhat, sizeof x);
    if (diag) *diag = dg;
    if (ahat_out) memcpy(ahat_out, st->ahat, (size_t)nv * sizeof(double));
    if (z_out) memcpy(z_out, z, (size_t)nv * sizeof(double));
    free(z);
    return n_kept;
}

/* ---- Alg. 1 as a whole, for one sample: scores and norms, then the decisions above ---- */
int32_t oracle_prune_step(const float *q, const float *k, const float *hidden,
                          int32_t n_heads, int32_t head_dim, int32_t d_model,
                          const oracle_sample *s, const oracle_params *p, int32_t mode,
                          oracle_state *st, int32_t *kept_idx, oracle_diag *diag,
                          double *attn_out, double *l1_out, double *ahat_out, double *z_out)
{
    const int32_t nv = s->n_2d + s->n_3d;
    double *a = (double *)malloc((size_t)nv * sizeof(double));
    double *l1 = NULL;

    oracle_salience(q, k, n_heads, head_dim, s, a);
    if (mode == ORACLE_MODE_ADAPTIVE) {
        l1 = (double *)malloc((size_t)nv * sizeof(double));
        oracle_l1norm(hidden, d_model, s, l1);
    }
    const int32_t n_kept = oracle_decide_step(a, l1, s, p, mode, st, kept_idx, diag, ahat_out, z_out);
    if (attn_out) memcpy(attn_out, a, (size_t)nv * sizeof(double));
    if (l1_out && l1) memcpy(l1_out, l1, (size_t)nv * sizeof(double));
    free(a); free(l1);
    return n_kept;
}

/* Threads the head loop of oracle_salience may use (reporting only). */
#ifdef _OPENMP
#include <omp.h>
int32_t oracle_num_threads(void) { return (int32_t)omp_get_max_threads(); }
void oracle_set_num_threads(int32_t n) { if (n >= 1) omp_set_num_threads((int)n); }
#else
int32_t oracle_num_threads(void) { return 1; }
void oracle_set_num_threads(int32_t n) { (void)n; }
#endif
