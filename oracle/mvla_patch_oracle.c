/*
 * mvla_patch_oracle.c -- plain fp64 CPU statement of Alg. 1 taken literally, patch by patch.
 *
 * TEST INFRASTRUCTURE ONLY (see mvla_patch_oracle.h).  Plain loops in the order of the paper.
 */
#include "mvla_patch_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

static int32_t vis_row(const oracle_sample *s, int32_t j)
{
    return j < s->n_2d ? s->off_2d + j : s->off_3d + (j - s->n_2d);
}

/* ---- Sec. 3.2.1: attention of every (head, text query) over the visual keys ---- */
void oracle_attention(const float *q, const float *k, int32_t n_heads, int32_t head_dim,
                      const oracle_sample *s, double *alpha)
{
    const int32_t H = n_heads, d = head_dim, nt = s->n_txt, nv = s->n_2d + s->n_3d;
    const int64_t row = (int64_t)H * d;
#pragma omp parallel for schedule(static)
    for (int32_t h = 0; h < H; ++h) {
        for (int32_t i = 0; i < nt; ++i) {
            double *out = alpha + ((size_t)h * nt + i) * nv;
            const float *qi = q + ((int64_t)s->seq_off + s->off_txt + i) * row + (int64_t)h * d;
            double mx = -INFINITY;
            for (int32_t j = 0; j < nv; ++j) {
                const float *kj = k + ((int64_t)s->seq_off + vis_row(s, j)) * row + (int64_t)h * d;
                double acc = 0.0;
                for (int32_t c = 0; c < d; ++c) acc += (double)qi[c] * (double)kj[c];
                out[j] = acc / sqrt((double)d);
                if (out[j] > mx) mx = out[j];
            }
            double den = 0.0;
            for (int32_t j = 0; j < nv; ++j) den += exp(out[j] - mx);
            for (int32_t j = 0; j < nv; ++j) out[j] = exp(out[j] - mx) / den;
        }
    }
}

/* ---- Eq. 3-4: alpha_3D = {alpha_3D}_para + {alpha_3D}_ortho with respect to alpha_2D ---- */
void oracle_ortho_decompose(const double *a2, const double *a3, int32_t n, double *para, double *ortho)
{
    double d32 = 0.0, d22 = 0.0;
    for (int32_t r = 0; r < n; ++r) {
        d32 += a3[r] * a2[r];
        d22 += a2[r] * a2[r];
    }
    const double c = d22 > 0.0 ? d32 / d22 : 0.0;       /* projection coefficient */
    for (int32_t r = 0; r < n; ++r) {
        para[r] = c * a2[r];
        ortho[r] = a3[r] - para[r];
    }
}

/* ---- Eq. 3-1, Eq. P2D, Eq. P3D for every patch (the terms inside "avg(sum_p ...)") ---- */
void oracle_patch_indicators(const double *alpha, int32_t rows_a, int32_t n_patch, const double *l1,
                             double *x)
{
    const int32_t P = n_patch, nv = 2 * n_patch;
    double *a2 = (double *)malloc((size_t)rows_a * sizeof(double));
    double *a3 = (double *)malloc((size_t)rows_a * sizeof(double));
    double *para = (double *)malloc((size_t)rows_a * sizeof(double));
    double *ortho = (double *)malloc((size_t)rows_a * sizeof(double));
    for (int32_t p = 0; p < P; ++p) {
        /* feature-norm shares of the patch's two tokens */
        const double f2 = l1[p], f3 = l1[P + p];
        x[4 * p + 0] = f2 / (f2 + f3);
        x[4 * p + 1] = f3 / (f2 + f3);
        /* attention vectors of the patch's two tokens: one entry per (head, text query) */
        for (int32_t r = 0; r < rows_a; ++r) {
            a2[r] = alpha[(size_t)r * nv + p];
            a3[r] = alpha[(size_t)r * nv + P + p];
        }
        oracle_ortho_decompose(a2, a3, rows_a, para, ortho);
        double n2 = 0.0, n3 = 0.0, no = 0.0;
        for (int32_t r = 0; r < rows_a; ++r) {
            n2 += fabs(a2[r]);
            n3 += fabs(a3[r]);
            no += fabs(ortho[r]);
        }
        x[4 * p + 2] = n2 / (n2 + n3);
        x[4 * p + 3] = no / (n2 + n3);
    }
    free(a2); free(a3); free(para); free(ortho);
}

/* ---- Sec. 4.2: 1-D K-Means, K = 3 ---- */
int32_t oracle_kmeans1d(const double *v, int32_t n, int32_t max_iter, int32_t *labels,
                        double centre[3], double *margin)
{
    double mn = INFINITY, mx = -INFINITY, sum = 0.0, mg = INFINITY;
    for (int32_t p = 0; p < n; ++p) {
        if (v[p] < mn) mn = v[p];
        if (v[p] > mx) mx = v[p];
        sum += v[p];
    }
    centre[0] = mn;
    centre[1] = n > 0 ? sum / n : 0.0;
    centre[2] = mx;
    for (int32_t p = 0; p < n; ++p) labels[p] = -1;
    int32_t it = 0;
    while (it < max_iter) {
        ++it;
        int32_t changed = 0;
        for (int32_t p = 0; p < n; ++p) {
            int32_t best = 0;
            double bd = fabs(v[p] - centre[0]), second = INFINITY;
            for (int32_t c = 1; c < 3; ++c) {
                const double dc = fabs(v[p] - centre[c]);
                if (dc < bd) { second = bd; bd = dc; best = c; }      /* strict: ties stay with the lower centre */
                else if (dc < second) second = dc;
            }
            if (second - bd < mg) mg = second - bd;
            if (labels[p] != best) { labels[p] = best; changed = 1; }
        }
        if (!changed) break;
        for (int32_t c = 0; c < 3; ++c) {
            double acc = 0.0;
            int32_t cnt = 0;
            for (int32_t p = 0; p < n; ++p)
                if (labels[p] == c) { acc += v[p]; ++cnt; }
            if (cnt > 0) centre[c] = acc / cnt;
        }
    }
    if (margin) *margin = mg;
    return it;
}

/* ---- Sec. 4.1: dual threshold on the smoothed 3D feature share of the patch ---- */
int32_t oracle_patch_c_s1(double mhat_s1_3d, double tau_2d, double tau_3d)
{
    if (mhat_s1_3d < tau_2d) return ORACLE_SET_2D;
    if (mhat_s1_3d > tau_3d) return ORACLE_SET_3D;
    return ORACLE_SET_2D | ORACLE_SET_3D;
}

/* ---- Sec. 4.2 / Alg. 1 stage 3 ---- */
int32_t oracle_patch_c_s2(int32_t label, double m2, double m3, double mu_2d, double mu_3d, double u,
                          const oracle_patch_params *p)
{
    const int32_t both = ORACLE_SET_2D | ORACLE_SET_3D;
    if (label == ORACLE_LABEL_BG)                       /* 90 % uniform random pruning */
        return u < p->bg_prune_prob ? 0 : both;
    if (label == ORACLE_LABEL_ROB) {
        if (m3 > mu_3d) return both;                    /* pure 3D reliance above the baseline */
        if (m2 > mu_2d) return ORACLE_SET_2D;           /* 2D texture dominant */
        return 0;
    }
    /* target object: dual protection unless 2D reliance is large and the 3D response near zero */
    if (m2 > p->obj_2d_min && m3 < p->eps_3d) return ORACLE_SET_2D;
    return both;
}

/* ---- Sec. 4.4: intersection, conflict resolution; empty C_S2 discards the patch ---- */
int32_t oracle_patch_fuse(int32_t c_s1, int32_t c_s2)
{
    if (c_s2 == 0) return 0;
    const int32_t cf = c_s2 & c_s1;
    return cf != 0 ? cf : c_s2;
}

static int cmp_i32(const void *pa, const void *pb)
{
    const int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

int32_t oracle_patch_select(const double *a, const double *x, const double *u, const oracle_sample *s,
                            const oracle_patch_params *p, oracle_patch_state *st, int32_t *labels,
                            int32_t *cand, int32_t *kept_idx, oracle_patch_diag *diag)
{
    const int32_t P = s->n_2d;
    oracle_patch_diag dg;
    memset(&dg, 0, sizeof dg);
    int32_t *lab = (int32_t *)malloc((size_t)(P > 0 ? P : 1) * sizeof(int32_t));
    double *mass = (double *)malloc((size_t)(P > 0 ? P : 1) * sizeof(double));

    /* stage 1 of Alg. 1: temporal predictor for each patch and indicator */
    const int32_t t = st->t + 1;
    oracle_state_update(t, p->window_k, p->beta, 4 * P, x, st->xhat);
    st->t = t;
    dg.t = t;

    /* stage 3 preparations: cluster the patches by their attention response; baselines */
    for (int32_t q = 0; q < P; ++q) mass[q] = a[q] + a[P + q];
    dg.iters = oracle_kmeans1d(mass, P, p->kmeans_max_iter, lab, dg.centre, &dg.kmeans_margin);
    double s2 = 0.0, s3 = 0.0;
    for (int32_t q = 0; q < P; ++q) {
        s2 += st->xhat[4 * q + 2];
        s3 += st->xhat[4 * q + 3];
    }
    dg.mu_2d = P > 0 ? s2 / P : 0.0;
    dg.mu_3d = P > 0 ? s3 / P : 0.0;

    int32_t n = 0;
    const int cold = (t == 1 && p->cold_start_full_keep);
    for (int32_t q = 0; q < P; ++q) {
        const double *xh = st->xhat + 4 * q;
        const int32_t c1 = oracle_patch_c_s1(xh[1], p->tau_2d, p->tau_3d);                 /* stage 2 */
        const int32_t c2 = oracle_patch_c_s2(lab[q], xh[2], xh[3], dg.mu_2d, dg.mu_3d, u[q], p); /* stage 3 */
        int32_t cf = oracle_patch_fuse(c1, c2);                                            /* stage 4 */
        if (cold) cf = ORACLE_SET_2D | ORACLE_SET_3D;           /* cold start: full unpruned tokens */
        if (cand) { cand[3 * q] = c1; cand[3 * q + 1] = c2; cand[3 * q + 2] = cf; }
        if (labels) labels[q] = lab[q];
        dg.n_label[lab[q]] += 1;
        if (cf & ORACLE_SET_2D) { if (kept_idx) kept_idx[n] = s->off_2d + q; ++n; ++dg.k_2d; }   /* Mask_2D^p = 1 */
        if (cf & ORACLE_SET_3D) { if (kept_idx) kept_idx[n] = s->off_3d + q; ++n; ++dg.k_3d; }   /* Mask_3D^p = 1 */
    }
    for (int32_t i = 0; i < s->n_txt; ++i) { if (kept_idx) kept_idx[n] = s->off_txt + i; ++n; }
    if (kept_idx) qsort(kept_idx, (size_t)n, sizeof(int32_t), cmp_i32);
    if (diag) *diag = dg;
    free(lab); free(mass);
    return n;
}

int32_t oracle_patch_step(const float *q, const float *k, const float *hidden, int32_t n_heads,
                          int32_t head_dim, int32_t d_model, const oracle_sample *s, const double *u,
                          const oracle_patch_params *p, oracle_patch_state *st, int32_t *labels,
                          int32_t *cand, int32_t *kept_idx, oracle_patch_diag *diag, double *attn_out,
                          double *x_out)
{
    const int32_t P = s->n_2d, nv = 2 * P, rows_a = n_heads * s->n_txt;
    if (s->n_3d != P) return -1;
    double *alpha = (double *)malloc((size_t)rows_a * nv * sizeof(double));
    double *a = (double *)malloc((size_t)nv * sizeof(double));
    double *l1 = (double *)malloc((size_t)nv * sizeof(double));
    double *x = (double *)malloc((size_t)4 * P * sizeof(double));

    oracle_attention(q, k, n_heads, head_dim, s, alpha);
    /* per-token score: mean over (head, text query) of the token's attention, as in oracle_salience */
    for (int32_t j = 0; j < nv; ++j) {
        double acc = 0.0;
        for (int32_t r = 0; r < rows_a; ++r) acc += alpha[(size_t)r * nv + j];
        a[j] = acc / (double)rows_a;
    }
    oracle_l1norm(hidden, d_model, s, l1);
    oracle_patch_indicators(alpha, rows_a, P, l1, x);
    const int32_t n = oracle_patch_select(a, x, u, s, p, st, labels, cand, kept_idx, diag);
    if (attn_out) memcpy(attn_out, a, (size_t)nv * sizeof(double));
    if (x_out) memcpy(x_out, x, (size_t)4 * P * sizeof(double));
    free(alpha); free(a); free(l1); free(x);
    return n;
}
