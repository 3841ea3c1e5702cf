/*
 * Reference oracle for one scheduled round of Lasso coordinate descent
 * (Lee, Kim, Ho, Gibson, Xing: "Structure-Aware Dynamic Scheduler for Parallel
 * Machine Learning", Section 2.1, Algorithm 1, Eq. 1 and Eq. 2).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, single-threaded CPU
 * program that takes the algorithm's steps in the paper's order, in FP64, so
 * that a reader can check it against the paper by eye.  It shares no code with
 * the CUDA library and must never be called from the product path.
 *
 * Every function is pinned by CPU tests against something other than itself
 * (closed forms, brute force, KKT conditions, enumeration of the sampling
 * distribution, an independent Philox implementation).  The one exception is
 * the free-running multi-round trajectory: a randomised iteration has no closed
 * form, so for it parity is unpinned beyond the converged optimum (KKT / brute
 * force) that it must reach.
 *
 * Notation follows the paper: N samples, J coefficients, P' candidates per
 * round (n_cand), P parallel updates per round (n_keep), eta, rho, lambda, and
 * C the "very large" initial change.  delta_j = |beta_j^(t_j-1) - beta_j^(t_j-2)|.
 *
 * X and y are the FP32 arrays the GPU sees, widened to double on the fly.
 * The only FP32 arithmetic is the sampling key (so_race_key), which is FP32 by
 * specification so that two independent implementations can agree bit for bit.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Design matrix: dense column-major or CSC, both FP32 storage.               */
/* ------------------------------------------------------------------------- */
typedef struct {
    int32_t layout;          /* 0 dense column-major, 1 CSC                    */
    int64_t n_rows, n_cols;  /* N, J                                           */
    int64_t ld;              /* dense: floats between column starts            */
    const float *values;     /* dense: [J][ld]; CSC: [nnz]                     */
    const int32_t *row_idx;  /* CSC: ascending inside a column                 */
    const int64_t *col_ptr;  /* CSC: [J+1]                                     */
} so_matrix;

/* x_j^T v for a dense double vector v of length N. */
static double col_dot_vec(const so_matrix *X, int64_t j, const double *v)
{
    double s = 0.0;
    if (X->layout == 0) {
        const float *x = X->values + j * X->ld;
        for (int64_t i = 0; i < X->n_rows; ++i) s += (double)x[i] * v[i];
    } else {
        for (int64_t p = X->col_ptr[j]; p < X->col_ptr[j + 1]; ++p)
            s += (double)X->values[p] * v[X->row_idx[p]];
    }
    return s;
}

/* x_j^T x_k. CSC columns are intersected by a two-pointer walk over sorted rows. */
static double col_dot_col(const so_matrix *X, int64_t j, int64_t k)
{
    double s = 0.0;
    if (X->layout == 0) {
        const float *a = X->values + j * X->ld, *b = X->values + k * X->ld;
        for (int64_t i = 0; i < X->n_rows; ++i) s += (double)a[i] * (double)b[i];
    } else {
        int64_t p = X->col_ptr[j], pe = X->col_ptr[j + 1];
        int64_t q = X->col_ptr[k], qe = X->col_ptr[k + 1];
        while (p < pe && q < qe) {
            int32_t rp = X->row_idx[p], rq = X->row_idx[q];
            if (rp == rq) { s += (double)X->values[p] * (double)X->values[q]; ++p; ++q; }
            else if (rp < rq) ++p;
            else ++q;
        }
    }
    return s;
}

/* n_j = ||x_j||^2 for every column. */
void so_colnorm2(const so_matrix *X, double *n2)
{
    for (int64_t j = 0; j < X->n_cols; ++j) n2[j] = col_dot_col(X, j, j);
}

/* ------------------------------------------------------------------------- */
/* Counter-based random numbers: Philox4x32-10 as published by Salmon, Moraes, */
/* Dror and Shaw ("Parallel random numbers: as easy as 1, 2, 3", SC'11).      */
/* ------------------------------------------------------------------------- */
void so_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4])
{
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;   /* golden-ratio Weyl increment */
        k1 += 0xBB67AE85u;   /* sqrt(3)-1 Weyl increment    */
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The random word of coefficient j in round t: key = seed, counter =
 * (j / 4, t low, t high, 0); coefficient j takes output word j mod 4. */
uint32_t so_draw_word(uint64_t seed, uint64_t t, uint64_t j)
{
    uint32_t ctr[4] = { (uint32_t)(j >> 2), (uint32_t)t, (uint32_t)(t >> 32), 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    so_philox4x32_10(ctr, key, out);
    return out[j & 3];
}

/* ------------------------------------------------------------------------- */
/* Sampling key (FP32 by specification).                                       */
/*                                                                             */
/* Drawing P' coefficients without replacement with p(j) proportional to w_j   */
/* (Algorithm 1's "draw a set of P' coefficients") is an exponential race:     */
/* give every j an independent unit exponential E_j, rank by T_j = E_j / w_j   */
/* ascending, take the first P'.  (Equivalent to Gumbel-top-k on ln w_j + G_j.)*/
/* Every operation below is one correctly rounded IEEE binary32 operation;     */
/* this file is compiled with -ffp-contract=off so none are fused.             */
/* ------------------------------------------------------------------------- */
static float f32_from_bits(uint32_t b) { float f; memcpy(&f, &b, 4); return f; }
static uint32_t f32_bits(float f) { uint32_t b; memcpy(&b, &f, 4); return b; }

/* 2*atanh(s) = 2s (1 + z/3 + z^2/5 + ... + z^8/17), z = s^2, for |s| <= 1/3. */
static float two_atanh_f32(float s)
{
    const float z = s * s;
    float p = f32_from_bits(0x3d70f0f1u);                 /* 1/17 */
    p = fmaf(p, z, f32_from_bits(0x3d888889u));           /* 1/15 */
    p = fmaf(p, z, f32_from_bits(0x3d9d89d9u));           /* 1/13 */
    p = fmaf(p, z, f32_from_bits(0x3dba2e8cu));           /* 1/11 */
    p = fmaf(p, z, f32_from_bits(0x3de38e39u));           /* 1/9  */
    p = fmaf(p, z, f32_from_bits(0x3e124925u));           /* 1/7  */
    p = fmaf(p, z, f32_from_bits(0x3e4ccccdu));           /* 1/5  */
    p = fmaf(p, z, f32_from_bits(0x3eaaaaabu));           /* 1/3  */
    const float r = z * p;
    const float s2 = s + s;
    return fmaf(s2, r, s2);
}

/* Unit exponential E = -ln(1 - v) from a 32-bit word, v = (x + 1/2) / 2^32. */
float so_unit_exponential_f32(uint32_t x)
{
    const float xf = (float)x;                                      /* round to nearest */
    float v = fmaf(xf, f32_from_bits(0x2f800000u) /* 2^-32 */, f32_from_bits(0x2f000000u) /* 2^-33 */);
    const float vmax = f32_from_bits(0x3f7fffffu);                  /* 1 - 2^-24 */
    if (v > vmax) v = vmax;
    if (v <= 0.5f) {
        /* -ln(1-v) = 2 atanh(v / (2 - v)); keeps full relative precision for small v */
        const float s = v / (2.0f - v);
        return two_atanh_f32(s);
    }
    /* q = 1 - v is exact; q = m 2^e with m in [sqrt(1/2), sqrt(2)); ln q = e ln2 + 2 atanh((m-1)/(m+1)) */
    const float q = 1.0f - v;
    const uint32_t qb = f32_bits(q);
    int32_t e = (int32_t)(qb >> 23) - 127;
    float m = f32_from_bits((qb & 0x007fffffu) | 0x3f800000u);
    if (m >= f32_from_bits(0x3fb504f3u) /* sqrt 2 */) { m = m * 0.5f; e += 1; }
    const float s = (m - 1.0f) / (m + 1.0f);
    const float a = two_atanh_f32(s);
    const float ef = (float)e;
    const float lo = fmaf(ef, f32_from_bits(0x3805fdf4u) /* ln2 low part */, a);
    const float lnq = fmaf(ef, f32_from_bits(0x3f317000u) /* ln2 high part */, lo);
    return -lnq;
}

/* Race time T_j = E_j / w_j with the priority weight w_j = delta_j^2 + eta
 * (Theorem 1's (delta beta_j)^2 with Algorithm 1's floor eta). */
float so_race_key(float delta_j, float eta, uint32_t x)
{
    const float w = fmaf(delta_j, delta_j, eta);
    return so_unit_exponential_f32(x) / w;
}

/* Other importance distributions p(j):
 *   mode 0  w_j = delta_j^2 + eta   (Theorem 1; so_race_key)
 *   mode 1  w_j = |delta_j| + eta   (Algorithm 1 as printed: p(j) ~ |beta_j^(t_j-2) - beta_j^(t_j-1)| + eta)
 *   mode 2  w_j = 1                 (uniform draw: the static and the random scheduler of the comparison, Section 5.1) */
float so_race_key_mode(float delta_j, float eta, uint32_t x, int32_t mode)
{
    if (mode == 0) return so_race_key(delta_j, eta, x);
    const float w = mode == 1 ? fabsf(delta_j) + eta : 1.0f;
    return so_unit_exponential_f32(x) / w;
}

typedef struct { uint32_t tbits; int32_t j; } so_keyed;

static int keyed_less(const void *pa, const void *pb)
{
    const so_keyed *a = (const so_keyed *)pa, *b = (const so_keyed *)pb;
    if (a->tbits != b->tbits) return a->tbits < b->tbits ? -1 : 1;   /* T >= 0: bit order = value order */
    return (a->j > b->j) - (a->j < b->j);                              /* ties to the smaller index */
}

/* Algorithm 1, "Draw a set U of P' coefficients": rank ALL J race keys and
 * return the first n_cand indices, best first.  Returns 0, or -1 on bad args. */
int so_sample(int64_t J, const double *delta, double eta, uint64_t seed, uint64_t t,
              int32_t n_cand, int32_t *cand, float *keys_out /* [J] or NULL */)
{
    if (J <= 0 || n_cand < 0 || n_cand > J) return -1;
    so_keyed *all = (so_keyed *)malloc((size_t)J * sizeof(so_keyed));
    if (!all) return -2;
    for (int64_t j = 0; j < J; ++j) {
        const float T = so_race_key((float)delta[j], (float)eta, so_draw_word(seed, t, (uint64_t)j));
        all[j].tbits = f32_bits(T);
        all[j].j = (int32_t)j;
        if (keys_out) keys_out[j] = T;
    }
    qsort(all, (size_t)J, sizeof(so_keyed), keyed_less);
    for (int32_t a = 0; a < n_cand; ++a) cand[a] = all[a].j;
    free(all);
    return 0;
}

/* The same draw under another importance distribution (so_race_key_mode). */
int so_sample_mode(int64_t J, const double *delta, double eta, uint64_t seed, uint64_t t,
                   int32_t n_cand, int32_t mode, int32_t *cand)
{
    if (J <= 0 || n_cand < 0 || n_cand > J || mode < 0 || mode > 2) return -1;
    so_keyed *all = (so_keyed *)malloc((size_t)J * sizeof(so_keyed));
    if (!all) return -2;
    for (int64_t j = 0; j < J; ++j) {
        const float T = so_race_key_mode((float)delta[j], (float)eta, so_draw_word(seed, t, (uint64_t)j), mode);
        all[j].tbits = f32_bits(T);
        all[j].j = (int32_t)j;
    }
    qsort(all, (size_t)J, sizeof(so_keyed), keyed_less);
    for (int32_t a = 0; a < n_cand; ++a) cand[a] = all[a].j;
    free(all);
    return 0;
}

/* STRADS ("Implementation Overview"): S scheduler threads, thread s owning a fixed,
 * disjoint set of J/S coefficients and sampling only from its own p_s(j).  The
 * assignment used here: thread s owns { j : j mod S == s } (the paper assigns at
 * random; the caller may permute the columns).  Ranks the race keys of the
 * coefficients of thread `s` only and returns the first n_cand, best first.
 * With S == 1 this is so_sample. */
int so_sample_part(int64_t J, const double *delta, double eta, uint64_t seed, uint64_t t,
                   int32_t S, int32_t s, int32_t n_cand, int32_t *cand)
{
    if (J <= 0 || S < 1 || s < 0 || s >= S || n_cand < 0) return -1;
    const int64_t members = (J - s + S - 1) / S;      /* |{ j < J : j mod S == s }| */
    if (n_cand > members) return -1;
    so_keyed *own = (so_keyed *)malloc((size_t)(members > 0 ? members : 1) * sizeof(so_keyed));
    if (!own) return -2;
    int64_t m = 0;
    for (int64_t j = s; j < J; j += S) {
        const float T = so_race_key((float)delta[j], (float)eta, so_draw_word(seed, t, (uint64_t)j));
        own[m].tbits = f32_bits(T);
        own[m].j = (int32_t)j;
        ++m;
    }
    qsort(own, (size_t)m, sizeof(so_keyed), keyed_less);
    for (int32_t a = 0; a < n_cand; ++a) cand[a] = own[a].j;
    free(own);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Dependency filter (Algorithm 1, "Choose a set B1 of <= P coefficients from  */
/* U such that |x_j^T x_k| <= rho"; strict form of SAP step 2).  Walk the      */
/* candidates best first; keep c when |corr(c,k)| < rho for every k already    */
/* kept; stop at P kept.  corr is the cosine x_c^T x_k / (||x_c|| ||x_k||),    */
/* which is x_c^T x_k itself on standardised columns.                          */
/*                                                                             */
/* follow / n_follow / tol implement the parity protocol for borderline pairs: */
/* a pair with | |corr| - rho | <= tol is "ambiguous".  A candidate that has   */
/* no clear conflict but at least one ambiguous pair is kept iff it appears in */
/* `follow` (the other implementation's kept list).  With follow == NULL the   */
/* plain strict rule applies.  min_margin receives the smallest | |corr|-rho | */
/* consulted.                                                                  */
/* ------------------------------------------------------------------------- */
int so_filter(const so_matrix *X, const double *n2, const int32_t *cand, int32_t n_cand,
              int32_t n_keep, double rho, const int32_t *follow, int32_t n_follow, double tol,
              int32_t *kept, int32_t *n_kept_out, int32_t *n_examined_out, double *min_margin)
{
    int32_t nk = 0, examined = 0;
    double mm = INFINITY;
    for (int32_t a = 0; a < n_cand && nk < n_keep; ++a) {
        const int32_t c = cand[a];
        ++examined;
        int clear_conflict = 0, ambiguous = 0;
        for (int32_t b = 0; b < nk; ++b) {
            const int32_t k = kept[b];
            const double den = sqrt(n2[c] * n2[k]);
            const double corr = den > 0.0 ? col_dot_col(X, c, k) / den : 0.0;
            const double margin = fabs(fabs(corr) - rho);
            if (margin < mm) mm = margin;
            if (follow && margin <= tol) ambiguous = 1;
            else if (fabs(corr) >= rho) { clear_conflict = 1; break; }
        }
        int keep;
        if (clear_conflict) keep = 0;
        else if (ambiguous) {
            keep = 0;
            for (int32_t f = 0; f < n_follow; ++f) if (follow[f] == c) { keep = 1; break; }
        } else keep = 1;
        if (keep) kept[nk++] = c;
    }
    *n_kept_out = nk;
    *n_examined_out = examined;
    if (min_margin) *min_margin = mm;
    return 0;
}

/* The filter with dependencies dropped at run time (SAP step 4: "removing dependencies between
 * variables that have reached zero"; Section 1, "Dynamic Block Structures": a coefficient that stays
 * zero does not affect the update of another, however correlated the two columns are).
 * A coefficient is dormant when it is zero and its last update left it there (beta_j = 0 and
 * delta_j = 0; a coefficient never updated has delta_j = C and is not dormant).  The coupling
 * d(x_j, x_k) of a pair with a dormant member is taken as 0: a dormant candidate is always kept and
 * blocks nobody; the rho test applies among the others exactly as in so_filter. */
int so_filter_dynamic(const so_matrix *X, const double *n2, const int32_t *cand, int32_t n_cand,
                      int32_t n_keep, double rho, const double *beta, const double *delta,
                      int32_t *kept, int32_t *n_kept_out, int32_t *n_examined_out)
{
    int32_t nk = 0, examined = 0;
    for (int32_t a = 0; a < n_cand && nk < n_keep; ++a) {
        const int32_t c = cand[a];
        ++examined;
        int keep = 1;
        if (!(beta[c] == 0.0 && delta[c] == 0.0)) {
            for (int32_t b = 0; b < nk; ++b) {
                const int32_t k = kept[b];
                if (beta[k] == 0.0 && delta[k] == 0.0) continue;
                const double den = sqrt(n2[c] * n2[k]);
                const double corr = den > 0.0 ? col_dot_col(X, c, k) / den : 0.0;
                if (fabs(corr) >= rho) { keep = 0; break; }
            }
        }
        if (keep) kept[nk++] = c;
    }
    *n_kept_out = nk;
    *n_examined_out = examined;
    return 0;
}

/* Correlation of two columns as the filter sees it (exposed for tests). */
double so_corr(const so_matrix *X, const double *n2, int64_t j, int64_t k)
{
    const double den = sqrt(n2[j] * n2[k]);
    return den > 0.0 ? col_dot_col(X, j, k) / den : 0.0;
}

/* ------------------------------------------------------------------------- */
/* Parallel update (Algorithm 1, "In parallel on P workers ... update beta_j   */
/* using Eq. 2").  With r = y - X beta, Eq. 2's argument                        */
/*   x_j^T y - sum_{k != j} x_j^T x_k beta_k  =  x_j^T r + n_j beta_j,          */
/* and for a column of squared norm n_j the coordinate minimiser is             */
/*   beta_j' = S(beta_j + x_j^T r / n_j, lambda / n_j),                         */
/* S(a, k) = sign(a) max(|a| - k, 0); n_j = 1 gives Eq. 2 as printed.           */
/* All kept coefficients are computed from the same pre-round r (the workers    */
/* run in parallel), then applied together.                                     */
/* ------------------------------------------------------------------------- */
static double soft_threshold(double a, double k)
{
    const double m = fabs(a) - k;
    if (m <= 0.0) return 0.0;
    return a > 0.0 ? m : -m;
}

int so_update(const so_matrix *X, const double *n2, double lambda, const int32_t *kept, int32_t n_kept,
              double *beta, double *resid, double *delta, double *dbeta /* [n_kept] */)
{
    for (int32_t a = 0; a < n_kept; ++a) {
        const int32_t j = kept[a];
        double d = 0.0;
        if (n2[j] > 0.0) {
            const double g = col_dot_vec(X, j, resid);
            const double z = beta[j] + g / n2[j];
            d = soft_threshold(z, lambda / n2[j]) - beta[j];
        }
        dbeta[a] = d;
    }
    for (int32_t a = 0; a < n_kept; ++a) {
        const int32_t j = kept[a];
        const double d = dbeta[a];
        beta[j] += d;
        delta[j] = fabs(d);             /* progress monitoring: refreshes p(j) for the next draw */
        if (d != 0.0) {
            if (X->layout == 0) {
                const float *x = X->values + j * X->ld;
                for (int64_t i = 0; i < X->n_rows; ++i) resid[i] -= (double)x[i] * d;
            } else {
                for (int64_t p = X->col_ptr[j]; p < X->col_ptr[j + 1]; ++p)
                    resid[X->row_idx[p]] -= (double)X->values[p] * d;
            }
        }
    }
    return 0;
}

/* Initial state of Algorithm 1: beta = 0 (so r = y) and a previous iterate C,
 * i.e. delta_j = |C - 0| = C for every coefficient. */
void so_init(const so_matrix *X, const float *y, double c_init, double *n2,
             double *beta, double *resid, double *delta)
{
    so_colnorm2(X, n2);
    for (int64_t j = 0; j < X->n_cols; ++j) { beta[j] = 0.0; delta[j] = c_init; }
    for (int64_t i = 0; i < X->n_rows; ++i) resid[i] = (double)y[i];
}

/* One whole round of Algorithm 1's loop body; t is the 0-based round index. */
int so_round(const so_matrix *X, const double *n2, double lambda, double eta, double rho,
             int32_t n_cand, int32_t n_keep, uint64_t seed, uint64_t t,
             double *beta, double *resid, double *delta,
             int32_t *cand /* [n_cand] */, int32_t *kept /* [n_keep] */, double *dbeta /* [n_keep] */,
             int32_t *counts /* [4]: n_cand, n_examined, n_kept, n_nonzero */)
{
    int rc = so_sample(X->n_cols, delta, eta, seed, t, n_cand, cand, NULL);
    if (rc) return rc;
    int32_t nk = 0, ne = 0;
    so_filter(X, n2, cand, n_cand, n_keep, rho, NULL, 0, 0.0, kept, &nk, &ne, NULL);
    so_update(X, n2, lambda, kept, nk, beta, resid, delta, dbeta);
    int32_t nz = 0;
    for (int32_t a = 0; a < nk; ++a) nz += dbeta[a] != 0.0;
    counts[0] = n_cand; counts[1] = ne; counts[2] = nk; counts[3] = nz;
    return 0;
}

/* One round under another schedule: weight_mode as so_race_key_mode; filter_mode 0 the rho test of
 * Algorithm 1, 1 none (the first P candidates: the random scheduler, which "does not perform
 * dependency checking"), 2 the rho test with dependencies dropped at run time (so_filter_dynamic).
 * weight_mode 2 with filter_mode 0 is the static scheduler of Section 5.1. */
int so_round_mode(const so_matrix *X, const double *n2, double lambda, double eta, double rho,
                  int32_t n_cand, int32_t n_keep, uint64_t seed, uint64_t t, int32_t weight_mode, int32_t filter_mode,
                  double *beta, double *resid, double *delta,
                  int32_t *cand, int32_t *kept, double *dbeta, int32_t *counts)
{
    int rc = so_sample_mode(X->n_cols, delta, eta, seed, t, n_cand, weight_mode, cand);
    if (rc) return rc;
    int32_t nk = 0, ne = 0;
    if (filter_mode == 0) {
        so_filter(X, n2, cand, n_cand, n_keep, rho, NULL, 0, 0.0, kept, &nk, &ne, NULL);
    } else if (filter_mode == 1) {
        nk = n_cand < n_keep ? n_cand : n_keep;
        for (int32_t a = 0; a < nk; ++a) kept[a] = cand[a];
        ne = nk;
    } else if (filter_mode == 2) {
        so_filter_dynamic(X, n2, cand, n_cand, n_keep, rho, beta, delta, kept, &nk, &ne);
    } else {
        return -1;
    }
    so_update(X, n2, lambda, kept, nk, beta, resid, delta, dbeta);
    int32_t nz = 0;
    for (int32_t a = 0; a < nk; ++a) nz += dbeta[a] != 0.0;
    counts[0] = n_cand; counts[1] = ne; counts[2] = nk; counts[3] = nz;
    return 0;
}

/* One round of STRADS with S scheduler threads taking turns ("thread 1 dispatches
 * first, then thread 2, ... before returning to thread 1"): round t is dispatched
 * by thread t mod S, which samples from its own coefficients; the rest of the round
 * is Algorithm 1's loop body unchanged. */
int so_round_part(const so_matrix *X, const double *n2, double lambda, double eta, double rho,
                  int32_t n_cand, int32_t n_keep, uint64_t seed, uint64_t t, int32_t S,
                  double *beta, double *resid, double *delta,
                  int32_t *cand, int32_t *kept, double *dbeta, int32_t *counts)
{
    if (S < 1) return -1;
    int rc = so_sample_part(X->n_cols, delta, eta, seed, t, S, (int32_t)(t % (uint64_t)S), n_cand, cand);
    if (rc) return rc;
    int32_t nk = 0, ne = 0;
    so_filter(X, n2, cand, n_cand, n_keep, rho, NULL, 0, 0.0, kept, &nk, &ne, NULL);
    so_update(X, n2, lambda, kept, nk, beta, resid, delta, dbeta);
    int32_t nz = 0;
    for (int32_t a = 0; a < nk; ++a) nz += dbeta[a] != 0.0;
    counts[0] = n_cand; counts[1] = ne; counts[2] = nk; counts[3] = nz;
    return 0;
}

/* Eq. 1 with squared loss, from the maintained residual:
 * F = 1/2 ||r||^2 + lambda ||beta||_1. */
double so_objective(int64_t N, int64_t J, const double *resid, const double *beta, double lambda)
{
    double sq = 0.0, l1 = 0.0;
    for (int64_t i = 0; i < N; ++i) sq += resid[i] * resid[i];
    for (int64_t j = 0; j < J; ++j) l1 += fabs(beta[j]);
    return 0.5 * sq + lambda * l1;
}

/* Eq. 1 recomputed from beta alone: r = y - X beta formed from scratch into
 * resid_out (drift check for the incrementally maintained residual). */
double so_objective_from_scratch(const so_matrix *X, const float *y, const double *beta,
                                 double lambda, double *resid_out)
{
    for (int64_t i = 0; i < X->n_rows; ++i) resid_out[i] = (double)y[i];
    for (int64_t j = 0; j < X->n_cols; ++j) {
        const double b = beta[j];
        if (b == 0.0) continue;
        if (X->layout == 0) {
            const float *x = X->values + j * X->ld;
            for (int64_t i = 0; i < X->n_rows; ++i) resid_out[i] -= (double)x[i] * b;
        } else {
            for (int64_t p = X->col_ptr[j]; p < X->col_ptr[j + 1]; ++p)
                resid_out[X->row_idx[p]] -= (double)X->values[p] * b;
        }
    }
    return so_objective(X->n_rows, X->n_cols, resid_out, beta, lambda);
}

/* x_j^T r for every column (used by the KKT checks in the tests). */
void so_gradient(const so_matrix *X, const double *resid, double *g)
{
    for (int64_t j = 0; j < X->n_cols; ++j) g[j] = col_dot_vec(X, j, resid);
}

/* ------------------------------------------------------------------------- */
/* Logistic loss (Section 2.1, remark after Eq. 1: "it is straightforward to   */
/* use other loss functions such as logistic-loss using the same approach      */
/* shown in" the Shotgun paper).  Labels y_i in {0, 1}, margin m = X beta,     */
/*   F(beta) = sum_i [ log(1 + exp(m_i)) - y_i m_i ] + lambda ||beta||_1.      */
/* The coordinate step is that of Shotgun for this loss: the second derivative */
/* of the loss along coordinate j is at most n_j / 4, so with g_j = x_j^T r,   */
/* r = y - sigma(m) (minus the gradient), the minimiser of the quadratic upper */
/* bound is                                                                    */
/*   beta_j' = S(beta_j + 4 g_j / n_j, 4 lambda / n_j).                        */
/* Everything else of the round (draw, filter, parallel application from one   */
/* snapshot, delta_j = |change|) is Algorithm 1 unchanged.  State: beta, the   */
/* margin m, and r = y - sigma(m), which plays the residual's part.            */
/* ------------------------------------------------------------------------- */
static double sigmoid(double m) { return m >= 0.0 ? 1.0 / (1.0 + exp(-m)) : exp(m) / (1.0 + exp(m)); }

void so_init_logistic(const so_matrix *X, const float *y, double c_init, double *n2,
                      double *beta, double *margin, double *resid, double *delta)
{
    so_colnorm2(X, n2);
    for (int64_t j = 0; j < X->n_cols; ++j) { beta[j] = 0.0; delta[j] = c_init; }
    for (int64_t i = 0; i < X->n_rows; ++i) { margin[i] = 0.0; resid[i] = (double)y[i] - 0.5; }
}

int so_update_logistic(const so_matrix *X, const float *y, const double *n2, double lambda,
                       const int32_t *kept, int32_t n_kept,
                       double *beta, double *margin, double *resid, double *delta, double *dbeta)
{
    for (int32_t a = 0; a < n_kept; ++a) {
        const int32_t j = kept[a];
        double d = 0.0;
        if (n2[j] > 0.0) {
            const double g = col_dot_vec(X, j, resid);
            d = soft_threshold(beta[j] + 4.0 * g / n2[j], 4.0 * lambda / n2[j]) - beta[j];
        }
        dbeta[a] = d;
    }
    for (int32_t a = 0; a < n_kept; ++a) {
        const int32_t j = kept[a];
        const double d = dbeta[a];
        beta[j] += d;
        delta[j] = fabs(d);
        if (d != 0.0) {
            if (X->layout == 0) {
                const float *x = X->values + j * X->ld;
                for (int64_t i = 0; i < X->n_rows; ++i) margin[i] += (double)x[i] * d;
            } else {
                for (int64_t p = X->col_ptr[j]; p < X->col_ptr[j + 1]; ++p)
                    margin[X->row_idx[p]] += (double)X->values[p] * d;
            }
        }
    }
    for (int64_t i = 0; i < X->n_rows; ++i) resid[i] = (double)y[i] - sigmoid(margin[i]);
    return 0;
}

double so_objective_logistic(int64_t N, int64_t J, const float *y, const double *margin,
                             const double *beta, double lambda)
{
    double loss = 0.0, l1 = 0.0;
    for (int64_t i = 0; i < N; ++i) {
        const double m = margin[i];
        loss += (m > 0.0 ? m : 0.0) + log1p(exp(-fabs(m))) - (double)y[i] * m;      /* log(1 + e^m) - y m */
    }
    for (int64_t j = 0; j < J; ++j) l1 += fabs(beta[j]);
    return loss + lambda * l1;
}

/* One whole round with the logistic loss (weight_mode / filter_mode as so_round_mode). */
int so_round_logistic(const so_matrix *X, const float *y, const double *n2, double lambda, double eta, double rho,
                      int32_t n_cand, int32_t n_keep, uint64_t seed, uint64_t t, int32_t weight_mode, int32_t filter_mode,
                      double *beta, double *margin, double *resid, double *delta,
                      int32_t *cand, int32_t *kept, double *dbeta, int32_t *counts)
{
    int rc = so_sample_mode(X->n_cols, delta, eta, seed, t, n_cand, weight_mode, cand);
    if (rc) return rc;
    int32_t nk = 0, ne = 0;
    if (filter_mode == 0) so_filter(X, n2, cand, n_cand, n_keep, rho, NULL, 0, 0.0, kept, &nk, &ne, NULL);
    else if (filter_mode == 1) { nk = n_cand < n_keep ? n_cand : n_keep; for (int32_t a = 0; a < nk; ++a) kept[a] = cand[a]; ne = nk; }
    else if (filter_mode == 2) so_filter_dynamic(X, n2, cand, n_cand, n_keep, rho, beta, delta, kept, &nk, &ne);
    else return -1;
    so_update_logistic(X, y, n2, lambda, kept, nk, beta, margin, resid, delta, dbeta);
    int32_t nz = 0;
    for (int32_t a = 0; a < nk; ++a) nz += dbeta[a] != 0.0;
    counts[0] = n_cand; counts[1] = ne; counts[2] = nk; counts[3] = nz;
    return 0;
}
