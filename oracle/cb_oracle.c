/*
 * CPU oracle for head-local weighted affine ridge mapping of KV caches.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against.  It shares no code, header, table or helper with
 * the CUDA path and is never called by it.  Everything is fp64; bf16 inputs are
 * widened exactly.  Loops are written in the order of the definitions they
 * follow (no blocking, no fusion) so they can be read against the paper.
 *
 * Notation (paper, Section 2.1 and Section 3.1): source model has L_s layers,
 * H_s KV heads of width d; target has L_t, H_t, d.  "comp" is 0 for keys, 1 for
 * values.  A map is one (comp, target layer l, target head h); its id is
 * m = (comp*L_t + l)*H_t + h.  Row-vector convention y_hat = x W + b.
 *
 * Pins (see tests/test_oracle_*.py): brute force on hand-checkable integers,
 * closed forms of the bias row/column, additivity over token splits, weight
 * scaling, equality with the centred two-pass estimator of Eq. "closedform",
 * textbook least squares for constant weights, exact recovery of (A, b),
 * identity recovery for X = Y, the effective-dimension bound, the coefficient
 * counts of Section 3.2 and the storage figures of Section 4.4; the full-head
 * and multi-layer statistics against a library matrix product on gathered
 * features; the general-width solve by exact recovery and its residual; the
 * ESS floor by the Kish identity and the floors printed in Section 4.1; the
 * two-pass centred statistics against a library weighted covariance, a hand
 * example, shift invariance and equality of the resulting map with both the
 * bias-column solve and the literal centred route; the rotary embedding
 * against a library implementation, the relative-position identity and a hand
 * example; the selector's probe R^2 against a library regression score and
 * closed cases (exact linear target: 1, independent target: ~0), the ranking
 * by brute force.
 * Parity unpinned by the paper (defined by this build, not by the paper): the
 * synthetic input laws, the nearest-depth single-layer match (k = 1), the
 * lambda_eff = lambda * s_w / n convention for weights that are not mean-one,
 * the rotate-half pairing of the rotary embedding, and the pooling of the
 * selector's R^2 over target channels (each is pinned as an implementation of
 * the stated convention; the convention itself is this build's reading).
 */
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* bf16 -> fp64, exact: a bf16 is the upper half of an IEEE binary32. */
static double orc_bf16(uint16_t v)
{
    uint32_t u = ((uint32_t)v) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* fp64 -> bf16, round to nearest even, via binary32 (double rounding avoided by
 * rounding the fp64 value directly on the bf16 grid). */
static uint16_t orc_to_bf16(double x)
{
    if (x != x) return 0x7fc0;
    double ax = fabs(x);
    uint16_t sign = (x < 0.0 || (x == 0.0 && 1.0 / x < 0.0)) ? 0x8000 : 0;
    if (ax == 0.0) return sign;
    if (isinf(ax)) return (uint16_t)(sign | 0x7f80);
    int e;
    double fr = frexp(ax, &e);        /* ax = fr * 2^e, fr in [0.5, 1) */
    int E = e - 1;                    /* ax = (2 fr) * 2^E, 2 fr in [1, 2) */
    if (E < -126) E = -126;           /* subnormal range of bf16 shares binary32's exponent floor */
    double ulp = ldexp(1.0, E - 7);   /* 8 significant bits */
    double q = ax / ulp;              /* exact scaling by a power of two */
    double r = nearbyint(q);          /* default rounding mode: nearest even */
    double y = r * ulp;
    if (y >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7f80);
    float f = (float)y;               /* exact: y has at most 8 significant bits */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    (void)fr;
    return (uint16_t)(sign | (uint16_t)((u >> 16) & 0x7fff));
}

void orc_bf16_decode(const uint16_t *in, double *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_bf16(in[i]);
}

void orc_bf16_encode(const double *in, uint16_t *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_to_bf16(in[i]);
}

/* ------------------------------------------------------------------------- */
/* Head match (Section 3.2: a(h) = h for aligned KV groups; one selected layer */
/* per target layer, nearest relative depth).                                 */
/* j(l) = round(l (L_s - 1) / (L_t - 1)) in integers, halves rounded up.       */
/* ------------------------------------------------------------------------- */
void orc_head_map(int32_t Ls, int32_t Hs, int32_t Lt, int32_t Ht,
                  int32_t *src_layer /* [Lt] */, int32_t *src_head /* [Ht] */)
{
    for (int32_t l = 0; l < Lt; ++l) {
        if (Lt == 1) { src_layer[l] = 0; continue; }
        int64_t num = 2 * (int64_t)l * (Ls - 1) + (Lt - 1);
        int64_t den = 2 * (int64_t)(Lt - 1);
        src_layer[l] = (int32_t)(num / den);
    }
    for (int32_t h = 0; h < Ht; ++h)
        src_head[h] = (int32_t)(((int64_t)h * Hs) / Ht);   /* identity when Hs == Ht */
}

/*
 * Static gather schedule (Section 2.3): maps grouped by the source head they
 * read, so the source block is fetched once per group.  Items are ordered by
 * (comp, source layer, source head); the maps of an item are in ascending id.
 * Only source heads with at least one map become items.
 * Returns the number of items; arrays must hold 2*Ls*Hs (items) / 2*Lt*Ht (maps).
 */
int32_t orc_work_list(int32_t Ls, int32_t Hs, int32_t Lt, int32_t Ht,
                      const int32_t *src_layer, const int32_t *src_head,
                      int32_t *item_comp, int32_t *item_layer, int32_t *item_head,
                      int32_t *item_begin /* [n_items+1] offsets into item_maps */,
                      int32_t *item_maps)
{
    int32_t n_items = 0, n_listed = 0;
    for (int32_t comp = 0; comp < 2; ++comp)
        for (int32_t j = 0; j < Ls; ++j)
            for (int32_t g = 0; g < Hs; ++g) {
                int32_t first = n_listed;
                for (int32_t l = 0; l < Lt; ++l)
                    for (int32_t h = 0; h < Ht; ++h)
                        if (src_layer[l] == j && src_head[h] == g)
                            item_maps[n_listed++] = (comp * Lt + l) * Ht + h;
                if (n_listed > first) {
                    item_comp[n_items] = comp;
                    item_layer[n_items] = j;
                    item_head[n_items] = g;
                    item_begin[n_items] = first;
                    ++n_items;
                }
            }
    item_begin[n_items] = n_listed;
    return n_items;
}

/* ------------------------------------------------------------------------- */
/* Weighted sufficient statistics, augmented form (Section 3.4, Eq. fusedstats */
/* before centring):                                                          */
/*   G = sum_t w_t xt_t xt_t^T  (p x p),  C = sum_t w_t xt_t y_t^T  (p x d),   */
/*   xt_t = [x_t, 1], p = d + 1, bias entry last.                              */
/* One map, fp64 rows.                                                        */
/* ------------------------------------------------------------------------- */
void orc_stats_f64(const double *X /* [n][d] */, const double *Y /* [n][d] */,
                   const double *w /* [n] */, int64_t n, int32_t d,
                   double *G /* [p][p] */, double *C /* [p][d] */)
{
    const int32_t p = d + 1;
    double *xt = (double *)malloc(sizeof(double) * (size_t)p);
    memset(G, 0, sizeof(double) * (size_t)p * p);
    memset(C, 0, sizeof(double) * (size_t)p * d);
    for (int64_t t = 0; t < n; ++t) {
        for (int32_t i = 0; i < d; ++i) xt[i] = X[t * d + i];
        xt[d] = 1.0;
        for (int32_t i = 0; i < p; ++i) {
            const double wx = w[t] * xt[i];
            for (int32_t j = 0; j < p; ++j) G[(size_t)i * p + j] += wx * xt[j];
            for (int32_t j = 0; j < d; ++j) C[(size_t)i * d + j] += wx * Y[t * d + j];
        }
    }
    free(xt);
}

/*
 * The same statistics for a list of maps read straight from strided bf16 KV
 * traces (element (layer, token, head, channel) at base + layer*sl + token*st +
 * head*sh + channel, strides in elements) and fp32 weights
 * w[comp][l][h][t] at w_comp + l*w_sl + h*w_sh + t.  Maps are independent, one
 * per OpenMP thread.
 */
void orc_stats_traces(const uint16_t *src_k, const uint16_t *src_v,
                      int64_t s_sl, int64_t s_st, int64_t s_sh,
                      const uint16_t *tgt_k, const uint16_t *tgt_v,
                      int64_t t_sl, int64_t t_st, int64_t t_sh,
                      const float *w_k, const float *w_v, int64_t w_sl, int64_t w_sh,
                      int64_t n_tokens, int32_t d, int32_t Lt, int32_t Ht,
                      const int32_t *src_layer, const int32_t *src_head,
                      const int32_t *maps, int32_t n_sel,
                      double *G /* [n_sel][p][p] */, double *C /* [n_sel][p][d] */)
{
    const int32_t p = d + 1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t s = 0; s < n_sel; ++s) {
        const int32_t m = maps[s];
        const int32_t comp = m / (Lt * Ht);
        const int32_t l = (m / Ht) % Lt;
        const int32_t h = m % Ht;
        const uint16_t *xs = (comp ? src_v : src_k) + (int64_t)src_layer[l] * s_sl + (int64_t)src_head[h] * s_sh;
        const uint16_t *ys = (comp ? tgt_v : tgt_k) + (int64_t)l * t_sl + (int64_t)h * t_sh;
        const float *ws = (comp ? w_v : w_k) + (int64_t)l * w_sl + (int64_t)h * w_sh;
        double *Gm = G + (size_t)s * p * p;
        double *Cm = C + (size_t)s * p * d;
        double *xt = (double *)malloc(sizeof(double) * (size_t)p);
        double *yt = (double *)malloc(sizeof(double) * (size_t)d);
        memset(Gm, 0, sizeof(double) * (size_t)p * p);
        memset(Cm, 0, sizeof(double) * (size_t)p * d);
        for (int64_t t = 0; t < n_tokens; ++t) {
            for (int32_t i = 0; i < d; ++i) xt[i] = orc_bf16(xs[t * s_st + i]);
            xt[d] = 1.0;
            for (int32_t i = 0; i < d; ++i) yt[i] = orc_bf16(ys[t * t_st + i]);
            const double wt = (double)ws[t];
            for (int32_t i = 0; i < p; ++i) {
                const double wx = wt * xt[i];
                double *gr = Gm + (size_t)i * p;
                double *cr = Cm + (size_t)i * d;
                for (int32_t j = 0; j < p; ++j) gr[j] += wx * xt[j];
                for (int32_t j = 0; j < d; ++j) cr[j] += wx * yt[j];
            }
        }
        free(xt);
        free(yt);
    }
}

/* ------------------------------------------------------------------------- */
/* Cholesky factorisation and solve, fp64, in place.  Returns 0, or r > 0 if   */
/* pivot r (1-based) is not positive.                                         */
/* ------------------------------------------------------------------------- */
static int32_t orc_cholesky(double *A, int32_t p)
{
    for (int32_t j = 0; j < p; ++j) {
        double s = A[(size_t)j * p + j];
        for (int32_t k = 0; k < j; ++k) s -= A[(size_t)j * p + k] * A[(size_t)j * p + k];
        if (!(s > 0.0)) return j + 1;
        const double ljj = sqrt(s);
        A[(size_t)j * p + j] = ljj;
        for (int32_t i = j + 1; i < p; ++i) {
            double v = A[(size_t)i * p + j];
            for (int32_t k = 0; k < j; ++k) v -= A[(size_t)i * p + k] * A[(size_t)j * p + k];
            A[(size_t)i * p + j] = v / ljj;
        }
    }
    return 0;
}

static void orc_cholesky_solve(const double *L, int32_t p, double *B, int32_t nrhs)
{
    for (int32_t c = 0; c < nrhs; ++c) {
        for (int32_t i = 0; i < p; ++i) {            /* L z = b */
            double v = B[(size_t)i * nrhs + c];
            for (int32_t k = 0; k < i; ++k) v -= L[(size_t)i * p + k] * B[(size_t)k * nrhs + c];
            B[(size_t)i * nrhs + c] = v / L[(size_t)i * p + i];
        }
        for (int32_t i = p - 1; i >= 0; --i) {       /* L^T x = z */
            double v = B[(size_t)i * nrhs + c];
            for (int32_t k = i + 1; k < p; ++k) v -= L[(size_t)k * p + i] * B[(size_t)k * nrhs + c];
            B[(size_t)i * nrhs + c] = v / L[(size_t)i * p + i];
        }
    }
}

/*
 * Ridge solve on augmented statistics (Section 3.1, Eq. closedform, written
 * for the bias-column form): (G + lambda_eff J) Theta = C, J = diag(1,..,1,0)
 * (the bias is not penalised), Theta = [W; b].
 * The paper states the objective for weights rescaled to mean one; rescaling w
 * by n / s_w is the same as keeping w and using lambda_eff = lambda * s_w / n
 * (s_w = G[d][d]).  raw_lambda != 0 uses lambda_eff = lambda instead.
 * Degenerate systems: info = failing pivot, Theta zero-filled.
 */
int32_t orc_ridge_solve(const double *G, const double *C, int32_t d, int64_t n,
                        double lambda, int32_t raw_lambda, double *Theta /* [p][d] */)
{
    const int32_t p = d + 1;
    double *A = (double *)malloc(sizeof(double) * (size_t)p * p);
    memcpy(A, G, sizeof(double) * (size_t)p * p);
    const double s_w = G[(size_t)d * p + d];
    const double lam = raw_lambda ? lambda : lambda * s_w / (double)n;
    for (int32_t i = 0; i < d; ++i) A[(size_t)i * p + i] += lam;
    int32_t info = orc_cholesky(A, p);
    if (info != 0) {
        memset(Theta, 0, sizeof(double) * (size_t)p * d);
    } else {
        memcpy(Theta, C, sizeof(double) * (size_t)p * d);
        orc_cholesky_solve(A, p, Theta, d);
    }
    free(A);
    return info;
}

void orc_ridge_solve_batch(const double *G, const double *C, int32_t n_maps, int32_t d, int64_t n,
                           double lambda, int32_t raw_lambda, double *Theta, int32_t *info)
{
    const int32_t p = d + 1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t m = 0; m < n_maps; ++m)
        info[m] = orc_ridge_solve(G + (size_t)m * p * p, C + (size_t)m * p * d, d, n, lambda, raw_lambda,
                                  Theta + (size_t)m * p * d);
}

/*
 * The paper's literal route (Section 3.1): rescale the weights to mean one,
 * weighted means x_bar = n^-1 sum w_i x_i, y_bar likewise, centred rows,
 * W = (Xc^T Dw Xc + lambda I)^-1 Xc^T Dw Yc, b = y_bar - x_bar W.
 * Used to check that the bias-column form above is the same estimator.
 */
int32_t orc_ridge_centered(const double *X, const double *Y, const double *w, int64_t n, int32_t d,
                           double lambda, double *Theta /* [d+1][d]: W then b */)
{
    double sw = 0.0;
    for (int64_t t = 0; t < n; ++t) sw += w[t];
    if (!(sw > 0.0)) { memset(Theta, 0, sizeof(double) * (size_t)(d + 1) * d); return 1; }
    const double scale = (double)n / sw;                 /* mean-one rescale */
    double *xb = (double *)calloc((size_t)d, sizeof(double));
    double *yb = (double *)calloc((size_t)d, sizeof(double));
    for (int64_t t = 0; t < n; ++t) {
        const double wt = w[t] * scale;
        for (int32_t i = 0; i < d; ++i) { xb[i] += wt * X[t * d + i]; yb[i] += wt * Y[t * d + i]; }
    }
    for (int32_t i = 0; i < d; ++i) { xb[i] /= (double)n; yb[i] /= (double)n; }
    double *A = (double *)calloc((size_t)d * d, sizeof(double));
    double *B = (double *)calloc((size_t)d * d, sizeof(double));
    double *xc = (double *)malloc(sizeof(double) * (size_t)d);
    double *yc = (double *)malloc(sizeof(double) * (size_t)d);
    for (int64_t t = 0; t < n; ++t) {
        const double wt = w[t] * scale;
        for (int32_t i = 0; i < d; ++i) { xc[i] = X[t * d + i] - xb[i]; yc[i] = Y[t * d + i] - yb[i]; }
        for (int32_t i = 0; i < d; ++i)
            for (int32_t j = 0; j < d; ++j) {
                A[(size_t)i * d + j] += wt * xc[i] * xc[j];
                B[(size_t)i * d + j] += wt * xc[i] * yc[j];
            }
    }
    for (int32_t i = 0; i < d; ++i) A[(size_t)i * d + i] += lambda;
    int32_t info = orc_cholesky(A, d);
    if (info == 0) {
        orc_cholesky_solve(A, d, B, d);
        memcpy(Theta, B, sizeof(double) * (size_t)d * d);
        for (int32_t j = 0; j < d; ++j) {
            double v = yb[j];
            for (int32_t i = 0; i < d; ++i) v -= xb[i] * B[(size_t)i * d + j];
            Theta[(size_t)d * d + j] = v;
        }
    } else {
        memset(Theta, 0, sizeof(double) * (size_t)(d + 1) * d);
    }
    free(A); free(B); free(xc); free(yc); free(xb); free(yb);
    return info;
}

/* ------------------------------------------------------------------------- */
/* Two-pass centred construction (Section 3.4, Eq. fusedstats): first the      */
/* weighted means of every map over ALL rows,                                  */
/*   s_w = sum_t w_t,  mu_x = sum_t w_t x_t / s_w,  mu_y = sum_t w_t y_t / s_w, */
/* then, in a second traversal,                                                */
/*   A = sum_t w_t (x_t - mu_x)(x_t - mu_x)^T,                                 */
/*   B = sum_t w_t (x_t - mu_x)(y_t - mu_y)^T.                                 */
/* Same trace addressing and map numbering as orc_stats_traces.  The weights   */
/* are used as given (not rescaled); a map whose weights sum to zero gets zero */
/* means.                                                                      */
/* ------------------------------------------------------------------------- */
void orc_means_traces(const uint16_t *src_k, const uint16_t *src_v,
                      int64_t s_sl, int64_t s_st, int64_t s_sh,
                      const uint16_t *tgt_k, const uint16_t *tgt_v,
                      int64_t t_sl, int64_t t_st, int64_t t_sh,
                      const float *w_k, const float *w_v, int64_t w_sl, int64_t w_sh,
                      int64_t n_tokens, int32_t d, int32_t Lt, int32_t Ht,
                      const int32_t *src_layer, const int32_t *src_head,
                      const int32_t *maps, int32_t n_sel,
                      double *sum_x /* [n_sel][d]: sum w x */, double *sum_y /* [n_sel][d] */,
                      double *s_w /* [n_sel] */)
{
    for (int32_t s = 0; s < n_sel; ++s) {
        const int32_t m = maps[s];
        const int32_t comp = m / (Lt * Ht);
        const int32_t l = (m / Ht) % Lt;
        const int32_t h = m % Ht;
        const uint16_t *xs = (comp ? src_v : src_k) + (int64_t)src_layer[l] * s_sl + (int64_t)src_head[h] * s_sh;
        const uint16_t *ys = (comp ? tgt_v : tgt_k) + (int64_t)l * t_sl + (int64_t)h * t_sh;
        const float *ws = (comp ? w_v : w_k) + (int64_t)l * w_sl + (int64_t)h * w_sh;
        double *ax = sum_x + (size_t)s * d, *ay = sum_y + (size_t)s * d;
        for (int32_t i = 0; i < d; ++i) ax[i] = ay[i] = 0.0;
        double sw = 0.0;
        for (int64_t t = 0; t < n_tokens; ++t) {
            const double wt = (double)ws[t];
            sw += wt;
            for (int32_t i = 0; i < d; ++i) {
                ax[i] += wt * orc_bf16(xs[t * s_st + i]);
                ay[i] += wt * orc_bf16(ys[t * t_st + i]);
            }
        }
        s_w[s] = sw;
    }
}

void orc_centered_stats_traces(const uint16_t *src_k, const uint16_t *src_v,
                               int64_t s_sl, int64_t s_st, int64_t s_sh,
                               const uint16_t *tgt_k, const uint16_t *tgt_v,
                               int64_t t_sl, int64_t t_st, int64_t t_sh,
                               const float *w_k, const float *w_v, int64_t w_sl, int64_t w_sh,
                               int64_t n_tokens, int32_t d, int32_t Lt, int32_t Ht,
                               const int32_t *src_layer, const int32_t *src_head,
                               const int32_t *maps, int32_t n_sel,
                               const double *mu_x /* [n_sel][d] */, const double *mu_y /* [n_sel][d] */,
                               double *A /* [n_sel][d][d] */, double *B /* [n_sel][d][d] */)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t s = 0; s < n_sel; ++s) {
        const int32_t m = maps[s];
        const int32_t comp = m / (Lt * Ht);
        const int32_t l = (m / Ht) % Lt;
        const int32_t h = m % Ht;
        const uint16_t *xs = (comp ? src_v : src_k) + (int64_t)src_layer[l] * s_sl + (int64_t)src_head[h] * s_sh;
        const uint16_t *ys = (comp ? tgt_v : tgt_k) + (int64_t)l * t_sl + (int64_t)h * t_sh;
        const float *ws = (comp ? w_v : w_k) + (int64_t)l * w_sl + (int64_t)h * w_sh;
        const double *mx = mu_x + (size_t)s * d, *my = mu_y + (size_t)s * d;
        double *Am = A + (size_t)s * d * d, *Bm = B + (size_t)s * d * d;
        double *xc = (double *)malloc(sizeof(double) * (size_t)d);
        double *yc = (double *)malloc(sizeof(double) * (size_t)d);
        memset(Am, 0, sizeof(double) * (size_t)d * d);
        memset(Bm, 0, sizeof(double) * (size_t)d * d);
        for (int64_t t = 0; t < n_tokens; ++t) {
            for (int32_t i = 0; i < d; ++i) {
                xc[i] = orc_bf16(xs[t * s_st + i]) - mx[i];
                yc[i] = orc_bf16(ys[t * t_st + i]) - my[i];
            }
            const double wt = (double)ws[t];
            for (int32_t i = 0; i < d; ++i) {
                const double wx = wt * xc[i];
                for (int32_t j = 0; j < d; ++j) {
                    Am[(size_t)i * d + j] += wx * xc[j];
                    Bm[(size_t)i * d + j] += wx * yc[j];
                }
            }
        }
        free(xc);
        free(yc);
    }
}

/*
 * The solve of the two-pass path (Section 3.4, last display; Section 3.1, Eq.
 * closedform): W = (A + lambda_eff I)^-1 B, b = mu_y - mu_x W, with the same
 * lambda_eff = lambda * s_w / n convention as orc_ridge_solve (weights not
 * rescaled to mean one), or lambda itself when raw_lambda != 0.
 */
int32_t orc_ridge_solve_centered(const double *A, const double *B, const double *mu_x, const double *mu_y,
                                 double s_w, int32_t d, int64_t n, double lambda, int32_t raw_lambda,
                                 double *Theta /* [d+1][d]: W then b */)
{
    const double lam = raw_lambda ? lambda : (n > 0 ? lambda * s_w / (double)n : lambda);
    double *M = (double *)malloc(sizeof(double) * (size_t)d * d);
    memcpy(M, A, sizeof(double) * (size_t)d * d);
    for (int32_t i = 0; i < d; ++i) M[(size_t)i * d + i] += lam;
    int32_t info = orc_cholesky(M, d);
    if (info == 0) {
        memcpy(Theta, B, sizeof(double) * (size_t)d * d);
        orc_cholesky_solve(M, d, Theta, d);
        for (int32_t j = 0; j < d; ++j) {
            double v = mu_y[j];
            for (int32_t i = 0; i < d; ++i) v -= mu_x[i] * Theta[(size_t)i * d + j];
            Theta[(size_t)d * d + j] = v;
        }
    } else {
        memset(Theta, 0, sizeof(double) * (size_t)(d + 1) * d);
    }
    free(M);
    return info;
}

/* ------------------------------------------------------------------------- */
/* Rotary position embedding at the boundary (Section 2.2 and Section 3.1:     */
/* source RoPE is removed before fitting, target RoPE restored after mapping,  */
/* so the map acts in content coordinates).  Keys only; values carry no RoPE.  */
/* Convention (the paper does not print one; this is the rotate-half form of   */
/* the RoFormer rotation used by the Llama / Qwen model families): channel i   */
/* < d/2 pairs with channel i + d/2, angle phi_i = pos * base^(-2 i / d),       */
/*   out_i       = x_i cos phi_i - x_{i+d/2} sin phi_i,                          */
/*   out_{i+d/2} = x_i sin phi_i + x_{i+d/2} cos phi_i;                          */
/* inverse != 0 rotates by -phi (removes the embedding).  Rows of width d.     */
/* ------------------------------------------------------------------------- */
void orc_rope_rotate(const double *in, double *out, int64_t n_rows, int32_t d,
                     const int32_t *pos, double base, int32_t inverse)
{
    const int32_t half = d / 2;
    for (int64_t t = 0; t < n_rows; ++t)
        for (int32_t i = 0; i < half; ++i) {
            const double phi = (double)pos[t] * pow(base, -2.0 * (double)i / (double)d);
            const double c = cos(phi), s = inverse ? -sin(phi) : sin(phi);
            const double a = in[t * d + i], b = in[t * d + i + half];
            out[t * d + i] = a * c - b * s;
            out[t * d + i + half] = a * s + b * c;
        }
}

/* ------------------------------------------------------------------------- */
/* Layer selector (Section 3.1, first paragraph): for a target layer, every    */
/* candidate source layer gets centred single-source-layer OLS probes under    */
/* the same head assignment; the held-in R^2 of a probe is                     */
/*   R^2 = 1 - sum_t w_t ||yc_t - xc_t W||^2 / sum_t w_t ||yc_t||^2            */
/* (xc, yc centred at the weighted means, W the least-squares solution,        */
/* residuals pooled over the d target channels: the paper does not say how the */
/* channels are combined; this is the variance-weighted multi-output R^2).     */
/* The layer's score is the mean over KV heads and K/V; the first k layers in  */
/* descending score (ties: lower index) are the selected set, returned in      */
/* ascending order.  lambda_rel > 0 adds lambda_rel * tr(A)/d to the diagonal  */
/* (0 = plain OLS).  Returns 0, or the failing pivot of the factorisation.     */
/* ------------------------------------------------------------------------- */
int32_t orc_probe_r2(const double *X, const double *Y, const double *w, int64_t n, int32_t d,
                     double lambda_rel, double *r2_out)
{
    double sw = 0.0;
    double *xb = (double *)calloc((size_t)d, sizeof(double));
    double *yb = (double *)calloc((size_t)d, sizeof(double));
    for (int64_t t = 0; t < n; ++t) {
        sw += w[t];
        for (int32_t i = 0; i < d; ++i) { xb[i] += w[t] * X[t * d + i]; yb[i] += w[t] * Y[t * d + i]; }
    }
    if (!(sw > 0.0)) { free(xb); free(yb); *r2_out = 0.0; return 1; }
    for (int32_t i = 0; i < d; ++i) { xb[i] /= sw; yb[i] /= sw; }
    double *A = (double *)calloc((size_t)d * d, sizeof(double));
    double *B = (double *)calloc((size_t)d * d, sizeof(double));
    for (int64_t t = 0; t < n; ++t)
        for (int32_t i = 0; i < d; ++i) {
            const double wx = w[t] * (X[t * d + i] - xb[i]);
            for (int32_t j = 0; j < d; ++j) {
                A[(size_t)i * d + j] += wx * (X[t * d + j] - xb[j]);
                B[(size_t)i * d + j] += wx * (Y[t * d + j] - yb[j]);
            }
        }
    double tr = 0.0;
    for (int32_t i = 0; i < d; ++i) tr += A[(size_t)i * d + i];
    for (int32_t i = 0; i < d; ++i) A[(size_t)i * d + i] += lambda_rel * tr / (double)d;
    int32_t info = orc_cholesky(A, d);
    if (info == 0) {
        orc_cholesky_solve(A, d, B, d);            /* B now holds W */
        double sse = 0.0, sst = 0.0;
        for (int64_t t = 0; t < n; ++t)
            for (int32_t j = 0; j < d; ++j) {
                double pred = 0.0;
                for (int32_t i = 0; i < d; ++i) pred += (X[t * d + i] - xb[i]) * B[(size_t)i * d + j];
                const double yc = Y[t * d + j] - yb[j];
                sse += w[t] * (yc - pred) * (yc - pred);
                sst += w[t] * yc * yc;
            }
        *r2_out = sst > 0.0 ? 1.0 - sse / sst : 0.0;
    } else {
        *r2_out = 0.0;
    }
    free(A); free(B); free(xb); free(yb);
    return info;
}

void orc_rank_layers(const double *scores /* [Lt][Ls] */, int32_t Lt, int32_t Ls, int32_t k, int32_t *sets /* [Lt][k] */)
{
    for (int32_t l = 0; l < Lt; ++l) {
        char *taken = (char *)calloc((size_t)Ls, 1);
        for (int32_t q = 0; q < k; ++q) {
            int32_t best = -1;
            for (int32_t j = 0; j < Ls; ++j)
                if (!taken[j] && (best < 0 || scores[(size_t)l * Ls + j] > scores[(size_t)l * Ls + best])) best = j;
            taken[best] = 1;
        }
        int32_t q = 0;
        for (int32_t j = 0; j < Ls; ++j)
            if (taken[j]) sets[(size_t)l * k + q++] = j;   /* ascending */
        free(taken);
    }
}

/* ------------------------------------------------------------------------- */
/* Online affine apply (Section 3.2): y_hat_t = x_t W + b per map, written to  */
/* a target cache.  Source rows come from strided bf16; output is fp64, and   */
/* optionally also rounded to bf16 (nearest even) as a decode-ready cache.    */
/* Output element (l, t, h, c) of component comp at                            */
/*   out[comp] + l*o_sl + t*o_st + h*o_sh + c.                                 */
/* ------------------------------------------------------------------------- */
void orc_apply(const uint16_t *src_k, const uint16_t *src_v, int64_t s_sl, int64_t s_st, int64_t s_sh,
               int64_t n_tokens, int32_t d, int32_t Lt, int32_t Ht,
               const int32_t *src_layer, const int32_t *src_head,
               const double *Theta /* [n_maps][p][d] */,
               const int32_t *maps, int32_t n_sel,
               double *out_k, double *out_v, uint16_t *out_k_bf16, uint16_t *out_v_bf16,
               int64_t o_sl, int64_t o_st, int64_t o_sh)
{
    const int32_t p = d + 1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t s = 0; s < n_sel; ++s) {
        const int32_t m = maps[s];
        const int32_t comp = m / (Lt * Ht);
        const int32_t l = (m / Ht) % Lt;
        const int32_t h = m % Ht;
        const uint16_t *xs = (comp ? src_v : src_k) + (int64_t)src_layer[l] * s_sl + (int64_t)src_head[h] * s_sh;
        const double *W = Theta + (size_t)m * p * d;
        double *o = (comp ? out_v : out_k);
        uint16_t *ob = (comp ? out_v_bf16 : out_k_bf16);
        for (int64_t t = 0; t < n_tokens; ++t) {
            const int64_t base = (int64_t)l * o_sl + t * o_st + (int64_t)h * o_sh;
            for (int32_t c = 0; c < d; ++c) {
                double v = W[(size_t)d * d + c];                       /* b */
                for (int32_t i = 0; i < d; ++i) v += orc_bf16(xs[t * s_st + i]) * W[(size_t)i * d + c];
                if (o) o[base + c] = v;
                if (ob) ob[base + c] = orc_to_bf16(v);
            }
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Full-head regressor (Section 3.1, Eq. "fullheadfeature"): the feature of a  */
/* target layer l concatenates every source KV head of the k selected source  */
/* layers S_l, layer-major then head then channel, bias last:                 */
/*   x_full = concat_{j in S_l, g in [H_s]} Z_{j,t,g},  p_f = k H_s d + 1.     */
/* One G (p_f x p_f) per (comp, l), shared by the layer's heads (weights are   */
/* per (comp, l, token) here), and one C (p_f x d) per target head.           */
/* Same definition of the statistics as above, written out for this feature.  */
/* ------------------------------------------------------------------------- */
void orc_fullhead_stats(const uint16_t *src /* one component: [Ls][T][Hs][d] */,
                        int64_t s_sl, int64_t s_st, int64_t s_sh,
                        const uint16_t *tgt /* one component */, int64_t t_sl, int64_t t_st, int64_t t_sh,
                        const float *w /* [T] weights of this (comp, l) */,
                        int64_t n_tokens, int32_t d, int32_t Hs, int32_t Ht, int32_t l,
                        const int32_t *layer_set /* [k] */, int32_t k,
                        double *G /* [pf][pf] */, double *C /* [Ht][pf][d] */)
{
    const int32_t nf = k * Hs * d, pf = nf + 1;
    memset(G, 0, sizeof(double) * (size_t)pf * pf);
    memset(C, 0, sizeof(double) * (size_t)Ht * pf * d);
    int nthreads = 1;
#ifdef _OPENMP
    nthreads = omp_get_max_threads();
#endif
    /* rows of G are independent given the token's feature vector: parallel over row blocks, tokens in order */
    double *xt_all = (double *)malloc(sizeof(double) * (size_t)pf);
    double *yt_all = (double *)malloc(sizeof(double) * (size_t)Ht * d);
    (void)nthreads;
    for (int64_t t = 0; t < n_tokens; ++t) {
        for (int32_t q = 0; q < k; ++q)
            for (int32_t g = 0; g < Hs; ++g)
                for (int32_t c = 0; c < d; ++c)
                    xt_all[(q * Hs + g) * d + c] =
                        orc_bf16(src[(int64_t)layer_set[q] * s_sl + t * s_st + (int64_t)g * s_sh + c]);
        xt_all[nf] = 1.0;
        for (int32_t h = 0; h < Ht; ++h)
            for (int32_t c = 0; c < d; ++c)
                yt_all[h * d + c] = orc_bf16(tgt[(int64_t)l * t_sl + t * t_st + (int64_t)h * t_sh + c]);
        const double wt = (double)w[t];
#pragma omp parallel for schedule(static)
        for (int32_t i = 0; i < pf; ++i) {
            const double wx = wt * xt_all[i];
            double *gr = G + (size_t)i * pf;
            for (int32_t j = 0; j < pf; ++j) gr[j] += wx * xt_all[j];
            for (int32_t h = 0; h < Ht; ++h) {
                double *cr = C + ((size_t)h * pf + i) * d;
                for (int32_t c = 0; c < d; ++c) cr[c] += wx * yt_all[h * d + c];
            }
        }
    }
    free(xt_all);
    free(yt_all);
}

/* Selected source layers of the full-head contrast: c = j(l) (nearest depth); S_l = {c-1, c, c+1, c+2}       */
/* (k consecutive layers starting one below c), shifted into [0, L_s - 1], ascending.                        */
void orc_fullhead_layer_sets(int32_t Ls, int32_t Lt, int32_t k, int32_t *sets /* [Lt][k] */)
{
    for (int32_t l = 0; l < Lt; ++l) {
        int32_t c = 0;
        if (Lt > 1) c = (int32_t)((2 * (int64_t)l * (Ls - 1) + (Lt - 1)) / (2 * (int64_t)(Lt - 1)));
        int32_t lo = c - 1;
        if (lo + k > Ls) lo = Ls - k;
        if (lo < 0) lo = 0;
        for (int32_t q = 0; q < k; ++q) sets[l * k + q] = lo + q;
    }
}

/* ------------------------------------------------------------------------- */
/* Effective-sample-size floor on the attention weights (Section 3.3).        */
/* For one (layer, head, component): raw sensitivities r_raw >= 0 over n       */
/* rows are mean-normalised (mean r = 1), CV^2 = mean (r_i - 1)^2, and the     */
/* weights are shrunk toward uniform, w_i = 1 + alpha (r_i - 1), with the      */
/* largest alpha in [0, 1] whose Kish effective sample size                    */
/*   n_eff = (sum w)^2 / sum w^2 = n / (1 + alpha^2 CV^2)                      */
/* stays at or above tau = min(n, 2 p) (p = feature width):                    */
/*   alpha* = 1 if CV^2 = 0, else min(1, sqrt((n / tau - 1) / CV^2)).          */
/* Returns alpha*; cv2_out (may be NULL) receives CV^2.  A row of zeros (no    */
/* sensitivity at all) gives uniform weights.                                 */
/* ------------------------------------------------------------------------- */
double orc_ess_weights(const double *r_raw, int64_t n, int64_t p_width, double *w, double *cv2_out)
{
    double mean = 0.0;
    for (int64_t i = 0; i < n; ++i) mean += r_raw[i];
    mean /= (double)n;
    if (!(mean > 0.0)) {
        for (int64_t i = 0; i < n; ++i) w[i] = 1.0;
        if (cv2_out) *cv2_out = 0.0;
        return 1.0;
    }
    double cv2 = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        const double r = r_raw[i] / mean;
        cv2 += (r - 1.0) * (r - 1.0);
    }
    cv2 /= (double)n;
    const double tau = (double)((n < 2 * p_width) ? n : 2 * p_width);
    double alpha = 1.0;
    if (cv2 > 0.0) {
        const double a = sqrt(((double)n / tau - 1.0) / cv2);
        alpha = a < 1.0 ? a : 1.0;
    }
    for (int64_t i = 0; i < n; ++i) w[i] = 1.0 + alpha * (r_raw[i] / mean - 1.0);
    if (cv2_out) *cv2_out = cv2;
    return alpha;
}

/* The ridge solve for a regressor of any width (several selected layers): G [p][p], C [p][dy], bias entry last and not */
/* penalised; same conventions as orc_ridge_solve.                                                                      */
int32_t orc_ridge_solve_pd(const double *G, const double *C, int32_t p, int32_t dy, int64_t n,
                           double lambda, int32_t raw_lambda, double *Theta /* [p][dy] */)
{
    double *A = (double *)malloc(sizeof(double) * (size_t)p * p);
    memcpy(A, G, sizeof(double) * (size_t)p * p);
    const double s_w = G[(size_t)(p - 1) * p + (p - 1)];
    const double lam = raw_lambda ? lambda : lambda * s_w / (double)n;
    for (int32_t i = 0; i < p - 1; ++i) A[(size_t)i * p + i] += lam;
    int32_t info = orc_cholesky(A, p);
    if (info != 0) {
        memset(Theta, 0, sizeof(double) * (size_t)p * dy);
    } else {
        memcpy(Theta, C, sizeof(double) * (size_t)p * dy);
        orc_cholesky_solve(A, p, Theta, dy);
    }
    free(A);
    return info;
}
