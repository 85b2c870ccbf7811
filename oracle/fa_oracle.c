/*
 * fa_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of what the hybrid-KV decode path of
 * FourierAttention computes.  It exists so that the CUDA library can be
 * checked against something written straight from the paper's definitions.
 * Only the test-suite, the smoke check and the benchmark's cpu_baseline /
 * reference arm may build, load or call this file.  It shares no code,
 * header, table or helper with the CUDA library, and it keeps its own
 * (natural, token-major) representation of the cache.
 *
 * Every function cites the passage of the paper it follows:
 *   Eq.1  init / local windows           (Sec. 3.3)
 *   Eq.2  middle slices by index sets    (Sec. 3.3)
 *   Eq.3  K^mc = F K^mn, V^mc = F V^mn   (Sec. 3.3)
 *   Eq.4  the real 2k x L matrix F       (Sec. 3.3)
 *   Eq.5  per-token coefficient update   (Sec. 3.3)
 *   Eq.6  reconstruction + attention     (Sec. 3.3)
 *   Sec. 3.4  dimension selection by reconstruction error
 *
 * Readings taken where the paper is silent or inconsistent (each one is
 * listed in the design notes of the repository):
 *   - the basis argument is the position of a token inside the middle
 *     segment, j = t - n_init, both in Eq.3 and Eq.5, so that appending
 *     equals recompressing;
 *   - the reconstruction weights are either the orthogonal ones
 *     (1/T for the constant row, 2/T for the others; norm == 0) or the
 *     paper's literal 1/k (norm == 1);
 *   - the tokens that leave the local window also append their kept
 *     dimensions to K^mu / V^mu;
 *   - no mask, q head g reads KV head g / (Hq / Hkv).
 *
 * Pins (tests/test_oracle_*.py): Gram matrix of F, numpy rfft / irfft,
 * exact recovery of in-span signals, append == recompress, reduction to
 * textbook softmax attention, brute force on tiny inputs, Eq.4 fixture.
 * The paper-literal 1/k scale has no independent pin beyond its closed-form
 * ratio to the orthogonal one: "parity unpinned" for that flag.
 *
 * Parallelism: optional OpenMP over independent rows only; no blocking,
 * fusion or re-association of the definitions.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define FO_PI 3.14159265358979323846264338327950288

typedef struct {
    int32_t B, Hq, Hkv, d;         /* batch, query heads, KV heads, head dim          */
    int32_t n_full_k, n_full_v;    /* |D^ku|, |D^vu|                                   */
    int32_t k;                     /* complex states; 2k real coefficients (Eq.4)      */
    int32_t norm;                  /* 0: orthogonal weights, 1: literal 1/k (Eq.6)     */
    int64_t T;                     /* period of the translated window                  */
    int32_t L_init, L_local;       /* Eq.1                                             */
    int32_t cap_mid;               /* rows allocated for K^mu / V^mu                   */
    double  scale;                 /* softmax scale                                    */
} fo_cfg;

/* The oracle's own cache: natural layouts, everything double. */
typedef struct {
    const int32_t *idx_full_k, *idx_comp_k;   /* [Hkv][n_full_k], [Hkv][d-n_full_k] */
    const int32_t *idx_full_v, *idx_comp_v;
    double *k_init, *v_init;       /* [B][Hkv][L_init][d]                  */
    double *k_local, *v_local;     /* [B][Hkv][L_local][d], oldest first   */
    double *k_mid, *v_mid;         /* [B][Hkv][cap_mid][n_full]  (K^mu)    */
    double *coef_k, *coef_v;       /* [B][Hkv][2k][d - n_full]   (K^mc)    */
    int32_t *n_init, *n_local, *n_mid;   /* [B] */
} fo_cache;

int fo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Eq.4: column j of F.  f[2n] = cos(2 pi n j / T), f[2n+1] = sin(2 pi n j / T).
 * The product n*j is reduced modulo T in integers before the division so the
 * angle keeps full precision at any position. */
void fo_basis_column(int64_t T, int32_t k, int64_t j, double *f)
{
    for (int32_t n = 0; n < k; ++n) {
        int64_t r = ((int64_t)n * j) % T;
        double ang = 2.0 * FO_PI * (double)r / (double)T;
        f[2 * n] = cos(ang);
        f[2 * n + 1] = sin(ang);
    }
}

/* Reconstruction weight of coefficient row m (Eq.6's 1/k, or the weights that
 * make F^T diag(w) F the identity on the span of the rows over a full period). */
double fo_weight(const fo_cfg *c, int32_t m)
{
    if (c->norm == 1) return 1.0 / (double)c->k;
    if (m == 0) return 1.0 / (double)c->T;
    if (m == 1) return 0.0;
    return 2.0 / (double)c->T;
}

static size_t off_win(const fo_cfg *c, int b, int h, int rows_per, int row)
{
    return ((((size_t)b * c->Hkv + h) * rows_per) + row) * (size_t)c->d;
}
static size_t off_mid(const fo_cfg *c, int b, int h, int nfull, int row)
{
    return ((((size_t)b * c->Hkv + h) * c->cap_mid) + row) * (size_t)nfull;
}
static size_t off_coef(const fo_cfg *c, int b, int h, int ncomp)
{
    return (((size_t)b * c->Hkv + h) * (size_t)(2 * c->k)) * (size_t)ncomp;
}

/* Eq.5 for one side (K or V) of one (b, h): the row x that leaves the local
 * window becomes middle token j; its kept dims join K^mu, its compressed dims
 * are folded into the coefficients with column j of F. */
static void fold_row(const fo_cfg *c, const double *x, const int32_t *idx_full,
                     const int32_t *idx_comp, int nfull, double *mid_row,
                     double *coef, int64_t j)
{
    int ncomp = c->d - nfull;
    for (int e = 0; e < nfull; ++e) mid_row[e] = x[idx_full[e]];
    double *f = (double *)malloc(sizeof(double) * 2 * (size_t)c->k);
    fo_basis_column(c->T, c->k, j, f);
    for (int m = 0; m < 2 * c->k; ++m)
        for (int e = 0; e < ncomp; ++e)
            coef[(size_t)m * ncomp + e] += f[m] * x[idx_comp[e]];
    free(f);
}

/* Eq.1-3: partition a prefilled K, V ([B][L][Hkv][d], double) into windows,
 * kept middle dims and Fourier coefficients of the compressed middle dims.
 * Returns 0, or -1 if the middle does not fit (cap_mid or T). */
int fo_compress(const fo_cfg *c, fo_cache *cache, const double *K, const double *V, int32_t L)
{
    int n_init = L < c->L_init ? L : c->L_init;
    int n_local = (L - n_init) < c->L_local ? (L - n_init) : c->L_local;
    int n_mid = L - n_init - n_local;
    if (n_mid > c->cap_mid || (int64_t)n_mid > c->T) return -1;
    int M = 2 * c->k;
    for (int b = 0; b < c->B; ++b) {
        cache->n_init[b] = n_init;
        cache->n_local[b] = n_local;
        cache->n_mid[b] = n_mid;
        for (int h = 0; h < c->Hkv; ++h) {
            for (int side = 0; side < 2; ++side) {
                const double *X = side == 0 ? K : V;
                int nfull = side == 0 ? c->n_full_k : c->n_full_v;
                int ncomp = c->d - nfull;
                const int32_t *idf = (side == 0 ? cache->idx_full_k : cache->idx_full_v) + (size_t)h * nfull;
                const int32_t *idc = (side == 0 ? cache->idx_comp_k : cache->idx_comp_v) + (size_t)h * ncomp;
                double *w_init = side == 0 ? cache->k_init : cache->v_init;
                double *w_local = side == 0 ? cache->k_local : cache->v_local;
                double *mid = side == 0 ? cache->k_mid : cache->v_mid;
                double *coef = (side == 0 ? cache->coef_k : cache->coef_v) + off_coef(c, b, h, ncomp);
#define XROW(t) (X + ((((size_t)b * L + (t)) * c->Hkv + h) * (size_t)c->d))
                /* Eq.1 */
                for (int t = 0; t < n_init; ++t)
                    memcpy(w_init + off_win(c, b, h, c->L_init, t), XROW(t), sizeof(double) * c->d);
                for (int t = 0; t < n_local; ++t)
                    memcpy(w_local + off_win(c, b, h, c->L_local, t), XROW(L - n_local + t), sizeof(double) * c->d);
                /* Eq.2, kept dims */
                for (int j = 0; j < n_mid; ++j)
                    for (int e = 0; e < nfull; ++e)
                        mid[off_mid(c, b, h, nfull, j) + e] = XROW(n_init + j)[idf[e]];
                /* Eq.3 with F from Eq.4: C[m][e] = sum_j F[m][j] X[n_init + j][D^c[e]] */
#pragma omp parallel for schedule(static)
                for (int n = 0; n < c->k; ++n) {
                    double *row_c = coef + (size_t)(2 * n) * ncomp;
                    double *row_s = coef + (size_t)(2 * n + 1) * ncomp;
                    for (int e = 0; e < ncomp; ++e) { row_c[e] = 0.0; row_s[e] = 0.0; }
                    for (int j = 0; j < n_mid; ++j) {
                        int64_t r = ((int64_t)n * j) % c->T;
                        double ang = 2.0 * FO_PI * (double)r / (double)c->T;
                        double fc = cos(ang), fs = sin(ang);
                        const double *x = XROW(n_init + j);
                        for (int e = 0; e < ncomp; ++e) {
                            row_c[e] += fc * x[idc[e]];
                            row_s[e] += fs * x[idc[e]];
                        }
                    }
                }
                (void)M;
#undef XROW
            }
        }
    }
    return 0;
}

/* Eq.5: push one token (k_new, v_new: [B][Hkv][d]).  Tokens fill the init
 * window first, then the local window; once the local window is full its
 * oldest row leaves and is folded into the middle.  Returns 0, or -1 when the
 * middle is out of room. */
int fo_append(const fo_cfg *c, fo_cache *cache, const double *k_new, const double *v_new)
{
    for (int b = 0; b < c->B; ++b) {
        int to_init = cache->n_init[b] < c->L_init;
        int evict = !to_init && cache->n_local[b] == c->L_local;
        if (evict && (cache->n_mid[b] >= c->cap_mid || (int64_t)cache->n_mid[b] >= c->T)) return -1;
    }
    for (int b = 0; b < c->B; ++b) {
        int to_init = cache->n_init[b] < c->L_init;
        int evict = !to_init && cache->n_local[b] == c->L_local;
        for (int h = 0; h < c->Hkv; ++h) {
            for (int side = 0; side < 2; ++side) {
                const double *x_new = (side == 0 ? k_new : v_new) + (((size_t)b * c->Hkv + h) * (size_t)c->d);
                int nfull = side == 0 ? c->n_full_k : c->n_full_v;
                int ncomp = c->d - nfull;
                const int32_t *idf = (side == 0 ? cache->idx_full_k : cache->idx_full_v) + (size_t)h * nfull;
                const int32_t *idc = (side == 0 ? cache->idx_comp_k : cache->idx_comp_v) + (size_t)h * ncomp;
                double *w_init = side == 0 ? cache->k_init : cache->v_init;
                double *w_local = side == 0 ? cache->k_local : cache->v_local;
                double *mid = side == 0 ? cache->k_mid : cache->v_mid;
                double *coef = (side == 0 ? cache->coef_k : cache->coef_v) + off_coef(c, b, h, ncomp);
                if (to_init) {
                    memcpy(w_init + off_win(c, b, h, c->L_init, cache->n_init[b]), x_new, sizeof(double) * c->d);
                    continue;
                }
                if (evict) {
                    int j = cache->n_mid[b];
                    if (c->L_local == 0) {
                        /* an empty local window: the new token leaves it at once */
                        fold_row(c, x_new, idf, idc, nfull, mid + off_mid(c, b, h, nfull, j), coef, j);
                        continue;
                    }
                    double *first = w_local + off_win(c, b, h, c->L_local, 0);
                    fold_row(c, first, idf, idc, nfull, mid + off_mid(c, b, h, nfull, j), coef, j);
                    memmove(first, first + c->d, sizeof(double) * (size_t)c->d * (c->L_local - 1));
                    memcpy(w_local + off_win(c, b, h, c->L_local, c->L_local - 1), x_new, sizeof(double) * c->d);
                } else {
                    memcpy(w_local + off_win(c, b, h, c->L_local, cache->n_local[b]), x_new, sizeof(double) * c->d);
                }
            }
        }
        if (to_init) cache->n_init[b] += 1;
        else if (evict) cache->n_mid[b] += 1;
        else cache->n_local[b] += 1;
    }
    return 0;
}

/* Eq.6, first and third line: the middle segment of one (b, h) side rebuilt
 * densely.  out: [n_mid][d].  Kept dims are copied from K^mu, compressed dims
 * are sum_m w_m F[m][j] C[m][e]. */
void fo_reconstruct(const fo_cfg *c, const fo_cache *cache, int b, int h, int side, double *out)
{
    int nfull = side == 0 ? c->n_full_k : c->n_full_v;
    int ncomp = c->d - nfull;
    int M = 2 * c->k;
    const int32_t *idf = (side == 0 ? cache->idx_full_k : cache->idx_full_v) + (size_t)h * nfull;
    const int32_t *idc = (side == 0 ? cache->idx_comp_k : cache->idx_comp_v) + (size_t)h * ncomp;
    const double *mid = side == 0 ? cache->k_mid : cache->v_mid;
    const double *coef = (side == 0 ? cache->coef_k : cache->coef_v) + off_coef(c, b, h, ncomp);
    int n_mid = cache->n_mid[b];
#pragma omp parallel
    {
        double *f = (double *)malloc(sizeof(double) * (size_t)M);
#pragma omp for schedule(static)
        for (int j = 0; j < n_mid; ++j) {
            double *row = out + (size_t)j * c->d;
            for (int e = 0; e < nfull; ++e) row[idf[e]] = mid[off_mid(c, b, h, nfull, j) + e];
            fo_basis_column(c->T, c->k, j, f);
            for (int e = 0; e < ncomp; ++e) {
                double acc = 0.0;
                for (int m = 0; m < M; ++m) acc += fo_weight(c, m) * f[m] * coef[(size_t)m * ncomp + e];
                row[idc[e]] = acc;
            }
        }
        free(f);
    }
}

/* Eq.6, remaining lines: K~ = cat(K^i, K~^m, K^l), V~ likewise, then softmax
 * attention of each query head over every cached token (no mask).
 * q, out: [B][Hq][d].  Heads outside [h_begin, h_end) are left untouched so a
 * caller can sample KV heads of a large problem. */
void fo_decode_heads(const fo_cfg *c, const fo_cache *cache, const double *q, double *out,
                     int h_begin, int h_end)
{
    int G = c->Hq / c->Hkv;
    for (int b = 0; b < c->B; ++b) {
        int n_init = cache->n_init[b], n_local = cache->n_local[b], n_mid = cache->n_mid[b];
        int n_tok = n_init + n_mid + n_local;
        double *Kt = (double *)malloc(sizeof(double) * (size_t)(n_tok > 0 ? n_tok : 1) * c->d);
        double *Vt = (double *)malloc(sizeof(double) * (size_t)(n_tok > 0 ? n_tok : 1) * c->d);
        double *s = (double *)malloc(sizeof(double) * (size_t)(n_tok > 0 ? n_tok : 1));
        for (int h = h_begin; h < h_end; ++h) {
            memcpy(Kt, cache->k_init + off_win(c, b, h, c->L_init, 0), sizeof(double) * (size_t)n_init * c->d);
            memcpy(Vt, cache->v_init + off_win(c, b, h, c->L_init, 0), sizeof(double) * (size_t)n_init * c->d);
            fo_reconstruct(c, cache, b, h, 0, Kt + (size_t)n_init * c->d);
            fo_reconstruct(c, cache, b, h, 1, Vt + (size_t)n_init * c->d);
            memcpy(Kt + (size_t)(n_init + n_mid) * c->d, cache->k_local + off_win(c, b, h, c->L_local, 0),
                   sizeof(double) * (size_t)n_local * c->d);
            memcpy(Vt + (size_t)(n_init + n_mid) * c->d, cache->v_local + off_win(c, b, h, c->L_local, 0),
                   sizeof(double) * (size_t)n_local * c->d);
            for (int g = h * G; g < (h + 1) * G; ++g) {
                const double *qg = q + (((size_t)b * c->Hq + g) * (size_t)c->d);
                double *og = out + (((size_t)b * c->Hq + g) * (size_t)c->d);
                double mx = -INFINITY;
                for (int i = 0; i < n_tok; ++i) {
                    double acc = 0.0;
                    for (int e = 0; e < c->d; ++e) acc += qg[e] * Kt[(size_t)i * c->d + e];
                    s[i] = c->scale * acc;
                    if (s[i] > mx) mx = s[i];
                }
                double den = 0.0;
                for (int i = 0; i < n_tok; ++i) { s[i] = exp(s[i] - mx); den += s[i]; }
                for (int e = 0; e < c->d; ++e) {
                    double acc = 0.0;
                    for (int i = 0; i < n_tok; ++i) acc += s[i] * Vt[(size_t)i * c->d + e];
                    og[e] = n_tok > 0 ? acc / den : 0.0;
                }
            }
        }
        free(Kt); free(Vt); free(s);
    }
}

void fo_decode(const fo_cfg *c, const fo_cache *cache, const double *q, double *out)
{
    fo_decode_heads(c, cache, q, out, 0, c->Hkv);
}

/* Sec. 3.4: compress and decompress EVERY dimension of one side of one
 * (b, h) over the middle segment and report the mean squared reconstruction
 * error per dimension.  X: [B][L][Hkv][d]; mse: [d].  The dimensions with the
 * smallest error are the ones to hold at fixed length. */
void fo_dim_mse(const fo_cfg *c, const double *X, int32_t L, int b, int h, double *mse)
{
    int n_init = L < c->L_init ? L : c->L_init;
    int n_local = (L - n_init) < c->L_local ? (L - n_init) : c->L_local;
    int n_mid = L - n_init - n_local;
    int M = 2 * c->k, d = c->d;
    double *coef = (double *)calloc((size_t)M * d, sizeof(double));
    double *f = (double *)malloc(sizeof(double) * (size_t)M);
#define XROW(t) (X + ((((size_t)b * L + (t)) * c->Hkv + h) * (size_t)d))
    for (int j = 0; j < n_mid; ++j) {
        fo_basis_column(c->T, c->k, j, f);
        const double *x = XROW(n_init + j);
        for (int m = 0; m < M; ++m)
            for (int e = 0; e < d; ++e) coef[(size_t)m * d + e] += f[m] * x[e];
    }
    for (int e = 0; e < d; ++e) mse[e] = 0.0;
    for (int j = 0; j < n_mid; ++j) {
        fo_basis_column(c->T, c->k, j, f);
        const double *x = XROW(n_init + j);
        for (int e = 0; e < d; ++e) {
            double acc = 0.0;
            for (int m = 0; m < M; ++m) acc += fo_weight(c, m) * f[m] * coef[(size_t)m * d + e];
            mse[e] += (acc - x[e]) * (acc - x[e]);
        }
    }
    for (int e = 0; e < d; ++e) mse[e] = n_mid > 0 ? mse[e] / n_mid : 0.0;
#undef XROW
    free(coef); free(f);
}

/* Sec. 3.4: indices of the n_full dimensions to KEEP (largest error), sorted
 * ascending; equal errors are broken towards the lower index being compressed
 * first, i.e. among equal errors the higher index is kept.  idx_full: [n_full],
 * idx_comp: [d - n_full], both ascending. */
void fo_select_dims(const double *mse, int d, int n_full, int32_t *idx_full, int32_t *idx_comp)
{
    /* rank dims by (mse ascending, index ascending); the first d - n_full are compressed */
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * (size_t)d);
    for (int i = 0; i < d; ++i) order[i] = i;
    for (int i = 1; i < d; ++i) {            /* insertion sort: stable */
        int32_t v = order[i]; int p = i - 1;
        while (p >= 0 && mse[order[p]] > mse[v]) { order[p + 1] = order[p]; --p; }
        order[p + 1] = v;
    }
    char *comp = (char *)calloc((size_t)d, 1);
    for (int i = 0; i < d - n_full; ++i) comp[order[i]] = 1;
    int a = 0, b2 = 0;
    for (int i = 0; i < d; ++i) { if (comp[i]) idx_comp[b2++] = i; else idx_full[a++] = i; }
    free(order); free(comp);
}
