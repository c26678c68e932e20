/*
 * CPU oracle for k-MIP self-attention  --  TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 restatement of what the method computes, used only by the
 * tests, the smoke check and the benchmark's cpu_baseline leg.  It shares no code
 * with the CUDA library and must never be called from the product path.
 *
 * What it follows:
 *   forward   Eq. 1 and Algorithm 1 lines 2-6 of the paper: for every head h and
 *             query node i, all inner products q_i . k_j over the nodes j of i's own
 *             graph (self included, Eq. 1 has no diagonal mask); keep the k largest
 *             (T_k: everything else is -inf); softmax of (kept score / sqrt(d_K));
 *             weighted sum of the kept V rows.  The 1/sqrt(d_K) factor sits outside
 *             T_k in Eq. 1 and in line 5 of Algorithm 1, so selection and the stored
 *             E_topk use the raw inner product.
 *   backward  chain rule through lines 4-6 of Algorithm 1 with the index set held
 *             constant (Sec. 3.1: the top-k indices are reused in the sparse backward;
 *             App. E: I_argtopk and E_topk need no recomputation).
 *
 * Readings where the paper is silent: ties are broken by the lower key index; the k
 * results are ordered by (score descending, index ascending); indices are global row
 * numbers of the concatenated batch; a graph with fewer than k nodes keeps all of them
 * and pads the remaining slots with index -1 / score -inf / weight 0; graphs of a
 * batch are separated by CSR offsets; NaN scores count as -inf.
 *
 * Inputs are float arrays (bf16- or fp32-valued); every product and sum is fp64.
 * Layout: Q, K, V, dOut, out, dQ, dK, dV : [N, H, d] row-major.
 *
 * Parity pins (tests/test_oracle_pins.py): k = n equals dense softmax attention
 * (library routine), k = 1 equals arg-max retrieval, exhaustive subset enumeration on
 * tiny cases, hand-derived closed-form fixtures, constant-V and identical-K cases,
 * permutation equivariance, CSR confinement, finite differences and autograd for the
 * backward.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define KMIP_ORACLE_OK 0
#define KMIP_ORACLE_BAD_ARG 1
#define KMIP_ORACLE_NOMEM 2

int kmip_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* q . k over d entries in fp64, index order (Algorithm 1 line 2, one entry of S). */
static double inner(const float *q, const float *kk, int d)
{
    double s = 0.0;
    for (int c = 0; c < d; ++c)
        s += (double)q[c] * (double)kk[c];
    return s;
}

/* Node range [lo, hi) of the graph that holds row i. */
static int graph_range(const int32_t *offs, int32_t G, int64_t N, int64_t i, int64_t *lo, int64_t *hi)
{
    if (offs == NULL) {
        *lo = 0;
        *hi = N;
        return 1;
    }
    for (int32_t g = 0; g < G; ++g)
        if ((int64_t)offs[g] <= i && i < (int64_t)offs[g + 1]) {
            *lo = offs[g];
            *hi = offs[g + 1];
            return 1;
        }
    return 0;
}

static int offsets_ok(const int32_t *offs, int32_t G, int64_t N)
{
    if (offs == NULL)
        return 1;
    if (G < 0 || offs[0] != 0 || (int64_t)offs[G] != N)
        return 0;
    for (int32_t g = 0; g < G; ++g)
        if (offs[g] > offs[g + 1])
            return 0;
    return 1;
}

/*
 * Row-wise top-k (Algorithm 1 line 3) as a partial insertion sort: walk the keys in
 * index order and keep a list of at most `keep` entries sorted by (score desc, index
 * asc).  A new score goes after every entry whose score is >= its own, so among equal
 * scores the lower index stays in front.
 */
static void topk_insert(double *ls, int64_t *li, int *len, int keep, double s, int64_t j)
{
    int p = *len;
    while (p > 0 && ls[p - 1] < s)
        --p;
    if (p >= keep)
        return;
    int last = (*len < keep) ? *len : keep - 1;
    for (int t = last; t > p; --t) {
        ls[t] = ls[t - 1];
        li[t] = li[t - 1];
    }
    ls[p] = s;
    li[p] = j;
    if (*len < keep)
        ++*len;
}

/* softmax over `n` kept scores scaled by 1/sqrt(d) (Algorithm 1 line 5). */
static void softmax_scaled(const double *s, int n, double scale, double *p)
{
    double m = -INFINITY, z = 0.0;
    for (int t = 0; t < n; ++t)
        if (s[t] > m)
            m = s[t];
    for (int t = 0; t < n; ++t) {
        p[t] = exp(scale * (s[t] - m));
        z += p[t];
    }
    for (int t = 0; t < n; ++t)
        p[t] /= z;
}

/*
 * Forward for the query rows listed in `rows` (rows == NULL: all N rows, n_rows = N).
 * Outputs are indexed by position in `rows`:
 *   out [n_rows, H, d] fp64, topk_idx [n_rows, H, k] int32, topk_score [n_rows, H, k] fp64,
 *   kth_gap [n_rows, H] fp64 (optional): score of the k-th kept key minus the best
 *   score left out (+inf when nothing is left out) -- how far the selection is from a tie.
 */
int kmip_oracle_forward_rows(const float *Q, const float *K, const float *V,
                             const int32_t *graph_offsets, int32_t G, int64_t N,
                             int32_t H, int32_t d, int32_t k,
                             const int64_t *rows, int64_t n_rows,
                             double *out, int32_t *topk_idx, double *topk_score, double *kth_gap)
{
    if (!Q || !K || !V || !out || !topk_idx || !topk_score || N < 0 || H < 1 || d < 1 || k < 1)
        return KMIP_ORACLE_BAD_ARG;
    if (!offsets_ok(graph_offsets, G, N))
        return KMIP_ORACLE_BAD_ARG;
    if (rows == NULL)
        n_rows = N;
    const double scale = 1.0 / sqrt((double)d);
    const int64_t HD = (int64_t)H * d;
    int failed = 0;

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        const int64_t i = rows ? rows[r] : r;
        int64_t lo, hi;
        double *ls = (double *)malloc(sizeof(double) * (size_t)(k + 1));
        int64_t *li = (int64_t *)malloc(sizeof(int64_t) * (size_t)(k + 1));
        double *p = (double *)malloc(sizeof(double) * (size_t)k);
        if (!ls || !li || !p || i < 0 || i >= N || !graph_range(graph_offsets, G, N, i, &lo, &hi)) {
            failed = 1;
        } else {
            for (int32_t h = 0; h < H; ++h) {
                const float *q = Q + i * HD + (int64_t)h * d;
                int len = 0;
                /* all scores of the row, reduced on the fly to the best k+1 */
                for (int64_t j = lo; j < hi; ++j) {
                    double s = inner(q, K + j * HD + (int64_t)h * d, d);
                    if (isnan(s))
                        s = -INFINITY;
                    topk_insert(ls, li, &len, k + 1, s, j);
                }
                const int keff = len < k ? len : k;
                int32_t *oi = topk_idx + (r * H + h) * (int64_t)k;
                double *os = topk_score + (r * H + h) * (int64_t)k;
                for (int t = 0; t < k; ++t) {
                    oi[t] = t < keff ? (int32_t)li[t] : -1;
                    os[t] = t < keff ? ls[t] : -INFINITY;
                }
                if (kth_gap)
                    kth_gap[r * H + h] = (len > k) ? ls[k - 1] - ls[k] : INFINITY;
                double *o = out + (r * H + h) * (int64_t)d;
                for (int c = 0; c < d; ++c)
                    o[c] = 0.0;
                if (keff > 0) {
                    softmax_scaled(ls, keff, scale, p);
                    /* gather the kept V rows and sum them with their weights (lines 4 and 6) */
                    for (int t = 0; t < keff; ++t) {
                        const float *v = V + li[t] * HD + (int64_t)h * d;
                        for (int c = 0; c < d; ++c)
                            o[c] += p[t] * (double)v[c];
                    }
                }
            }
        }
        free(ls);
        free(li);
        free(p);
    }
    return failed ? KMIP_ORACLE_BAD_ARG : KMIP_ORACLE_OK;
}

/*
 * Diagnostic of the paper's App. I ("cumulative attention weight"): how much of the FULL softmax
 * over all keys of the query's graph falls on the k keys with the largest scores,
 *   mass[i,h] = sum_{t<k} softmax_j(q_i.k_j / sqrt(d))_(t)     (1 when the graph has <= k nodes).
 * Plain definition: every score of the row, a stable log-sum-exp over all of them, and the sum of
 * the k largest probabilities.  mass [n_rows, H] fp64, indexed by position in `rows`.
 */
static int cmp_desc(const void *a, const void *b)
{
    const double x = *(const double *)a, y = *(const double *)b;
    return (x < y) - (x > y);
}

int kmip_oracle_topk_mass(const float *Q, const float *K, const int32_t *graph_offsets, int32_t G, int64_t N,
                          int32_t H, int32_t d, int32_t k, const int64_t *rows, int64_t n_rows, double *mass)
{
    if (!Q || !K || !mass || N < 0 || H < 1 || d < 1 || k < 1)
        return KMIP_ORACLE_BAD_ARG;
    if (!offsets_ok(graph_offsets, G, N))
        return KMIP_ORACLE_BAD_ARG;
    if (rows == NULL)
        n_rows = N;
    const double scale = 1.0 / sqrt((double)d);
    const int64_t HD = (int64_t)H * d;
    int failed = 0;

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        const int64_t i = rows ? rows[r] : r;
        int64_t lo, hi;
        if (i < 0 || i >= N || !graph_range(graph_offsets, G, N, i, &lo, &hi)) {
            failed = 1;
            continue;
        }
        const int64_t n = hi - lo;
        double *s = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
        if (!s) {
            failed = 1;
            continue;
        }
        for (int32_t h = 0; h < H; ++h) {
            const float *q = Q + i * HD + (int64_t)h * d;
            double m = -INFINITY, z = 0.0, top = 0.0;
            for (int64_t j = lo; j < hi; ++j) {
                s[j - lo] = scale * inner(q, K + j * HD + (int64_t)h * d, d);
                if (s[j - lo] > m)
                    m = s[j - lo];
            }
            for (int64_t j = 0; j < n; ++j)
                z += exp(s[j] - m);
            qsort(s, (size_t)n, sizeof(double), cmp_desc);
            for (int64_t t = 0; t < n && t < k; ++t)
                top += exp(s[t] - m);
            mass[r * H + h] = n > 0 ? top / z : 0.0;
        }
        free(s);
    }
    return failed ? KMIP_ORACLE_BAD_ARG : KMIP_ORACLE_OK;
}

/*
 * Attention dropout on the k softmax weights (the paper trains with it: 0.5 on the LRGB and
 * City-Networks models, 0.0 on point clouds; App. H): each weight is kept with probability
 * 1 - drop and divided by 1 - drop ("inverted" dropout), independently per (query, head, slot).
 * The draw for slot t of query i, head h is a counter-based uniform: the splitmix64 finaliser
 * of seed + (pair + 1) * 0x9E3779B97F4A7C15 with pair = (i*H + h)*k + t, top 24 bits / 2^24;
 * the weight is kept when the uniform is >= drop.  Returns the factor the weight is multiplied by.
 */
static double dropout_factor(double drop, uint64_t seed, int64_t i, int32_t H, int32_t h, int32_t k, int t)
{
    if (drop <= 0.0)
        return 1.0;
    const uint64_t pair = ((uint64_t)i * (uint64_t)H + (uint64_t)h) * (uint64_t)k + (uint64_t)t;
    uint64_t z = seed + (pair + 1u) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z = z ^ (z >> 31);
    const double u = (double)(z >> 40) / 16777216.0;
    return u >= drop ? 1.0 / (1.0 - drop) : 0.0;
}

/*
 * Lines 4-6 of Algorithm 1 for an index set supplied by the caller (any order, -1 = empty
 * slot); the scores of the listed keys are recomputed in fp64.  With drop > 0 the softmax
 * weights go through dropout_factor (slot = position in idx) before the weighted sum.
 *   idx [n_rows, H, k], out [n_rows, H, d], score_out [n_rows, H, k] (optional).
 */
int kmip_oracle_forward_given_idx_dropout(const float *Q, const float *K, const float *V,
                                          int64_t N, int32_t H, int32_t d, int32_t k,
                                          const int64_t *rows, int64_t n_rows, const int32_t *idx,
                                          double drop, uint64_t seed, double *out, double *score_out)
{
    if (!Q || !K || !V || !idx || !out || N < 0 || H < 1 || d < 1 || k < 1)
        return KMIP_ORACLE_BAD_ARG;
    if (rows == NULL)
        n_rows = N;
    const double scale = 1.0 / sqrt((double)d);
    const int64_t HD = (int64_t)H * d;
    int failed = 0;

#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_rows; ++r) {
        const int64_t i = rows ? rows[r] : r;
        double *s = (double *)malloc(sizeof(double) * (size_t)k);
        double *p = (double *)malloc(sizeof(double) * (size_t)k);
        int64_t *jj = (int64_t *)malloc(sizeof(int64_t) * (size_t)k);
        int *slot = (int *)malloc(sizeof(int) * (size_t)k);
        if (!s || !p || !jj || !slot || i < 0 || i >= N) {
            failed = 1;
        } else {
            for (int32_t h = 0; h < H; ++h) {
                const int32_t *ii = idx + (r * H + h) * (int64_t)k;
                const float *q = Q + i * HD + (int64_t)h * d;
                int n = 0;
                for (int t = 0; t < k; ++t) {
                    if (score_out)
                        score_out[(r * H + h) * (int64_t)k + t] = -INFINITY;
                    if (ii[t] < 0)
                        continue;
                    if (ii[t] >= N) {
                        failed = 1;
                        continue;
                    }
                    jj[n] = ii[t];
                    slot[n] = t;
                    s[n] = inner(q, K + jj[n] * HD + (int64_t)h * d, d);
                    if (score_out)
                        score_out[(r * H + h) * (int64_t)k + t] = s[n];
                    ++n;
                }
                double *o = out + (r * H + h) * (int64_t)d;
                for (int c = 0; c < d; ++c)
                    o[c] = 0.0;
                if (n > 0) {
                    softmax_scaled(s, n, scale, p);
                    for (int t = 0; t < n; ++t) {
                        const float *v = V + jj[t] * HD + (int64_t)h * d;
                        const double w = p[t] * dropout_factor(drop, seed, i, H, h, k, slot[t]);
                        for (int c = 0; c < d; ++c)
                            o[c] += w * (double)v[c];
                    }
                }
            }
        }
        free(s);
        free(p);
        free(jj);
        free(slot);
    }
    return failed ? KMIP_ORACLE_BAD_ARG : KMIP_ORACLE_OK;
}

int kmip_oracle_forward_given_idx(const float *Q, const float *K, const float *V,
                                  int64_t N, int32_t H, int32_t d, int32_t k,
                                  const int64_t *rows, int64_t n_rows, const int32_t *idx,
                                  double *out, double *score_out)
{
    return kmip_oracle_forward_given_idx_dropout(Q, K, V, N, H, d, k, rows, n_rows, idx, 0.0, 0, out, score_out);
}

/*
 * Backward through lines 4-6 of Algorithm 1 with the selection held constant.
 * With s_t = q_i . k_{j_t}, p = softmax(s / sqrt(d)), o_i = sum_t p_t v_{j_t} and upstream g_i:
 *   dP_t = g_i . v_{j_t}          D = sum_t p_t dP_t        dS_t = p_t (dP_t - D) / sqrt(d)
 *   dQ_i += dS_t k_{j_t}          dK_{j_t} += dS_t q_i      dV_{j_t} += p_t g_i
 * idx [N, H, k] (-1 = empty slot).  dQ, dK, dV [N, H, d] fp64, overwritten.
 * Heads touch disjoint columns, so the loop over heads is the parallel one.
 * With dropout (factor f_t of dropout_factor, a constant of the backward pass) the output is
 * o_i = sum_t f_t p_t v_{j_t}, so dP_t = f_t (g_i . v_{j_t}) and dV_{j_t} += f_t p_t g_i;
 * D, dS, dQ and dK keep their form.
 */
int kmip_oracle_backward_dropout(const float *Q, const float *K, const float *V, const float *dOut,
                                 const int32_t *idx, int64_t N, int32_t H, int32_t d, int32_t k,
                                 double drop, uint64_t seed, double *dQ, double *dK, double *dV)
{
    if (!Q || !K || !V || !dOut || !idx || !dQ || !dK || !dV || N < 0 || H < 1 || d < 1 || k < 1)
        return KMIP_ORACLE_BAD_ARG;
    const double scale = 1.0 / sqrt((double)d);
    const int64_t HD = (int64_t)H * d;
    memset(dQ, 0, sizeof(double) * (size_t)(N * HD));
    memset(dK, 0, sizeof(double) * (size_t)(N * HD));
    memset(dV, 0, sizeof(double) * (size_t)(N * HD));
    int failed = 0;

#pragma omp parallel for schedule(static, 1)
    for (int32_t h = 0; h < H; ++h) {
        double *s = (double *)malloc(sizeof(double) * (size_t)k);
        double *p = (double *)malloc(sizeof(double) * (size_t)k);
        double *dP = (double *)malloc(sizeof(double) * (size_t)k);
        int64_t *jj = (int64_t *)malloc(sizeof(int64_t) * (size_t)k);
        double *f = (double *)malloc(sizeof(double) * (size_t)k);
        if (!s || !p || !dP || !jj || !f) {
            failed = 1;
        } else {
            for (int64_t i = 0; i < N; ++i) {
                const int32_t *ii = idx + (i * H + h) * (int64_t)k;
                const float *q = Q + i * HD + (int64_t)h * d;
                const float *g = dOut + i * HD + (int64_t)h * d;
                int n = 0;
                for (int t = 0; t < k; ++t) {
                    if (ii[t] < 0)
                        continue;
                    if (ii[t] >= N) {
                        failed = 1;
                        continue;
                    }
                    jj[n] = ii[t];
                    f[n] = dropout_factor(drop, seed, i, H, h, k, t);
                    s[n] = inner(q, K + jj[n] * HD + (int64_t)h * d, d);
                    ++n;
                }
                if (n == 0)
                    continue;
                softmax_scaled(s, n, scale, p);
                double D = 0.0;
                for (int t = 0; t < n; ++t) {
                    dP[t] = f[t] * inner(g, V + jj[t] * HD + (int64_t)h * d, d);
                    D += p[t] * dP[t];
                }
                for (int t = 0; t < n; ++t) {
                    const double dS = scale * p[t] * (dP[t] - D);
                    const float *kr = K + jj[t] * HD + (int64_t)h * d;
                    double *dq = dQ + i * HD + (int64_t)h * d;
                    double *dk = dK + jj[t] * HD + (int64_t)h * d;
                    double *dv = dV + jj[t] * HD + (int64_t)h * d;
                    for (int c = 0; c < d; ++c) {
                        dq[c] += dS * (double)kr[c];
                        dk[c] += dS * (double)q[c];
                        dv[c] += f[t] * p[t] * (double)g[c];
                    }
                }
            }
        }
        free(s);
        free(p);
        free(dP);
        free(jj);
        free(f);
    }
    return failed ? KMIP_ORACLE_BAD_ARG : KMIP_ORACLE_OK;
}

int kmip_oracle_backward(const float *Q, const float *K, const float *V, const float *dOut,
                         const int32_t *idx, int64_t N, int32_t H, int32_t d, int32_t k,
                         double *dQ, double *dK, double *dV)
{
    return kmip_oracle_backward_dropout(Q, K, V, dOut, idx, N, H, d, k, 0.0, 0, dQ, dK, dV);
}
