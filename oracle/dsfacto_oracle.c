/*
 * CPU ORACLE for the DS-FACTO epoch (doubly-separable factorization machines, arXiv 2004.13940).
 *
 * TEST INFRASTRUCTURE ONLY.  This is the slow, plain statement of what the paper's method
 * computes, used by the tests, the smoke check and the bench's CPU-baseline leg to judge the CUDA
 * library.  It shares no code, header, table or helper with the CUDA path and is never called by
 * the product.  All arithmetic is fp64; inputs arrive as fp32 (exactly representable) and the
 * initial parameters are rounded to fp32 so that both sides start from identical values.
 *
 * What each routine follows
 *   oracle_init_params   Algorithm 1, initialisation line: w = 0, V ~ N(0, 0.01) (0.01 read as
 *                        the standard deviation); draws are SplitMix64 outputs + Box-Muller
 *   oracle_bucket        Section 4.2 / figure "communication pattern": p x p partition of X into
 *                        (row-block, column-block) tiles, diagonal first, column ownership rotating
 *                        so that row block r works on column block (r+s) mod p in inner round s
 *   oracle_score         eq. (fm_model2): w0 + sum_j w_j x_ij + 1/2 sum_k[(sum_j v_jk x_ij)^2
 *                        - sum_j v_jk^2 x_ij^2]
 *   oracle_refresh       eq. (compute_a_jk) for a_ik, eq. (fm_model2) for f_i, the multiplier G_i
 *                        defined after eq. (updates_v), and the objective eq. (fm_obj)
 *   oracle_sgd_phase     eqs. (dsfacto_sgdupdatew) and (dsfacto_sgdupdatev) applied per nonzero in
 *                        the stratified order, with G and A frozen (Section 4.2, "Handling the
 *                        staleness ...": the auxiliaries are recomputed after the update step)
 *   oracle_epoch         one outer iteration t of Algorithm 1 in its synchronous (DSGD-style) form:
 *                        the update loop, then the recompute loop
 *   oracle_epoch_segmented  the same epoch with the recompute loop run after every R inner rounds
 *                        (Section 4.2: stale G, A slow convergence, hence the recompute)
 *   oracle_evaluate      the quantities the experiments plot on held-out rows (Section 5, the
 *                        convergence figures): mean loss, and RMSE (regression) or accuracy
 *                        (classification) of the scores eq. (fm_model2)
 *
 * Readings of points the paper leaves garbled or open (each also listed in the design notes):
 *   - update = gradient descent on eq. (fm_obj): theta <- theta - eta_s (G * df/dtheta + lambda theta);
 *     the printed "+ lambda w" outside eta is taken as a typesetting slip
 *   - eta_s = eta / N (the objective carries 1/N, the printed updates do not)
 *   - squared loss l = 1/2 (f-y)^2 so that its derivative is the printed G = f - y;
 *     logistic loss l = log(1 + exp(-y f)), y in {+1,-1}
 *   - w0 <- w0 - eta_s sum_i G_i once per epoch, before the strata (the printed w0 update lost
 *     its multiplier; df/dw0 = 1)
 *   - inside a tile: columns ascending, rows ascending within a column (incremental gradient
 *     descent, i.e. a fixed sweep rather than sampling)
 *
 * Parity status: every routine here is pinned by tests/test_oracle_*.py against brute force,
 * finite differences, closed forms or invariants; the numerical trajectory values themselves are
 * printed nowhere in the paper.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_SQUARED 0
#define ORACLE_LOGISTIC 1
#define ORACLE_INIT_SIGMA 0.01

/* ---- SplitMix64 (Steele, Lea, Flood 2014): the c-th output of the stream seeded with `seed` ---- */
uint64_t oracle_splitmix64_at(uint64_t seed, uint64_t c) {
    uint64_t z = seed + (c + 1) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
static double to_unit(uint64_t u) { return ((double)(u >> 11) + 0.5) / 9007199254740992.0; }

/* element e = j*K + k uses outputs 2e and 2e+1; Box-Muller, cosine branch */
double oracle_init_value(uint64_t seed, uint64_t e) {
    double u1 = to_unit(oracle_splitmix64_at(seed, 2 * e));
    double u2 = to_unit(oracle_splitmix64_at(seed, 2 * e + 1));
    double z = sqrt(-2.0 * log(u1)) * cos(2.0 * 3.14159265358979323846 * u2);
    return (double)(float)(ORACLE_INIT_SIGMA * z);
}

void oracle_init_params(int32_t d, int32_t K, uint64_t seed, double *w0, double *w, double *V) {
    *w0 = 0.0;
    for (int32_t j = 0; j < d; ++j) {
        w[j] = 0.0;
        for (int32_t k = 0; k < K; ++k)
            V[(size_t)j * K + k] = oracle_init_value(seed, (uint64_t)j * (uint64_t)K + (uint64_t)k);
    }
}

/* ---- partition ---- */
static int64_t row_block(int64_t i, int64_t n, int64_t p) { return (int64_t)(((__int128)i * p) / n); }
static int64_t col_block(int64_t j, int64_t d, int64_t p) { return (int64_t)(((__int128)j * p) / d); }

typedef struct { int32_t j, i; float x; } entry_t;
static int cmp_entry(const void *a, const void *b) {
    const entry_t *ea = (const entry_t *)a, *eb = (const entry_t *)b;
    if (ea->j != eb->j) return ea->j < eb->j ? -1 : 1;
    if (ea->i != eb->i) return ea->i < eb->i ? -1 : 1;
    return 0;
}

/* Tile (r,c) belongs to inner round s = (c - r) mod p; tiles are stored in order (s, r); inside a
 * tile entries are ordered by (column, row).  tile_ptr has p*p+1 entries. */
int oracle_bucket(int64_t n, int32_t d, int32_t p, const int64_t *indptr, const int32_t *indices,
                  const float *values, int64_t *tile_ptr, int32_t *rows, int32_t *cols, float *vals) {
    const int64_t nt = (int64_t)p * p;
    const int64_t nnz = indptr[n];
    int64_t *fill = (int64_t *)calloc((size_t)nt + 1, sizeof(int64_t));
    entry_t *ent = (entry_t *)malloc(sizeof(entry_t) * (size_t)(nnz > 0 ? nnz : 1));
    if (!fill || !ent) { free(fill); free(ent); return -1; }
    for (int64_t t = 0; t <= nt; ++t) tile_ptr[t] = 0;
    for (int64_t i = 0; i < n; ++i) {
        int64_t r = row_block(i, n, p);
        for (int64_t e = indptr[i]; e < indptr[i + 1]; ++e) {
            int64_t c = col_block(indices[e], d, p);
            int64_t s = ((c - r) % p + p) % p;
            tile_ptr[s * p + r + 1] += 1;
        }
    }
    for (int64_t t = 0; t < nt; ++t) tile_ptr[t + 1] += tile_ptr[t];
    for (int64_t t = 0; t < nt; ++t) fill[t] = tile_ptr[t];
    for (int64_t i = 0; i < n; ++i) {
        int64_t r = row_block(i, n, p);
        for (int64_t e = indptr[i]; e < indptr[i + 1]; ++e) {
            int64_t c = col_block(indices[e], d, p);
            int64_t s = ((c - r) % p + p) % p;
            int64_t at = fill[s * p + r]++;
            ent[at].j = indices[e]; ent[at].i = (int32_t)i; ent[at].x = values[e];
        }
    }
    for (int64_t t = 0; t < nt; ++t)
        qsort(ent + tile_ptr[t], (size_t)(tile_ptr[t + 1] - tile_ptr[t]), sizeof(entry_t), cmp_entry);
    for (int64_t e = 0; e < nnz; ++e) { rows[e] = ent[e].i; cols[e] = ent[e].j; vals[e] = ent[e].x; }
    free(fill); free(ent);
    return 0;
}

/* ---- model ---- */
/* eq. (fm_model2) for one sparse row; also returns a_k = sum_j v_jk x_j (k < K) through `a`,
 * lin = sum_j w_j x_j and q = sum_j sum_k v_jk^2 x_j^2 */
static double score_row(int32_t K, int64_t len, const int32_t *idx, const float *val, double w0,
                        const double *w, const double *V, double *a, double *lin_out, double *q_out) {
    double lin = 0.0, q = 0.0;
    for (int32_t k = 0; k < K; ++k) a[k] = 0.0;
    for (int64_t t = 0; t < len; ++t) {
        const double x = (double)val[t];
        const double *v = V + (size_t)idx[t] * K;
        lin += w[idx[t]] * x;
        for (int32_t k = 0; k < K; ++k) {
            a[k] += v[k] * x;
            q += v[k] * v[k] * x * x;
        }
    }
    double sq = 0.0;
    for (int32_t k = 0; k < K; ++k) sq += a[k] * a[k];
    if (lin_out) *lin_out = lin;
    if (q_out) *q_out = q;
    return w0 + lin + 0.5 * (sq - q);
}

void oracle_score(int64_t m, int32_t K, const int64_t *indptr, const int32_t *indices,
                  const float *values, double w0, const double *w, const double *V, double *out) {
#pragma omp parallel
    {
        double *a = (double *)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
#pragma omp for schedule(static)
        for (int64_t i = 0; i < m; ++i)
            out[i] = score_row(K, indptr[i + 1] - indptr[i], indices + indptr[i], values + indptr[i],
                               w0, w, V, a, NULL, NULL);
        free(a);
    }
}

static double loss_value(int32_t loss, double f, double y) {
    if (loss == ORACLE_SQUARED) return 0.5 * (f - y) * (f - y);
    double m = y * f;                          /* log(1+exp(-m)) without overflow */
    return (m > 0.0 ? 0.0 : -m) + log1p(exp(-fabs(m)));
}
static double multiplier(int32_t loss, double f, double y) {
    if (loss == ORACLE_SQUARED) return f - y;
    return -y / (1.0 + exp(y * f));
}

/* Recompute loop of Algorithm 1 for all rows: A (n x K), lin, q, f, per-row loss, G; and the
 * scalars sum_i G_i, mean loss, objective eq. (fm_obj).  out3 = {sumG, mean loss, objective}. */
void oracle_refresh(int64_t n, int32_t d, int32_t K, int32_t loss, double lambda_w, double lambda_v,
                    const int64_t *indptr, const int32_t *indices, const float *values, const float *y,
                    double w0, const double *w, const double *V, double *A, double *lin, double *q,
                    double *f, double *lossv, double *G, double *out3) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        f[i] = score_row(K, indptr[i + 1] - indptr[i], indices + indptr[i], values + indptr[i], w0, w, V,
                         A + (size_t)i * K, lin + i, q + i);
        lossv[i] = loss_value(loss, f[i], (double)y[i]);
        G[i] = multiplier(loss, f[i], (double)y[i]);
    }
    double sumG = 0.0, suml = 0.0, w2 = 0.0, v2 = 0.0;
    for (int64_t i = 0; i < n; ++i) { sumG += G[i]; suml += lossv[i]; }
    for (int32_t j = 0; j < d; ++j) w2 += w[j] * w[j];
    for (size_t e = 0; e < (size_t)d * K; ++e) v2 += V[e] * V[e];
    out3[0] = sumG;
    out3[1] = n > 0 ? suml / (double)n : 0.0;
    out3[2] = out3[1] + 0.5 * lambda_w * w2 + 0.5 * lambda_v * v2;
}

/* Update loop of Algorithm 1, synchronous form, inner rounds s0 <= s < s1: in round s the p tiles
 * (r, (r+s) mod p) touch disjoint rows and disjoint columns, so they run in parallel.  Each stored
 * entry applies eqs. (dsfacto_sgdupdatew) / (dsfacto_sgdupdatev) once with frozen G_i, a_ik. */
void oracle_sgd_rounds(int32_t K, int32_t p, int32_t s0, int32_t s1, double eta_s, double lambda_w,
                       double lambda_v, const int64_t *tile_ptr, const int32_t *rows, const int32_t *cols,
                       const float *vals, const double *A, const double *G, double *w, double *V) {
    for (int32_t s = s0; s < s1; ++s) {
#pragma omp parallel for schedule(dynamic, 1)
        for (int32_t r = 0; r < p; ++r) {
            const int64_t t = (int64_t)s * p + r;
            for (int64_t e = tile_ptr[t]; e < tile_ptr[t + 1]; ++e) {
                const int32_t i = rows[e], j = cols[e];
                const double x = (double)vals[e];
                const double g = G[i];
                const double *a = A + (size_t)i * K;
                double *v = V + (size_t)j * K;
                w[j] = w[j] - eta_s * (g * x + lambda_w * w[j]);
                for (int32_t k = 0; k < K; ++k)
                    v[k] = v[k] - eta_s * (g * (x * a[k] - v[k] * x * x) + lambda_v * v[k]);
            }
        }
    }
}

/* The whole update loop: rounds 0..p-1. */
void oracle_sgd_phase(int32_t K, int32_t p, double eta_s, double lambda_w, double lambda_v,
                      const int64_t *tile_ptr, const int32_t *rows, const int32_t *cols,
                      const float *vals, const double *A, const double *G, double *w, double *V) {
    oracle_sgd_rounds(K, p, 0, p, eta_s, lambda_w, lambda_v, tile_ptr, rows, cols, vals, A, G, w, V);
}

/* One epoch: w0 step with the frozen multipliers, the p strata, then the recompute pass. */
void oracle_epoch(int64_t n, int32_t d, int32_t K, int32_t p, int32_t loss, double eta_s,
                  double lambda_w, double lambda_v, const int64_t *indptr, const int32_t *indices,
                  const float *values, const float *y, const int64_t *tile_ptr, const int32_t *rows,
                  const int32_t *cols, const float *vals, double *w0, double *w, double *V, double *A,
                  double *lin, double *q, double *f, double *lossv, double *G, double *out3) {
    *w0 = *w0 - eta_s * out3[0];
    oracle_sgd_phase(K, p, eta_s, lambda_w, lambda_v, tile_ptr, rows, cols, vals, A, G, w, V);
    oracle_refresh(n, d, K, loss, lambda_w, lambda_v, indptr, indices, values, y, *w0, w, V, A, lin, q, f,
                   lossv, G, out3);
}

/* Second schedule: shorter staleness.  Section 4.2 ("Handling the staleness ...") recomputes G and A
 * after the update step because stale auxiliaries slow convergence; this variant applies the same
 * recompute after every `every` inner rounds instead of after all p (every <= 0 or >= p gives
 * oracle_epoch).  Reading for w0, which belongs to no column block: before a segment of m rounds it
 * takes the share m/p of its epoch step with the multipliers frozen for that segment,
 * w0 <- w0 - eta_s (m/p) sum_i G_i, so that the shares add up to the one step of oracle_epoch. */
void oracle_epoch_segmented(int64_t n, int32_t d, int32_t K, int32_t p, int32_t loss, int32_t every,
                            double eta_s, double lambda_w, double lambda_v, const int64_t *indptr,
                            const int32_t *indices, const float *values, const float *y,
                            const int64_t *tile_ptr, const int32_t *rows, const int32_t *cols,
                            const float *vals, double *w0, double *w, double *V, double *A, double *lin,
                            double *q, double *f, double *lossv, double *G, double *out3) {
    if (every <= 0 || every > p) every = p;
    for (int32_t s0 = 0; s0 < p; s0 += every) {
        const int32_t s1 = s0 + every < p ? s0 + every : p;
        *w0 = *w0 - eta_s * ((double)(s1 - s0) / (double)p) * out3[0];
        oracle_sgd_rounds(K, p, s0, s1, eta_s, lambda_w, lambda_v, tile_ptr, rows, cols, vals, A, G, w, V);
        oracle_refresh(n, d, K, loss, lambda_w, lambda_v, indptr, indices, values, y, *w0, w, V, A, lin, q,
                       f, lossv, G, out3);
    }
}

/* The same epoch restricted to ONE column j, computed straight from the CSR data and the
 * parameters at the start of the epoch, without building tiles or the full auxiliaries: the rows
 * holding column j are visited in the stratified order (round of the tile, then row), and for
 * each the frozen a_i, G_i are evaluated from the starting parameters.  Used to spot-check
 * full-size runs.  Output: wj_out (1), vj_out (K).  Returns the number of entries applied. */
int64_t oracle_column_epoch(int64_t n, int32_t d, int32_t K, int32_t p, int32_t loss, double eta_s,
                            double lambda_w, double lambda_v, const int64_t *indptr,
                            const int32_t *indices, const float *values, const float *y, double w0,
                            const double *w, const double *V, int32_t j, double *wj_out, double *vj_out) {
    const int64_t c = col_block(j, d, p);
    int64_t count = 0;
    double *a = (double *)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
    double wj = w[j];
    for (int32_t k = 0; k < K; ++k) vj_out[k] = V[(size_t)j * K + k];
    for (int64_t s = 0; s < p; ++s) {
        const int64_t r = ((c - s) % p + p) % p;
        /* rows of block r: smallest i with floor(i*p/n) = r  ..  smallest i with floor(i*p/n) = r+1 */
        int64_t lo = (int64_t)(((__int128)r * n + p - 1) / p);
        int64_t hi = (int64_t)(((__int128)(r + 1) * n + p - 1) / p);
        for (int64_t i = lo; i < hi; ++i) {
            int64_t b = indptr[i], e = indptr[i + 1], pos = -1;
            for (int64_t t = b; t < e; ++t) if (indices[t] == j) { pos = t; break; }
            if (pos < 0) continue;
            const double x = (double)values[pos];
            const double fi = score_row(K, e - b, indices + b, values + b, w0, w, V, a, NULL, NULL);
            const double g = multiplier(loss, fi, (double)y[i]);
            wj = wj - eta_s * (g * x + lambda_w * wj);
            for (int32_t k = 0; k < K; ++k)
                vj_out[k] = vj_out[k] - eta_s * (g * (x * a[k] - vj_out[k] * x * x) + lambda_v * vj_out[k]);
            ++count;
        }
    }
    *wj_out = wj;
    free(a);
    return count;
}

/* Held-out evaluation (Section 5: the convergence figures plot objective, test RMSE for the
 * regression sets and test accuracy for the classification sets).  m rows as CSR with labels y.
 * out2[0] = (1/m) sum_i l(f_i, y_i) with the loss of the model;
 * out2[1] = sqrt((1/m) sum_i (f_i - y_i)^2)          for the squared loss (RMSE),
 *         = (1/m) #{ i : y_i f_i > 0 }                for the logistic loss (accuracy; the predicted
 *           class is the sign of the score, and a score of exactly 0 predicts neither class). */
void oracle_evaluate(int64_t m, int32_t K, int32_t loss, const int64_t *indptr, const int32_t *indices,
                     const float *values, const float *y, double w0, const double *w, const double *V,
                     double *out2) {
    double suml = 0.0, sumsq = 0.0, correct = 0.0;
    double *a = (double *)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
    for (int64_t i = 0; i < m; ++i) {
        const double f = score_row(K, indptr[i + 1] - indptr[i], indices + indptr[i], values + indptr[i],
                                   w0, w, V, a, NULL, NULL);
        const double yi = (double)y[i];
        suml += loss_value(loss, f, yi);
        sumsq += (f - yi) * (f - yi);
        if (yi * f > 0.0) correct += 1.0;
    }
    free(a);
    out2[0] = m > 0 ? suml / (double)m : 0.0;
    if (loss == ORACLE_SQUARED) out2[1] = m > 0 ? sqrt(sumsq / (double)m) : 0.0;
    else out2[1] = m > 0 ? correct / (double)m : 0.0;
}
