/*
 * Seeded synthetic sparse data sets (CSR + labels) shaped like factorization-machine workloads.
 *
 * This file only synthesises INPUTS: sparsity structure, feature values and labels.  It contains
 * none of the training method (no tile schedule, no auxiliary variables, no SGD step).  Both the
 * CPU oracle and the CUDA library are fed from arrays produced here; neither links this file.
 *
 * Every random draw is a pure function of (seed, stream, row, slot), so the output does not
 * depend on the number of OpenMP threads.
 *
 * Structures
 *   0 uniform : each row holds `len` distinct columns, uniform over [0,d)
 *   1 zipf    : row length uniform in [len_min,len_max]; column = perm[rank], rank ~ Zipf(s) over d
 *               ids, distinct within the row by rejection
 *   2 fields  : n_fields nonzeros per row, field f draws rank ~ Zipf(s) over field_range ids and
 *               maps it through a per-field permutation into [f*field_range,(f+1)*field_range)
 * Values      0 N(0,1) | 1 U(-1,1) | 2 lognormal(0,1) then row L2-normalised | 3 all 1.0
 * Labels      0 planted score + N(0,noise^2) | 1 sign(planted score), flipped w.p. `flip`
 *             2 +1 w.p. sigmoid(planted score + bias) else -1 | 3 the raw planted score
 * The planted score is a second-order factorization machine with K* factors whose parameters
 * are themselves seeded draws (w* ~ N(0,w_scale^2), V* ~ N(0,v_scale^2), optionally restricted
 * to a random `support_frac` of the columns).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int64_t n;
    int32_t d;
    uint64_t seed;
    int32_t structure;
    int32_t len_min, len_max;
    int32_t n_fields, field_range;
    double zipf_s;
    int32_t value_kind;
    int32_t label_kind;
    int32_t k_star;
    double w_scale, v_scale, support_frac;
    double noise, flip, bias;
} wl_spec;

enum { ST_LEN = 1, ST_COL = 2, ST_VAL = 3, ST_LABEL = 4, ST_PLANT_W = 5, ST_PLANT_V = 6,
       ST_SUPPORT = 7, ST_PERM = 8 };

static inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
static inline uint64_t draw(uint64_t seed, uint64_t stream, uint64_t a, uint64_t b) {
    uint64_t h = mix64(seed ^ (stream * 0xD6E8FEB86659FD93ull));
    h = mix64(h ^ a);
    return mix64(h + b * 0xA0761D6478BD642Full);
}
static inline double unit(uint64_t u) { return ((double)(u >> 11) + 0.5) * (1.0 / 9007199254740992.0); }
static inline double gauss(uint64_t seed, uint64_t stream, uint64_t a, uint64_t b) {
    double u1 = unit(draw(seed, stream, a, 2 * b));
    double u2 = unit(draw(seed, stream, a, 2 * b + 1));
    return sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925 * u2);
}

/* inverse-CDF Zipf sampler with a guide table */
typedef struct { int32_t R; double *cdf; int32_t *guide; int32_t G; } zipf_t;

static int zipf_init(zipf_t *z, int32_t R, double s) {
    z->R = R;
    z->cdf = (double *)malloc(sizeof(double) * (size_t)R);
    int32_t G = 1; while (G < 2 * R) G <<= 1;
    z->G = G;
    z->guide = (int32_t *)malloc(sizeof(int32_t) * (size_t)(G + 1));
    if (!z->cdf || !z->guide) return -1;
    double tot = 0.0;
    for (int32_t r = 0; r < R; ++r) { tot += pow((double)(r + 1), -s); z->cdf[r] = tot; }
    for (int32_t r = 0; r < R; ++r) z->cdf[r] /= tot;
    z->cdf[R - 1] = 1.0;
    int32_t r = 0;
    for (int32_t g = 0; g <= G; ++g) {
        double t = (double)g / (double)G;
        while (r < R - 1 && z->cdf[r] < t) ++r;
        z->guide[g] = r;
    }
    return 0;
}
static void zipf_free(zipf_t *z) { free(z->cdf); free(z->guide); }
static inline int32_t zipf_rank(const zipf_t *z, double u) {
    int32_t g = (int32_t)(u * (double)z->G);
    if (g >= z->G) g = z->G - 1;
    int32_t r = z->guide[g];
    while (r < z->R - 1 && z->cdf[r] < u) ++r;
    return r;
}

static void make_perm(int32_t *perm, int32_t R, uint64_t seed, uint64_t which) {
    for (int32_t i = 0; i < R; ++i) perm[i] = i;
    for (int32_t i = R - 1; i > 0; --i) {
        uint64_t u = draw(seed, ST_PERM, which, (uint64_t)i);
        int32_t j = (int32_t)(u % (uint64_t)(i + 1));
        int32_t t = perm[i]; perm[i] = perm[j]; perm[j] = t;
    }
}

static inline int32_t row_len(const wl_spec *sp, int64_t i) {
    if (sp->structure == 2) return sp->n_fields;
    int32_t span = sp->len_max - sp->len_min + 1;
    if (span <= 1) return sp->len_min;
    return sp->len_min + (int32_t)(draw(sp->seed, ST_LEN, (uint64_t)i, 0) % (uint64_t)span);
}

static void sort_i32(int32_t *a, int32_t m) {
    for (int32_t i = 1; i < m; ++i) {
        int32_t v = a[i], j = i - 1;
        while (j >= 0 && a[j] > v) { a[j + 1] = a[j]; --j; }
        a[j + 1] = v;
    }
}

/* number of stored entries per row -> indptr (n+1) */
int wl_row_pointers(const wl_spec *sp, int64_t *indptr) {
    if (sp->n < 0 || sp->d <= 0) return -1;
    if (sp->structure != 2 && (sp->len_min < 0 || sp->len_max < sp->len_min || sp->len_max > sp->d)) return -1;
    if (sp->structure == 2 && (int64_t)sp->n_fields * sp->field_range > sp->d) return -1;
    indptr[0] = 0;
    for (int64_t i = 0; i < sp->n; ++i) indptr[i + 1] = indptr[i] + row_len(sp, i);
    return 0;
}

/* fills indices/values (sized by wl_row_pointers) and y (n) */
int wl_fill(const wl_spec *sp, const int64_t *indptr, int32_t *indices, float *values, float *y) {
    const int64_t n = sp->n;
    const int32_t d = sp->d;
    const int32_t ks = sp->k_star;
    zipf_t zf; memset(&zf, 0, sizeof zf);
    int32_t *perm = NULL;
    int rc = 0;
    if (sp->structure == 1) {
        if (zipf_init(&zf, d, sp->zipf_s)) return -2;
        perm = (int32_t *)malloc(sizeof(int32_t) * (size_t)d);
        if (!perm) return -2;
        make_perm(perm, d, sp->seed, 0);
    } else if (sp->structure == 2) {
        if (zipf_init(&zf, sp->field_range, sp->zipf_s)) return -2;
        perm = (int32_t *)malloc(sizeof(int32_t) * (size_t)sp->n_fields * (size_t)sp->field_range);
        if (!perm) return -2;
        for (int32_t f = 0; f < sp->n_fields; ++f)
            make_perm(perm + (size_t)f * sp->field_range, sp->field_range, sp->seed, (uint64_t)f + 1);
    }
    /* planted parameters */
    float *wst = (float *)malloc(sizeof(float) * (size_t)d);
    float *vst = (float *)malloc(sizeof(float) * (size_t)d * (size_t)(ks > 0 ? ks : 1));
    if (!wst || !vst) { rc = -2; goto done; }
#pragma omp parallel for schedule(static)
    for (int32_t j = 0; j < d; ++j) {
        int on = 1;
        if (sp->support_frac < 1.0) on = unit(draw(sp->seed, ST_SUPPORT, (uint64_t)j, 0)) < sp->support_frac;
        wst[j] = on ? (float)(sp->w_scale * gauss(sp->seed, ST_PLANT_W, (uint64_t)j, 0)) : 0.0f;
        for (int32_t k = 0; k < ks; ++k)
            vst[(size_t)j * ks + k] = on ? (float)(sp->v_scale * gauss(sp->seed, ST_PLANT_V, (uint64_t)j, (uint64_t)k)) : 0.0f;
    }

#pragma omp parallel
    {
        double *acc = (double *)malloc(sizeof(double) * (size_t)(ks > 0 ? ks : 1));
#pragma omp for schedule(dynamic, 4096)
        for (int64_t i = 0; i < n; ++i) {
            const int64_t b = indptr[i];
            const int32_t len = (int32_t)(indptr[i + 1] - b);
            int32_t *cols = indices + b;
            float *vals = values + b;
            /* ---- columns ---- */
            if (sp->structure == 2) {
                for (int32_t f = 0; f < len; ++f) {
                    int32_t r = zipf_rank(&zf, unit(draw(sp->seed, ST_COL, (uint64_t)i, (uint64_t)f)));
                    cols[f] = f * sp->field_range + perm[(size_t)f * sp->field_range + r];
                }
            } else {
                int32_t got = 0;
                uint64_t attempt = 0;
                while (got < len) {
                    double u = unit(draw(sp->seed, ST_COL, (uint64_t)i, attempt++));
                    int32_t c;
                    if (sp->structure == 1) c = perm[zipf_rank(&zf, u)];
                    else { c = (int32_t)(u * (double)d); if (c >= d) c = d - 1; }
                    int dup = 0;
                    for (int32_t t = 0; t < got; ++t) if (cols[t] == c) { dup = 1; break; }
                    if (!dup) cols[got++] = c;
                }
                sort_i32(cols, len);
            }
            /* ---- values ---- */
            double nrm = 0.0;
            for (int32_t t = 0; t < len; ++t) {
                double v;
                switch (sp->value_kind) {
                case 0: v = gauss(sp->seed, ST_VAL, (uint64_t)i, (uint64_t)t); break;
                case 1: v = 2.0 * unit(draw(sp->seed, ST_VAL, (uint64_t)i, (uint64_t)t)) - 1.0; break;
                case 2: v = exp(gauss(sp->seed, ST_VAL, (uint64_t)i, (uint64_t)t)); break;
                default: v = 1.0;
                }
                vals[t] = (float)v;
                nrm += v * v;
            }
            if (sp->value_kind == 2 && nrm > 0.0) {
                double inv = 1.0 / sqrt(nrm);
                for (int32_t t = 0; t < len; ++t) vals[t] = (float)((double)vals[t] * inv);
            }
            /* ---- label from the planted model (values as stored, i.e. fp32-rounded) ---- */
            double lin = 0.0, sq = 0.0;
            for (int32_t k = 0; k < ks; ++k) acc[k] = 0.0;
            for (int32_t t = 0; t < len; ++t) {
                const double x = (double)vals[t];
                const int32_t c = cols[t];
                lin += (double)wst[c] * x;
                for (int32_t k = 0; k < ks; ++k) {
                    double vx = (double)vst[(size_t)c * ks + k] * x;
                    acc[k] += vx; sq += vx * vx;
                }
            }
            double pair = -sq;
            for (int32_t k = 0; k < ks; ++k) pair += acc[k] * acc[k];
            const double score = lin + 0.5 * pair;
            double lab;
            switch (sp->label_kind) {
            case 0: lab = score + sp->noise * gauss(sp->seed, ST_LABEL, (uint64_t)i, 0); break;
            case 1: {
                lab = score >= 0.0 ? 1.0 : -1.0;
                if (unit(draw(sp->seed, ST_LABEL, (uint64_t)i, 7)) < sp->flip) lab = -lab;
            } break;
            case 2: {
                double pr = 1.0 / (1.0 + exp(-(score + sp->bias)));
                lab = unit(draw(sp->seed, ST_LABEL, (uint64_t)i, 7)) < pr ? 1.0 : -1.0;
            } break;
            default: lab = score;
            }
            y[i] = (float)lab;
        }
        free(acc);
    }
done:
    free(wst); free(vst); free(perm);
    if (zf.cdf) zipf_free(&zf);
    return rc;
}
