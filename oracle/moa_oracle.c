/*
 * moa_oracle.c -- plain CPU oracle (test infrastructure, see moa_oracle.h).
 *
 * One (batch item, query head) at a time, exactly the three steps of Algorithm 1:
 *   Step I   (eq. (1)):  s[l] = scale * sum_j q[j] * K[l][j]
 *   Step II  (eq. (2)):  m = max_l s[l];  e[l] = exp(s[l] - m);  Z = sum_l e[l];
 *                        a[l] = e[l] / Z
 *   Step III (eq. (3)):  out[d] = sum_l a[l] * V[l][d]
 * with the O(n) scratch vectors s and a kept explicitly.  No blocking, no online
 * softmax, no splitting of the sequence, no SIMD: the shape of this code is meant to be
 * checkable against the paper by eye and to differ from the GPU kernels.
 * OpenMP parallelism is over the independent (batch, head) problems only.
 */
#include "moa_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int dims_ok(int batch, int h_q, int h_kv, int n, int d_k, int d_v)
{
    if (batch < 1 || h_q < 1 || h_kv < 1 || n < 1 || d_k < 1 || d_v < 1) return 0;
    if (h_q % h_kv != 0) return 0;
    return 1;
}

/* One head, everything in double.  q: d_k values, Kg: rows x d_k, Vg: rows x d_v.
 * The *_f32in variant below differs only in the type the inputs are read as. */
static void one_head_f64(const double *q, const double *Kg, const double *Vg, double *out,
                         int rows, int d_k, int d_v, double scale, double *s, double *a)
{
    /* Step I */
    for (int l = 0; l < rows; l++) {
        double dot = 0.0;
        for (int j = 0; j < d_k; j++) dot += q[j] * Kg[(size_t)l * d_k + j];
        s[l] = scale * dot;
    }
    /* Step II */
    double m = -INFINITY;
    for (int l = 0; l < rows; l++) if (s[l] > m) m = s[l];
    double Z = 0.0;
    for (int l = 0; l < rows; l++) { a[l] = exp(s[l] - m); Z += a[l]; }
    for (int l = 0; l < rows; l++) a[l] = a[l] / Z;
    /* Step III */
    for (int d = 0; d < d_v; d++) {
        double acc = 0.0;
        for (int l = 0; l < rows; l++) acc += a[l] * Vg[(size_t)l * d_v + d];
        out[d] = acc;
    }
}

static void one_head_f32in(const float *q, const float *Kg, const float *Vg, float *out,
                           int rows, int d_k, int d_v, double scale, double *s, double *a)
{
    for (int l = 0; l < rows; l++) {
        double dot = 0.0;
        for (int j = 0; j < d_k; j++)
            dot += (double)q[j] * (double)Kg[(size_t)l * d_k + j];
        s[l] = scale * dot;
    }
    double m = -INFINITY;
    for (int l = 0; l < rows; l++) if (s[l] > m) m = s[l];
    double Z = 0.0;
    for (int l = 0; l < rows; l++) { a[l] = exp(s[l] - m); Z += a[l]; }
    for (int l = 0; l < rows; l++) a[l] = a[l] / Z;
    for (int d = 0; d < d_v; d++) {
        double acc = 0.0;
        for (int l = 0; l < rows; l++) acc += a[l] * (double)Vg[(size_t)l * d_v + d];
        out[d] = (float)acc;              /* the single rounding to fp32 */
    }
}

int moa_oracle_decode_varlen(const float *q, const float *K, const float *V, float *out,
                             int batch, int h_q, int h_kv, const int32_t *seq_lens,
                             int n_max, int d_k, int d_v, double scale)
{
    if (!q || !K || !V || !out || !seq_lens) return -1;
    if (!dims_ok(batch, h_q, h_kv, n_max, d_k, d_v)) return -1;
    for (int b = 0; b < batch; b++)
        if (seq_lens[b] < 1 || seq_lens[b] > n_max) return -1;
    const int group = h_q / h_kv;         /* g_s: query heads per K/V head */
    int failed = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)n_max);
        double *a = (double *)malloc(sizeof(double) * (size_t)n_max);
        if (!s || !a) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (long bg = 0; bg < (long)batch * h_q; bg++) {
            if (!s || !a) continue;
            const int b = (int)(bg / h_q), g = (int)(bg % h_q);
            const int g_kv = g / group;   /* psi-selection of the K/V slab */
            const size_t slab = (size_t)b * h_kv + g_kv;
            one_head_f32in(q + (size_t)bg * d_k,
                           K + slab * (size_t)n_max * d_k,
                           V + slab * (size_t)n_max * d_v,
                           out + (size_t)bg * d_v,
                           seq_lens[b], d_k, d_v, scale, s, a);
        }
        free(s);
        free(a);
    }
    return failed ? -1 : 0;
}

int moa_oracle_decode(const float *q, const float *K, const float *V, float *out,
                      int batch, int h_q, int h_kv, int n, int d_k, int d_v, double scale)
{
    if (batch < 1 || n < 1) return -1;
    int32_t *lens = (int32_t *)malloc(sizeof(int32_t) * (size_t)batch);
    if (!lens) return -1;
    for (int b = 0; b < batch; b++) lens[b] = n;
    int rc = moa_oracle_decode_varlen(q, K, V, out, batch, h_q, h_kv, lens, n, d_k, d_v,
                                      scale);
    free(lens);
    return rc;
}

int moa_oracle_decode_f64(const double *q, const double *K, const double *V, double *out,
                          int batch, int h_q, int h_kv, int n, int d_k, int d_v,
                          double scale)
{
    if (!q || !K || !V || !out) return -1;
    if (!dims_ok(batch, h_q, h_kv, n, d_k, d_v)) return -1;
    const int group = h_q / h_kv;
    double *s = (double *)malloc(sizeof(double) * (size_t)n);
    double *a = (double *)malloc(sizeof(double) * (size_t)n);
    if (!s || !a) { free(s); free(a); return -1; }
    for (int b = 0; b < batch; b++)
        for (int g = 0; g < h_q; g++) {
            const int g_kv = g / group;
            const size_t slab = (size_t)b * h_kv + g_kv;
            const size_t bg = (size_t)b * h_q + g;
            one_head_f64(q + bg * d_k, K + slab * (size_t)n * d_k,
                         V + slab * (size_t)n * d_v, out + bg * d_v,
                         n, d_k, d_v, scale, s, a);
        }
    free(s);
    free(a);
    return 0;
}

/* One head in single precision: the same three steps as one_head_f32in, with every
 * product, sum, exponential and division rounded to fp32 (eqs. (1)-(3) as stated: the
 * weights are normalised, a[l] = e[l] / Z, before Step III uses them). */
static void one_head_f32(const float *q, const float *Kg, const float *Vg, float *out,
                         int rows, int d_k, int d_v, float scale, float *s, float *a)
{
    for (int l = 0; l < rows; l++) {                         /* Step I, eq. (1) */
        float dot = 0.0f;
        for (int j = 0; j < d_k; j++) dot += q[j] * Kg[(size_t)l * d_k + j];
        s[l] = scale * dot;
    }
    float m = -INFINITY;                                     /* Step II, eq. (2) */
    for (int l = 0; l < rows; l++) if (s[l] > m) m = s[l];
    float Z = 0.0f;
    for (int l = 0; l < rows; l++) { a[l] = expf(s[l] - m); Z += a[l]; }
    for (int l = 0; l < rows; l++) a[l] = a[l] / Z;
    for (int d = 0; d < d_v; d++) {                          /* Step III, eq. (3) */
        float acc = 0.0f;
        for (int l = 0; l < rows; l++) acc += a[l] * Vg[(size_t)l * d_v + d];
        out[d] = acc;
    }
}

int moa_oracle_decode_f32(const float *q, const float *K, const float *V, float *out,
                          int batch, int h_q, int h_kv, int n, int d_k, int d_v,
                          float scale)
{
    if (!q || !K || !V || !out) return -1;
    if (!dims_ok(batch, h_q, h_kv, n, d_k, d_v)) return -1;
    const int group = h_q / h_kv;
    int failed = 0;
#pragma omp parallel
    {
        float *s = (float *)malloc(sizeof(float) * (size_t)n);
        float *a = (float *)malloc(sizeof(float) * (size_t)n);
        if (!s || !a) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (long bg = 0; bg < (long)batch * h_q; bg++) {
            if (!s || !a) continue;
            const int b = (int)(bg / h_q), g = (int)(bg % h_q);
            const size_t slab = (size_t)b * h_kv + g / group;     /* psi-selection */
            one_head_f32(q + (size_t)bg * d_k, K + slab * (size_t)n * d_k,
                         V + slab * (size_t)n * d_v, out + (size_t)bg * d_v,
                         n, d_k, d_v, scale, s, a);
        }
        free(s);
        free(a);
    }
    return failed ? -1 : 0;
}

int moa_oracle_kv_append(float *K, float *V, const float *k_new, const float *v_new,
                         const int32_t *pos, int batch, int h_kv, int n_max,
                         int d_k, int d_v)
{
    if (!K || !V || !k_new || !v_new || !pos) return -1;
    if (batch < 1 || h_kv < 1 || n_max < 1 || d_k < 1 || d_v < 1) return -1;
    for (int b = 0; b < batch; b++)
        if (pos[b] < 0 || pos[b] >= n_max) return -1;
    for (int b = 0; b < batch; b++)
        for (int h = 0; h < h_kv; h++) {
            const size_t slab = (size_t)b * h_kv + h;
            /* the new row starts at flat offset t*d inside its slab */
            memcpy(K + (slab * (size_t)n_max + (size_t)pos[b]) * d_k,
                   k_new + slab * d_k, sizeof(float) * (size_t)d_k);
            memcpy(V + (slab * (size_t)n_max + (size_t)pos[b]) * d_v,
                   v_new + slab * d_v, sizeof(float) * (size_t)d_v);
        }
    return 0;
}

long long moa_oracle_min_bytes(int batch, int h_q, int h_kv, long long n, int d_k, int d_v)
{
    const long long per_token = (long long)d_k + d_v;   /* one K row + one V row */
    const long long kv = (long long)h_kv * n * per_token;
    const long long q_and_out = (long long)h_q * per_token;
    return (long long)batch * (kv + q_and_out) * 4;
}

int moa_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
