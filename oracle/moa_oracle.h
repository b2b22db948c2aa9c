/*
 * moa_oracle.h -- CPU oracle for single-query decode attention over a KV cache.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a deliberately plain, slow restatement of the
 * paper's definition (Decode DNF, eqs. (1)-(3), Algorithm 1; cache append eqs. (4),(5);
 * GQA psi-selection).  It exists so that the CUDA library can be checked against
 * something that shares no code with it.  Only tests, the smoke check and the
 * benchmark's cpu-baseline leg may call it; the product path never does.
 *
 * All arrays are host memory, row-major, owned by the caller.
 *   q   [batch, h_q,  d_k]
 *   K   [batch, h_kv, n_max, d_k]      (n_max == n for the dense entry points)
 *   V   [batch, h_kv, n_max, d_v]
 *   out [batch, h_q,  d_v]
 * Query head g uses K/V head  g_kv = g / (h_q / h_kv)   (contiguous groups).
 *
 * Every function is pinned by tests against the paper's worked examples, closed
 * forms, invariants and an independent brute force; none is "parity unpinned".
 *
 * Return value: 0 on success, -1 on an invalid argument (nothing written).
 */
#ifndef MOA_ORACLE_H
#define MOA_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Algorithm 1 with fp32 inputs/outputs and every intermediate (products, sums, exp,
 * division) in double; one rounding to fp32 at the end.  The parity reference. */
int moa_oracle_decode(const float *q, const float *K, const float *V, float *out,
                      int batch, int h_q, int h_kv, int n, int d_k, int d_v,
                      double scale);

/* Same, but sequence b attends over rows [0, seq_lens[b]) of a cache whose row
 * capacity (stride between heads) is n_max.  1 <= seq_lens[b] <= n_max. */
int moa_oracle_decode_varlen(const float *q, const float *K, const float *V, float *out,
                             int batch, int h_q, int h_kv, const int32_t *seq_lens,
                             int n_max, int d_k, int d_v, double scale);

/* All-double variant (inputs and outputs double): used to compare the oracle's
 * arithmetic with brute force at ~1e-13 before any fp32 rounding enters. */
int moa_oracle_decode_f64(const double *q, const double *K, const double *V, double *out,
                          int batch, int h_q, int h_kv, int n, int d_k, int d_v,
                          double scale);

/* Algorithm 1 (eqs. (1)-(3)) with every intermediate in single precision: what a
 * straightforward fp32 CPU implementation of the definition gives.  A timing baseline and
 * a sanity band for the fp32 error; not the parity reference. */
int moa_oracle_decode_f32(const float *q, const float *K, const float *V, float *out,
                          int batch, int h_q, int h_kv, int n, int d_k, int d_v,
                          float scale);

/* Cache append, eqs. (4),(5): row pos[b] of every (b, kv-head) slab of K (V) receives
 * k_new[b,h,:] (v_new[b,h,:]) as a raw 32-bit copy; nothing else changes.
 * Returns -1 (nothing written) if any pos[b] is outside [0, n_max). */
int moa_oracle_kv_append(float *K, float *V, const float *k_new, const float *v_new,
                         const int32_t *pos, int batch, int h_kv, int n_max,
                         int d_k, int d_v);

/* Proposition 1 lifted over batch and heads with the GQA factor:
 *   batch * (h_kv * n * (d_k + d_v) + h_q * (d_k + d_v)) * 4 bytes. */
long long moa_oracle_min_bytes(int batch, int h_q, int h_kv, long long n, int d_k, int d_v);

/* Number of OpenMP threads the decode entry points will use. */
int moa_oracle_threads(void);

#ifdef __cplusplus
}
#endif
#endif
