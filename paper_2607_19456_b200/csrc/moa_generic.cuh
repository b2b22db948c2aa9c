// moa_generic.cuh -- the catch-all decode kernel, the append kernel and the length
// counter kernels.
//
// The generic decode kernel handles any d_k <= MOA_MAX_DK, d_v <= MOA_MAX_DV, any group
// size and pointers that are only 4-byte aligned (for example the d = 2, 3 shapes of the
// paper's worked examples).  One CTA per (batch, query head); its warps take cached rows
// round-robin with lanes striding the feature axis (adjacent lanes read adjacent floats),
// each warp runs the online form of Steps I-III of Algorithm 1 and the warps' states are
// merged once at the end.  It needs no workspace and is not tuned.
#pragma once

#include "moa_device.cuh"

namespace moa {

constexpr int kGenericWarps = 8;
constexpr int kGenericDvSlots = MOA_MAX_DV / 32;

__global__ void __launch_bounds__(kGenericWarps * 32) generic_decode_kernel(const DecodeArgs a)
{
    extern __shared__ float gsm[];
    float *sq = gsm;                                    // [d_k] query, pre-scaled
    float *so = gsm + a.d_k;                            // [warps][d_v]
    float *sml = so + kGenericWarps * a.d_v;            // [warps][2]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x / a.h_q, g = blockIdx.x % a.h_q;
    const int len = seq_len_of(a, b);
    if (len == 0) return;                               // out-of-range length: untouched
    const int h = g / a.g_s;
    const float *Kg = a.K + (size_t)b * a.k_sb + (size_t)h * a.k_sh;
    const float *Vg = a.V + (size_t)b * a.v_sb + (size_t)h * a.v_sh;
    const float *qg = a.q + ((size_t)b * a.h_q + g) * a.d_k;

    for (int j = threadIdx.x; j < a.d_k; j += blockDim.x) sq[j] = qg[j] * a.qscale;
    __syncthreads();

    float o[kGenericDvSlots];
#pragma unroll
    for (int i = 0; i < kGenericDvSlots; ++i) o[i] = 0.f;
    float m = -INFINITY, l = 0.f;

    for (int row = warp; row < len; row += kGenericWarps) {
        const float *kr = Kg + (size_t)row * a.k_sr;
        float dot = 0.f;
        for (int j = lane; j < a.d_k; j += 32) dot = fmaf(sq[j], kr[j], dot);
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
        const float m_new = fmaxf(m, dot);
        const float alpha = exp2_diff(m, m_new);
        const float p = exp2_diff(dot, m_new);
        l = fmaf(l, alpha, p);
        m = m_new;
        const float *vr = Vg + (size_t)row * a.v_sr;
#pragma unroll
        for (int i = 0; i < kGenericDvSlots; ++i) {
            const int d = lane + 32 * i;
            if (d < a.d_v) o[i] = fmaf(o[i], alpha, p * vr[d]);
        }
    }
#pragma unroll
    for (int i = 0; i < kGenericDvSlots; ++i) {
        const int d = lane + 32 * i;
        if (d < a.d_v) so[warp * a.d_v + d] = o[i];
    }
    if (lane == 0) { sml[warp * 2] = m; sml[warp * 2 + 1] = l; }
    __syncthreads();
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kGenericWarps; ++w) M = fmaxf(M, sml[w * 2]);
    float L = 0.f;
#pragma unroll
    for (int w = 0; w < kGenericWarps; ++w) L = fmaf(sml[w * 2 + 1], exp2_diff(sml[w * 2], M), L);
    const bool partial = a.partial_out != nullptr;
    float *og = partial ? a.partial_out + ((size_t)b * a.h_q + g) * (size_t)(a.d_v + 4)
                        : a.out + ((size_t)b * a.h_q + g) * a.d_v;
    for (int d = threadIdx.x; d < a.d_v; d += blockDim.x) {
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < kGenericWarps; ++w)
            acc = fmaf(so[w * a.d_v + d], exp2_diff(sml[w * 2], M), acc);
        og[d] = partial ? acc : acc / L;
    }
    if (partial && threadIdx.x == 0) { og[a.d_v] = M; og[a.d_v + 1] = L; }
}

// Merge `nparts` unnormalised triples per (batch, query head) row -- the results of decode
// calls over disjoint row ranges of the same sequences -- into the normalised output.
// parts: [nparts][rows][d_v + 4] (o[d_v], m, l, 2 pad); merged in part order.  One block per row.
__global__ void __launch_bounds__(128) combine_partials_kernel(const float *parts, int nparts, float *out,
                                                               long long rows, int d_v)
{
    const long long r = blockIdx.x;
    const size_t ps = (size_t)d_v + 4, part_stride = (size_t)rows * ps;
    const float *base = parts + (size_t)r * ps;
    float M = -INFINITY;
    for (int i = 0; i < nparts; ++i) M = fmaxf(M, base[(size_t)i * part_stride + d_v]);
    float L = 0.f, Lc = 0.f;
    for (int i = 0; i < nparts; ++i)
        comp_fma(L, Lc, base[(size_t)i * part_stride + d_v + 1], exp2_diff(base[(size_t)i * part_stride + d_v], M));
    for (int d = threadIdx.x; d < d_v; d += blockDim.x) {
        float acc = 0.f, accc = 0.f;
        for (int i = 0; i < nparts; ++i)
            comp_fma(acc, accc, base[(size_t)i * part_stride + d], exp2_diff(base[(size_t)i * part_stride + d_v], M));
        out[(size_t)r * d_v + d] = acc / L;
    }
}

// Raise MOA_STATUS_SEQLEN_RANGE if any sequence length (after the bias) is outside
// [1, n_max].  One thread per batch item.
__global__ void check_lens_kernel(const int32_t *lens, int bias, int batch, int n_max)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch) {
        const int len = lens[b] + bias;
        if (len < 1 || len > n_max) raise_status(MOA_STATUS_SEQLEN_RANGE);
    }
}

// Element strides of one cache: batch item, kv head, row.
struct CacheStrides { long long sb, sh, sr; };

// Cache append, eqs. (4),(5): one thread per 32-bit word of the new K row and V row of
// one (batch, kv head); words are moved as raw bit patterns.
__global__ void __launch_bounds__(256) kv_append_kernel(uint32_t *K, uint32_t *V,
                                                        const uint32_t *k_new,
                                                        const uint32_t *v_new,
                                                        const int32_t *pos, int batch, int h_kv,
                                                        int n_max, int d_k, int d_v,
                                                        CacheStrides ks, CacheStrides vs)
{
    const int per = d_k + d_v;
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (long long)batch * h_kv * per) return;
    const int w = (int)(t % per);
    const long long slab = t / per;                     // b * h_kv + h
    const int b = (int)(slab / h_kv), h = (int)(slab % h_kv);
    const int p = pos[b];
    if (p < 0 || p >= n_max) {
        if (w == 0 && h == 0) raise_status(MOA_STATUS_APPEND_RANGE);
        return;
    }
    if (w < d_k) K[(size_t)b * ks.sb + (size_t)h * ks.sh + (size_t)p * ks.sr + w] = k_new[(size_t)slab * d_k + w];
    else V[(size_t)b * vs.sb + (size_t)h * vs.sh + (size_t)p * vs.sr + (w - d_k)] = v_new[(size_t)slab * d_v + (w - d_k)];
}

// lens[b] += delta.  With `guard_n_max` > 0 the increment is applied only to lengths in
// [0, guard_n_max - 1] (the fused step leaves the length of a skipped item unchanged).
__global__ void lens_add_kernel(int32_t *lens, int batch, int delta, int guard_n_max)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch) {
        const int v = lens[b];
        if (guard_n_max <= 0 || (v >= 0 && v < guard_n_max)) lens[b] = v + delta;
    }
}

}  // namespace moa
