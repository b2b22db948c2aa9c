// moa_stream.cuh -- the split-sequence streaming decode kernel and its combine kernel.
//
// Steps I-III of Algorithm 1 (eqs. (1)-(3)) in online-softmax form, for the g_s query
// heads that share one K/V head (psi-selection, section 6.1), with each K/V element
// fetched from HBM once for the whole group.
//
// Decomposition.  The cached rows of every (batch, kv head) unit are cut into row blocks
// of R rows; all blocks of all units form one flat list that is dealt to the CTAs in
// equal contiguous ranges (one persistent CTA per SM), so every SM streams the same
// number of bytes whatever the batch, head count or (ragged) sequence lengths are.
// Inside a CTA the blocks go round-robin to the warps.  Each warp owns a private ring of
// S shared-memory stages filled by 1-D bulk asynchronous copies (one K block + one V
// block per stage, completion on an mbarrier) and keeps S-1 copies in flight while it
// computes; there is no producer warp and no block-wide synchronisation in the
// streaming loop.  A warp keeps its own running (max, sum, weighted-V) state; when the
// CTA's range crosses a unit boundary the warps' states are merged through shared
// memory and written either as the final output (the CTA saw the whole unit) or as a
// partial (m, l, o) triple into the CTA's slot of the workspace.  The CTA that delivers the
// last partial of a split unit (found with a completion counter) merges that unit's
// partials in CTA order, so the result does not depend on which CTA does it; with more than
// kTicketCtas CTAs a second tiny kernel does the merging instead.  The same launch can
// also perform the cache append of the step's new (k, v) row and advance the lengths.
#pragma once

#include "moa_device.cuh"

namespace moa {

template <int D_, int G_, int RV_, int S_, int W_>
struct StreamCfg {
    static constexpr int D = D_;              // d_k == d_v
    static constexpr int G = G_;              // query heads per kv head handled (power of 2)
    static constexpr int RV = RV_;            // row slots per lane per block
    static constexpr int S = S_;              // ring stages per warp
    static constexpr int W = W_;              // warps per CTA
    static constexpr int LPR = D / 4;         // lanes that share one row (float4 each)
    static constexpr int RPI = 32 / LPR;      // rows covered by one warp-wide 512-byte read
    static constexpr int R = RV * RPI;        // rows per block
    static constexpr int NV = G * RV;         // per-lane partial scores before the reduce
    static constexpr int VW = W * RPI;        // independent softmax states per CTA
    static constexpr int PS = D + 4;          // floats per partial: o[D], m, l, 2 pad
    static constexpr int STAGE_FLOATS = 2 * R * D;
    static constexpr int THREADS = W * 32;
    static_assert(D == 32 || D == 64 || D == 128, "row must be 128, 256 or 512 bytes");
    static_assert(NV >= 4 && NV <= 32 && NV <= LPR && (NV & (NV - 1)) == 0, "bad NV");
    static_assert(NV % 4 == 0, "p is fetched as float4");
    static_assert(G * LPR <= THREADS, "merge uses one thread per (head, float4)");

    // shared-memory carve-up (byte offsets)
    static constexpr size_t OFF_RING = 0;
    static constexpr size_t OFF_MERGE_O = OFF_RING + sizeof(float) * W * S * STAGE_FLOATS;
    static constexpr size_t OFF_MERGE_ML = OFF_MERGE_O + sizeof(float) * VW * G * D;
    static constexpr size_t OFF_P = OFF_MERGE_ML + sizeof(float) * VW * G * 2;
    static constexpr size_t OFF_A = OFF_P + sizeof(float) * VW * NV;
    static constexpr size_t OFF_BAR = (OFF_A + sizeof(float) * VW * G + 15) / 16 * 16;
    static constexpr size_t SMEM_BYTES = OFF_BAR + sizeof(uint64_t) * W * S;
};

// Sum NV per-lane values across the LPR lanes of a row group.  Each step halves the
// number of live values by swapping halves with the partner lane, so the whole reduce
// costs NV-1 shuffles (plus log2(LPR/NV) for the final butterfly).  On return every lane
// holds the complete sum for value index (lane % NV).
template <int NV, int LPR>
__device__ __forceinline__ float transpose_reduce(float (&v)[NV], int lane)
{
#pragma unroll
    for (int half = NV / 2; half >= 1; half >>= 1) {
        const bool upper = (lane & half) != 0;
#pragma unroll
        for (int i = 0; i < half; ++i) {
            const float send = upper ? v[i] : v[i + half];
            const float keep = upper ? v[i + half] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, half);
        }
    }
    float r = v[0];
#pragma unroll
    for (int mask = NV; mask < LPR; mask <<= 1) r += __shfl_xor_sync(0xffffffffu, r, mask);
    return r;
}

__device__ __forceinline__ float dot4(const float4 &a, const float4 &b)
{
    return fmaf(a.x, b.x, fmaf(a.y, b.y, fmaf(a.z, b.z, a.w * b.w)));
}

template <class C>
__global__ void __launch_bounds__(C::THREADS, 1) stream_decode_kernel(const DecodeArgs a)
{
    constexpr int D = C::D, G = C::G, RV = C::RV, S = C::S, W = C::W, LPR = C::LPR,
                  RPI = C::RPI, R = C::R, NV = C::NV, VW = C::VW, PS = C::PS;
    extern __shared__ __align__(128) unsigned char smem[];
    float *ring = reinterpret_cast<float *>(smem + C::OFF_RING);
    float *merge_o = reinterpret_cast<float *>(smem + C::OFF_MERGE_O);
    float *merge_ml = reinterpret_cast<float *>(smem + C::OFF_MERGE_ML);
    float *pbuf = reinterpret_cast<float *>(smem + C::OFF_P);
    float *abuf = reinterpret_cast<float *>(smem + C::OFF_A);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::OFF_BAR);
    __shared__ int s_last;                    // "this CTA completed a counter" broadcast
    __shared__ int s_pref[kPrefixBatch + 1];  // per-item block prefix for ragged batches

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane / LPR;               // which of the RPI rows of a 512-byte read
    const int vw = warp * RPI + sub;          // this lane's softmax state index
    const int vi = lane & (NV - 1);           // score value this lane owns after the reduce
    const int my_g = vi / RV, my_r = vi % RV;
    const int my_row = my_r * RPI + sub;      // its row inside the block
    const bool owner = (lane % LPR) < NV;     // first copy of the value inside the row group
    const int h_stored = a.h_kv / a.kv_share; // K/V heads as stored

    launch_dependents();
    if (tid < W * S) mbar_init(smem_u32(&bars[tid]), 1);
    mbar_fence_init();
    grid_dependency_wait();                   // lengths, cache rows, counters, partial slots of the previous step
    __syncthreads();

    const int *pref = nullptr;
    if (a.seq_lens != nullptr && a.batch <= kPrefixBatch) {
        if (warp == 0) build_block_prefix<R>(a, s_pref, lane);
        __syncthreads();
        pref = s_pref;
    }
    const long long total = pref ? (long long)pref[a.batch] * a.h_kv : total_blocks<R>(a, lane);
    const long long bpc = (total + gridDim.x - 1) / gridDim.x;
    const long long c0 = (long long)blockIdx.x * bpc;
    const long long c1 = (c0 + bpc < total) ? c0 + bpc : total;

    if (c0 < c1) {                            // uniform for the whole CTA
    float *my_ring = ring + (size_t)warp * S * C::STAGE_FLOATS;
    const uint32_t my_bar0 = smem_u32(&bars[warp * S]);

    // ---- load side: this warp's blocks are c0+warp, c0+warp+W, ... ---------------------
    long long jl = c0 + warp;
    int kl = 0;
    Cursor lc = cursor_at<R>(a, (jl < c1) ? jl : c0, pref);
    auto issue_next_load = [&]() {
        while (jl >= lc.first + lc.ub) cursor_next_unit<R>(a, lc);
        const int row0 = (int)(jl - lc.first) * R;
        const int nr = (lc.len - row0 < R) ? lc.len - row0 : R;
        // Fused append: the unit's last row is the token being appended.  It is fetched from
        // k_new / v_new (never from the cache), and this warp also stores it into the cache.
        const bool has_new = (a.k_new != nullptr) && (row0 + nr == lc.len);
        const int nr_cache = has_new ? nr - 1 : nr;
        const int hs = lc.h / a.kv_share;      // stored kv head
        const size_t slab = (size_t)lc.b * h_stored + hs;
        const float *Ksrc = a.K + (size_t)lc.b * a.k_sb + (size_t)hs * a.k_sh + (size_t)row0 * D;
        const float *Vsrc = a.V + (size_t)lc.b * a.v_sb + (size_t)hs * a.v_sh + (size_t)row0 * D;
        if (lane == 0) {
            const int stage = kl % S;
            const uint32_t bar = my_bar0 + 8u * stage;
            const uint32_t dst = smem_u32(my_ring + (size_t)stage * C::STAGE_FLOATS);
            const uint32_t bytes = (uint32_t)nr_cache * D * 4u;
            mbar_expect_tx(bar, 2u * (uint32_t)nr * D * 4u);
            const bool skip = (jl == a.skip_copy_block);     // test hook: nothing is copied, the wait expires
            if (nr_cache > 0 && !skip) {
                bulk_g2s(dst, Ksrc, bytes, bar);
                bulk_g2s(dst + R * D * 4u, Vsrc, bytes, bar);
            }
            if (has_new && !skip) {
                bulk_g2s(dst + bytes, a.k_new + slab * D, D * 4u, bar);
                bulk_g2s(dst + R * D * 4u + bytes, a.v_new + slab * D, D * 4u, bar);
            }
        }
        if (has_new && (lc.h % a.kv_share) == 0 && lane < LPR) {
            const size_t in_unit = (size_t)nr_cache * D + lane * 4;
            *reinterpret_cast<float4 *>(a.Kw + (Ksrc - a.K) + in_unit) =
                *reinterpret_cast<const float4 *>(a.k_new + slab * D + lane * 4);
            *reinterpret_cast<float4 *>(a.Vw + (Vsrc - a.V) + in_unit) =
                *reinterpret_cast<const float4 *>(a.v_new + slab * D + lane * 4);
        }
        jl += W;
        ++kl;
    };
#pragma unroll 1
    for (int i = 0; i < S && jl < c1; ++i) issue_next_load();

    // ---- compute side ------------------------------------------------------------------
    Cursor cc = cursor_at<R>(a, c0, pref);
    float4 qreg[G];
    float4 o[G];
    float m_run, l_run;
    auto begin_unit = [&]() {
        const float *qb = a.q + (size_t)cc.b * a.h_q * D;
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            const int qh = query_head(a, cc.h, g);
            if (qh >= 0) t = *reinterpret_cast<const float4 *>(qb + (size_t)qh * D + (lane % LPR) * 4);
            qreg[g] = make_float4(t.x * a.qscale, t.y * a.qscale, t.z * a.qscale, t.w * a.qscale);
            o[g] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        m_run = -INFINITY;
        l_run = 0.f;
    };

    // Merge the VW running states of this CTA for the unit under `cc` and emit either the
    // final output rows or this CTA's partial triple.  Called by every warp, in the same
    // order, once per unit the CTA touches.  When completion counters are in use, the CTA
    // that delivers the last partial of a split unit also merges that unit's partials.
    auto finish_unit = [&]() {
        float l_tot = l_run;                   // sum over the RV lanes holding one head
#pragma unroll
        for (int off = 1; off < RV; off <<= 1) l_tot += __shfl_xor_sync(0xffffffffu, l_tot, off);
        if (owner && my_r == 0) {
            merge_ml[(vw * G + my_g) * 2 + 0] = m_run;
            merge_ml[(vw * G + my_g) * 2 + 1] = l_tot;
        }
#pragma unroll
        for (int g = 0; g < G; ++g)
            *reinterpret_cast<float4 *>(merge_o + ((size_t)(vw * G + g)) * D + (lane % LPR) * 4) = o[g];
        __syncthreads();
        const long long seg_begin = (c0 > cc.first) ? c0 : cc.first;
        const long long unit_end = cc.first + cc.ub;
        const long long seg_end = (c1 < unit_end) ? c1 : unit_end;
        const bool complete = (seg_begin == cc.first) && (seg_end == unit_end);
        if (tid < G * LPR) {
            const int g = tid / LPR, d4 = tid % LPR;
            float M = -INFINITY;
#pragma unroll 4
            for (int v = 0; v < VW; ++v) M = fmaxf(M, merge_ml[(v * G + g) * 2]);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), accc = acc;
            float L = 0.f, Lc = 0.f;
#pragma unroll 4
            for (int v = 0; v < VW; ++v) {
                const float f = exp2_diff(merge_ml[(v * G + g) * 2], M);
                const float4 t = *reinterpret_cast<const float4 *>(merge_o + ((size_t)(v * G + g)) * D + d4 * 4);
                comp_fma4(acc, accc, t, f);
                comp_fma(L, Lc, merge_ml[(v * G + g) * 2 + 1], f);
            }
            if (complete) {
                const int qh = query_head(a, cc.h, g);
                if (qh >= 0) emit_columns(a, (size_t)cc.b * a.h_q + qh, D, d4, acc, M, L);
            } else {
                const int slot = (seg_begin == c0) ? 0 : 1;
                float *dst = a.ws + (((size_t)blockIdx.x * 2 + slot) * G + g) * PS;
                *reinterpret_cast<float4 *>(dst + d4 * 4) = acc;
                if (d4 == 0) { dst[D] = M; dst[D + 1] = L; }
            }
        }
        __syncthreads();
        if (!complete && a.tickets != nullptr) {
            const long long c_first = cc.first / bpc, c_last = (unit_end - 1) / bpc;
            if (tid == 0) {
                __threadfence();               // this CTA's partial is visible before it is counted
                const unsigned arrived = ticket_arrive(&a.tickets[c_first], a.ticket_tag);
                const int last = (arrived == (unsigned)(c_last - c_first));
                if (last) a.tickets[c_first] = 0ull;
                s_last = last;
            }
            __syncthreads();
            if (s_last) {                          // uniform for the CTA
                __threadfence();
                merge_unit_partials<D>(a, merge_o, VW * G * D, G, c_first, c_last, bpc, cc.first, cc.b, cc.h, tid,
                                       C::THREADS);
            }
        }
    };

    auto process_block = [&](const float *stage_base, int nr, auto full_tag) {
        constexpr bool FULL = decltype(full_tag)::value;
        const float4 *sK = reinterpret_cast<const float4 *>(stage_base);
        const float4 *sV = sK + R * D / 4;
        float v[NV];
#pragma unroll
        for (int r = 0; r < RV; ++r) {
            float4 k4 = sK[r * 32 + lane];
            if (!FULL && (r * RPI + sub >= nr)) k4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int g = 0; g < G; ++g) v[g * RV + r] = dot4(qreg[g], k4);
        }
        float s = transpose_reduce<NV, LPR>(v, lane);
        if (!FULL && my_row >= nr) s = -INFINITY;
        float bm = s;
#pragma unroll
        for (int off = 1; off < RV; off <<= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, off));
        const float m_new = fmaxf(m_run, bm);
        const float alpha = exp2_diff(m_run, m_new);
        const float p = exp2_diff(s, m_new);
        l_run = fmaf(l_run, alpha, p);
        m_run = m_new;
        float *myP = pbuf + (size_t)vw * NV;
        float *myA = abuf + (size_t)vw * G;
        if (owner) {
            myP[vi] = p;
            if (my_r == 0) myA[my_g] = alpha;
        }
        __syncwarp();
        float pr[NV];
#pragma unroll
        for (int i = 0; i < NV / 4; ++i) {
            const float4 t = reinterpret_cast<const float4 *>(myP)[i];
            pr[4 * i] = t.x; pr[4 * i + 1] = t.y; pr[4 * i + 2] = t.z; pr[4 * i + 3] = t.w;
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float al = myA[g];
            o[g].x *= al; o[g].y *= al; o[g].z *= al; o[g].w *= al;
        }
#pragma unroll
        for (int r = 0; r < RV; ++r) {
            float4 v4 = sV[r * 32 + lane];
            if (!FULL && (r * RPI + sub >= nr)) v4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float pg = pr[g * RV + r];
                o[g].x = fmaf(pg, v4.x, o[g].x); o[g].y = fmaf(pg, v4.y, o[g].y);
                o[g].z = fmaf(pg, v4.z, o[g].z); o[g].w = fmaf(pg, v4.w, o[g].w);
            }
        }
    };

    begin_unit();
    bool failed = false;
    int k = 0;
#pragma unroll 1
    for (long long j = c0 + warp; j < c1; j += W, ++k) {
        while (j >= cc.first + cc.ub) {
            finish_unit();
            cursor_next_unit<R>(a, cc);
            begin_unit();
        }
        const int stage = k % S;
        if (!failed && !mbar_wait_bounded(my_bar0 + 8u * stage, (uint32_t)(k / S) & 1u, a.wait_limit)) {
            failed = true;
            if (lane == 0) raise_status(MOA_STATUS_WAIT_TIMEOUT);
        }
        if (!failed) {
            const int row0 = (int)(j - cc.first) * R;
            const int nr = (cc.len - row0 < R) ? cc.len - row0 : R;
            const float *stage_base = my_ring + (size_t)stage * C::STAGE_FLOATS;
            if (nr == R) process_block(stage_base, nr, std::true_type{});
            else process_block(stage_base, nr, std::false_type{});
        }
        __syncwarp();                          // all lanes are done with this stage
        if (!failed && jl < c1) issue_next_load();
    }
    while (cc.first + cc.ub < c1) {            // units after this warp's last block
        finish_unit();
        cursor_next_unit<R>(a, cc);
        begin_unit();
    }
    finish_unit();
    }  // c0 < c1

    // ---- whole-grid completion: range report and length advance by the last CTA ---------
    if (a.tickets != nullptr) {
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            const unsigned done = ticket_arrive(&a.tickets[kTicketCtas], a.ticket_tag);
            const int last = (done == gridDim.x - 1);
            if (last) a.tickets[kTicketCtas] = 0ull;
            s_last = last;
        }
        __syncthreads();
        if (s_last && a.seq_lens != nullptr) {   // every CTA has finished reading the lengths
            for (int b = tid; b < a.batch; b += blockDim.x) {
                const int raw = a.seq_lens[b];
                const int len = raw + a.len_bias;
                if (len < 1 || len > a.n_max) {
                    raise_status(MOA_STATUS_SEQLEN_RANGE | (a.k_new != nullptr ? MOA_STATUS_APPEND_RANGE : 0));
                } else if (a.lens_rw != nullptr) {
                    a.lens_rw[b] = raw + 1;
                }
            }
        }
    }
}

// Merge the partial triples of every unit that was split across CTAs.  One warp per
// (batch, query head); lanes over float4 columns of the output row.  The decomposition
// (total, blocks per CTA, unit -> CTA range, slot rule) is recomputed with the same
// arithmetic as in the streaming kernel.
template <int D, int R>
__global__ void __launch_bounds__(128) stream_combine_kernel(const DecodeArgs a, int num_ctas, int G)
{
    constexpr int LPR = D / 4, PS = D + 4;
    const int lane = threadIdx.x & 31;
    const long long wid = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= (long long)a.batch * a.h_q) return;
    const int b = (int)(wid / a.h_q), gq = (int)(wid % a.h_q);
    const int in_stored = gq % a.g_total;      // head inside its stored K/V head
    const int h = (gq / a.g_total) * a.kv_share + in_stored / a.g_s, g = in_stored % a.g_s;

    const long long total = total_blocks<R>(a, lane);
    const long long bpc = (total + num_ctas - 1) / num_ctas;
    const int len = seq_len_of(a, b);
    const int ub = blocks_of<R>(len);
    if (ub == 0) {                             // out-of-range length: report, leave out untouched
        if (gq == 0 && lane == 0) raise_status(MOA_STATUS_SEQLEN_RANGE);
        return;
    }
    long long before = 0;                      // blocks of batch items < b
    if (a.seq_lens == nullptr) {
        before = (long long)b * a.h_kv * ub;
    } else {
        for (int base = 0; base < b; base += 32) {
            const int bb = base + lane;
            int nb = (bb < b) ? blocks_of<R>(seq_len_of(a, bb)) : 0;
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) nb += __shfl_xor_sync(0xffffffffu, nb, off);
            before += (long long)nb * a.h_kv;
        }
    }
    const long long first = before + (long long)h * ub;
    const long long c_first = first / bpc, c_last = (first + ub - 1) / bpc;
    if (c_first == c_last) return;             // written directly by the streaming kernel

    auto slot_ptr = [&](long long c) {
        const int slot = (first <= c * bpc) ? 0 : 1;
        return a.ws + (((size_t)c * 2 + slot) * G + g) * PS;
    };
    float M = -INFINITY;
    for (long long c = c_first; c <= c_last; ++c) M = fmaxf(M, slot_ptr(c)[D]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), accc = acc;
    float L = 0.f, Lc = 0.f;
    for (long long c = c_first; c <= c_last; ++c) {
        const float *p = slot_ptr(c);
        const float f = exp2_diff(p[D], M);
        comp_fma(L, Lc, p[D + 1], f);
        if (lane < LPR) {
            const float4 t = *reinterpret_cast<const float4 *>(p + lane * 4);
            comp_fma4(acc, accc, t, f);
        }
    }
    if (lane < LPR) emit_columns(a, (size_t)b * a.h_q + gq, D, lane, acc, M, L);
}

}  // namespace moa
