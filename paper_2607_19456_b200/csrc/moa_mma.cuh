// moa_mma.cuh -- split-sequence streaming decode kernel for groups of 8 or 16 query
// heads per K/V head, with the two contractions on the warp-level tensor-core MMA.
//
// Steps I-III of Algorithm 1 (eqs. (1)-(3)) in online-softmax form with the psi-selection
// of section 6.1, as in the FMA streaming kernel, and with the same decomposition: the
// cached rows of every (batch, kv head) unit are cut into 16-row tiles, all tiles form one
// flat list dealt to persistent CTAs in equal contiguous ranges, every warp owns a private
// ring of shared-memory stages filled by bulk asynchronous copies, split units are merged
// by the CTA that delivers the last partial.  What differs is the arithmetic of a tile, and
// that (at d = 128) warps work in pairs: one warp owns the K tiles (scores, online softmax),
// its partner the V tiles (weighted sum); probabilities and rescale factors pass from one to
// the other through a double-buffered shared-memory slot guarded by two mbarriers each way.
// At d = 64 one warp does both halves of a tile, one after the other.
// With 8 query heads per fetched row the FMA kernel is bound by instruction issue, not by
// HBM; here a warp computes
//     S^T [16 rows x 8 heads]   = K_tile [16 x d]  * Q^T [d x 8]        (m16n8k8, TF32)
//     O^T [d features x 8 heads] += V_tile^T [d x 16] * P^T [16 x 8]
// Every product is formed three times (hi*hi + lo*hi + hi*lo, where hi is the value cut to
// TF32 and lo the remainder), which restores fp32-grade accuracy.  The split happens in
// registers, on the fragments a thread has just loaded, so a K/V element crosses shared
// memory once (tensor-core instructions that take their operands from shared memory
// would need the lo parts written back, several times the traffic).  Accumulator chains
// are kept short (a tile's products start from zero and are added to fp32 running
// values with ordinary FMAs), because the tensor core's accumulation is not rounded to
// nearest.
//
// Fragment bookkeeping.  The contraction index of an MMA and the order of rows and
// features may be permuted freely as long as both operands agree, which is used to load
// every fragment with 128-bit shared-memory reads: lane (g = lane/4, t = lane%4) reads,
// of a K row, the float4 chunks t, t+4, t+8, ... (each chunk feeds two k-steps) and, of V
// rows 2t, 2t+1, 2t+8, 2t+9, the chunks g, g+8, g+16, g+24 (each chunk feeds two 16-feature
// output tiles).  A tile is fetched by one tiled bulk-tensor copy per operand (an SM retires
// only about one bulk copy per 70 cycles whatever its size, so copies are kept large): the
// cache is described as [d/32 column groups][rows][32 floats] with the 128-byte swizzle,
// so a tile lands as d/32 sub-tiles of [16 rows][128 bytes] whose 16-byte chunks are
// XOR-ed with the row number, and with the row <-> fragment-slot assignment used below
// both read patterns are free of bank conflicts.
#pragma once

#include <cuda.h>

#include "moa_device.cuh"
#include "moa_tc.cuh"

namespace moa {

template <int DK_, int DV_, int S_, int P_, bool PAIRED_, int NT_>
struct MmaCfg {
    static constexpr int DK = DK_, DV = DV_;  // they may differ in paired mode (each warp owns one operand)
    static constexpr int D = DV;              // output row length (partials, merge buffers)
    static constexpr int NT = NT_;            // 8-head column tiles of the score matrix
    static constexpr int G = 8 * NT;          // query heads per (virtual) kv head
    static constexpr int S = S_;              // ring stages per warp
    static constexpr bool PAIRED = PAIRED_;   // a tile is worked on by a warp pair / by one warp
    static constexpr int P = P_;              // independent tile streams (pairs or single warps) per CTA
    static constexpr int W = PAIRED ? 2 * P : P;   // warps per CTA
    static constexpr int R = 16;              // rows per tile
    static constexpr int LPR = DV / 4;        // float4 per output row
    static constexpr int NJ = DK / 16;        // K chunks a lane reads per row (2 k-steps each)
    static constexpr int NU = DV / 32;        // V chunks a lane reads per row (2 feature tiles each)
    static constexpr int MT = DV / 16;        // 16-feature output tiles
    static constexpr int DMAX = DK > DV ? DK : DV;
    static constexpr int SUBT = R * 32;       // floats of one [16 rows][32 floats] sub-tile
    static constexpr int STAGE_FLOATS = PAIRED ? R * DMAX : 2 * R * D;   // one operand's tile / K tile + V tile
    static constexpr int PT_STRIDE = 20;      // floats between heads in a P^T hand-over buffer
    static constexpr int PBUF_FLOATS = G * PT_STRIDE + G;   // P^T [8 heads][16 rows] + alpha [8 heads]
    static constexpr int PS = D + 4;          // floats per partial: o[D], m, l, 2 pad
    static constexpr int THREADS = W * 32;
    static_assert((DK == 64 || DK == 128) && (DV == 64 || DV == 128), "rows must be 256 or 512 bytes");
    static_assert(PAIRED || DK == DV, "one warp per tile handles equal row lengths only");
    static_assert(NT == 1 || NT == 2, "8 or 16 heads");
    static_assert(G * LPR <= 4 * THREADS, "merge_unit_partials handles four items per thread");
    static_assert((STAGE_FLOATS * 4) % 1024 == 0, "swizzled sub-tiles need 1024-byte alignment");

    static constexpr size_t OFF_RING = 0;             // from the 1024-byte aligned base
    static constexpr size_t OFF_MERGE_O = OFF_RING + sizeof(float) * W * S * STAGE_FLOATS;
    static constexpr size_t OFF_MERGE_ML = OFF_MERGE_O + sizeof(float) * P * 8 * D;   // 8 heads at a time
    static constexpr size_t OFF_PBUF = OFF_MERGE_ML + sizeof(float) * P * 8 * 2;
    static constexpr size_t OFF_BAR = (OFF_PBUF + sizeof(float) * P * 2 * PBUF_FLOATS + 15) / 16 * 16;
    static constexpr int NBAR = W * S + 4 * P;        // tile landed; per pair: P^T ready x2, P^T consumed x2 (paired mode)
    static constexpr size_t SMEM_BYTES = OFF_BAR + sizeof(uint64_t) * NBAR + 1024;   // + alignment slack
};

__device__ __forceinline__ void mma_tf32_16x8x8(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// x = hi + lo (+ at most 2^-23 of x): hi the nearest TF32 value (10 mantissa bits kept), lo the
// remainder rounded to TF32 as well, so that the tensor core, which ignores the low 13 bits of
// an operand, has nothing left to cut off and the rounding errors have no preferred sign.
struct Split4 {
    uint32_t h[4], l[4];
};
__device__ __forceinline__ Split4 split4(const float4 &v)
{
    Split4 s;
    const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t hb = (__float_as_uint(x[i]) + 0x1000u) & 0xFFFFE000u;
        s.h[i] = hb;
        s.l[i] = (__float_as_uint(x[i] - __uint_as_float(hb)) + 0x1000u) & 0xFFFFE000u;
    }
    return s;
}

// D += A * B with both operands split; the two small terms go to accumulators of their own
// (three independent chains, so that consecutive MMAs never wait for one another).
__device__ __forceinline__ void mma3(float (&acc_hh)[4], float (&acc_lh)[4], float (&acc_hl)[4],
                                     const uint32_t (&ah)[4], const uint32_t (&al)[4], uint32_t bh0, uint32_t bh1,
                                     uint32_t bl0, uint32_t bl1)
{
    mma_tf32_16x8x8(acc_hh, ah[0], ah[1], ah[2], ah[3], bh0, bh1);
    mma_tf32_16x8x8(acc_lh, al[0], al[1], al[2], al[3], bh0, bh1);
    mma_tf32_16x8x8(acc_hl, ah[0], ah[1], ah[2], ah[3], bl0, bl1);
}

// Per-thread running state of the two halves of a tile's work.
template <int NJ, int NT>
struct ScoreState {
    uint32_t qh[NT][NJ][4], ql[NT][NJ][4];   // Q^T fragments of head 8nt+g (chunk t+4j of the scaled query row), split
    float m_run[2 * NT], l_run[2 * NT];      // heads 8nt+2t, 8nt+2t+1: running maximum, this thread's share of the sum
};
template <int MT, int NT>
struct PvState {
    float om[MT][NT][4];                     // O^T fragments: features (by 16-feature tile) x heads 8nt+2t, 8nt+2t+1
};

template <class C>
__global__ void __launch_bounds__(C::THREADS, 1)
mma_decode_kernel(const __grid_constant__ CUtensorMap tmapK, const __grid_constant__ CUtensorMap tmapV, const DecodeArgs a)
{
    constexpr int D = C::D, DK = C::DK, G = C::G, NT = C::NT, S = C::S, P = C::P, R = C::R, LPR = C::LPR, NJ = C::NJ, NU = C::NU,
                  MT = C::MT, SUBT = C::SUBT, PS = C::PS, PTS = C::PT_STRIDE;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char *const smem_m = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    float *ring = reinterpret_cast<float *>(smem_m + C::OFF_RING);
    float *merge_o = reinterpret_cast<float *>(smem_m + C::OFF_MERGE_O);
    float *merge_ml = reinterpret_cast<float *>(smem_m + C::OFF_MERGE_ML);
    float *pbuf_all = reinterpret_cast<float *>(smem_m + C::OFF_PBUF);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_m + C::OFF_BAR);
    __shared__ int s_last;
    __shared__ int s_pref[kPrefixBatch + 1];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    // Paired mode: the two warps of a pair work on the same tiles, the score warp (even) turns a
    // K tile into probabilities, the weighted-sum warp (odd) multiplies them into the V tile one
    // or two tiles later; each fetches its own operand into its own ring.  It halves the
    // registers a warp needs (d = 128).  Single mode: one warp does both, one after the other,
    // on a stage that holds the K and the V tile; fewer fixed costs per tile (d = 64).
    constexpr bool PAIRED = C::PAIRED;
    const int pair = PAIRED ? (warp >> 1) : warp;
    const bool is_pv = PAIRED && (warp & 1) != 0;
    // MMA row index m (0..7) <-> tile row: the two rows read in one shared-memory phase (g even
    // and odd) lie four rows apart, which the swizzle turns into disjoint halves of the banks.
    const int rowA = (g >> 1) + 4 * (g & 1), rowB = rowA + 8;
    const int h_stored = a.h_kv / a.kv_share;

    launch_dependents();
    if (tid < C::NBAR) mbar_init(smem_u32(&bars[tid]), 1);
    if (tid == 0) { tc::prefetch_tmap(&tmapK); tc::prefetch_tmap(&tmapV); }
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
    float *my_pbuf = pbuf_all + (size_t)pair * 2 * C::PBUF_FLOATS;
    const uint32_t bar_pfull0 = smem_u32(&bars[C::W * S + 4 * pair]), bar_pfree0 = bar_pfull0 + 16u;
    const CUtensorMap *my_map = is_pv ? &tmapV : &tmapK;
    const int my_d = is_pv ? D : DK;            // row length of this warp's operand
    const float *my_new = is_pv ? a.v_new : a.k_new;
    float *my_cache = is_pv ? a.Vw : a.Kw;

    // ---- load side: this pair's tiles are c0+pair, c0+pair+P, ... ------------------------
    long long jl = c0 + pair;
    int kl = 0;
    Cursor lc = cursor_at<R>(a, (jl < c1) ? jl : c0, pref);
    // The 16-head configuration is at the register limit: what only the fused append needs is
    // recomputed there instead of being carried through the loop (the other configurations are
    // 5 % faster with the values carried).
    constexpr bool LEAN = (C::NT == 2);
    const long long sb_keep = is_pv ? a.v_sb : a.k_sb, sh_keep = is_pv ? a.v_sh : a.k_sh, sr_keep = is_pv ? a.v_sr : a.k_sr;
    size_t slab_keep = 0;                      // stored (batch, kv head) of the unit under lc
    int hs = 0;                                // its stored kv head
    bool writes_new = false;                   // this virtual head stores the appended row
    auto load_unit_changed = [&]() {
        hs = lc.h / a.kv_share;
        if (!LEAN) slab_keep = (size_t)lc.b * h_stored + hs;
        writes_new = (a.k_new != nullptr) && (lc.h == hs * a.kv_share);
    };
    load_unit_changed();
    auto issue_next_load = [&]() {
        if (jl >= lc.first + lc.ub) {
            do cursor_next_unit<R>(a, lc); while (jl >= lc.first + lc.ub);
            load_unit_changed();
        }
        const int row0 = (int)(jl - lc.first) * R;
        if (lane == 0) {
            const int stage = kl % S;
            const uint32_t bar = my_bar0 + 8u * stage;
            // A box is always transferred whole: rows past the slab's capacity read as zero, rows
            // past the live length are masked later.
            const uint32_t dst = smem_u32(my_ring + (size_t)stage * C::STAGE_FLOATS);
            mbar_expect_tx(bar, PAIRED ? (uint32_t)R * my_d * 4u : (uint32_t)C::STAGE_FLOATS * 4u);
            tc::tma_load_5d(dst, my_map, 0, row0, 0, hs, lc.b, bar);
            if (!PAIRED) tc::tma_load_5d(dst + R * D * 4u, &tmapV, 0, row0, 0, hs, lc.b, bar);
        }
        // Fused append: the unit's last row is the token being appended.  The warp that fetches
        // the tile holding it also stores it into the cache (K by the score warp, V by the other);
        // the tile's copy of that row is replaced from k_new / v_new before use.
        if (writes_new && row0 + R >= lc.len && lane * 4 < my_d) {
            const size_t slab = LEAN ? (size_t)lc.b * h_stored + hs : slab_keep;   // (b, stored kv head) of the dense new rows
            const long long my_sb = LEAN ? (is_pv ? a.v_sb : a.k_sb) : sb_keep, my_sh = LEAN ? (is_pv ? a.v_sh : a.k_sh) : sh_keep,
                            my_sr = LEAN ? (is_pv ? a.v_sr : a.k_sr) : sr_keep;
            const size_t dst = (size_t)lc.b * my_sb + (size_t)hs * my_sh + (size_t)(lc.len - 1) * my_sr + lane * 4;
            *reinterpret_cast<float4 *>(my_cache + dst) = *reinterpret_cast<const float4 *>(my_new + slab * my_d + lane * 4);
            if (!PAIRED) {
                const size_t dstv = (size_t)lc.b * a.v_sb + (size_t)hs * a.v_sh + (size_t)(lc.len - 1) * a.v_sr + lane * 4;
                *reinterpret_cast<float4 *>(a.Vw + dstv) = *reinterpret_cast<const float4 *>(a.v_new + slab * D + lane * 4);
            }
        }
        jl += P;
        ++kl;
    };
#pragma unroll 1
    for (int i = 0; i < S && jl < c1; ++i) issue_next_load();

    // ---- compute side ------------------------------------------------------------------
    Cursor cc = cursor_at<R>(a, c0, pref);
    // float offset, inside a tile, of 16-byte chunk `ch` of row r
    auto chunk_at = [](int r, int ch) { return (ch >> 3) * SUBT + r * 32 + (((ch & 7) ^ (r & 7)) << 2); };

    // Merge the P running states of this CTA for the unit under `cc` (each pair has published
    // (m, l) and O through `publish`) and emit either the final output rows or this CTA's
    // partial triple; with completion counters in use, the CTA that delivers the last partial
    // of a split unit also merges that unit's partials.
    auto finish_unit = [&](auto publish) {
        const long long seg_begin = (c0 > cc.first) ? c0 : cc.first;
        const long long unit_end = cc.first + cc.ub;
        const long long seg_end = (c1 < unit_end) ? c1 : unit_end;
        const bool complete = (seg_begin == cc.first) && (seg_end == unit_end);
#pragma unroll 1
        for (int hb = 0; hb < NT; ++hb) {          // eight heads at a time through the merge buffers
            publish(hb);
            __syncthreads();
            for (int idx = tid; idx < 8 * LPR; idx += C::THREADS) {
                const int h8 = idx / LPR, d4 = idx % LPR, hg = 8 * hb + h8;
                float M = -INFINITY;
#pragma unroll
                for (int v = 0; v < P; ++v) M = fmaxf(M, merge_ml[(v * 8 + h8) * 2]);
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), accc = acc;
                float L = 0.f, Lc = 0.f;
#pragma unroll
                for (int v = 0; v < P; ++v) {
                    const float f = exp2_diff(merge_ml[(v * 8 + h8) * 2], M);
                    const float4 x = *reinterpret_cast<const float4 *>(merge_o + ((size_t)(v * 8 + h8)) * D + d4 * 4);
                    comp_fma4(acc, accc, x, f);
                    comp_fma(L, Lc, merge_ml[(v * 8 + h8) * 2 + 1], f);
                }
                if (complete) {
                    const int qh = query_head<NT == 1>(a, cc.h, hg);
                    if (qh >= 0) emit_columns(a, (size_t)cc.b * a.h_q + qh, D, d4, acc, M, L);
                } else {
                    const int slot = (seg_begin == c0) ? 0 : 1;
                    float *dst = a.ws + (((size_t)blockIdx.x * 2 + slot) * G + hg) * PS;
                    *reinterpret_cast<float4 *>(dst + d4 * 4) = acc;
                    if (d4 == 0) { dst[D] = M; dst[D + 1] = L; }
                }
            }
            __syncthreads();
        }
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
                merge_unit_partials<D, NT == 1>(a, merge_o, P * 8 * D, G, c_first, c_last, bpc, cc.first, cc.b, cc.h, tid,
                                       C::THREADS);
            }
        }
    };

    // One loop for both roles: walk this pair's tiles, closing units on the way.  `begin`,
    // `publish` and `tile` are the role's parts.
    auto run = [&](auto begin, auto publish, auto tile) {
        begin();
        bool failed = false;
        int k = 0;
#pragma unroll 1
        for (long long j = c0 + pair; j < c1; j += P, ++k) {
            while (j >= cc.first + cc.ub) {
                finish_unit(publish);
                cursor_next_unit<R>(a, cc);
                begin();
            }
            const int stage = k % S;
            if (!failed && !mbar_test_wait(my_bar0 + 8u * stage, (uint32_t)(k / S) & 1u) &&
                !mbar_wait_bounded(my_bar0 + 8u * stage, (uint32_t)(k / S) & 1u)) {
                failed = true;
                if (lane == 0) raise_status(MOA_STATUS_WAIT_TIMEOUT);
            }
            if (!failed) {
                const int row0 = (int)(j - cc.first) * R;
                const int nr = (cc.len - row0 < R) ? cc.len - row0 : R;
                float *tile_base = my_ring + (size_t)stage * C::STAGE_FLOATS;
                if ((a.k_new != nullptr) && (row0 + nr == cc.len)) {
                    // the appended token is this tile's last row: take it from k_new / v_new
                    if (lane * 4 < my_d) {
                        const size_t cslab = (size_t)cc.b * h_stored + cc.h / a.kv_share;
                        *reinterpret_cast<float4 *>(tile_base + chunk_at(nr - 1, lane)) =
                            *reinterpret_cast<const float4 *>(my_new + cslab * my_d + lane * 4);
                        if (!PAIRED)
                            *reinterpret_cast<float4 *>(tile_base + R * D + chunk_at(nr - 1, lane)) =
                                *reinterpret_cast<const float4 *>(a.v_new + cslab * D + lane * 4);
                    }
                    tc::fence_async_smem();        // plain stores to the stage precede its next bulk copy
                    __syncwarp();
                }
                if (nr == R) failed = !tile(tile_base, nr, k, std::true_type{});
                else failed = !tile(tile_base, nr, k, std::false_type{});
                if (failed && lane == 0) raise_status(MOA_STATUS_WAIT_TIMEOUT);
            }
            __syncwarp();                          // all lanes are done with this stage
            if (!failed && jl < c1) issue_next_load();
        }
        while (cc.first + cc.ub < c1) {            // units after this pair's last tile
            finish_unit(publish);
            cursor_next_unit<R>(a, cc);
            begin();
        }
        finish_unit(publish);
    };

    // ================= score part: S^T = K_tile * Q^T, online softmax, P^T hand-over ==========
    // State: Q^T fragments of head g (chunk t+4j of the scaled query row, split), running
    // maximum and this thread's share of the sum for heads 2t and 2t+1.
    auto score_begin = [&](ScoreState<NJ, NT> &st) {
        const float *qb = a.q + (size_t)cc.b * a.h_q * DK;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int qh = query_head<NT == 1>(a, cc.h, 8 * nt + g);
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (qh >= 0) v = *reinterpret_cast<const float4 *>(qb + (size_t)qh * DK + (t + 4 * j) * 4);
                const Split4 s = split4(make_float4(v.x * a.qscale, v.y * a.qscale, v.z * a.qscale, v.w * a.qscale));
#pragma unroll
                for (int i = 0; i < 4; ++i) { st.qh[nt][j][i] = s.h[i]; st.ql[nt][j][i] = s.l[i]; }
            }
        }
#pragma unroll
        for (int i = 0; i < 2 * NT; ++i) { st.m_run[i] = -INFINITY; st.l_run[i] = 0.f; }
    };
    auto score_publish = [&](const ScoreState<NJ, NT> &st, int hb) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            float l = (NT == 2 && hb == 1) ? st.l_run[2 + i] : st.l_run[i];
            const float m = (NT == 2 && hb == 1) ? st.m_run[2 + i] : st.m_run[i];
            l += __shfl_xor_sync(0xffffffffu, l, 4);
            l += __shfl_xor_sync(0xffffffffu, l, 8);
            l += __shfl_xor_sync(0xffffffffu, l, 16);
            if (g == 0) {
                merge_ml[(pair * 8 + 2 * t + i) * 2 + 0] = m;
                merge_ml[(pair * 8 + 2 * t + i) * 2 + 1] = l;
            }
        }
    };
    auto score_tile = [&](ScoreState<NJ, NT> &st, const float *sK, int nr, int k, auto full_tag) -> bool {
        constexpr bool FULL = decltype(full_tag)::value;
        // 2*NJ k-steps.  The warp-level MMA accumulates with truncation, and what a truncation
        // costs is set by the size of the accumulator, so the large hi*hi products of a score are
        // spread over NCH short chains (four k-steps each at d = 128 with one head tile) that are
        // added in fp32 afterwards; the two small cross terms share one chain each.  A K fragment
        // is loaded and split once and used for all head tiles.
        constexpr int NCH = (NT == 1) ? 4 : 2;
        float sh[NT][NCH][4], sl[NT][4], sm[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                sl[nt][i] = 0.f; sm[nt][i] = 0.f;
#pragma unroll
                for (int c = 0; c < NCH; ++c) sh[nt][c][i] = 0.f;
            }
#pragma unroll
        for (int j = 0; j < NJ; ++j) {
            const Split4 ka = split4(*reinterpret_cast<const float4 *>(sK + chunk_at(rowA, t + 4 * j)));
            const Split4 kb = split4(*reinterpret_cast<const float4 *>(sK + chunk_at(rowB, t + 4 * j)));
#pragma unroll
            for (int e = 0; e < 2; ++e) {          // elements (2e, 2e+1) of the chunk are k-slots (t, t+4)
                const uint32_t ah[4] = {ka.h[2 * e], kb.h[2 * e], ka.h[2 * e + 1], kb.h[2 * e + 1]};
                const uint32_t al[4] = {ka.l[2 * e], kb.l[2 * e], ka.l[2 * e + 1], kb.l[2 * e + 1]};
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
                    mma3(sh[nt][(2 * j + e) % NCH], sl[nt], sm[nt], ah, al, st.qh[nt][j][2 * e],
                         st.qh[nt][j][2 * e + 1], st.ql[nt][j][2 * e], st.ql[nt][j][2 * e + 1]);
            }
        }
        float alpha[NT][2], p[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            // this thread's scores: rows rowA (0,1) and rowB (2,3) of heads 8nt+2t (0,2) and 8nt+2t+1 (1,3)
            float s[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if constexpr (NCH == 4)
                    s[i] = ((sh[nt][0][i] + sh[nt][1][i]) + (sh[nt][2][i] + sh[nt][3][i])) + (sl[nt][i] + sm[nt][i]);
                else
                    s[i] = (sh[nt][0][i] + sh[nt][1][i]) + (sl[nt][i] + sm[nt][i]);
            }
            if (!FULL) {
                if (rowA >= nr) { s[0] = -INFINITY; s[1] = -INFINITY; }
                if (rowB >= nr) { s[2] = -INFINITY; s[3] = -INFINITY; }
            }
            // online softmax per head (row maximum across the 8 lanes with the same t)
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                float bm = fmaxf(s[i], s[i + 2]);
                bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 4));
                bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 8));
                bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 16));
                const float m_new = fmaxf(st.m_run[2 * nt + i], bm);
                alpha[nt][i] = exp2_diff(st.m_run[2 * nt + i], m_new);
                p[nt][i] = exp2_diff(s[i], m_new);
                p[nt][i + 2] = exp2_diff(s[i + 2], m_new);
                st.l_run[2 * nt + i] = fmaf(st.l_run[2 * nt + i], alpha[nt][i], p[nt][i] + p[nt][i + 2]);
                st.m_run[2 * nt + i] = m_new;
            }
        }
        // P^T and the rescale factors go to the weighted-sum part through one of two buffers:
        // lane (g, t) there fetches rows 2t, 2t+1, 2t+8, 2t+9 of a head (the rows whose V it
        // loads) with one 128-bit read
        const int b = k & 1, use = k >> 1;
        if (PAIRED && use >= 1 && !mbar_wait_bounded(bar_pfree0 + 8u * b, (uint32_t)(use - 1) & 1u)) return false;
        float *pt = my_pbuf + b * C::PBUF_FLOATS;
        const int pa = 4 * ((rowA >> 1) & 3) + (rowA & 1), pb = pa + 2;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            float *ph = pt + (8 * nt + 2 * t) * PTS;
            ph[pa] = p[nt][0];
            ph[PTS + pa] = p[nt][1];
            ph[pb] = p[nt][2];
            ph[PTS + pb] = p[nt][3];
            if (g == 0) { pt[G * PTS + 8 * nt + 2 * t] = alpha[nt][0]; pt[G * PTS + 8 * nt + 2 * t + 1] = alpha[nt][1]; }
        }
        __syncwarp();
        if (PAIRED && lane == 0) tc::mbar_arrive(bar_pfull0 + 8u * b);
        return true;
    };

    // ================= weighted-sum part: O^T += V_tile^T * P^T ================================
    // State: O^T fragments, features (by 16-feature tile) x heads 2t, 2t+1.
    auto pv_begin = [&](PvState<MT, NT> &st) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) st.om[mt][nt][i] = 0.f;
    };
    auto pv_publish = [&](const PvState<MT, NT> &st, int hb) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            // output tile mt = 2u+e holds features 32u + 4g + 2e (+1) of heads 2t (+1)
            const int f = 32 * (mt >> 1) + 4 * g + 2 * (mt & 1);
            float *o0 = merge_o + ((size_t)(pair * 8 + 2 * t)) * D + f;
            const float (&o)[4] = (NT == 2 && hb == 1) ? st.om[mt][NT - 1] : st.om[mt][0];
            o0[0] = o[0]; o0[D] = o[1]; o0[1] = o[2]; o0[D + 1] = o[3];
        }
    };
    auto pv_tile = [&](PvState<MT, NT> &st, const float *sV, int nr, int k, auto full_tag) -> bool {
        constexpr bool FULL = decltype(full_tag)::value;
        const int b = k & 1, use = k >> 1;
        if (PAIRED && !mbar_test_wait(bar_pfull0 + 8u * b, (uint32_t)use & 1u) &&
            !mbar_wait_bounded(bar_pfull0 + 8u * b, (uint32_t)use & 1u)) return false;
        const float *pt = my_pbuf + b * C::PBUF_FLOATS;
        Split4 pp[NT];
        float alpha[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            pp[nt] = split4(*reinterpret_cast<const float4 *>(pt + (8 * nt + g) * PTS + 4 * t));
            alpha[nt][0] = pt[G * PTS + 8 * nt + 2 * t];
            alpha[nt][1] = pt[G * PTS + 8 * nt + 2 * t + 1];
        }
        __syncwarp();
        if (PAIRED && lane == 0) tc::mbar_arrive(bar_pfree0 + 8u * b);
        // 16 features at a time; a tile's products start from zero and are then added to the
        // running values, rescaled by alpha; a V fragment is loaded and split once for all head tiles
#pragma unroll
        for (int u = 0; u < NU; ++u) {
            Split4 v[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = 2 * t + (i & 1) + 8 * (i >> 1);
                float4 x = *reinterpret_cast<const float4 *>(sV + chunk_at(r, g + 8 * u));
                if (!FULL && r >= nr) x = make_float4(0.f, 0.f, 0.f, 0.f);
                v[i] = split4(x);
            }
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int mt = 2 * u + e;
                uint32_t ah[2][4], al[2][4];       // rows (2t+8kp, 2t+1+8kp) are k-slots (t, t+4)
#pragma unroll
                for (int kp = 0; kp < 2; ++kp) {
                    ah[kp][0] = v[2 * kp].h[2 * e]; ah[kp][1] = v[2 * kp].h[2 * e + 1];
                    ah[kp][2] = v[2 * kp + 1].h[2 * e]; ah[kp][3] = v[2 * kp + 1].h[2 * e + 1];
                    al[kp][0] = v[2 * kp].l[2 * e]; al[kp][1] = v[2 * kp].l[2 * e + 1];
                    al[kp][2] = v[2 * kp + 1].l[2 * e]; al[kp][3] = v[2 * kp + 1].l[2 * e + 1];
                }
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    float oh[4] = {0.f, 0.f, 0.f, 0.f}, ol[4] = {0.f, 0.f, 0.f, 0.f}, ox[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int kp = 0; kp < 2; ++kp)
                        mma3(oh, ol, ox, ah[kp], al[kp], pp[nt].h[2 * kp], pp[nt].h[2 * kp + 1], pp[nt].l[2 * kp],
                             pp[nt].l[2 * kp + 1]);
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        st.om[mt][nt][i] = fmaf(st.om[mt][nt][i], alpha[nt][i & 1], oh[i] + (ol[i] + ox[i]));
                }
            }
        }
        return true;
    };

    if (!PAIRED) {
        ScoreState<NJ, NT> ss;
        PvState<MT, NT> ps;
        run([&]() { score_begin(ss); pv_begin(ps); }, [&](int hb) { score_publish(ss, hb); pv_publish(ps, hb); },
            [&](const float *tile_base, int nr, int k, auto full_tag) -> bool {
                return score_tile(ss, tile_base, nr, k, full_tag) && pv_tile(ps, tile_base + R * D, nr, k, full_tag);
            });
    } else if (!is_pv) {
        ScoreState<NJ, NT> ss;
        run([&]() { score_begin(ss); }, [&](int hb) { score_publish(ss, hb); },
            [&](const float *tile_base, int nr, int k, auto full_tag) -> bool {
                return score_tile(ss, tile_base, nr, k, full_tag);
            });
    } else {
        PvState<MT, NT> ps;
        run([&]() { pv_begin(ps); }, [&](int hb) { pv_publish(ps, hb); },
            [&](const float *tile_base, int nr, int k, auto full_tag) -> bool {
                return pv_tile(ps, tile_base, nr, k, full_tag);
            });
    }
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

}  // namespace moa
