// moa_grouped.cuh -- tensor-core decode kernel for large head groups (MQA / wide GQA).
//
// When GH = h_q/h_kv query heads share one K/V head, Steps I and III of Algorithm 1
// (eqs. (1),(3)) are dense contractions per tile of cached rows:
//     S^T[rows x GH] = K_tile[rows x d] * Q^T[d x GH],   O^T[d x GH] += V_tile^T[d x rows] * P^T[rows x GH]
// and at GH >= 16 the fp32 FMA pipes, not HBM, would bound the kernel.  Here both products
// run on the 5th-generation tensor cores (tcgen05.mma, kind::tf32, accumulators in tensor
// memory) with a three-term error-compensated split so that the result keeps fp32 accuracy:
//     x = hi + lo,  hi = x with the low 13 mantissa bits cleared (exactly what the tensor
//     core keeps of an fp32 operand),  a*b ~= a_hi*b_hi + a_lo*b_hi + a_hi*b_lo.
// The hi and lo parts of the small operand (Q, P) are stacked along N so one instruction
// covers two terms; the lo part of the streamed operand (K, V) is produced in place in
// the shared-memory buffer after the hi product has consumed it, so it costs no space.
//
// Orientation: the 128 cached rows of a tile are the M dimension, so a thread of the
// softmax group owns one cached row and all GH heads of it.  Step II (eq. (2)) uses a
// per-head reference m_ref instead of the exact running maximum (any reference gives the
// same value; it only has to keep exp2 in range): m_ref is raised, and the accumulators
// rescaled, only when a score exceeds it by more than 2^16.
//
// Roles (512 threads): warp 0 TMA producer, warps 1 and 2 MMA issuers (warp 1 also owns the
// TMEM allocation), warps 4-11 softmax (warp w works on TMEM lane quarter w % 4, i.e. cached
// rows 32*(w%4).., and on the lower (w < 8) or upper half of the heads), warps 3 and 12-15
// turn K chunks into their lo parts.  V chunks are turned into their lo parts by the
// softmax warps themselves: they would otherwise idle exactly while the weighted-sum
// products of the previous tile wait for that conversion.  Every hand-off is an mbarrier; every wait is bounded.
#pragma once

#include <cuda.h>

#include "moa_device.cuh"
#include "moa_tc.cuh"

namespace moa {

template <int GH_>
struct GroupedCfg {
    static constexpr int GH = GH_;
    static constexpr int D = 128;
    static constexpr int TILE = 128;               // cached rows per tile = MMA M
    static constexpr int N1 = 2 * GH;              // hi|lo stacked operand rows
    static constexpr int NBUF = GH == 64 ? 6 : (GH == 32 ? 10 : 12);   // 16 KB K/V chunk buffers
    static constexpr int CHUNK = 16384;
    static constexpr int OPCH = N1 * 128;          // bytes of one 32-wide k-chunk of the Q / P operand
    static constexpr int THREADS = 512;            // 16 warps, see the role list above
    static constexpr int KCONV_WARPS = 5;          // warps 3, 12..15 convert K chunks
    static constexpr int VCONV_WARPS = 8;          // the softmax warps convert V chunks
    static constexpr int NSOFT = 256;              // softmax threads (warps 4..11)
    static constexpr int HH = GH / 2;              // heads per softmax thread
    static constexpr int PW = HH < 16 ? HH : 16;   // heads handled per TMEM read
    static constexpr int PS = D + 4;               // floats per partial row: o[D], m, l, pad
    static constexpr uint32_t OFF_Q = 0;
    static constexpr uint32_t OFF_P = OFF_Q + 4 * OPCH;
    static constexpr uint32_t OFF_RING = OFF_P + 4 * OPCH;
    static constexpr uint32_t OFF_MREF = OFF_RING + NBUF * CHUNK;
    static constexpr uint32_t OFF_ALPHA = OFF_MREF + GH * 4;
    static constexpr uint32_t OFF_TMAX = OFF_ALPHA + GH * 4;
    static constexpr uint32_t OFF_LRED = OFF_TMAX + GH * 4;
    static constexpr uint32_t OFF_BAR = OFF_LRED + 4 * GH * 4;      // lred: [4 row quarters][GH]
    static constexpr int NBAR = 7 * NBUF + 2 + 2 + 4 + 1;   // full/hi/lo per chunk kind, empty, and the tile barriers
    static constexpr uint32_t OFF_TMEM = OFF_BAR + NBAR * 8;
    static constexpr uint32_t OFF_ABORT = OFF_TMEM + 4;
    static constexpr uint32_t OFF_ACC = OFF_ABORT + 4;        // "weighted sum of this tile adds to the accumulator"
    static constexpr size_t SMEM_BYTES = OFF_ACC + 4;
    static constexpr int FOLD_EVERY = 4;           // tiles accumulated by the tensor core between folds
    static_assert(GH == 16 || GH == 32 || GH == 64, "group size");
    static_assert(OFF_RING % 1024 == 0, "swizzled tiles need 1024-byte alignment");
};

struct GroupedArgs {
    const float *q;      // [batch, h_q, 128]
    float *out;          // [batch, h_q, 128]
    float *ws;           // partial slots [units][splits][GH][PS]
    int batch, h_q, h_kv, n;
    int g_s;             // query heads per (virtual) kv head; smaller than GH only on the 64-lane kernel (padded group)
    int h_kv_stored;     // K/V heads as stored; h_kv above counts virtual heads of GH query heads
    int share;           // virtual heads per stored K/V head (h_kv = h_kv_stored * share)
    int splits;          // sequence splits per unit
    int tiles_per_split;
    float qscale;        // scale * log2(e)
    float *partial_out;  // nullptr, or [batch, h_q, 132]: unnormalised triples instead of `out`
    // ---- ragged caches and the fused step (all null / zero for a dense decode) ----
    const int32_t *seq_lens;   // device [batch] or nullptr: sequence b has seq_lens[b] + len_bias rows (n = capacity)
    int len_bias;
    float *tailK, *tailV;      // [stored units][128][128]: zero-padded copy of every unit's last tile, or nullptr
    int flat;                  // 0, or the grid size: ragged caches, CTAs are dealt to the units in proportion
                               // to their lengths (see flat_share)
    int pair;                  // 64-lane kernel on rows of 64 features: two consecutive cached rows form one row of
                               // 128 (n counts such pairs, lengths are given in cached rows), a head takes two
                               // pseudo-heads (even rows, odd rows); ragged caches only with share == 1
    int g_total;               // pair mode: query heads per stored K/V head (<= share * g_s: the last virtual head
                               // of a stored one may hold fewer than g_s)
};

// Cached rows of sequence b (rows of 64 features in pair mode); 0 for an out-of-range length.
__device__ __forceinline__ int grouped_len_rows(const GroupedArgs &a, int b)
{
    const int cap = a.pair ? 2 * a.n : a.n;
    if (a.seq_lens == nullptr) return cap;
    const int len = a.seq_lens[b] + a.len_bias;
    return (len >= 1 && len <= cap) ? len : 0;
}
// Rows of sequence b as this kernel family sees them (pair mode: rows of 128 = pairs of cached
// rows, the last one possibly half filled); 0 for an out-of-range length.
__device__ __forceinline__ int grouped_len(const GroupedArgs &a, int b)
{
    const int rows = grouped_len_rows(a, b);
    return a.pair ? (rows + 1) >> 1 : rows;
}

// Ragged caches, `flat` mode (share == 1): the grid's CTAs are dealt to the units in
// proportion to their tile counts, every unit getting at least one:
//     s_u = 1 + floor(extra * tiles_u / total),   extra = grid - units,   capped at tiles_u,
// and CTA c works on split (c - first_u) of the unit u whose CTA range contains c; its
// partial goes to slot c.  Every CTA and the combine kernel recompute this from the lengths.
struct FlatShare {
    int unit, first, count;    // unit == -1: a CTA past the last unit's range
};
// Warp-collective (all 32 lanes, same arguments); every lane gets the answer.
__device__ __forceinline__ FlatShare flat_share(const GroupedArgs &a, int grid, int want_cta, int want_unit, int lane)
{
    const int units = a.batch * a.h_kv_stored;
    long long total = 0;
    for (int b = lane; b < a.batch; b += 32) total += (long long)((grouped_len(a, b) + 127) / 128) * a.h_kv_stored;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) total += __shfl_xor_sync(0xffffffffu, total, off);
    const long long extra = grid > units ? grid - units : 0;
    int first = 0;
    for (int base = 0; base < units; base += 32) {
        const int u = base + lane;
        int cnt = 0;
        if (u < units) {
            const int tiles = (grouped_len(a, u / a.h_kv_stored) + 127) / 128;
            long long c = 1 + (total > 0 ? extra * tiles / total : 0);
            if (c > tiles) c = tiles > 0 ? tiles : 1;
            cnt = (int)c;
        }
        int incl = cnt;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += t;
        }
        const int mine = first + incl - cnt;
        const bool hit = u < units && (u == want_unit || (want_cta >= mine && want_cta < mine + cnt));
        const unsigned m = __ballot_sync(0xffffffffu, hit);
        if (m != 0u) {
            const int src = __ffs(m) - 1;
            return FlatShare{base + src, __shfl_sync(0xffffffffu, mine, src), __shfl_sync(0xffffffffu, cnt, src)};
        }
        first += __shfl_sync(0xffffffffu, incl, 31);
    }
    return FlatShare{-1, first, 0};
}

// Ragged caches: rows past a sequence's length hold arbitrary bits (possibly NaN), and a zero
// probability does not neutralise them inside a tensor-core product.  So the last, partly
// filled tile of every unit is first copied into a scratch tile with its unused rows zeroed,
// and the main kernel fetches that tile from there.  For the fused step the row being
// appended (the unit's last row) is taken from k_new / v_new and also stored into the cache
// (eqs. (4),(5)).  Eight blocks per stored (batch, kv head), 16 rows of 128 floats each.
__global__ void __launch_bounds__(256) grouped_tail_kernel(const GroupedArgs a, const float *K, const float *V, float *Kw,
                                                           float *Vw, const float *k_new, const float *v_new)
{
    // The main kernel that follows may be scheduled while this one runs (programmatic dependent
    // launch): it only waits for this grid before it fetches the tiles copied here.
    launch_dependents();
    const int unit = blockIdx.x >> 3, part = blockIdx.x & 7, b = unit / a.h_kv_stored;
    const int len = grouped_len(a, b);
    // pair mode: a row of 128 is two cached rows of 64; `halves` counts the cached rows of the tile
    const int rows_real = grouped_len_rows(a, b);
    if (len == 0) {
        if (threadIdx.x == 0 && part == 0 && (unit % a.h_kv_stored) == 0)
            raise_status(MOA_STATUS_SEQLEN_RANGE | (k_new != nullptr ? MOA_STATUS_APPEND_RANGE : 0));
        return;
    }
    const int row0 = ((len - 1) / 128) * 128, valid = len - row0;
    const int halves = a.pair ? rows_real - 2 * row0 : 2 * valid;     // 64-float half rows that hold data
    const int new_half = halves - 1;                                  // pair mode: the appended cached row
    const float4 *srcK = reinterpret_cast<const float4 *>(K + ((size_t)unit * a.n + row0) * 128);
    const float4 *srcV = reinterpret_cast<const float4 *>(V + ((size_t)unit * a.n + row0) * 128);
    float4 *dstK = reinterpret_cast<float4 *>(a.tailK + (size_t)unit * 128 * 128);
    float4 *dstV = reinterpret_cast<float4 *>(a.tailV + (size_t)unit * 128 * 128);
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i = part * 512 + threadIdx.x; i < (part + 1) * 512; i += blockDim.x) {
        const int r = i >> 5, c = i & 31;
        const int half = 2 * r + (c >> 4);
        float4 k = zero, v = zero;
        if (half < halves) {
            if (k_new != nullptr && (a.pair ? half == new_half : r == valid - 1)) {
                k = a.pair ? reinterpret_cast<const float4 *>(k_new + (size_t)unit * 64)[c & 15]
                           : reinterpret_cast<const float4 *>(k_new + (size_t)unit * 128)[c];
                v = a.pair ? reinterpret_cast<const float4 *>(v_new + (size_t)unit * 64)[c & 15]
                           : reinterpret_cast<const float4 *>(v_new + (size_t)unit * 128)[c];
                reinterpret_cast<float4 *>(Kw + ((size_t)unit * a.n + row0) * 128)[i] = k;
                reinterpret_cast<float4 *>(Vw + ((size_t)unit * a.n + row0) * 128)[i] = v;
            } else {
                k = srcK[i];
                v = srcV[i];
            }
        }
        dstK[i] = k;
        dstV[i] = v;
    }
}

// Bounded mbarrier wait that also gives up when another role has already failed.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    // test_wait polls without suspending the thread: the hand-offs of this kernel are short
    // and on the critical path, so a prompt wake-up matters more than the issue slots
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        if (mbar_test_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    raise_status(MOA_STATUS_WAIT_TIMEOUT);
    return false;
}

__device__ __forceinline__ uint32_t ordered_bits(float x)      // monotone float -> uint
{
    const uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t u)
{
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}
__device__ __forceinline__ float tf32_hi(float x) { return __uint_as_float(__float_as_uint(x) & 0xFFFFE000u); }
// Nearest TF32 value (10 mantissa bits kept, the rest rounded away).  Operands this library
// writes itself are split as hi = tf32_rn(x), lo = tf32_rn(x - hi): nothing is left for the
// tensor core to cut off, and the rounding errors (at most 2^-23 of x) have no preferred sign.
// A streamed operand is multiplied as loaded, i.e. with hi = tf32_hi(x) (what the tensor core
// keeps of an fp32 word), and its remainder x - tf32_hi(x) is left to the tensor core's cut.
__device__ __forceinline__ float tf32_rn(float x) { return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u); }

__device__ __forceinline__ void named_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ bool named_or(int id, int n, bool pred)
{
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %3, 0;\n\tbar.red.or.pred p, %1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(r) : "r"(id), "r"(n), "r"((uint32_t)pred) : "memory");
    return r != 0;
}

// The order in which 16 KB chunks travel through the ring, shared by producer, issuer and
// converters: K(0), then for every tile t: K(t+1) (if any) followed by V(t).
struct ChunkSeq {
    int T;          // tiles of this CTA
    int t;          // tile of the current group
    bool is_k;      // group kind
    int c;          // chunk inside the group, 0..3
    int seq;        // running chunk number (ring position = seq % NBUF)
    bool done;
    __device__ __forceinline__ explicit ChunkSeq(int tiles) : T(tiles), t(0), is_k(true), c(0), seq(0), done(tiles <= 0) {}
    // Skip whole groups of the other kind (used by an issuer that handles one kind only).
    __device__ __forceinline__ void skip_to_kind(bool want_k)
    {
        while (!done && is_k != want_k) { next(); next(); next(); next(); }
    }
    __device__ __forceinline__ void next()
    {
        ++seq;
        if (++c < 4) return;
        c = 0;
        if (is_k) {                     // after K(0) comes K(1) or V(0); after K(t+1) comes V(t)
            if (t == 0 && T > 1 && seq == 4) { t = 1; return; }     // K(0) -> K(1)
            is_k = false;
            t = (t == 0) ? 0 : t - 1;
        } else {                        // after V(t): K(t+2) if it exists, else V(t+1), else done
            if (t + 2 < T) { is_k = true; t = t + 2; }
            else if (t + 1 < T) { t = t + 1; }
            else done = true;
        }
    }
};

template <class C>
__global__ void __launch_bounds__(C::THREADS, 1)
grouped_decode_kernel(const __grid_constant__ CUtensorMap tmapK, const __grid_constant__ CUtensorMap tmapV,
                      const __grid_constant__ CUtensorMap tmapKt, const __grid_constant__ CUtensorMap tmapVt,
                      const GroupedArgs a)
{
    constexpr int GH = C::GH, N1 = C::N1, NBUF = C::NBUF, PS = C::PS;
    extern __shared__ __align__(1024) unsigned char smem_g[];
    unsigned char *const smem = smem_g;
    float *mref = reinterpret_cast<float *>(smem + C::OFF_MREF);
    float *alpha_s = reinterpret_cast<float *>(smem + C::OFF_ALPHA);
    uint32_t *tmax = reinterpret_cast<uint32_t *>(smem + C::OFF_TMAX);
    float *lred = reinterpret_cast<float *>(smem + C::OFF_LRED);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::OFF_BAR);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::OFF_TMEM);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_ABORT);
    volatile uint32_t *acc_flag = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_ACC);

    const uint32_t sbase = smem_u32(smem);
    const uint32_t sQ = sbase + C::OFF_Q, sP = sbase + C::OFF_P, sRing = sbase + C::OFF_RING;
    // A ring buffer is used by K chunks and V chunks in turn, but the roles of one kind never
    // look at the other kind's chunks.  A parity wait is only safe for a waiter that sees
    // every phase of its barrier, so "data landed", "hi product done" and "lo part ready"
    // exist once per kind; each role keeps one parity bit per buffer for its own kind.
    auto bar_full = [&](bool k, int b) { return smem_u32(&bars[(k ? 0 : NBUF) + b]); };
    auto bar_hi = [&](bool k, int b) { return smem_u32(&bars[(k ? 2 : 3) * NBUF + b]); };
    auto bar_lo = [&](bool k, int b) { return smem_u32(&bars[(k ? 4 : 5) * NBUF + b]); };
    auto bar_empty = [&](int b) { return smem_u32(&bars[6 * NBUF + b]); };
    auto bar_sfull = [&](int s) { return smem_u32(&bars[7 * NBUF + s]); };
    auto bar_sfree = [&](int s) { return smem_u32(&bars[7 * NBUF + 2 + s]); };
    auto bar_pfull = [&](int c) { return smem_u32(&bars[7 * NBUF + 4 + c]); };
    const uint32_t bar_pvdone = smem_u32(&bars[7 * NBUF + 8]);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // CTA order: the virtual heads that share one stored K/V head are neighbours, so they run
    // at the same time and the second reader of a chunk finds it in L2.
    int sub = blockIdx.x % a.share;
    int split = (blockIdx.x / a.share) % a.splits;
    int sunit = blockIdx.x / (a.share * a.splits);                // stored (batch, kv head)
    int splits_u = a.splits;
    if (a.flat) {                                  // warp 0 walks the lengths, all take its answer
        int *s_share = reinterpret_cast<int *>(lred);    // (the reduction scratch is not in use yet)
        if (warp == 0) {
            const FlatShare f = flat_share(a, (int)gridDim.x, (int)blockIdx.x, -1, lane);
            if (lane == 0) { s_share[0] = f.unit; s_share[1] = f.first; s_share[2] = f.count; }
        }
        __syncthreads();
        if (s_share[0] < 0) return;
        sub = 0; sunit = s_share[0]; split = (int)blockIdx.x - s_share[1]; splits_u = s_share[2];
    }
    const int b = sunit / a.h_kv_stored, h = (sunit % a.h_kv_stored) * a.share + sub;   // virtual head
    const int unit = sunit;                                         // tensor-map coordinate
    const int len_b = grouped_len(a, b);           // 0: out-of-range length, the item is skipped
    const int tiles_total = (len_b + C::TILE - 1) / C::TILE;
    const int tiles_per_split = a.seq_lens ? (tiles_total + splits_u - 1) / splits_u : a.tiles_per_split;
    const int tile0 = split * tiles_per_split;
    int T = tiles_total - tile0;
    if (T > tiles_per_split) T = tiles_per_split;
    if (T <= 0) return;                            // an empty split (uniform for the CTA)
    // the unit's last tile comes from the zero-padded scratch copy when there is one
    const int tail_t = (a.tailK != nullptr) ? tiles_total - 1 - tile0 : -1;

    // ---- set-up --------------------------------------------------------------------------
    if (tid == 0) {
        for (int i = 0; i < NBUF; ++i) {
            for (int k = 0; k < 2; ++k) {
                mbar_init(bar_full(k != 0, i), 1); mbar_init(bar_hi(k != 0, i), 1);
                mbar_init(bar_lo(k != 0, i), k != 0 ? C::KCONV_WARPS : C::VCONV_WARPS);
            }
            mbar_init(bar_empty(i), 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(bar_sfull(i), 1); mbar_init(bar_sfree(i), 8); }
        for (int i = 0; i < 4; ++i) mbar_init(bar_pfull(i), 2);
        mbar_init(bar_pvdone, 1);
        mbar_fence_init();
        *abort_flag = 0;
        *acc_flag = 0u;
        tc::prefetch_tmap(&tmapK);
        tc::prefetch_tmap(&tmapV);
        if (a.tailK != nullptr) { tc::prefetch_tmap(&tmapKt); tc::prefetch_tmap(&tmapVt); }
    }
    if (warp == 1) tc::tmem_alloc(smem_u32(tmem_slot), 512);
    // Q operand: rows 0..GH-1 hold hi(q*qscale), rows GH..2GH-1 the lo parts; K-major, 4
    // chunks of 32 features, 128-byte swizzle.
    {
        const float *qb = a.q + ((size_t)b * a.h_q + (size_t)h * GH) * 128;
        for (int i = tid; i < GH * 128; i += C::THREADS) {
            const int g = i >> 7, k = i & 127;
            const float x = qb[i] * a.qscale;
            const float hi = tf32_rn(x);
            const uint32_t chunk = (uint32_t)(k >> 5) * C::OPCH, col = (uint32_t)(k & 31) * 4;
            *reinterpret_cast<float *>(smem + C::OFF_Q + chunk + tc::swz128(g, col)) = hi;
            *reinterpret_cast<float *>(smem + C::OFF_Q + chunk + tc::swz128(GH + g, col)) = tf32_rn(x - hi);
        }
        if (tid < GH) mref[tid] = -INFINITY;
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    auto tS_of = [tmem](int sb) -> uint32_t { return tmem + (uint32_t)(sb & 1) * 128u; };   // two score buffers
    const uint32_t tO = tmem + 256u;           // per-tile weighted sum [hi | lo] written by the tensor core
    const uint32_t tOm = tmem + 384u;          // fp32 master copy of the weighted sum, GH columns
    const int row_base = tile0 * C::TILE;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            for (ChunkSeq s(T); !s.done; s.next()) {
                const int buf = s.seq % NBUF, use = s.seq / NBUF;
                if (use > 0 && !wait_or_abort(bar_empty(buf), (uint32_t)(use - 1) & 1u, abort_flag)) break;
                const uint32_t dst = sRing + (uint32_t)buf * C::CHUNK;
                const uint32_t fb = bar_full(s.is_k, buf);
                mbar_expect_tx(fb, C::CHUNK);
                const bool tail = (s.t == tail_t);
                const int row = tail ? 0 : row_base + s.t * C::TILE;
                if (s.is_k) {
                    tc::tma_load_3d(dst, tail ? &tmapKt : &tmapK, 32 * s.c, row, unit, fb);
                } else {
                    for (int dg = 0; dg < 4; ++dg)
                        tc::tma_load_3d(dst + dg * 4096, tail ? &tmapVt : &tmapV, 32 * dg, row + 32 * s.c, unit, fb);
                }
            }
        }
    } else if (warp == 1 || warp == 2) {
        // ================= MMA issuers =================
        // Two single-thread issuers feed the tensor core: warp 1 the score products (K chunks,
        // accumulators S), warp 2 the weighted-sum products (V chunks, accumulator O).  Each
        // keeps two cursors over its chunks: `hi` (next chunk whose raw data is multiplied) and
        // `lo` (next chunk whose in-place lo part is multiplied) and issues whichever is
        // ready, so a chunk waiting for its converters never holds up the ones behind it.
        // A lone thread retires an instruction every few cycles, so the issue path is kept to
        // a handful of instructions per MMA (descriptor words are advanced, not rebuilt).
        {
            // Polling a barrier costs a shared-memory round trip of a few hundred cycles, far
            // more than issuing a product, so the whole warp polls: lane s checks the barrier
            // that step s of the current group waits for, one ballot tells lane 0 how many of
            // the next steps can go, and lane 0 issues them back to back.
            const bool kind_k = (warp == 1);
            const uint32_t idesc_hi = kind_k ? tc::idesc_tf32(128, N1, false, false) : tc::idesc_tf32(128, N1, true, false);
            const uint32_t idesc_lo = kind_k ? tc::idesc_tf32(128, GH, false, false) : tc::idesc_tf32(128, GH, true, false);
            // descriptor words: [addr>>4 | lbo>>4 << 16] and [sbo>>4 | version << 14 | layout << 29]
            const uint32_t a_hiword = kind_k ? (64u | (1u << 14) | (2u << 29)) : (32u | (1u << 14) | (1u << 29));
            const uint32_t a_base = (sRing >> 4) | (kind_k ? (1u << 16) : (256u << 16));
            const uint32_t a_step = kind_k ? 2u : 64u;                 // 32 B / 1024 B per k-step
            const uint32_t b_hiword = 64u | (1u << 14) | (2u << 29);
            const uint32_t b_base = ((kind_k ? sQ : sP) >> 4) | (1u << 16);
            // Issue order inside a group of four chunks is fixed (hi0 hi1 hi2 lo0 hi3 lo1 lo2 lo3):
            // the hi*lo and lo*hi terms share accumulator columns and the tensor core's
            // accumulation is not associative, so a timing-dependent order would make the
            // result differ from run to run.  The two-chunk lag gives the converters time.
            // In the chunk sequence the K groups sit at group indices 0,1,3,5,... and the V
            // groups at 2,4,...,2T-2,2T-1; a group's first chunk is number 4*index.
            // step s of a group: is it a hi product, and of which chunk?
            const bool my_is_hi = (lane < 3) || (lane == 4);
            const int my_c = my_is_hi ? (lane < 3 ? lane : 3) : (lane == 3 ? 0 : lane - 4);
            bool ok = true;
            uint32_t par = 0;                      // per ring buffer: parity of this kind's next use
            uint32_t idle = 0;
            for (int t = 0; ok && t < T; ++t) {
                const int gi = kind_k ? (t == 0 ? 0 : 2 * t - 1) : (t < T - 1 ? 2 * t + 2 : 2 * T - 1);
                const int b0 = (4 * gi) % NBUF;
                const uint32_t d_hi = kind_k ? tS_of(t) : tO;
                // ---- group dependencies: the score buffer is free / all probabilities are stored
                // (chunk 0 of a weighted sum may overwrite the whole accumulator, which every
                // softmax warp reads while folding, so all of them have to be done)
                for (;;) {
                    bool r = true;
                    if (kind_k) { if (t >= 2 && lane == 0) r = mbar_test_wait(bar_sfree(t & 1), (uint32_t)(t / 2 - 1) & 1u); }
                    else if (lane < 4) r = mbar_test_wait(bar_pfull(lane), (uint32_t)t & 1u);
                    if (__all_sync(0xffffffffu, r)) break;
                    if (++idle >= kWaitLimit) { if (lane == 0) { *abort_flag = 1; raise_status(MOA_STATUS_WAIT_TIMEOUT); } ok = false; break; }
                    if ((idle & 255u) == 255u && *abort_flag) { ok = false; break; }
                }
                if (!ok) break;
                idle = 0;
                const uint32_t acc_first = kind_k ? 0u : *acc_flag;   // does the tile add to the accumulator?
                // this lane's barrier for its step
                const int my_buf = (b0 + my_c >= NBUF) ? b0 + my_c - NBUF : b0 + my_c;
                const uint32_t my_bar = my_is_hi ? bar_full(kind_k, my_buf) : bar_lo(kind_k, my_buf);
                const uint32_t my_par = (par >> my_buf) & 1u;
                int step = 0;
                while (step < 8) {
                    const bool r = (lane < 8 && lane >= step) ? mbar_test_wait(my_bar, my_par) : false;
                    const uint32_t m = __ballot_sync(0xffffffffu, r) >> step;
                    const int run = __ffs(~m) - 1;               // consecutive ready steps from `step`
                    if (run == 0) {
                        if (++idle >= kWaitLimit) { if (lane == 0) { *abort_flag = 1; raise_status(MOA_STATUS_WAIT_TIMEOUT); } ok = false; break; }
                        if ((idle & 255u) == 255u && *abort_flag) { ok = false; break; }
                        continue;
                    }
                    idle = 0;
                    if (lane == 0) {
                        tc::fence_after_sync();
#pragma unroll
                        for (int sidx = 0; sidx < 8; ++sidx) {
                            if (sidx < step || sidx >= step + run) continue;
                            const bool is_hi = (sidx < 3) || (sidx == 4);
                            const int c = is_hi ? (sidx < 3 ? sidx : 3) : (sidx == 3 ? 0 : sidx - 4);
                            const int buf = (b0 + c >= NBUF) ? b0 + c - NBUF : b0 + c;
                            const uint32_t a_lo = a_base + (uint32_t)buf * (C::CHUNK >> 4);
                            const uint32_t b_lo = b_base + (uint32_t)c * (C::OPCH >> 4);
                            if (is_hi) {
                                // the first product of a tile overwrites the accumulator unless the
                                // softmax group said to keep adding (it folds the weighted sum into an
                                // fp32 master copy every few tiles, because the tensor core
                                // accumulates with truncation)
                                tc::mma_tf32_ss(d_hi, tc::pack64(a_lo, a_hiword), tc::pack64(b_lo, b_hiword), idesc_hi,
                                                (uint32_t)c | acc_first);
#pragma unroll
                                for (uint32_t ks = 1; ks < 4; ++ks)
                                    tc::mma_tf32_ss(d_hi, tc::pack64(a_lo + ks * a_step, a_hiword),
                                                    tc::pack64(b_lo + ks * 2u, b_hiword), idesc_hi, 1u);
                                tc::mma_commit(bar_hi(kind_k, buf));
                            } else {
#pragma unroll
                                for (uint32_t ks = 0; ks < 4; ++ks)
                                    tc::mma_tf32_ss(d_hi + GH, tc::pack64(a_lo + ks * a_step, a_hiword),
                                                    tc::pack64(b_lo + ks * 2u, b_hiword), idesc_lo, 1u);
                                tc::mma_commit(bar_empty(buf));
                                if (c == 3) tc::mma_commit(kind_k ? bar_sfull(t & 1) : bar_pvdone);
                            }
                        }
                    }
                    step += run;
                    __syncwarp();
                }
                // this kind has now used the four buffers once more
#pragma unroll
                for (int c = 0; c < 4; ++c) par ^= 1u << ((b0 + c >= NBUF) ? b0 + c - NBUF : b0 + c);
            }
        }
    } else if (warp >= 4 && warp < 12) {
        // ================= softmax group: thread = (cached row, half of the heads) =================
        constexpr int HH = C::HH, PW = C::PW, NP = HH / PW, NS = C::NSOFT;
        const int q4 = warp & 3;                     // TMEM lane quarter = rows 32*q4 .. 32*q4+31 of the tile
        const int h0 = (warp < 8) ? 0 : HH;          // first head of this thread
        const int st = tid - 128;                    // 0..255 inside the group
        const int row_in_tile = q4 * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
        float lsum[HH], p[HH];
#pragma unroll
        for (int g = 0; g < HH; ++g) lsum[g] = 0.f;
        unsigned char *pch = smem + C::OFF_P + (uint32_t)q4 * C::OPCH;     // this row quarter's P chunk
        bool ok = true;
        uint32_t par_v = 0;                          // per ring buffer: parity of the next V use
        bool have_master = false;                    // has anything been folded into the master copy?
        // Turn the four V chunks of tile tv into their lo parts, each as soon as its hi
        // product has completed (all 256 threads: four float4 each per chunk).
        auto convert_v = [&](int tv) -> bool {
            const int seq0 = 4 * (tv < T - 1 ? 2 * tv + 2 : 2 * T - 1);
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                const int buf = (seq0 + c) % NBUF;
                const uint32_t ph = (par_v >> buf) & 1u;
                par_v ^= 1u << buf;
                if (!wait_or_abort(bar_hi(false, buf), ph, abort_flag)) return false;
                float4 *pv = reinterpret_cast<float4 *>(smem + C::OFF_RING + (uint32_t)buf * C::CHUNK);
                float4 v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) v[i] = pv[st + i * NS];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    v[i].x -= tf32_hi(v[i].x); v[i].y -= tf32_hi(v[i].y);
                    v[i].z -= tf32_hi(v[i].z); v[i].w -= tf32_hi(v[i].w);
                    pv[st + i * NS] = v[i];
                }
                tc::fence_async_smem();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(bar_lo(false, buf));
            }
            return true;
        };
        for (int t = 0; ok && t < T; ++t) {
            const int sb = t & 1;
            if (t > 0) ok = convert_v(t - 1);        // (a failure is shared at the vote just below)
            ok = ok && wait_or_abort(bar_sfull(sb), (uint32_t)(t >> 1) & 1u, abort_flag);
            if (named_or(1, NS, !ok)) { ok = false; break; }     // leave together or not at all
            tc::fence_after_sync();
            const bool valid = (row_base + t * C::TILE + row_in_tile) < len_b;
            // scores of this row against the current references; probabilities are formed at
            // once (they are only wrong if the reference has to be raised, which is rare)
            float vmax = -INFINITY;
#pragma unroll
            for (int j = 0; j < NP; ++j) {
                uint32_t hi[PW], lo[PW];
                tc::tmem_ld_piece<PW>(tS_of(sb) + lane_addr + h0 + PW * j, hi);
                tc::tmem_ld_piece<PW>(tS_of(sb) + lane_addr + GH + h0 + PW * j, lo);
                tc::tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < PW; ++i) {
                    const float x = (__uint_as_float(hi[i]) + __uint_as_float(lo[i])) - mref[h0 + PW * j + i];
                    vmax = fmaxf(vmax, x);
                    p[PW * j + i] = valid ? fast_exp2(x) : 0.f;
                }
            }
            const bool raise = named_or(1, NS, valid && (vmax > 16.0f));
            if (raise) {
                // ---- exact per-head maximum of this tile
                if (st < GH) tmax[st] = 0u;
                named_sync(1, NS);
#pragma unroll
                for (int j = 0; j < NP; ++j) {
                    uint32_t hi[PW], lo[PW];
                    tc::tmem_ld_piece<PW>(tS_of(sb) + lane_addr + h0 + PW * j, hi);
                    tc::tmem_ld_piece<PW>(tS_of(sb) + lane_addr + GH + h0 + PW * j, lo);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < PW; ++i) {
                        const float sv = valid ? (__uint_as_float(hi[i]) + __uint_as_float(lo[i])) : -INFINITY;
                        const uint32_t m = __reduce_max_sync(0xffffffffu, ordered_bits(sv));
                        if (lane == 0) atomicMax(&tmax[h0 + PW * j + i], m);
                    }
                }
                named_sync(1, NS);
                if (st < GH) {
                    const float old = mref[st];
                    const float nw = fmaxf(old, from_ordered_bits(tmax[st]));
                    alpha_s[st] = exp2_diff(old, nw);
                    mref[st] = nw;
                }
                named_sync(1, NS);
#pragma unroll
                for (int j = 0; j < NP; ++j) {        // probabilities again, against the new references
                    uint32_t hi[PW], lo[PW];
                    tc::tmem_ld_piece<PW>(tS_of(sb) + lane_addr + h0 + PW * j, hi);
                    tc::tmem_ld_piece<PW>(tS_of(sb) + lane_addr + GH + h0 + PW * j, lo);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < PW; ++i) {
                        const float x = (__uint_as_float(hi[i]) + __uint_as_float(lo[i])) - mref[h0 + PW * j + i];
                        p[PW * j + i] = valid ? fast_exp2(x) : 0.f;
                    }
                }
#pragma unroll
                for (int g = 0; g < HH; ++g) lsum[g] *= alpha_s[h0 + g];
            }
            // the score buffer is free again
            tc::fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(bar_sfree(sb));
#pragma unroll
            for (int g = 0; g < HH; ++g) lsum[g] += p[g];
            // The previous tile's weighted sum is complete, so the P buffers are free.  Every
            // FOLD_EVERY tiles, and whenever the references were raised, the accumulator is
            // folded into the fp32 master copy (the tensor core accumulates with truncation, so
            // its chains are kept short) and the next tile starts it afresh.
            if (t > 0) {
                ok = wait_or_abort(bar_pvdone, (uint32_t)(t - 1) & 1u, abort_flag);
                if (named_or(1, NS, !ok)) { ok = false; break; }
                tc::fence_after_sync();
                const bool fold = raise || (t % C::FOLD_EVERY) == 0;
                if (fold) {
#pragma unroll
                    for (int j = 0; j < NP; ++j) {
                        uint32_t hi[PW], lo[PW], ms[PW];
                        tc::tmem_ld_piece<PW>(tO + lane_addr + h0 + PW * j, hi);
                        tc::tmem_ld_piece<PW>(tO + lane_addr + GH + h0 + PW * j, lo);
                        if (have_master) tc::tmem_ld_piece<PW>(tOm + lane_addr + h0 + PW * j, ms);
                        tc::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < PW; ++i) {
                            float add = __uint_as_float(hi[i]) + __uint_as_float(lo[i]);
                            if (have_master) add += __uint_as_float(ms[i]);
                            if (raise) add *= alpha_s[h0 + PW * j + i];
                            ms[i] = __float_as_uint(add);
                        }
                        tc::tmem_st_piece<PW>(tOm + lane_addr + h0 + PW * j, ms);
                    }
                    tc::tmem_st_wait();
                    have_master = true;
                }
                if (st == 0) *acc_flag = fold ? 0u : 1u;     // read by the issuer after the P barriers
            }
            // probabilities, split into hi|lo, as the K-major B operand of this row quarter
#pragma unroll
            for (int g = 0; g < HH; ++g) {
                const float ph = tf32_rn(p[g]);
                *reinterpret_cast<float *>(pch + tc::swz128(h0 + g, lane * 4)) = ph;
                *reinterpret_cast<float *>(pch + tc::swz128(GH + h0 + g, lane * 4)) = tf32_rn(p[g] - ph);
            }
            tc::fence_before_sync();
            tc::fence_async_smem();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(bar_pfull(q4));
        }
        // ---- epilogue: this split's partial (m_ref, l, o) per head
        if (ok) {                            // (ok is uniform across the group here)
            ok = convert_v(T - 1) && wait_or_abort(bar_pvdone, (uint32_t)(T - 1) & 1u, abort_flag);
            if (named_or(1, NS, !ok)) ok = false;
        }
        if (ok) {
            tc::fence_after_sync();
#pragma unroll
            for (int g = 0; g < HH; ++g) {
                float v = lsum[g];
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
                if (lane == 0) lred[q4 * GH + h0 + g] = v;
            }
            named_sync(1, NS);
            float *slot = a.flat ? a.ws + ((size_t)blockIdx.x * GH) * PS
                                 : a.ws + ((((size_t)b * a.h_kv + h) * a.splits + split) * GH) * PS;
            const int d = row_in_tile;               // TMEM lane of O^T = output feature
#pragma unroll
            for (int j = 0; j < NP; ++j) {
                uint32_t hi[PW], lo[PW], ms[PW];
                tc::tmem_ld_piece<PW>(tO + lane_addr + h0 + PW * j, hi);
                tc::tmem_ld_piece<PW>(tO + lane_addr + GH + h0 + PW * j, lo);
                if (have_master) tc::tmem_ld_piece<PW>(tOm + lane_addr + h0 + PW * j, ms);
                tc::tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < PW; ++i) {
                    float add = __uint_as_float(hi[i]) + __uint_as_float(lo[i]);
                    if (have_master) add += __uint_as_float(ms[i]);
                    slot[(size_t)(h0 + PW * j + i) * PS + d] = add;
                }
            }
            if (st < GH) {
                slot[(size_t)st * PS + 128] = mref[st];
                slot[(size_t)st * PS + 129] = (lred[st] + lred[GH + st]) + (lred[2 * GH + st] + lred[3 * GH + st]);
            }
        }
    } else {
        // ================= K converters: chunk -> its lo part, in place =================
        constexpr int TT = C::KCONV_WARPS * 32;                        // 160 threads
        constexpr int FULL = (C::CHUNK / 16) / TT;                     // float4 every thread handles
        const int ct = (warp == 3 ? 0 : warp - 11) * 32 + lane;
        bool ok = true;
        uint32_t par = 0;                          // per ring buffer: parity of the next K use
        for (ChunkSeq s(T); ok && !s.done; s.next()) {
            if (!s.is_k) continue;
            const int buf = s.seq % NBUF;
            const uint32_t ph = (par >> buf) & 1u;
            par ^= 1u << buf;
            ok = wait_or_abort(bar_hi(true, buf), ph, abort_flag);
            if (!ok) break;
            float4 *p = reinterpret_cast<float4 *>(smem + C::OFF_RING + (uint32_t)buf * C::CHUNK);
            float4 v[FULL + 1];
#pragma unroll
            for (int i = 0; i < FULL; ++i) v[i] = p[ct + i * TT];
            const bool extra = ct + FULL * TT < C::CHUNK / 16;
            if (extra) v[FULL] = p[ct + FULL * TT];
#pragma unroll
            for (int i = 0; i <= FULL; ++i) {
                v[i].x -= tf32_hi(v[i].x); v[i].y -= tf32_hi(v[i].y);
                v[i].z -= tf32_hi(v[i].z); v[i].w -= tf32_hi(v[i].w);
            }
#pragma unroll
            for (int i = 0; i < FULL; ++i) p[ct + i * TT] = v[i];
            if (extra) p[ct + FULL * TT] = v[FULL];
            tc::fence_async_smem();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(bar_lo(true, buf));
        }
    }

    tc::fence_before_sync();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem, 512);
}

// Merge the per-split partials of the grouped kernels.  One block of four warps per (batch,
// query head): warp w accumulates the splits w, w+4, ... (in that order) against the global
// maximum, which every warp first reads from all splits in parallel; the four sums are then
// added in warp order, so the result is reproducible.  A split row is 132 floats
// (o[128], m, l, 2 pad); with many splits per unit the merge is a chain of dependent L2
// reads, which is why it is cut four ways.
template <int GH>
__global__ void __launch_bounds__(128) grouped_combine_kernel(const GroupedArgs a)
{
    constexpr int PS = 132;
    __shared__ float4 s_acc[4][32], s_accc[4][32];
    __shared__ float s_l[4], s_lc[4];
    grid_dependency_wait();                        // the partials of the main kernel (a no-op for an ordinary launch)
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long wid = blockIdx.x;
    const int b = (int)(wid / a.h_q), gq = (int)(wid % a.h_q);
    const int h = gq / a.g_s, g = gq % a.g_s;      // (partial slots are GH apart, the heads of a unit a.g_s)
    const int unit = b * a.h_kv + h;
    const int len_b = grouped_len(a, b);
    if (len_b == 0) {                              // out-of-range length: report, leave out untouched
        if (gq == 0 && threadIdx.x == 0) raise_status(MOA_STATUS_SEQLEN_RANGE);
        return;
    }
    const int tiles_total = (len_b + 127) / 128;
    int splits_u = a.splits;
    size_t first_slot = (size_t)unit * a.splits;
    if (a.flat) {
        const FlatShare f = flat_share(a, a.flat, -1, unit, lane);      // a.flat holds the grid size
        splits_u = f.count;
        first_slot = (size_t)f.first;
    }
    const int tiles_per_split = a.seq_lens ? (tiles_total + splits_u - 1) / splits_u : a.tiles_per_split;
    const int used = (tiles_total + tiles_per_split - 1) / tiles_per_split;   // non-empty splits
    const float *base = a.ws + (first_slot * GH + g) * PS;
    const size_t stride = (size_t)GH * PS;
    float M = -INFINITY;
    for (int s0 = 0; s0 < used; s0 += 32) {
        float m = (s0 + lane < used) ? base[(size_t)(s0 + lane) * stride + 128] : -INFINITY;
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
        M = fmaxf(M, m);
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), accc = acc;
    float L = 0.f, Lc = 0.f;
#pragma unroll 4
    for (int sp = warp; sp < used; sp += 4) {
        const float *row = base + (size_t)sp * stride;
        const float f = exp2_diff(row[128], M);
        comp_fma(L, Lc, row[129], f);
        const float4 t = *reinterpret_cast<const float4 *>(row + lane * 4);
        comp_fma4(acc, accc, t, f);
    }
    // (sum, compensation) of the four warps, added in warp order with the same care
    s_acc[warp][lane] = acc; s_accc[warp][lane] = accc;
    if (lane == 0) { s_l[warp] = L; s_lc[warp] = Lc; }
    __syncthreads();
    if (warp != 0) return;
    acc = s_acc[0][lane]; accc = s_accc[0][lane];
    L = s_l[0]; Lc = s_lc[0];
#pragma unroll
    for (int w = 1; w < 4; ++w) {
        comp_fma4(acc, accc, s_acc[w][lane], 1.0f);
        comp_fma4(acc, accc, s_accc[w][lane], -1.0f);
        comp_fma(L, Lc, s_l[w], 1.0f);
        comp_fma(L, Lc, s_lc[w], -1.0f);
    }
    if (a.partial_out != nullptr) {
        float *dst = a.partial_out + ((size_t)b * a.h_q + gq) * 132;
        *reinterpret_cast<float4 *>(dst + lane * 4) = acc;
        if (lane == 0) { dst[128] = M; dst[129] = L; }
        return;
    }
    const float inv = 1.0f / L;
    *reinterpret_cast<float4 *>(a.out + ((size_t)b * a.h_q + gq) * 128 + lane * 4) =
        make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
}

// Merge for the 64-lane kernel in pair mode (rows of 64 features): a head's result is spread over
// two pseudo-heads, 2j (even cached rows: features 0..63 of its 128-wide partial are meaningful)
// and 2j+1 (odd rows: features 64..127), each with a maximum and a sum of its own, times the
// splits of the unit.  One block of four warps per (batch, query head), as in the kernel above:
// warp w takes the partials w, w+4, ... in (split, parity) order against the global maximum,
// the four compensated sums are added in warp order.
__global__ void __launch_bounds__(128) grouped_pair_combine_kernel(const GroupedArgs a)
{
    constexpr int PS = 132, GH = 64;
    __shared__ float2 s_acc[4][32], s_accc[4][32];
    __shared__ float s_l[4], s_lc[4];
    grid_dependency_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long wid = blockIdx.x;
    const int b = (int)(wid / a.h_q), gq = (int)(wid % a.h_q);
    const int in_stored = gq % a.g_total;          // head inside its stored K/V head
    const int vh = (gq / a.g_total) * a.share + in_stored / a.g_s;   // virtual kv head (a.h_kv of them per batch item)
    const int j = in_stored % a.g_s;               // head inside the virtual head
    const int len_b = grouped_len(a, b);
    if (len_b == 0) {                              // out-of-range length: report, leave out untouched
        if (gq == 0 && threadIdx.x == 0) raise_status(MOA_STATUS_SEQLEN_RANGE);
        return;
    }
    const int tiles_total = (len_b + 127) / 128;
    int splits_u = a.splits;
    size_t first_slot = ((size_t)b * a.h_kv + vh) * a.splits;
    if (a.flat) {                                  // ragged caches (share == 1): slots follow the CTAs
        const FlatShare f = flat_share(a, a.flat, -1, b * a.h_kv + vh, lane);
        splits_u = f.count;
        first_slot = (size_t)f.first;
    }
    const int tiles_per_split = a.seq_lens ? (tiles_total + splits_u - 1) / splits_u : a.tiles_per_split;
    const int used = (tiles_total + tiles_per_split - 1) / tiles_per_split;          // non-empty splits
    const float *base = a.ws + (first_slot * GH + 2 * j) * PS;
    const size_t stride = (size_t)GH * PS;
    float M = -INFINITY;
    for (int i = lane; i < 2 * used; i += 32) M = fmaxf(M, base[(size_t)(i >> 1) * stride + (size_t)(i & 1) * PS + 128]);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    float2 acc = make_float2(0.f, 0.f), accc = acc;
    float L = 0.f, Lc = 0.f;
#pragma unroll 4
    for (int i = warp; i < 2 * used; i += 4) {
        const float *row = base + (size_t)(i >> 1) * stride + (size_t)(i & 1) * PS;
        const float f = exp2_diff(row[128], M);
        comp_fma(L, Lc, row[129], f);
        const float2 t = *reinterpret_cast<const float2 *>(row + 64 * (i & 1) + 2 * lane);
        comp_fma(acc.x, accc.x, t.x, f);
        comp_fma(acc.y, accc.y, t.y, f);
    }
    s_acc[warp][lane] = acc; s_accc[warp][lane] = accc;
    if (lane == 0) { s_l[warp] = L; s_lc[warp] = Lc; }
    __syncthreads();
    if (warp != 0) return;
    acc = s_acc[0][lane]; accc = s_accc[0][lane];
    L = s_l[0]; Lc = s_lc[0];
#pragma unroll
    for (int w = 1; w < 4; ++w) {
        comp_fma(acc.x, accc.x, s_acc[w][lane].x, 1.0f);
        comp_fma(acc.x, accc.x, s_accc[w][lane].x, -1.0f);
        comp_fma(acc.y, accc.y, s_acc[w][lane].y, 1.0f);
        comp_fma(acc.y, accc.y, s_accc[w][lane].y, -1.0f);
        comp_fma(L, Lc, s_l[w], 1.0f);
        comp_fma(L, Lc, s_lc[w], -1.0f);
    }
    const float inv = 1.0f / L;
    *reinterpret_cast<float2 *>(a.out + ((size_t)b * a.h_q + gq) * 64 + 2 * lane) = make_float2(acc.x * inv, acc.y * inv);
}

}  // namespace moa
