// moa_grouped64.cuh -- tensor-core decode kernel for groups of up to 64 query heads per K/V head
// (MQA and large GQA groups), with the small operands (Q, P) resident in tensor memory.
//
// Steps I and III of Algorithm 1 (eqs. (1),(3)) per tile of 128 cached rows, heads on the
// M axis:
//     S[heads x rows] = Q[heads x d] * K_tile^T,      O[heads x d] += P[heads x rows] * V_tile
// on tcgen05.mma (kind::tf32) with the three-term split x = hi + lo that keeps fp32 accuracy.
// The A operand is read from tensor memory: its 128 lanes hold, for every head, one lane with
// the hi part and one lane with the lo part of that head's row ("stacked" operand), so that
//     [Q_hi; Q_lo] * K_hi^T  gives  Q_hi*K_hi  in the hi lanes and  Q_lo*K_hi  in the lo lanes,
//     [Q_hi; Q_lo] * K_lo^T  gives  Q_hi*K_lo  in the hi lanes (and the negligible lo*lo term),
// and likewise for [P_hi; P_lo] and V.  Only the streamed operand (K and V chunks, the B
// operand) lives in shared memory, where it is read once as loaded (the tensor core keeps
// exactly the hi part of an fp32 word) and once after an in-place conversion to its lo part.
// Compared with both operands in shared memory this halves the operand traffic of every
// product and frees 128 KB for the chunk ring, which is what bounds that arrangement.
//
// Lanes: quadrant w (lanes 32w..32w+31) holds heads 16w..16w+15; lane 32w+j (j < 16) the hi
// part of head 16w+j, lane 32w+16+j its lo part.  A thread of the softmax group owns one
// lane, so the two parts of a head meet by one shuffle inside a warp.
//
// Tensor memory (512 columns): Q (128), two score/probability regions (128 each; the
// probabilities of a tile overwrite its scores), O (128).
//
// Accuracy: the tensor core accumulates with truncation, and what a truncation costs is set by
// the size of the accumulator, so small terms are never added on top of large ones.  The K_hi
// products of a tile are read out of its region by the softmax group before the K_lo products
// start the region afresh, and the two are added in fp32 (two chains of 16 steps per score); the
// weighted sum of every tile starts from zero and is folded into fp32 running values held in
// registers (online softmax, eq. (2) with a running maximum per head).
//
// A thread that issues tcgen05.mma cannot look at a barrier without draining the tensor pipe,
// so a scheduler thread does the waiting and releases batches of 16 products by number (all four
// chunks of a group landed -> hi products; their four conversions done -> lo products); the
// issuing thread derives everything else from that number: a chunk group always occupies the
// same four ring buffers, so the descriptors are a run-time base plus compile-time offsets.
//
// Roles (768 threads): warp 0 TMA producer, warp 3 MMA issuer (and owner of the tensor
// memory allocation), warp 22 batch scheduler, warps 4-19 softmax (warp w: lane quadrant w % 4,
// columns 32 * ((w-4)/4) .. +31 of a 128-column region), warps 1, 2, 20, 21 turn chunks into
// their lo parts (none of them on the issuer's scheduler quarter), warp 23 idles.  After the
// set-up the softmax warpgroups take registers from the others (setmaxnreg): they hold the
// running weighted sum and a tile's K_hi products at once.  Every hand-off is an mbarrier;
// every wait is bounded.
#pragma once

#include "moa_grouped.cuh"

namespace moa {

// Bounded wait for the roles that are not on the tensor core's critical path: try_wait lets
// the hardware suspend the thread, so a waiting warp takes no issue slots from the issuer.
__device__ __forceinline__ bool wait_suspended(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 15u) == 15u && *abort_flag) return false;
    }
    *abort_flag = 1;
    raise_status(MOA_STATUS_WAIT_TIMEOUT);
    return false;
}

__device__ __forceinline__ uint4 lds_volatile_v4(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.volatile.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_volatile_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w)
{
    asm volatile("st.volatile.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

struct Grouped64Cfg {
    static constexpr int GH = 64;
    static constexpr int D = 128;
    static constexpr int TILE = 128;
    static constexpr int NBUF = 12;                // 16 KB chunk buffers: three groups of four, so that a group always sits in the same buffers
    static constexpr int NG = 4;                   // groups of four chunks with barriers of their own (> NBUF / 4)
    static constexpr int CHUNK = 16384;
    static constexpr int THREADS = 768;            // 24 warps = 6 warpgroups (register reallocation works on whole warpgroups)
    static constexpr int CONV_WARPS = 4;
    static constexpr int SOFT_WARPS = 16;
    static constexpr int PS = D + 4;
    static constexpr uint32_t OFF_RING = 0;
    static constexpr uint32_t OFF_MX = OFF_RING + NBUF * CHUNK;     // [2 tiles][4 column quarters][64 heads] tile maxima
    static constexpr uint32_t OFF_LX = OFF_MX + 2 * 4 * 64 * 4;     // [4 column quarters][64 heads] sums
    static constexpr uint32_t OFF_BAR = OFF_LX + 4 * 64 * 4;
    static constexpr int NBAR = 2 * NBUF + 2 * NG + 2 + 1 + 1;
    static constexpr uint32_t OFF_TMEM = OFF_BAR + NBAR * 8;
    static constexpr uint32_t OFF_ABORT = OFF_TMEM + 4;
    static constexpr uint32_t OFF_SHARE = OFF_ABORT + 4;            // flat mode: unit, first CTA, CTA count
    static constexpr uint32_t OFF_QCNT = OFF_SHARE + 16;            // batches published / batches taken
    static constexpr size_t SMEM_BYTES = OFF_QCNT + 16;
};

// Batch number -> what it multiplies: operand kind, hi or lo pass, tile, chunk group (ring order).
struct Batch64 {
    bool is_k, is_hi;
    int t, g;
    __device__ __forceinline__ Batch64(int i, int T)
    {
        if (i < 2) { is_k = true; t = 0; is_hi = (i == 0); }
        else {
            const int jj = i - 2, r = jj & 3;
            t = jj >> 2;
            if (t >= T - 1) { is_k = false; t = T - 1; is_hi = (r == 0); }
            else { is_k = (r == 0 || r == 2); is_hi = (r < 2); if (is_k) t += 1; }
        }
        g = is_k ? (t == 0 ? 0 : 2 * t - 1) : (t < T - 1 ? 2 * t + 2 : 2 * T - 1);
    }
};

// The sixteen products of one batch: group slot SLOT of the ring (buffers 4*SLOT .. 4*SLOT+3), K
// chunks (K-major B operand) or V chunks (MN-major).  `ring_lo` is the ring's shared-memory
// address >> 4; all other descriptor fields are constants.  Issued by one thread.
template <bool IS_K, int SLOT>
__device__ __forceinline__ void issue_batch64(uint32_t d, uint32_t a0, uint32_t ring_lo, uint32_t acc0,
                                              uint32_t bar_first, uint32_t bar_mid, uint32_t bar_end)
{
    // descriptor words: [addr>>4 | lbo>>4 << 16] and [sbo>>4 | version << 14 | layout << 29]
    constexpr uint32_t hiword = IS_K ? (64u | (1u << 14) | (2u << 29)) : (32u | (1u << 14) | (1u << 29));
    constexpr uint32_t lbo = IS_K ? (1u << 16) : (256u << 16);
    constexpr uint32_t step = IS_K ? 2u : 64u;                       // descriptor step per k-step
    constexpr uint32_t idesc = tc::idesc_tf32(128, 128, false, !IS_K);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (uint32_t ks = 0; ks < 4; ++ks) {
            const uint32_t lo = ring_lo + (lbo + (uint32_t)(4 * SLOT + c) * (Grouped64Cfg::CHUNK >> 4) + ks * step);
            tc::mma_tf32_ts(d, a0 + (32u * c + 8u * ks), tc::pack64(lo, hiword), idesc, (c == 0 && ks == 0) ? acc0 : 1u);
        }
        // hi batch: one commit per pair of chunks (bar_first = 0: none after chunks 0 and 2);
        // lo batch: one per chunk, so that the producer can refill buffer by buffer
        if (bar_first != 0u) tc::mma_commit(bar_first + 8u * (uint32_t)c);
        else if (c == 1) tc::mma_commit(bar_mid);
    }
    if (bar_first == 0u) tc::mma_commit(bar_end);
}

__global__ void __launch_bounds__(Grouped64Cfg::THREADS, 1)
grouped64_decode_kernel(const __grid_constant__ CUtensorMap tmapK, const __grid_constant__ CUtensorMap tmapV,
                        const __grid_constant__ CUtensorMap tmapKt, const __grid_constant__ CUtensorMap tmapVt,
                        const GroupedArgs a)
{
    using C = Grouped64Cfg;
    constexpr int GH = C::GH, NBUF = C::NBUF, NG = C::NG, PS = C::PS;
    extern __shared__ __align__(1024) unsigned char smem_g64[];
    unsigned char *const smem = smem_g64;
    float *mx = reinterpret_cast<float *>(smem + C::OFF_MX);
    float *lx = reinterpret_cast<float *>(smem + C::OFF_LX);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + C::OFF_BAR);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::OFF_TMEM);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_ABORT);
    int *s_share = reinterpret_cast<int *>(smem + C::OFF_SHARE);
    volatile int *q_ready = reinterpret_cast<volatile int *>(smem + C::OFF_QCNT);

    const uint32_t sRing = smem_u32(smem) + C::OFF_RING;
    // Per ring buffer (every role sees every use of every buffer, so one parity bit per use):
    auto bar_hi = [&](int b) { return smem_u32(&bars[b]); };                 // the chunk's hi product is complete
    auto bar_empty = [&](int b) { return smem_u32(&bars[NBUF + b]); };       // its lo product is complete
    // Per group of four chunks (group g uses slot g % NG; the ring holds fewer than NG groups):
    auto bar_gfull = [&](int g) { return smem_u32(&bars[2 * NBUF + g]); };            // all four chunks landed
    auto bar_glo = [&](int g) { return smem_u32(&bars[2 * NBUF + NG + g]); };         // all four lo parts in place
    auto bar_pfull = [&](int s) { return smem_u32(&bars[2 * NBUF + 2 * NG + s]); };   // probabilities stored
    const uint32_t bar_ofree = smem_u32(&bars[2 * NBUF + 2 * NG + 2]);                // weighted sum of a tile folded
    const uint32_t bar_shread = smem_u32(&bars[2 * NBUF + 2 * NG + 3]);               // K_hi products of a tile read out

    // "The product of a whole tile is complete" is the completion of the lo product of the last
    // chunk of its group (a second tcgen05.commit at the end of a batch costs the issuer about
    // 250 cycles of tensor time, measured).  Group index of the K / V chunks of tile t in ring
    // order; ring buffer and use count of a group's last chunk.
    auto group_k = [](int t) { return t == 0 ? 0 : 2 * t - 1; };
    auto group_v = [](int t, int tiles) { return t < tiles - 1 ? 2 * t + 2 : 2 * tiles - 1; };
    auto bar_group_done = [&](int g) { return bar_empty((4 * g + 3) % NBUF); };
    auto par_group_done = [](int g) { return (uint32_t)((4 * g + 3) / Grouped64Cfg::NBUF) & 1u; };
    auto bar_group_hi = [&](int g) { return bar_hi((4 * g + 3) % NBUF); };            // ... of its hi products (same parity)
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int split = (int)blockIdx.x % a.splits;
    int sunit = (int)blockIdx.x / a.splits;                       // stored (batch, kv head)
    int splits_u = a.splits;
    if (a.flat) {                                  // warp 0 walks the lengths, all take its answer
        if (warp == 0) {
            const FlatShare f = flat_share(a, (int)gridDim.x, (int)blockIdx.x, -1, lane);
            if (lane == 0) { s_share[0] = f.unit; s_share[1] = f.first; s_share[2] = f.count; }
        }
        __syncthreads();
        if (s_share[0] < 0) return;
        sunit = s_share[0]; split = (int)blockIdx.x - s_share[1]; splits_u = s_share[2];
    }
    // pair mode: `sunit` counts virtual kv heads (a.share per stored one, 32 query heads each)
    const int unit = a.pair ? sunit / a.share : sunit;              // tensor-map coordinate: stored (batch, kv head)
    const int b = a.pair ? sunit / a.h_kv : sunit / a.h_kv_stored;
    const int h = a.pair ? sunit % a.h_kv : sunit % a.h_kv_stored;  // (virtual) kv head inside the batch item
    const int len_b = grouped_len(a, b);           // 0: out-of-range length, the item is skipped
    const int rows_b = grouped_len_rows(a, b);     // (pair mode: cached rows of 64 features)
    const int tiles_total = (len_b + C::TILE - 1) / C::TILE;
    const int tiles_per_split = a.seq_lens ? (tiles_total + splits_u - 1) / splits_u : a.tiles_per_split;
    const int tile0 = split * tiles_per_split;
    int T = tiles_total - tile0;
    if (T > tiles_per_split) T = tiles_per_split;
    if (T <= 0) return;                            // an empty split (uniform for the CTA)
    const int tail_t = (a.tailK != nullptr) ? tiles_total - 1 - tile0 : -1;
    const int row_base = tile0 * C::TILE;
    // ---- set-up --------------------------------------------------------------------------
    if (tid == 0) {
        for (int i = 0; i < NBUF; ++i) { mbar_init(bar_hi(i), 1); mbar_init(bar_empty(i), 1); }
        for (int g = 0; g < NG; ++g) {
            mbar_init(bar_gfull(g), 4);            // one arrival (with its byte count) per chunk
            mbar_init(bar_glo(g), 4);              // one warp per chunk
        }
        for (int i = 0; i < 2; ++i) mbar_init(bar_pfull(i), C::SOFT_WARPS);
        mbar_init(bar_ofree, C::SOFT_WARPS); mbar_init(bar_shread, C::SOFT_WARPS);
        mbar_fence_init();
        *abort_flag = 0;
        *q_ready = 0;
        tc::prefetch_tmap(&tmapK);
        tc::prefetch_tmap(&tmapV);
        if (a.tailK != nullptr) { tc::prefetch_tmap(&tmapKt); tc::prefetch_tmap(&tmapVt); }
    }
    if (warp == 3) tc::tmem_alloc(smem_u32(tmem_slot), 512);
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    // Launched with programmatic stream serialisation, this kernel may start while its
    // predecessor in the stream is still running (the streaming kernels let their successor go
    // early).  With a tail-copy kernel in front, that kernel is the only one (it was launched
    // after everything before it had completed) and only the tail tiles come from it; without
    // one, wait here, before the first access to global memory.
    if (a.tailK == nullptr) grid_dependency_wait();
    // The first ring-full of chunks needs nothing but the barriers: the producer starts those
    // loads now, so that they travel while the query operand is being built.
    ChunkSeq pseq(T);                              // the producer's position (warp 0, lane 0)
    bool tail_ready = false;                       // the grid that wrote the tail copies is complete
    auto issue_load = [&](const ChunkSeq &s) {
        const int buf = s.seq % NBUF;
        const uint32_t dst = sRing + (uint32_t)buf * C::CHUNK;
        const uint32_t fb = bar_gfull((s.seq >> 2) % NG);
        mbar_expect_tx(fb, C::CHUNK);
        const bool tail = (s.t == tail_t);
        const int row = tail ? 0 : row_base + s.t * C::TILE;
        // Launched with programmatic stream serialisation, this kernel may have started while the
        // tail-copy kernel before it was still running; nothing else it reads comes from there.
        if (tail && !tail_ready) { grid_dependency_wait(); tail_ready = true; }
        if (s.is_k) {
            tc::tma_load_3d(dst, tail ? &tmapKt : &tmapK, 32 * s.c, row, unit, fb);
        } else {
            for (int dg = 0; dg < 4; ++dg)
                tc::tma_load_3d(dst + dg * 4096, tail ? &tmapVt : &tmapV, 32 * dg, row + 32 * s.c, unit, fb);
        }
    };
    if (warp == 0 && lane == 0)
        for (; !pseq.done && pseq.seq < NBUF; pseq.next()) issue_load(pseq);
    const uint32_t tmem = *tmem_slot;
    const uint32_t tQ = tmem, tO = tmem + 384u;
    auto tSP_of = [tmem](int t) -> uint32_t { return tmem + 128u + (uint32_t)(t & 1) * 128u; };

    // softmax-group coordinates (also used for the Q operand, which that group writes)
    const bool is_soft = warp >= 4 && warp < 20;
    const int qd = warp & 3;                       // lane quadrant
    const int sub = (warp - 4) >> 2;               // which 32 columns of a 128-column region
    const int col0 = 32 * sub;
    const uint32_t lane_addr = (uint32_t)(qd * 32) << 16;
    const int head = 16 * qd + (lane & 15);
    const bool is_lo = (lane & 16) != 0;
    // rows (of 128) this lane's head attends over: in pair mode pseudo-head 2j sees the even cached
    // rows, pseudo-head 2j+1 the odd ones, so an odd length gives the latter one row less
    const int len_m = a.pair ? (rows_b + 1 - (head & 1)) >> 1 : len_b;
    if (is_soft) {
        // Q operand: this lane's part (hi or lo) of (scale * log2 e) * q[head], columns = features
        // (a group of fewer than 64 heads is padded: the lanes of the missing heads hold zeros)
        // Pair mode (rows of 64 features, two cached rows per 128-wide row): pseudo-head 2j holds
        // q of head j in features 0..63 and zeros in 64..127 (it sees the even cached rows),
        // pseudo-head 2j+1 the other way round.
        const int qhead = a.pair ? head >> 1 : head;
        // pair mode: head inside its stored K/V head (virtual head h % share of stored head h / share)
        const int q_in_stored = a.pair ? (h % a.share) * a.g_s + qhead : 0;
        const bool has_q = qhead < a.g_s && (!a.pair || ((sub >> 1) == (head & 1) && q_in_stored < a.g_total));
        const float *qb = a.pair ? a.q + ((size_t)b * a.h_q + (size_t)(h / a.share) * a.g_total + q_in_stored) * 64 + 32 * (sub & 1)
                                 : a.q + ((size_t)b * a.h_q + (size_t)h * a.g_s + head) * 128 + col0;
        uint32_t v[32];
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
            const float4 x4 = has_q ? *reinterpret_cast<const float4 *>(qb + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            const float xs[4] = {x4.x * a.qscale, x4.y * a.qscale, x4.z * a.qscale, x4.w * a.qscale};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float hi = tf32_rn(xs[k]);
                v[i + k] = __float_as_uint(is_lo ? tf32_rn(xs[k] - hi) : hi);
            }
        }
        tc::tmem_st32(tQ + lane_addr + col0, v);
        tc::tmem_st_wait();
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    // 24 warps x 80 registers at launch; the two warpgroups without softmax work (warps 0-3 and
    // 20-23) hand 32 registers per thread back to the pool of the CTA, from which the four softmax warpgroups
    // take 16 each (only registers that were handed back can be taken).
    if (!is_soft) asm volatile("setmaxnreg.dec.sync.aligned.u32 48;");

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            for (; !pseq.done; pseq.next()) {
                const int buf = pseq.seq % NBUF, use = pseq.seq / NBUF;
                if (use > 0 && !wait_suspended(bar_empty(buf), (uint32_t)(use - 1) & 1u, abort_flag)) break;
                issue_load(pseq);
            }
        }
    } else if (warp == 22) {
        // ================= batch scheduler (one thread) =================
        // The thread that issues tcgen05.mma cannot look at a barrier between two products without
        // draining the tensor pipe, so the waiting is done here.  Batches of 16 products, in the order
        //     K_hi(0) K_lo(0)  [K_hi(t+1) V_hi(t) K_lo(t+1) V_lo(t)] for t = 0..T-2  V_hi(T-1) V_lo(T-1):
        // between the hi and the lo batch of a group runs a batch of the other operand, which is
        // the time the converters have.  Batch i is released (q_ready = i + 1) once everything
        // it reads is complete; the issuer derives the rest from i.
        if (lane == 0) {
            const int nbatch = 4 * T;
            bool ok = true;
            for (int i = 0; ok && i < nbatch; ++i) {
                const Batch64 bt(i, T);
                const int gs = bt.g % NG;
                const uint32_t gpar = (uint32_t)(bt.g / NG) & 1u;
                // hi products need the four chunks (a weighted sum also the tile's probabilities and
                // the fold of the previous tile's weighted sum, which the softmax group does after
                // storing the probabilities); lo products the four conversions
                if (bt.is_hi) {
                    ok = wait_or_abort(bar_gfull(gs), gpar, abort_flag);
                    if (ok && !bt.is_k)
                        ok = (bt.t > 0) ? wait_or_abort(bar_ofree, (uint32_t)(bt.t - 1) & 1u, abort_flag)
                                        : wait_or_abort(bar_pfull(0), 0u, abort_flag);
                } else {
                    ok = wait_or_abort(bar_glo(gs), gpar, abort_flag);
                    // the K_lo products overwrite the K_hi products of the tile: those must have been read
                    if (ok && bt.is_k) ok = wait_or_abort(bar_shread, (uint32_t)bt.t & 1u, abort_flag);
                }
                if (!ok) break;
                __threadfence_block();
                *q_ready = i + 1;
            }
        }
    } else if (warp == 3) {
        // ================= MMA issuer (one thread) =================
        // Everything a batch needs is a function of its number: operand (K or V), tile, group and
        // with it the ring buffers (a group always occupies the same four), so the sixteen
        // descriptors of a batch are one run-time base plus compile-time offsets.  Commits: a hi
        // batch signals after its second and its fourth chunk (the converters of a pair of chunks
        // wait for the pair), a lo batch after every chunk (the producer refills buffer by buffer:
        // a group-wise refill starts the loads too late to cover their latency).
        if (lane == 0) {
            const int nbatch = 4 * T;
            const uint32_t ring_lo = sRing >> 4;
            bool ok = true;
            for (int i = 0; ok && i < nbatch; ++i) {
                const Batch64 bt(i, T);
                const uint32_t d = bt.is_k ? tSP_of(bt.t) : tO;
                const uint32_t a0 = bt.is_k ? tQ : tSP_of(bt.t);
                const uint32_t acc0 = (bt.is_hi || bt.is_k) ? 0u : 1u;    // only the V_lo products continue an accumulation
                const int slot = bt.g % 3, buf0 = 4 * slot;
                const uint32_t bar_first = bt.is_hi ? 0u : bar_empty(buf0);     // lo batch: barriers of the four buffers (8 bytes apart)
                const uint32_t bar_mid = bar_hi(buf0 + 1), bar_end = bar_hi(buf0 + 3);
                for (uint32_t it = 0; *q_ready <= i; ++it)             // the operands of this batch are complete
                    if (it >= kWaitLimit || ((it & 255u) == 255u && *abort_flag)) {
                        if (it >= kWaitLimit) { *abort_flag = 1; raise_status(MOA_STATUS_WAIT_TIMEOUT); }
                        ok = false;
                        break;
                    }
                if (!ok) break;
                __threadfence_block();
                tc::fence_after_sync();
                switch ((bt.is_k ? 0 : 3) + slot) {
                case 0: issue_batch64<true, 0>(d, a0, ring_lo, acc0, bar_first, bar_mid, bar_end); break;
                case 1: issue_batch64<true, 1>(d, a0, ring_lo, acc0, bar_first, bar_mid, bar_end); break;
                case 2: issue_batch64<true, 2>(d, a0, ring_lo, acc0, bar_first, bar_mid, bar_end); break;
                case 3: issue_batch64<false, 0>(d, a0, ring_lo, acc0, bar_first, bar_mid, bar_end); break;
                case 4: issue_batch64<false, 1>(d, a0, ring_lo, acc0, bar_first, bar_mid, bar_end); break;
                default: issue_batch64<false, 2>(d, a0, ring_lo, acc0, bar_first, bar_mid, bar_end); break;
                }
            }
        }
    } else if (is_soft) {
        // ================= softmax group: thread = (lane of the stacked operand, 32 columns) ==========
        asm volatile("setmaxnreg.inc.sync.aligned.u32 96;");
        uint64_t Om[16];                           // running weighted sum: this lane's part, features col0..col0+31, in pairs
#pragma unroll
        for (int i = 0; i < 16; ++i) Om[i] = 0ull;
        float m_run = -INFINITY, l_run = 0.f, alpha_prev = 0.f;
        bool ok = true;
        auto fold = [&](float alpha) {             // Om = alpha * Om + (weighted sum of the last tile)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                uint32_t o[16];
                tc::tmem_ld16(tO + lane_addr + col0 + 16 * hf, o);
                tc::tmem_ld_wait();
                const uint64_t al2 = pack2(__float_as_uint(alpha), __float_as_uint(alpha));
#pragma unroll
                for (int i = 0; i < 8; ++i) Om[8 * hf + i] = fma2(Om[8 * hf + i], al2, pack2(o[2 * i], o[2 * i + 1]));
            }
        };
        for (int t = 0; t < T; ++t) {
            const uint32_t tSP = tSP_of(t) + lane_addr + col0;
            const int row0 = row_base + t * C::TILE + col0;
            float sc[16];                              // scores: the hi lane of a head columns 0..15, the lo lane 16..31
            // Scores of this lane's head against 32 cached rows.  The two lanes of a head hold the
            // terms of its hi and of its lo query part; they share the work: the hi lane takes
            // columns 0..15, the lo lane columns 16..31, each gets the other lane's terms for its
            // columns by shuffle and hands back the part of the probabilities the other lane stores.
            {
                // the K_hi products of the tile are read out before the K_lo products start the
                // region afresh; the two are added here in fp32
                uint32_t xa[32];
                ok = ok && wait_suspended(bar_group_hi(group_k(t)), par_group_done(group_k(t)), abort_flag);
                tc::fence_after_sync();                // (after a failed wait the values are not used)
                tc::tmem_ld32(tSP, xa);
                tc::tmem_ld_wait();
                tc::fence_before_sync();
                __syncwarp();
                if (ok && lane == 0) tc::mbar_arrive(bar_shread);
                ok = ok && wait_suspended(bar_group_done(group_k(t)), par_group_done(group_k(t)), abort_flag);
                // (a warp whose wait has failed keeps walking through the tiles with the others, so that
                // the barriers of its quadrant stay balanced; every later wait returns at once)
                tc::fence_after_sync();
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {       // 16 columns at a time, to stay within the registers
                    uint32_t xb[16];
                    tc::tmem_ld16(tSP + 16 * hf, xb);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        unpack2(add2(pack2(xa[16 * hf + 2 * i], xa[16 * hf + 2 * i + 1]), pack2(xb[2 * i], xb[2 * i + 1])),
                                xa[16 * hf + 2 * i], xa[16 * hf + 2 * i + 1]);
                }
#pragma unroll
                for (int i = 0; i < 16; i += 2) {    // each lane sends what the other needs; sums two at a time
                    const uint32_t o0 = __shfl_xor_sync(0xffffffffu, is_lo ? xa[i] : xa[16 + i], 16);
                    const uint32_t o1 = __shfl_xor_sync(0xffffffffu, is_lo ? xa[i + 1] : xa[17 + i], 16);
                    uint32_t s0, s1;
                    unpack2(add2(pack2(is_lo ? xa[16 + i] : xa[i], is_lo ? xa[17 + i] : xa[i + 1]), pack2(o0, o1)), s0, s1);
                    sc[i] = __uint_as_float(s0);
                    sc[i + 1] = __uint_as_float(s1);
                }
            }
            float vmax = -INFINITY;
            const int rowc = row0 + (is_lo ? 16 : 0);
            const bool full_tile = (row0 + 32 <= len_m);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                if (!full_tile && rowc + i >= len_m) sc[i] = -INFINITY;
                vmax = fmaxf(vmax, sc[i]);
            }
            vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, 16));
            // maximum over the tile: the other columns belong to the other warps of the quadrant
            float *mxt = mx + (t & 1) * 256;
            if (!is_lo) mxt[sub * 64 + head] = vmax;
            named_sync(1 + qd, 128);
            // (never -inf: in pair mode a sequence of one row leaves the odd pseudo-heads without a score)
            const float m_new = fmaxf(fmaxf(fmaxf(m_run, mxt[head]), fmaxf(fmaxf(mxt[64 + head], mxt[128 + head]), mxt[192 + head])),
                                      -3.0e38f);
            const float alpha = exp2_diff(m_run, m_new);
            m_run = m_new;
            // probabilities of this lane's 16 columns, split: the lane keeps its own part (hi or lo)
            // and hands the other part to the other lane of the head; 16 columns at a time (the hi
            // lane's columns first), to stay within the registers
            float lsum;
            {
                uint32_t x[32];
                const uint64_t m2 = pack2(__float_as_uint(m_new), __float_as_uint(m_new));
                uint64_t ls2 = 0ull;
#pragma unroll
                for (int i = 0; i < 16; i += 2) {       // two columns at a time (packed subtractions and additions)
                    uint32_t d0, d1;
                    unpack2(sub2(pack2(__float_as_uint(sc[i]), __float_as_uint(sc[i + 1])), m2), d0, d1);
                    const float p0 = fast_exp2(__uint_as_float(d0)), p1 = fast_exp2(__uint_as_float(d1));
                    const uint64_t p2 = pack2(__float_as_uint(p0), __float_as_uint(p1));
                    ls2 = add2(ls2, p2);
                    const uint64_t ph2 = p2 & 0xFFFFE000FFFFE000ull;          // hi parts (what the tensor core keeps)
                    uint32_t ph0, ph1, pl0, pl1;
                    unpack2(ph2, ph0, ph1);
                    unpack2(sub2(p2, ph2), pl0, pl1);
                    const uint32_t g0 = __shfl_xor_sync(0xffffffffu, is_lo ? ph0 : pl0, 16);
                    const uint32_t g1 = __shfl_xor_sync(0xffffffffu, is_lo ? ph1 : pl1, 16);
                    x[i] = is_lo ? g0 : ph0;                                   // columns 0..15: own (hi lane) or received (lo lane)
                    x[i + 1] = is_lo ? g1 : ph1;
                    x[16 + i] = is_lo ? pl0 : g0;                              // columns 16..31
                    x[16 + i + 1] = is_lo ? pl1 : g1;
                }
                uint32_t l0, l1;
                unpack2(ls2, l0, l1);
                lsum = __uint_as_float(l0) + __uint_as_float(l1);
                tc::tmem_st32(tSP, x);
            }
            tc::tmem_st_wait();
            tc::fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(bar_pfull(t & 1));
            l_run = fmaf(l_run, alpha, lsum);
            // fold the previous tile's weighted sum into the running values
            if (t > 0) {
                ok = wait_suspended(bar_group_done(group_v(t - 1, T)), par_group_done(group_v(t - 1, T)), abort_flag);
                if (ok) {
                    tc::fence_after_sync();
                    fold(alpha_prev);
                    tc::fence_before_sync();
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(bar_ofree);
                }
            }
            alpha_prev = alpha;
        }
        // ---- epilogue: last fold, then this split's partial (m, l, o) per head
        if (ok) ok = wait_suspended(bar_group_done(group_v(T - 1, T)), par_group_done(group_v(T - 1, T)), abort_flag);
        if (named_or(1 + qd, 128, !ok)) ok = false;
        if (ok) {
            tc::fence_after_sync();
            fold(alpha_prev);
            const float l_pair = l_run + __shfl_xor_sync(0xffffffffu, l_run, 16);   // each lane summed 16 of the 32 columns
            if (!is_lo) lx[sub * 64 + head] = l_pair;
            named_sync(1 + qd, 128);
            const bool qhead_ok = a.pair ? ((head >> 1) < a.g_s && (h % a.share) * a.g_s + (head >> 1) < a.g_total)
                                         : head < a.g_s;
            float *slot = (a.flat ? a.ws + ((size_t)blockIdx.x * GH) * PS
                                  : a.ws + ((((size_t)b * a.h_kv + h) * a.splits + split) * GH) * PS) + (size_t)head * PS;
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
                uint32_t w[4];
                unpack2(Om[i / 2], w[0], w[1]);
                unpack2(Om[i / 2 + 1], w[2], w[3]);
                float4 v;
                v.x = __uint_as_float(w[0]) + __shfl_xor_sync(0xffffffffu, __uint_as_float(w[0]), 16);
                v.y = __uint_as_float(w[1]) + __shfl_xor_sync(0xffffffffu, __uint_as_float(w[1]), 16);
                v.z = __uint_as_float(w[2]) + __shfl_xor_sync(0xffffffffu, __uint_as_float(w[2]), 16);
                v.w = __uint_as_float(w[3]) + __shfl_xor_sync(0xffffffffu, __uint_as_float(w[3]), 16);
                if (!is_lo && qhead_ok) *reinterpret_cast<float4 *>(slot + col0 + i) = v;
            }
            if (sub == 0 && !is_lo && qhead_ok) {
                slot[128] = m_run;
                slot[129] = (lx[head] + lx[64 + head]) + (lx[128 + head] + lx[192 + head]);
            }
        }
    } else if (warp != 23) {
        // ================= converters: chunk -> its lo part, in place =================
        // Each of the four converter warps takes every fourth chunk, so that four conversions are in flight: a
        // conversion is a chain of barrier wait, 16 KB of loads, 16 KB of stores and barrier
        // arrival, and one team alone (about 750 cycles per chunk, 8 chunks per tile) was what the
        // lo batches waited for.
        constexpr int TT = 32;                                         // threads of a team
        constexpr int PER = (C::CHUNK / 16) / TT;                      // float4 every thread handles
        const int team = (warp < 4) ? warp - 1 : warp - 18;           // warps 1, 2, 20, 21
        const int ct = lane;
        bool ok = true;
        for (ChunkSeq s(T); ok && !s.done; s.next()) {
            if ((s.seq & 3) != team) continue;
            const int buf = s.seq % NBUF, use = s.seq / NBUF;
            ok = wait_suspended(bar_hi(buf | 1), (uint32_t)use & 1u, abort_flag);    // one commit per pair of chunks
            if (!ok) break;
            float4 *p = reinterpret_cast<float4 *>(smem + C::OFF_RING + (uint32_t)buf * C::CHUNK);
#pragma unroll
            for (int part = 0; part < 4; ++part) {
                float4 v[PER / 4];
#pragma unroll
                for (int i = 0; i < PER / 4; ++i) v[i] = p[ct + (part * (PER / 4) + i) * TT];
#pragma unroll
                for (int i = 0; i < PER / 4; ++i) {       // lo = x - hi(x), two floats per instruction
                    const uint64_t a01 = pack2(__float_as_uint(v[i].x), __float_as_uint(v[i].y));
                    const uint64_t a23 = pack2(__float_as_uint(v[i].z), __float_as_uint(v[i].w));
                    uint32_t w[4];
                    unpack2(sub2(a01, a01 & 0xFFFFE000FFFFE000ull), w[0], w[1]);
                    unpack2(sub2(a23, a23 & 0xFFFFE000FFFFE000ull), w[2], w[3]);
                    p[ct + (part * (PER / 4) + i) * TT] = make_float4(__uint_as_float(w[0]), __uint_as_float(w[1]),
                                                                      __uint_as_float(w[2]), __uint_as_float(w[3]));
                }
            }
            tc::fence_async_smem();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(bar_glo((s.seq >> 2) % NG));
        }
    }

    tc::fence_before_sync();
    __syncthreads();
    launch_dependents();                           // the combine kernel may be scheduled; it waits for this grid itself
    if (warp == 3) tc::tmem_dealloc(tmem, 512);
}

}  // namespace moa
