// moa_device.cuh -- small device-side building blocks shared by the kernels of libmoa:
// mbarrier + bulk-async-copy wrappers (inline PTX, sm_100a), bounded waits, the device
// status word and the work cursor that maps a flat row-block index to (batch, kv head,
// first row).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "moa.h"

namespace moa {

// One status word per device, OR-ed into by kernels, read and cleared by
// moa_device_status().
__device__ int g_status_word;

__device__ __forceinline__ void raise_status(int bits) { atomicOr(&g_status_word, bits); }

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier -------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Non-blocking probe of a phase (try_wait may suspend the thread for a while when the phase
// is not complete; a thread that polls several barriers in turn must not do that).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// ---- programmatic dependent launch ------------------------------------------------------
// The streaming kernels are launched so that the next kernel in the stream may be scheduled
// while this one is still running (its CTAs take the SMs that this kernel's CTAs leave).
// launch_dependents allows that; grid_dependency_wait blocks until the previous kernel in
// the stream has completed and its writes are visible, and is placed before the first read
// of anything that kernel may have written.  Both are no-ops for an ordinary launch.
__device__ __forceinline__ void launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Every spin in this library is bounded: after kWaitLimit unsuccessful polls the caller
// gives up, raises MOA_STATUS_WAIT_TIMEOUT and leaves without touching the data.
constexpr uint32_t kWaitLimit = 1u << 22;

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit = kWaitLimit)
{
    for (uint32_t it = 0; it < limit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// ---- bulk asynchronous copy global -> shared (TMA engine, 1-D) --------------------------
// dst and src 16-byte aligned, bytes a positive multiple of 16.  Completion is signalled
// on the mbarrier as `bytes` transaction bytes.  Every CTA fetches its own tile (plain
// copies into the issuing CTA's shared memory only).
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes,
                                         uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// exp2(a - b) that is 0 when a is -inf (an empty partial), whatever b is.
__device__ __forceinline__ float exp2_diff(float a, float b)
{
    return (a == -INFINITY) ? 0.0f : fast_exp2(a - b);
}

// ---- packed single precision (two fp32 values per instruction, sm_100) --------------------
// The role warps of the tensor-core kernel are bound by instruction issue; additions,
// subtractions and fused multiply-adds on pairs of floats halve those instructions.  Same
// rounding (to nearest) as the scalar instructions, so results do not change.
__device__ __forceinline__ uint64_t pack2(uint32_t lo, uint32_t hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, uint32_t &lo, uint32_t &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

// ---- compensated accumulation for the merges -------------------------------------------
// A merge adds up to a thousand partial triples.  When the softmax mass sits on a few rows,
// one partial is of order 1 and the rest are tiny, and every plain addition would round at
// the size of the large one: the error grows like the square root of the number of
// partials.  The merges therefore keep a running compensation (Kahan): s += x * f with the
// rounding error of each addition carried into the next.
__device__ __forceinline__ void comp_fma(float &s, float &c, float x, float f)
{
    const float y = fmaf(x, f, -c);
    const float t = s + y;
    c = (t - s) - y;
    s = t;
}
__device__ __forceinline__ void comp_fma4(float4 &s, float4 &c, const float4 &x, float f)
{
    comp_fma(s.x, c.x, x.x, f); comp_fma(s.y, c.y, x.y, f);
    comp_fma(s.z, c.z, x.z, f); comp_fma(s.w, c.w, x.w, f);
}

// ---- problem description passed to the decode kernels ----------------------------------
struct DecodeArgs {
    const float *q;           // [batch, h_q, d_k]
    const float *K;           // [batch, h_kv, n_max, d_k]
    const float *V;           // [batch, h_kv, n_max, d_v]
    float *out;               // [batch, h_q, d_v]
    float *ws;                // partial slots (streaming kernels) or nullptr
    const int32_t *seq_lens;  // device [batch] or nullptr (= every length is n_max)
    int32_t len_bias;         // added to every seq_lens[b] (fused step: attend over len+1)
    int batch, h_q;
    int h_kv;                 // kv heads as the kernels count them (virtual heads, see kv_share)
    int g_s;                  // query heads per (virtual) kv head
    int kv_share;             // consecutive virtual kv heads that read the same stored K/V head
    int g_total;              // query heads per stored K/V head (<= kv_share * g_s: the last virtual head of a
                              // stored one may hold fewer than g_s)
    int n_max;                // row capacity of every (batch, kv head) slab
    int d_k, d_v;
    // Element strides of the caches: batch item, stored kv head, row.  The dense layout is
    // (h_kv * n_max * d, n_max * d, d); the 1-D bulk copies need a row stride of exactly d.
    long long k_sb, k_sh, k_sr;
    long long v_sb, v_sh, v_sr;
    float qscale;             // scale * log2(e): scores live in the log2 domain
    // ---- fused step (all null/zero for a plain decode) ----
    float *Kw, *Vw;           // writable K / V when the new row is appended by the decode kernel
    const float *k_new;       // [batch, stored kv heads, d_k] row appended at index seq_lens[b]
    const float *v_new;       // [batch, stored kv heads, d_v]
    int32_t *lens_rw;         // lengths advanced by one when the whole grid is done, or nullptr
    unsigned long long *tickets;   // completion counters (kTicketStride words at the end of the
                                   // workspace), or nullptr: partials are merged by a second kernel
    unsigned long long ticket_tag; // what one arrival adds to a counter word: (launch tag << 20) + 1
    float *partial_out;       // nullptr, or [batch, h_q, d_v + 4]: emit the unnormalised triple
                              // (o[d_v], m, l, 2 pad) instead of the normalised output row
    uint32_t wait_limit;      // polls after which a wait on a tile's arrival gives up (FMA streaming kernel)
    long long skip_copy_block;// test hook: the copies of this row block are announced but never
                              // issued, so the wait for them runs out (-1: off)
};

// Query head (inside its batch item) that is head g of virtual kv head h, or -1 if that slot is
// padding.  The virtual heads of a stored K/V head take its g_total heads in runs of g_s.
// SHORTCUT: take the common case (one virtual head per stored one) without the divisions.  The
// 16-head warp-MMA configuration, which sits at the register limit, is measurably faster (8 %)
// with the one general form, every other kernel with the shortcut.
template <bool SHORTCUT = true>
__device__ __forceinline__ int query_head(const DecodeArgs &a, int h, int g)
{
    if (SHORTCUT && a.kv_share == 1) return g < a.g_s ? h * a.g_s + g : -1;
    const int in_stored = (h % a.kv_share) * a.g_s + g;
    return (g < a.g_s && in_stored < a.g_total) ? (h / a.kv_share) * a.g_total + in_stored : -1;
}

// Final emission of one float4 column group of a (batch, query head) row: the normalised
// output, or -- for a caller that merges several row ranges itself (sequence split across
// GPUs) -- the unnormalised weighted sum with its reference maximum (log2 domain) and sum.
__device__ __forceinline__ void emit_columns(const DecodeArgs &a, size_t bh, int D, int d4, const float4 &acc,
                                             float M, float L)
{
    if (a.partial_out != nullptr) {
        float *dst = a.partial_out + bh * (size_t)(D + 4);
        *reinterpret_cast<float4 *>(dst + d4 * 4) = acc;
        if (d4 == 0) { dst[D] = M; dst[D + 1] = L; }
    } else {
        const float inv = 1.0f / L;
        *reinterpret_cast<float4 *>(a.out + bh * (size_t)D + d4 * 4) =
            make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    }
}

// Completion counters of one launch: word c counts the CTAs that have delivered their
// partial for the split unit whose first segment lies in CTA c; the last word counts CTAs
// that have finished altogether.  The counters live at the end of the workspace the call
// was given, so calls with workspaces of their own never share one.  A workspace's contents
// are undefined on entry, so a counter proves that it belongs to the launch: every arrival
// adds `inc` = (tag << 20) + 1, where tag is a process-wide launch number (44 bits, never
// zero); a word is a live counter of this launch after j arrivals exactly when it equals
// j * inc.  Zero is the state before the first arrival; anything else is a leftover and is
// replaced.  Whoever brings a counter to its final value resets the word to zero, which keeps
// a captured launch (whose tag is frozen) replayable.  The ordinary path is one atomicAdd per
// arrival; the compare-and-swap only runs on a leftover, i.e. once per word of a workspace
// that was handed over uninitialised.
constexpr int kTicketCtas = 1024;
constexpr int kTicketStride = kTicketCtas + 1;
constexpr size_t kTicketBytes = (size_t)kTicketStride * sizeof(unsigned long long);
constexpr unsigned long long kTicketCountMask = (1ull << 20) - 1ull;

// Count one arrival on `word`; returns the number of arrivals of this launch before this one.
__device__ __forceinline__ unsigned ticket_arrive(unsigned long long *word, unsigned long long inc)
{
    unsigned long long old = atomicAdd(word, inc);
    for (;;) {
        const unsigned long long j = old & kTicketCountMask;
        if (old == j * inc) return (unsigned)j;
        // A leftover (to which the increment above was added in vain): claim the word as the
        // first arrival, or count again if another CTA has claimed it meanwhile.
        const unsigned long long seen = *reinterpret_cast<volatile unsigned long long *>(word);
        const unsigned long long js = seen & kTicketCountMask;
        if (seen == js * inc) { old = atomicAdd(word, inc); continue; }
        if (atomicCAS(word, seen, inc) == seen) return 0u;
        old = ~0ull;                            // lost the race: look again
    }
}

// Length of sequence b as the kernels see it; 0 for an out-of-range length (the item is
// then skipped by construction: it owns no row blocks).
__device__ __forceinline__ int seq_len_of(const DecodeArgs &a, int b)
{
    if (a.seq_lens == nullptr) return a.n_max;
    const int len = a.seq_lens[b] + a.len_bias;
    return (len >= 1 && len <= a.n_max) ? len : 0;
}

// ---- work cursor -----------------------------------------------------------------------
// The sequence axis of every (batch b, kv head h) "unit" is cut into row blocks of R
// rows; blocks are numbered unit by unit (b major, h minor).  A cursor remembers the unit
// that contains a block index and can only move forward.
struct Cursor {
    int b, h;          // current unit
    int len;           // rows in this unit's sequence
    int ub;            // row blocks in this unit
    long long first;   // flat index of the unit's first block
};

template <int R>
__device__ __forceinline__ int blocks_of(int len) { return (len + R - 1) / R; }

// Total number of row blocks (warp-collective; every lane gets the result).
template <int R>
__device__ __forceinline__ long long total_blocks(const DecodeArgs &a, int lane)
{
    if (a.seq_lens == nullptr) return (long long)a.batch * a.h_kv * blocks_of<R>(a.n_max);
    long long tot = 0;
    for (int base = 0; base < a.batch; base += 32) {
        const int b = base + lane;
        int nb = (b < a.batch) ? blocks_of<R>(seq_len_of(a, b)) : 0;
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) nb += __shfl_xor_sync(0xffffffffu, nb, off);
        tot += (long long)nb * a.h_kv;
    }
    return tot;
}

// Largest batch whose per-item block prefix is kept in shared memory by the streaming
// kernel (larger batches scan the lengths in global memory instead).
constexpr int kPrefixBatch = 1024;

// Fill pref[0..batch] with the exclusive prefix sum of blocks_of(len_b) (per kv head).
// Called by one full warp; the caller synchronises the block afterwards.
template <int R>
__device__ __forceinline__ void build_block_prefix(const DecodeArgs &a, int *pref, int lane)
{
    int run = 0;
    for (int base = 0; base < a.batch; base += 32) {
        const int b = base + lane;
        const int nb = (b < a.batch) ? blocks_of<R>(seq_len_of(a, b)) : 0;
        int inc = nb;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += t;
        }
        if (b < a.batch) pref[b] = run + inc - nb;
        run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) pref[a.batch] = run;
}

// Position a cursor on the unit containing block j (0 <= j < total).  Warp-uniform.
// `pref` is the shared-memory prefix built by build_block_prefix, or nullptr.
template <int R>
__device__ __forceinline__ Cursor cursor_at(const DecodeArgs &a, long long j, const int *pref = nullptr)
{
    Cursor c;
    if (a.seq_lens != nullptr && pref != nullptr) {
        int lo = 0, hi = a.batch;              // find b with h_kv*pref[b] <= j < h_kv*pref[b+1]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if ((long long)pref[mid] * a.h_kv <= j) lo = mid; else hi = mid;
        }
        while (lo < a.batch - 1 && pref[lo + 1] == pref[lo]) ++lo;   // skip items without blocks
        const int ub = pref[lo + 1] - pref[lo];
        const long long first = (long long)pref[lo] * a.h_kv;
        c.b = lo;
        c.ub = ub;
        c.len = seq_len_of(a, lo);
        c.h = ub > 0 ? (int)((j - first) / ub) : 0;
        c.first = first + (long long)c.h * ub;
        return c;
    }
    if (a.seq_lens == nullptr) {
        const int ub = blocks_of<R>(a.n_max);
        const long long u = j / ub;
        c.b = (int)(u / a.h_kv);
        c.h = (int)(u % a.h_kv);
        c.len = a.n_max;
        c.ub = ub;
        c.first = u * ub;
        return c;
    }
    long long first = 0;
    int b = 0;
    for (; b < a.batch; ++b) {
        const int len = seq_len_of(a, b);
        const int ub = blocks_of<R>(len);
        const long long span = (long long)ub * a.h_kv;
        if (j < first + span) {
            c.b = b;
            c.h = (int)((j - first) / ub);
            c.len = len;
            c.ub = ub;
            c.first = first + (long long)c.h * ub;
            return c;
        }
        first += span;
    }
    c.b = a.batch; c.h = 0; c.len = 0; c.ub = 0; c.first = first;   // past the end
    return c;
}

// Move to the next unit that owns at least one block (or past the end: b == batch).
template <int R>
__device__ __forceinline__ void cursor_next_unit(const DecodeArgs &a, Cursor &c)
{
    c.first += c.ub;
    for (;;) {
        if (++c.h == a.h_kv) {
            c.h = 0;
            if (++c.b >= a.batch) { c.b = a.batch; c.len = 0; c.ub = 0; return; }
            c.len = seq_len_of(a, c.b);
            c.ub = blocks_of<R>(c.len);
        }
        if (c.ub > 0) return;
    }
}

// ---- merge of a split unit's partials by the CTA that delivered the last one -------------
// The partial triples (m, l, o[D]) of the unit live in slots of `a.ws`, one per CTA c in
// [c_first, c_last] (slot 0 or 1 of that CTA: 0 if the unit starts before the CTA's range).
// They are merged in CTA order, so the result does not depend on which CTA does it.  The
// (m, l) pairs are first fetched by all threads at once into `stage` (one L2 round trip
// instead of one per partial); `stage_floats` bounds how many partials are handled per
// round, further rounds continue the same online merge.  Ends with a block barrier.
template <int D, bool SHORTCUT = true>
__device__ __forceinline__ void merge_unit_partials(const DecodeArgs &a, float *stage, int stage_floats, int G,
                                                    long long c_first, long long c_last, long long bpc,
                                                    long long unit_first, int b, int h, int tid, int nthreads)
{
    constexpr int LPR = D / 4, PS = D + 4;
    const int ns = (int)(c_last - c_first) + 1;
    const int per_round = stage_floats / (2 * G);
    auto slot_of = [&](long long c, int hg) {
        const int slot = (unit_first <= c * bpc) ? 0 : 1;
        return a.ws + (((size_t)c * 2 + slot) * G + hg) * PS;
    };
    // thread -> (head, float4 column); with fewer threads than G * LPR a thread takes several
    constexpr int kMaxItems = 4;
    float M[kMaxItems], L[kMaxItems], Lc[kMaxItems];
    float4 acc[kMaxItems], accc[kMaxItems];
#pragma unroll
    for (int it = 0; it < kMaxItems; ++it) {
        M[it] = -INFINITY; L[it] = 0.f; Lc[it] = 0.f;
        acc[it] = make_float4(0.f, 0.f, 0.f, 0.f); accc[it] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int base = 0; base < ns; base += per_round) {
        const int cnt = (ns - base < per_round) ? ns - base : per_round;
        for (int i = tid; i < cnt * G; i += nthreads) {
            const float *p = slot_of(c_first + base + i / G, i % G);
            stage[2 * i] = __ldcg(p + D);
            stage[2 * i + 1] = __ldcg(p + D + 1);
        }
        __syncthreads();
#pragma unroll
        for (int it = 0; it < kMaxItems; ++it) {
            const int idx = tid + it * nthreads;
            if (idx < G * LPR) {
                const int hg = idx / LPR, d4 = idx % LPR;
                float Mn = M[it];
                for (int i = 0; i < cnt; ++i) Mn = fmaxf(Mn, stage[(i * G + hg) * 2]);
                const float keep = exp2_diff(M[it], Mn);
                acc[it].x *= keep; acc[it].y *= keep; acc[it].z *= keep; acc[it].w *= keep;
                accc[it].x *= keep; accc[it].y *= keep; accc[it].z *= keep; accc[it].w *= keep;
                L[it] *= keep; Lc[it] *= keep;
                M[it] = Mn;
#pragma unroll 8
                for (int i = 0; i < cnt; ++i) {      // partials in CTA order; the loads are independent
                    const float f = exp2_diff(stage[(i * G + hg) * 2], Mn);
                    comp_fma(L[it], Lc[it], stage[(i * G + hg) * 2 + 1], f);
                    const float4 x = __ldcg(reinterpret_cast<const float4 *>(slot_of(c_first + base + i, hg) + d4 * 4));
                    comp_fma4(acc[it], accc[it], x, f);
                }
            }
        }
        __syncthreads();                       // the stage is rewritten by the next round / next unit
    }
#pragma unroll
    for (int it = 0; it < kMaxItems; ++it) {
        const int idx = tid + it * nthreads;
        if (idx < G * LPR) {
            const int hg = idx / LPR, d4 = idx % LPR;
            const int qh = query_head<SHORTCUT>(a, h, hg);
            if (qh >= 0) emit_columns(a, (size_t)b * a.h_q + qh, D, d4, acc[it], M[it], L[it]);
        }
    }
}

}  // namespace moa
