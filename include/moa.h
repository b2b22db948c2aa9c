/*
 * moa.h -- C ABI of libmoa: single-query decode attention over a KV cache on one
 * NVIDIA B200 (sm_100a), with GQA/MQA head grouping and the O(d_k+d_v) cache append.
 *
 * What is computed (per batch item b and query head g, fp32, row-major):
 *     g_kv   = g / (h_q / h_kv)                         GQA psi-selection (section 6.1)
 *     s[l]   = scale * sum_j q[b,g,j] * K[b,g_kv,l,j]   Step I,   eq. (1)
 *     a[l]   = exp(s[l]-max s) / sum_l exp(s[l]-max s)  Step II,  eq. (2)
 *     out[b,g,d] = sum_l a[l] * V[b,g_kv,l,d]           Step III, eq. (3)  (Algorithm 1)
 * and the append  K[b,h,pos_b,:] <- k_new[b,h,:],  V likewise      eqs. (4),(5).
 *
 * Conventions
 *  - Unless a parameter says HOST, every pointer is a DEVICE pointer on the current
 *    device, owned by the caller; the library never frees or retains it.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls
 *    enqueue work on it and return without synchronising, unless stated otherwise.
 *  - Every step runs in CUDA kernels of this library.  There is no CPU fallback: on a
 *    machine without a usable GPU the compute entry points return MOA_ERR_CUDA.
 *  - Arguments are validated on the host before anything is launched; on a non-zero
 *    return nothing has been written.
 *  - Results are deterministic: no floating-point atomics, fixed merge order.
 *  - Threads: every entry point may be called from any host thread; the library's host
 *    state is guarded by one internal lock (calls are serialised on the host while they
 *    enqueue their work; moa_decode_attn_host holds the lock until its copies are done).
 *    Calls that can overlap on the GPU must not share a workspace: the entry points that
 *    take no workspace argument share one library-owned buffer per device and therefore
 *    must be ordered with respect to each other (one stream, or events between streams).
 *    moa_set_option changes process-wide state and is meant for tests and tuning runs.
 */
#ifndef MOA_H
#define MOA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- return codes ---------------------------------------------------------------- */
#define MOA_OK               0
#define MOA_ERR_INVALID      1  /* null pointer, dimension < 1, h_q % h_kv != 0, non-finite scale */
#define MOA_ERR_UNSUPPORTED  2  /* d_k or d_v above the compiled maximum (MOA_MAX_DK / MOA_MAX_DV) */
#define MOA_ERR_ALIGN        3  /* a float pointer that is not 4-byte aligned */
#define MOA_ERR_CAPACITY     4  /* a size beyond a fixed capacity known on the host */
#define MOA_ERR_WORKSPACE    5  /* workspace missing or smaller than moa_workspace_bytes() */
#define MOA_ERR_CUDA         6  /* a CUDA runtime call failed (no device, launch error, ...) */

#define MOA_MAX_DK 1024
#define MOA_MAX_DV 512

/* ---- device status bits (see moa_device_status) ----------------------------------- */
#define MOA_STATUS_APPEND_RANGE  1  /* append: pos[b] outside [0,n_max); that row was skipped */
#define MOA_STATUS_SEQLEN_RANGE  2  /* decode: seq_lens[b] outside [1,n_max]; that item's out untouched */
#define MOA_STATUS_WAIT_TIMEOUT  4  /* a bounded in-kernel wait expired; results of that call are invalid */

/*
 * Decode attention over a dense cache (problem statement of section 2; batch/head
 * lifting of section 2 "Formal Inputs"; GQA of section 6).
 *   q   [batch, h_q,  d_k]       K [batch, h_kv, n, d_k]
 *   out [batch, h_q,  d_v]       V [batch, h_kv, n, d_v]
 * n >= 1 cached tokens.  `scale` is applied once, to the dot product (any finite value).
 * Scratch for split-sequence partial results comes from a per-device buffer owned by
 * the library (allocated on first use, outside any stream capture; grown on demand;
 * released by moa_release).  Calls that may overlap on one device must instead use
 * moa_decode_attn_varlen with their own workspace.
 */
int moa_decode_attn(const float *q, const float *K, const float *V, float *out,
                    int batch, int h_q, int h_kv, int n, int d_k, int d_v,
                    float scale, void *stream);

/*
 * Decode attention over a pre-allocated cache with per-sequence lengths (the cache of
 * section 5.3 lifted over a batch): K [batch,h_kv,n_max,d_k], V [batch,h_kv,n_max,d_v];
 * sequence b attends over rows [0, seq_lens[b]).  seq_lens is a device int32[batch]
 * read by the kernels at execution time (so a captured graph can be replayed while the
 * lengths advance) and never modified.  seq_lens == NULL means every length is n_max.
 * A length outside [1, n_max] sets MOA_STATUS_SEQLEN_RANGE and leaves that item's rows
 * of `out` untouched.
 * `workspace`: device memory, 256-byte aligned, at least moa_workspace_bytes(...) bytes,
 * owned by the caller, contents undefined on entry and exit (it holds the partial results
 * of split sequences and the completion counters of the in-kernel merge, which tolerate
 * arbitrary initial contents); it must not be shared by calls that can overlap on the
 * GPU.  The call allocates nothing.
 */
int moa_decode_attn_varlen(const float *q, const float *K, const float *V, float *out,
                           int batch, int h_q, int h_kv, const int32_t *seq_lens,
                           int n_max, int d_k, int d_v, float scale,
                           void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same decode for `layers` independent caches of one shape (the per-token accounting of
 * the paper's introduction counts one such call per transformer layer): q, K, V, out are
 * HOST arrays of `layers` device pointers, each with the layout of moa_decode_attn.  The
 * launches go to `stream` back to back; the first error is returned and later layers are
 * not launched.  (In a real model the layers of one token depend on each other; this entry
 * point is for measuring the attention traffic of a whole token in one call.)
 */
int moa_decode_attn_layers(const float *const *q, const float *const *K, const float *const *V,
                           float *const *out, int layers, int batch, int h_q, int h_kv, int n,
                           int d_k, int d_v, float scale, void *stream);

/*
 * Sequence split across devices (the paper treats leading batch/head dimensions as
 * independent outer indices, section 2; a split of the *sequence* axis is not in the paper
 * and rests on the shift invariance of eq. (2), like the split inside one device).
 *
 * moa_decode_attn_partial: same arguments and layouts as moa_decode_attn, over the n rows
 * this device holds, but instead of the normalised output it writes, per (batch, query
 * head), the unnormalised triple
 *     partial [batch, h_q, d_v + 4] :  o[d_v] = sum_l 2^(s2[l] - m) V[l,:],  m,  l = sum_l 2^(s2[l] - m),  2 pad
 * with s2 = log2(e) * scale * <q, K[l,:]> and m a reference value >= every s2[l] seen
 * (device memory, owned by the caller, 16-byte aligned when q/K/V are).
 *
 * moa_combine_partials: merges nparts such triples, laid out [nparts][batch][h_q][d_v+4]
 * (e.g. the result of an all-gather), in part order, into out [batch, h_q, d_v]:
 *     M = max_i m_i,  out = sum_i 2^(m_i - M) o_i / sum_i 2^(m_i - M) l_i.
 * The result equals moa_decode_attn over the concatenated rows up to fp32 rounding.
 * One kernel launch; device pointers; nothing is allocated.
 */
int moa_decode_attn_partial(const float *q, const float *K, const float *V, float *partial,
                            int batch, int h_q, int h_kv, int n, int d_k, int d_v,
                            float scale, void *stream);
int moa_combine_partials(const float *partials, int nparts, float *out, int batch, int h_q,
                         int d_v, void *stream);

/* Workspace size in bytes that moa_decode_attn_varlen needs for these dimensions on the
 * current device (0 on invalid dimensions).  Host-only arithmetic plus one device
 * attribute query. */
size_t moa_workspace_bytes(int batch, int h_q, int h_kv, int n_max, int d_k, int d_v);

/*
 * Cache append (eqs. (4),(5); Proposition 2): for every (b, h) copy the 32-bit patterns
 * of k_new[b,h,:] into K[b,h,pos[b],:] and of v_new[b,h,:] into V[b,h,pos[b],:].
 * Exactly (d_k+d_v)*4 bytes are read and written per (b,h); no other element changes.
 *   K [batch,h_kv,n_max,d_k]  V [batch,h_kv,n_max,d_v]
 *   k_new [batch,h_kv,d_k]    v_new [batch,h_kv,d_v]      pos: device int32[batch]
 * pos[b] outside [0,n_max) sets MOA_STATUS_APPEND_RANGE and skips item b.
 * pos is not modified (the caller owns the lengths; see moa_lens_add).
 */
int moa_kv_append(float *K, float *V, const float *k_new, const float *v_new,
                  const int32_t *pos, int batch, int h_kv, int n_max, int d_k, int d_v,
                  void *stream);

/* lens[b] += delta for b < batch, on the stream (the length counter of the cache of
 * section 5.3, kept on the device so that a decode loop needs no host round trip). */
int moa_lens_add(int32_t *lens, int batch, int delta, void *stream);

/*
 * One autoregressive step (the append-then-attend order of section 5.3's decode loop;
 * per-step cost M_step of section 5.2) in a single call:
 *   append (k_new, v_new) at row lens[b], then attend q over rows [0, lens[b]+1),
 *   then lens[b] += 1.
 * lens is a device int32[batch] that the call updates; all other arguments as above.
 * Requires lens[b] in [0, n_max-1]; otherwise the status bits above are set, the item
 * is skipped and its length is left unchanged.
 * For d_k == d_v in {32, 64, 128} (or d_k != d_v, both in {64, 128}) and 16-byte-aligned
 * pointers all three parts run in one kernel launch (the streaming kernel takes the new row from k_new/v_new, stores it into
 * the cache, and the last CTA to finish advances the lengths); otherwise in three.
 * `workspace` as for moa_decode_attn_varlen.
 * The call allocates nothing and needs no host round trip, so a sequence of steps can be
 * captured into a CUDA graph and replayed (after one uncaptured call on the device, which
 * does the library's one-time set-up); the captured pointers are those of the call.
 */
int moa_decode_step(const float *q, float *K, float *V, const float *k_new,
                    const float *v_new, float *out, int32_t *lens,
                    int batch, int h_q, int h_kv, int n_max, int d_k, int d_v, float scale,
                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same step without touching the lengths: append (k_new, v_new) at row pos[b], then
 * attend q over rows [0, pos[b]+1).  pos is a device int32[batch] that is only read.
 * (Eqs. (4),(5) followed by Algorithm 1 on the extended cache.)
 */
int moa_append_decode(const float *q, float *K, float *V, const float *k_new,
                      const float *v_new, float *out, const int32_t *pos,
                      int batch, int h_q, int h_kv, int n_max, int d_k, int d_v, float scale,
                      void *workspace, size_t workspace_bytes, void *stream);

/*
 * Caches that are not densely packed (section 5.3 pre-allocates the cache once; a serving
 * stack often carves K and V out of one larger allocation, keeps the heads innermost, or
 * shares one prefix between batch items).  Element (b, h, i, t) of K lives at
 *   K + b*k_strides[0] + h*k_strides[1] + i*k_strides[2] + t
 * and likewise for V with v_strides; both are HOST arrays of three element counts
 * {batch stride, kv-head stride, row stride}.  The feature axis is always contiguous.
 * Strides must be >= 0 and at most 2^40, the row stride at least the row length; a zero batch or head
 * stride (the same rows read for every item) is allowed for caches that are only read.
 * q, out, k_new, v_new stay dense.  The computation is Algorithm 1 on the addressed rows;
 * seq_lens (device int32[batch]) may be NULL: every sequence then has n_max rows.
 *   - every stride a multiple of 4, row stride == row length: the kernels of the dense
 *     calls (the tcgen05 kernel excepted, its groups run on the warp-MMA kernel);
 *   - every stride a multiple of 4, larger row stride, d_k and d_v in {64, 128}: the
 *     warp-MMA kernel (its tiled copies take any stride), groups padded to 8 heads;
 *   - anything else: the catch-all kernel.
 * `workspace` as for moa_decode_attn_varlen (moa_workspace_bytes covers these calls);
 * moa_decode_attn_strided also accepts workspace == NULL and then uses (and may grow)
 * the library-owned workspace like moa_decode_attn.
 * moa_kv_append_strided and moa_decode_step_strided are moa_kv_append and moa_decode_step
 * on such a cache; they refuse zero batch/head strides (MOA_ERR_INVALID).
 */
int moa_decode_attn_strided(const float *q, const float *K, const float *V, float *out,
                            const int32_t *seq_lens, int batch, int h_q, int h_kv, int n_max,
                            int d_k, int d_v, float scale, const long long *k_strides,
                            const long long *v_strides, void *workspace,
                            size_t workspace_bytes, void *stream);
int moa_kv_append_strided(float *K, float *V, const float *k_new, const float *v_new,
                          const int32_t *pos, int batch, int h_kv, int n_max, int d_k, int d_v,
                          const long long *k_strides, const long long *v_strides, void *stream);
int moa_decode_step_strided(const float *q, float *K, float *V, const float *k_new,
                            const float *v_new, float *out, int32_t *lens, int batch, int h_q,
                            int h_kv, int n_max, int d_k, int d_v, float scale,
                            const long long *k_strides, const long long *v_strides,
                            void *workspace, size_t workspace_bytes, void *stream);

/*
 * Host-buffer convenience call: q, K, V, out are HOST pointers (pinned memory gives
 * full copy bandwidth).  Copies the inputs to library-owned device staging buffers,
 * runs moa_decode_attn and copies `out` back; synchronises before returning.
 * Staging buffers are grown on demand and kept until moa_release.
 */
int moa_decode_attn_host(const float *q, const float *K, const float *V, float *out,
                         int batch, int h_q, int h_kv, int n, int d_k, int d_v,
                         float scale);

/*
 * Decode attention for callers that must not allocate device memory.  (The paper has no
 * counterpart to this entry point; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs after a process has handed all of its device memory to
 * a framework's pooling allocator (a cudaMalloc issued then fails or fragments the pool),
 * code inside a latency-critical serving loop where the implicit device-wide
 * synchronisation of cudaMalloc/cudaFree would stall every other stream, and plug-in
 * callbacks whose host framework forbids allocation calls while its own work is in
 * flight.  moa_decode_attn may call cudaMalloc on its first use (or when a larger problem
 * arrives) and moa_decode_attn_varlen pushes the scratch buffer onto the caller; this
 * variant does neither.
 *
 * Same arguments, layouts, results and return codes as moa_decode_attn.  The scratch for
 * the split-sequence partial results lives in a fixed array of
 * MOA_NOALLOC_SCRATCH_BYTES bytes that is part of the library image: every GPU that
 * loads the library holds that much memory until the process exits.  The call issues no
 * cudaMalloc, cudaFree or other allocating routine.
 *  - The array holds the partial slots of the largest plan the library compiles (two slots
 *    of 16 heads x 132 floats per streaming CTA, one CTA per SM: 2.5 MB on a 148-SM part)
 *    plus the completion counters.  A problem whose scratch need still exceeds
 *    MOA_NOALLOC_SCRATCH_BYTES (a part with many more SMs, or MOA_OPT_NUM_CTAS raised far
 *    above the SM count) is rejected with MOA_ERR_CAPACITY before anything is launched.
 *  - The first call on each device looks up the device address of the array (one
 *    cudaGetSymbolAddress with that device current) and keeps it; make that first call
 *    before starting any stream capture on that device.
 *  - The array is shared by every call on the device and keeps whatever the previous call
 *    left in it.  Nothing in it has to start at zero: each call writes every slot it later
 *    reads.  Two calls that can overlap on the GPU (different streams, no dependency
 *    between them) would race on it; order them, or give one of them its own workspace
 *    through moa_decode_attn_varlen.
 */
#define MOA_NOALLOC_SCRATCH_BYTES (4u << 20)
int moa_decode_attn_noalloc(const float *q, const float *K, const float *V, float *out,
                            int batch, int h_q, int h_kv, int n, int d_k, int d_v,
                            float scale, void *stream);

/* Synchronise `stream`, copy the device status word to *status_out (HOST int) and
 * clear it.  Zero means no kernel of this library reported a problem since the last
 * call. */
int moa_device_status(void *stream, int *status_out);

/* The paper's DRAM-traffic model (Proposition 1, with the h_kv/h_q factor of section 6
 * and lifted over the batch):  batch*(h_kv*n*(d_k+d_v) + h_q*(d_k+d_v))*4 bytes.
 * Host-only. */
long long moa_min_bytes(int batch, int h_q, int h_kv, long long n, int d_k, int d_v);

/* Free every library-owned device buffer on the current device (synchronises). */
int moa_release(void);

/* Text for a return code.  Host-only; the string is static. */
const char *moa_strerror(int code);

/*
 * Tuning and test hooks (host-only state, per process).
 *   MOA_OPT_FORCE_PATH : 0 = automatic, otherwise one of the MOA_PATH_* values below;
 *                        a forced path that cannot handle the shape returns
 *                        MOA_ERR_UNSUPPORTED.
 *   MOA_OPT_NUM_CTAS   : 0 = one streaming CTA per SM, otherwise that many.
 *   MOA_OPT_GROUPED_HEADS : query heads per CTA of the tensor-core kernel (16, 32 or 64;
 *                        0 = automatic).  Larger groups are cut into neighbouring CTAs.
 *   MOA_OPT_DEPENDENT_LAUNCH : 1 (default) = the streaming kernels are launched with
 *                        programmatic stream serialisation, 0 = ordinary launches.  Every
 *                        kernel of the library waits for its predecessor in the stream
 *                        before its first access to global memory, so calls in one stream
 *                        are ordered as usual; a kernel of the caller's that is itself
 *                        launched with programmatic stream serialisation right after a
 *                        library call has to do the same (cudaGridDependencySynchronize).
 *   MOA_OPT_GROUPED_OPERANDS : 0 (default) = groups of 17..64 heads may use the tensor-core kernel
 *                        that keeps the query and probability operands in tensor memory
 *                        (64 head lanes, smaller groups padded); 1 = only the kernel with
 *                        these operands in shared memory (groups of exactly 16, 32, 64).
 *   MOA_OPT_WAIT_LIMIT : number of polls after which the FMA streaming kernel gives up waiting
 *                        for a tile it has requested (0 = the built-in limit of 2^22 polls).
 *                        When a wait runs out the kernel sets MOA_STATUS_WAIT_TIMEOUT, stops
 *                        consuming and returns; the results of that call are invalid.
 *   MOA_OPT_TEST_SKIP_COPY : test hook for exactly that path: the copies of the row block with
 *                        this flat index are announced but never issued (nothing is in flight,
 *                        nothing out of bounds), so the wait for them runs out (-1 = off).
 * moa_last_path() reports which kernel family the last successful decode call used.
 */
#define MOA_OPT_FORCE_PATH 1
#define MOA_OPT_NUM_CTAS   2
#define MOA_OPT_GROUPED_HEADS 3
#define MOA_OPT_DEPENDENT_LAUNCH 4
#define MOA_OPT_GROUPED_OPERANDS 5
#define MOA_OPT_WAIT_LIMIT 7
#define MOA_OPT_TEST_SKIP_COPY 8
#define MOA_PATH_GENERIC   1   /* any d_k, d_v, alignment: one CTA per (batch, query head) */
#define MOA_PATH_STREAM    2   /* split-sequence streaming kernel on the FMA units, d in {32,64,128} */
#define MOA_PATH_GROUPED   3   /* tcgen05 tensor-core kernels: groups of 17..64 heads (16 when forced) at d = 128, dense layout;
                                  groups of 17..64 heads at d = 64 when the capacity is even (ragged caches and the
                                  fused step: 17..32) */
#define MOA_PATH_MMA       4   /* streaming kernel with warp-level MMA, 8 or 16 heads per fetched row (larger groups in
                                  several passes), d_k, d_v in {64,128} */
int moa_set_option(int option, int value);
int moa_last_path(void);

/*
 * Launch accounting for benchmarks (host-only state plus CUDA events; off by default).
 * moa_profile(1) clears the counters and starts counting every kernel the library
 * launches.  moa_profile(2) does the same and also brackets each launch of the dominant
 * decode kernel (streaming, grouped or generic) with a pair of CUDA events on the caller's
 * stream (at most MOA_PROFILE_MAX_EVENTS pairs are kept; later launches are counted but
 * not timed).  The events cost a few microseconds per launch, so a throughput
 * measurement should use mode 1.
 * moa_profile_read synchronises the device and reports the summed event time of the
 * timed decode-kernel launches in milliseconds, how many of them were timed, and the
 * total number of kernels launched since moa_profile(1).  Any pointer may be NULL.
 * moa_profile_launch_ms reports the event time of the index-th timed launch (for a median
 * or a histogram).  moa_profile(0) stops counting.
 */
#define MOA_PROFILE_MAX_EVENTS 8192
int moa_profile(int enable);
int moa_profile_read(double *decode_kernel_ms, long long *decode_kernel_launches,
                     long long *all_kernel_launches);
int moa_profile_launch_ms(long long index, double *ms);

#ifdef __cplusplus
}
#endif
#endif /* MOA_H */
