// moa_api.cu -- the extern "C" boundary of libmoa: argument validation, kernel
// selection, workspace management and launches.  See include/moa.h for the contract.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <atomic>
#include <mutex>
#include <type_traits>
#include <utility>

#include "moa.h"
#include "moa_device.cuh"
#include "moa_generic.cuh"
#include "moa_stream.cuh"
#include "moa_mma.cuh"
#include "moa_grouped.cuh"
#include "moa_grouped64.cuh"

namespace moa {

constexpr int kMaxDevices = 64;
constexpr float kLog2e = 1.4426950408889634f;

struct DeviceState {
    int sm_count = 0;
    void *ws = nullptr;          // library-owned workspace (moa_decode_attn)
    size_t ws_bytes = 0;
    void *stage[4] = {nullptr, nullptr, nullptr, nullptr};   // host-API staging: q K V out
    size_t stage_bytes[4] = {0, 0, 0, 0};
    cudaStream_t host_stream = nullptr;
};
static DeviceState g_dev[kMaxDevices];
// Host state of the library (the table above, the options, the launch accounting) is guarded
// by one lock, taken by every entry point that reads or changes it; launches are issued
// under it, so calls from several host threads are serialised on the host side only.
static std::recursive_mutex g_mu;
typedef std::lock_guard<std::recursive_mutex> Lock;
// Tag of the next launch that merges its partials in the kernel (see ticket_arrive).
static std::atomic<unsigned long long> g_launch_tag{1};
static int g_force_path = 0;
static int g_num_ctas = 0;
static int g_last_path = 0;

// ---- launch accounting (moa_profile) ----------------------------------------------------
static bool g_prof_on = false;
static bool g_prof_events = false;    // also bracket the dominant kernel with CUDA events
static long long g_prof_all = 0;          // kernels launched while profiling
static long long g_prof_timed = 0;        // decode-kernel launches bracketed by events
static cudaEvent_t *g_prof_ev = nullptr;  // 2 * MOA_PROFILE_MAX_EVENTS events, created lazily

struct TimedLaunch {                      // RAII: event before / after the dominant kernel
    cudaStream_t st;
    long long slot = -1;
    explicit TimedLaunch(cudaStream_t s) : st(s)
    {
        if (!g_prof_on || !g_prof_events || g_prof_timed >= MOA_PROFILE_MAX_EVENTS) return;
        if (!g_prof_ev) {
            g_prof_ev = new cudaEvent_t[2 * MOA_PROFILE_MAX_EVENTS]();
            for (int i = 0; i < 2 * MOA_PROFILE_MAX_EVENTS; ++i)
                if (cudaEventCreate(&g_prof_ev[i]) != cudaSuccess) { cudaGetLastError(); g_prof_ev[i] = nullptr; }
        }
        slot = g_prof_timed;
        if (g_prof_ev[2 * slot]) cudaEventRecord(g_prof_ev[2 * slot], st);
    }
    ~TimedLaunch()
    {
        if (slot < 0) return;
        if (g_prof_ev[2 * slot + 1]) cudaEventRecord(g_prof_ev[2 * slot + 1], st);
        ++g_prof_timed;
    }
};
static inline void count_launch(int n = 1) { if (g_prof_on) g_prof_all += n; }

static int g_dependent_launch = 1;   // MOA_OPT_DEPENDENT_LAUNCH
static int g_wait_limit = 0;         // MOA_OPT_WAIT_LIMIT: 0 = the built-in limit
static long long g_skip_copy_block = -1;   // MOA_OPT_TEST_SKIP_COPY

// Launch with programmatic stream serialisation: the kernel may start while its predecessor
// in the stream is still running and synchronises with it on the device (griddepcontrol.wait).
template <class... KArgs, class... Args>
static cudaError_t launch_dependent(void (*kernel)(KArgs...), int grid, int threads, size_t smem, cudaStream_t st,
                                    Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_dependent_launch ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

static int current_device(DeviceState **st)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return MOA_ERR_CUDA;
    }
    DeviceState &s = g_dev[dev];
    if (s.sm_count == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
            cudaGetLastError();
            return MOA_ERR_CUDA;
        }
        s.sm_count = n;
    }
    *st = &s;
    return MOA_OK;
}

static bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static int validate_dims(int batch, int h_q, int h_kv, int n, int d_k, int d_v)
{
    if (batch < 1 || h_q < 1 || h_kv < 1 || n < 1 || d_k < 1 || d_v < 1) return MOA_ERR_INVALID;
    if (h_q % h_kv != 0) return MOA_ERR_INVALID;
    if (d_k > MOA_MAX_DK || d_v > MOA_MAX_DV) return MOA_ERR_UNSUPPORTED;
    return MOA_OK;
}

// ---- cache layout ------------------------------------------------------------------------
struct Layout {
    CacheStrides k, v;      // element strides: batch item, kv head, row
    bool dense;             // exactly [batch, h_kv, n_max, d]
    bool rows_contig;       // row stride == row length for both caches
    bool vec4;              // every stride a multiple of 4 elements (16 bytes)
};

static Layout dense_layout(int h_kv, int n_max, int d_k, int d_v)
{
    Layout l;
    l.k = {(long long)h_kv * n_max * d_k, (long long)n_max * d_k, (long long)d_k};
    l.v = {(long long)h_kv * n_max * d_v, (long long)n_max * d_v, (long long)d_v};
    l.dense = l.rows_contig = true;
    l.vec4 = (d_k % 4 == 0) && (d_v % 4 == 0);
    return l;
}

// Layout from caller-supplied strides {batch, head, row}; false if they are unusable.
static bool strided_layout(const long long *ks, const long long *vs, int h_kv, int n_max, int d_k, int d_v, Layout *out)
{
    if (!ks || !vs) return false;
    for (int i = 0; i < 3; ++i)
        if (ks[i] < 0 || vs[i] < 0 || ks[i] > (1LL << 40) || vs[i] > (1LL << 40)) return false;
    if (ks[2] < d_k || vs[2] < d_v) return false;        // rows may not overlap
    Layout l;
    l.k = {ks[0], ks[1], ks[2]};
    l.v = {vs[0], vs[1], vs[2]};
    const Layout d = dense_layout(h_kv, n_max, d_k, d_v);
    l.dense = l.k.sb == d.k.sb && l.k.sh == d.k.sh && l.k.sr == d.k.sr && l.v.sb == d.v.sb && l.v.sh == d.v.sh &&
              l.v.sr == d.v.sr;
    l.rows_contig = (l.k.sr == d_k) && (l.v.sr == d_v);
    l.vec4 = true;
    for (int i = 0; i < 3; ++i)
        if (ks[i] % 4 != 0 || vs[i] % 4 != 0) l.vec4 = false;
    *out = l;
    return true;
}

// ---- streaming-kernel plan -------------------------------------------------------------
struct StreamPlan {
    bool ok = false;
    int D = 0;       // feature size (d_v; equal to d_k except in `mixed` plans)
    int Dk = 0;      // d_k
    int G = 0;       // heads per (virtual) kv head handled by one CTA pass
    int share = 1;   // virtual kv heads per physical kv head (g_s = share * G when g_s > 8)
    int R = 0;       // rows per block of the chosen configuration
    bool mma = false;  // groups of 8 heads: the contractions run on the warp-level MMA
};

static int stream_group(int g_s, int *share)
{
    if (g_s <= 8) {                      // pad to a power of two
        int G = 1;
        while (G < g_s) G <<= 1;
        *share = 1;
        return G;
    }
    *share = (g_s + 7) / 8;              // virtual kv heads of 8 query heads; the last may hold fewer
    return 8;
}

static int rows_per_block(int D, int G)
{
    if (D == 128) return (G == 8) ? 4 : 8;
    if (D == 64) return (G == 1 || G == 2) ? 16 : (G == 4 ? 8 : 4);
    return 32 / G;                       // D == 32
}

// Which of the two streaming kernels a call uses is part of the plan, because the row-block
// size (and with it the whole decomposition) differs.  MOA_PATH_STREAM forces the FMA kernel.
static bool mma_allowed() { return g_force_path != MOA_PATH_STREAM; }

static StreamPlan plan_stream(int g_s, int d_k, int d_v, bool rows_contig = true)
{
    StreamPlan p;
    p.Dk = d_k;
    if (d_k != d_v || !rows_contig || (g_force_path == MOA_PATH_MMA && d_k >= 64)) {
        // Unequal row lengths: only the paired mode of the warp-MMA kernel handles them (every
        // warp owns one operand), in groups of 8 heads.  Rows that are not contiguous in memory
        // (a row stride larger than the row) need tiled copies, which only that kernel issues:
        // small groups are padded to 8 heads, which costs no extra memory traffic.
        if (!mma_allowed() || (d_k != 64 && d_k != 128) || (d_v != 64 && d_v != 128)) return p;
        p.D = d_v;
        p.G = 8;
        p.share = g_s > 8 ? (g_s + 7) / 8 : 1;   // (the last virtual head of a stored one may hold fewer than 8)
        if (d_k == d_v && g_s > 8 && g_s < 16) { p.G = 16; p.share = 1; }
        else if (d_k == d_v && g_s >= 16) { p.G = 16; p.share = (g_s + 15) / 16; }
        p.mma = true;
        p.R = 16;
        p.ok = true;
        return p;
    }
    if (d_k != 32 && d_k != 64 && d_k != 128) return p;
    p.D = d_k;
    p.G = stream_group(g_s, &p.share);
    p.mma = mma_allowed() && p.G == 8 && p.D >= 64;
    if (p.mma && g_s >= 16) { p.G = 16; p.share = (g_s + 15) / 16; }   // two 8-head tiles per fetched row (the last virtual head may hold fewer)
    if (mma_allowed() && p.D >= 64 && g_s > 8 && g_s < 16) {         // 9..15 heads: one padded 16-head group
        p.G = 16; p.share = 1; p.mma = true;
    }
    p.R = p.mma ? 16 : rows_per_block(p.D, p.G);
    p.ok = true;
    return p;
}

static int stream_num_ctas(const DeviceState &s) { return g_num_ctas > 0 ? g_num_ctas : s.sm_count; }

// CTAs actually launched.  Cutting a unit across CTAs costs a counter round trip and a merge
// (about 2 us), which only pays when it removes more streaming time than that: units of up
// to 16 row blocks (128 KB of K and V) are left whole, one or more per CTA (measured: the
// 256-row single-head step takes 6.7 us on one CTA, 8.2 us on two).  Larger units are cut,
// but never into more than one CTA per 8 row blocks (one block per warp).
static int stream_grid(const DeviceState &s, const StreamPlan &p, int batch, int h_kv, int n_max)
{
    const int cap = stream_num_ctas(s);
    if (g_num_ctas > 0) return cap;
    const long long per_unit = (n_max + p.R - 1) / p.R;
    const long long units = (long long)batch * h_kv * p.share;
    const long long want = per_unit <= 16 ? units : (units * per_unit + 7) / 8;
    return (int)(want < cap ? (want < 1 ? 1 : want) : cap);
}

// Workspace of a streaming launch: two partial slots per CTA, then (256-byte aligned) the
// completion counters of the in-kernel merge.
static size_t stream_slot_bytes(const StreamPlan &p, int num_ctas)
{
    return ((size_t)num_ctas * 2 * p.G * (p.D + 4) * sizeof(float) + 255) / 256 * 256;
}
static size_t stream_ws_bytes(const StreamPlan &p, int num_ctas)
{
    return stream_slot_bytes(p, num_ctas) + (num_ctas <= kTicketCtas ? kTicketBytes : 0);
}

template <class C>
static cudaError_t launch_stream_cfg(const DecodeArgs &a, int num_ctas, cudaStream_t st)
{
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(stream_decode_kernel<C>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    {
        TimedLaunch t(st);
        launch_dependent(stream_decode_kernel<C>, num_ctas, C::THREADS, C::SMEM_BYTES, st, a);
    }
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || a.tickets != nullptr) return e;
    const long long warps = (long long)a.batch * a.h_q;
    const int blocks = (int)((warps + 3) / 4);
    stream_combine_kernel<C::D, C::R><<<blocks, 128, 0, st>>>(a, num_ctas, C::G);
    count_launch();
    return cudaGetLastError();
}

static bool make_rows_map(CUtensorMap *m, const float *base, int D, int n_max, int heads, int batch,
                          const CacheStrides &cs);

template <class C>
static cudaError_t launch_mma_cfg(const DecodeArgs &a, int num_ctas, cudaStream_t st)
{
    CUtensorMap mk, mv;
    const int h_stored = a.h_kv / a.kv_share;
    if (!make_rows_map(&mk, a.K, C::DK, a.n_max, h_stored, a.batch, CacheStrides{a.k_sb, a.k_sh, a.k_sr}) ||
        !make_rows_map(&mv, a.V, C::DV, a.n_max, h_stored, a.batch, CacheStrides{a.v_sb, a.v_sh, a.v_sr}))
        return cudaErrorInvalidValue;
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(mma_decode_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    {
        TimedLaunch t(st);
        launch_dependent(mma_decode_kernel<C>, num_ctas, C::THREADS, C::SMEM_BYTES, st, mk, mv, a);
    }
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || a.tickets != nullptr) return e;
    const long long warps = (long long)a.batch * a.h_q;
    stream_combine_kernel<C::D, C::R><<<(int)((warps + 3) / 4), 128, 0, st>>>(a, num_ctas, C::G);
    count_launch();
    return cudaGetLastError();
}

static cudaError_t launch_stream(const StreamPlan &p, const DecodeArgs &a, int num_ctas,
                                 cudaStream_t st)
{
    if (p.mma) {                         //                                     D   S  P  paired
        if (p.Dk != p.D) {               //                     d_k  d_v  S  P  paired NT
            if (p.Dk == 128) return launch_mma_cfg<MmaCfg<128, 64, 3, 4, true, 1>>(a, num_ctas, st);
            return launch_mma_cfg<MmaCfg<64, 128, 3, 4, true, 1>>(a, num_ctas, st);
        }
        if (p.D == 128 && p.G == 16) return launch_mma_cfg<MmaCfg<128, 128, 3, 4, true, 2>>(a, num_ctas, st);
        if (p.D == 128) return launch_mma_cfg<MmaCfg<128, 128, 3, 4, true, 1>>(a, num_ctas, st);
        if (p.G == 16) return launch_mma_cfg<MmaCfg<64, 64, 2, 8, false, 2>>(a, num_ctas, st);
        return launch_mma_cfg<MmaCfg<64, 64, 2, 8, false, 1>>(a, num_ctas, st);
    }
    // The heavier configurations (many FMAs per fetched byte) run 16 warps per CTA: with
    // eight, two warps per scheduler cannot hide the shuffle and FMA latencies.  The lightest
    // (one or two heads per row) run 12 warps with two stages each, measured 2-3 % faster
    // than 8 warps with three.
    //                                   D    G  RV  S  W
    if (p.D == 128) {
        switch (p.G) {
        case 1: return launch_stream_cfg<StreamCfg<128, 1, 8, 2, 12>>(a, num_ctas, st);
        case 2: return launch_stream_cfg<StreamCfg<128, 2, 8, 2, 12>>(a, num_ctas, st);
        case 4: return launch_stream_cfg<StreamCfg<128, 4, 8, 3, 8>>(a, num_ctas, st);
        default: return launch_stream_cfg<StreamCfg<128, 8, 4, 2, 16>>(a, num_ctas, st);
        }
    }
    if (p.D == 64) {
        switch (p.G) {
        case 1: return launch_stream_cfg<StreamCfg<64, 1, 8, 2, 12>>(a, num_ctas, st);
        case 2: return launch_stream_cfg<StreamCfg<64, 2, 8, 2, 12>>(a, num_ctas, st);
        case 4: return launch_stream_cfg<StreamCfg<64, 4, 4, 2, 16>>(a, num_ctas, st);
        default: return launch_stream_cfg<StreamCfg<64, 8, 2, 4, 16>>(a, num_ctas, st);
        }
    }
    switch (p.G) {                       // D == 32: eight lanes per row, four rows per 512-byte read
    case 1: return launch_stream_cfg<StreamCfg<32, 1, 8, 3, 8>>(a, num_ctas, st);
    case 2: return launch_stream_cfg<StreamCfg<32, 2, 4, 3, 16>>(a, num_ctas, st);
    case 4: return launch_stream_cfg<StreamCfg<32, 4, 2, 5, 16>>(a, num_ctas, st);
    default: return launch_stream_cfg<StreamCfg<32, 8, 1, 8, 16>>(a, num_ctas, st);
    }
}

// ---- grouped (tensor-core) plan -----------------------------------------------------------
struct GroupedPlan {
    bool ok = false;
    int GH = 0;          // query heads per CTA (per virtual kv head)
    int share = 1;       // virtual kv heads per stored kv head
    int splits = 1, tiles_per_split = 1;
    size_t ws_bytes = 0;        // partial slots
    size_t tail_bytes = 0;      // scratch copies of every unit's last tile (ragged caches, fused step)
    size_t ws_ragged() const { return (ws_bytes + 255) / 256 * 256 + tail_bytes; }
};
static int g_grouped_heads = 0;   // MOA_OPT_GROUPED_HEADS: 0 = automatic
static int g_grouped_operands = 0;   // MOA_OPT_GROUPED_OPERANDS

static GroupedPlan plan_grouped(const DeviceState &s, int batch, int h_q, int h_kv, int n, int d_k, int d_v)
{
    GroupedPlan p;
    const int g_s = h_q / h_kv;
    if (d_k != 128 || d_v != 128) return p;
    // Any group of 17 to 64 heads runs on the kernel with 64 head lanes (missing heads are zero
    // lanes): its time per tile does not depend on the number of heads, and from 17 heads on it
    // beats the warp-MMA kernel's passes over groups of 8 or 16.
    const bool lanes64 = (g_grouped_operands == 0) && g_s > 16 && g_s <= 64 && (g_grouped_heads == 0 || g_grouped_heads == 64);
    if (!lanes64 && g_s != 16 && g_s != 32 && g_s != 64) return p;
    // Groups of 16 are faster as two groups of 8 on the warp-MMA streaming kernel (the K/V tile
    // is read twice, the second time from L2); this kernel takes them only when forced.
    if (g_s == 16 && g_force_path != MOA_PATH_GROUPED) return p;
    const long long units = (long long)batch * h_kv;
    if (units > 0x7fffffffLL / 256 || (long long)n > 0x7fffffffLL - 256) return p;
    // One CTA takes the whole group (measured faster than cutting a group of 64 into two
    // neighbouring CTAs of 32 heads that read the same rows through L2).
    p.GH = lanes64 ? 64 : g_s;
    if (!lanes64 && (g_grouped_heads == 16 || g_grouped_heads == 32 || g_grouped_heads == 64))
        if (g_grouped_heads <= g_s) p.GH = g_grouped_heads;
    p.share = lanes64 ? 1 : g_s / p.GH;
    const long long ctas_per_split = units * p.share;
    const int tiles = (n + 127) / 128;
    long long splits = ctas_per_split >= s.sm_count ? 1 : s.sm_count / ctas_per_split;
    if (splits > tiles) splits = tiles;
    p.splits = (int)splits;
    p.tiles_per_split = (tiles + p.splits - 1) / p.splits;
    p.ws_bytes = (size_t)units * p.share * p.splits * p.GH * 132 * sizeof(float);
    const size_t flat_slots = (size_t)(units > s.sm_count ? units : s.sm_count);   // one partial per CTA in flat mode
    if (p.share == 1 && flat_slots * p.GH * 132 * sizeof(float) > p.ws_bytes) p.ws_bytes = flat_slots * p.GH * 132 * sizeof(float);
    p.tail_bytes = (size_t)units * 2 * 128 * 128 * sizeof(float);
    p.ok = true;
    return p;
}

typedef CUresult (*TmapEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                 const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static TmapEncodeFn tmap_encoder()
{
    static TmapEncodeFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        fn = reinterpret_cast<TmapEncodeFn>(p);
    }
    return fn;
}

// Tensor map over a cache [units][n][128] fp32 with boxes of 32 features x box_rows rows.
static bool make_cache_map(CUtensorMap *m, const float *base, long long units, int n, int box_rows,
                           CUtensorMapSwizzle swz)
{
    TmapEncodeFn enc = tmap_encoder();
    if (!enc) return false;
    cuuint64_t dims[3] = {128, (cuuint64_t)n, (cuuint64_t)units};
    cuuint64_t strides[2] = {512, (cuuint64_t)n * 512};
    cuuint32_t box[3] = {32, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map over a cache [batch][stored kv heads][n_max rows][D floats] with arbitrary element
// strides, seen as (32 floats, row, D/32 column groups, head, batch item): one box of 16 rows
// lands as D/32 swizzled [16 rows][128 bytes] sub-tiles; rows past n_max read as zero.
static bool make_rows_map(CUtensorMap *m, const float *base, int D, int n_max, int heads, int batch,
                          const CacheStrides &cs)
{
    TmapEncodeFn enc = tmap_encoder();
    if (!enc) return false;
    cuuint64_t dims[5] = {32, (cuuint64_t)n_max, (cuuint64_t)(D / 32), (cuuint64_t)heads, (cuuint64_t)batch};
    cuuint64_t strides[4] = {(cuuint64_t)cs.sr * 4, 128, (cuuint64_t)cs.sh * 4, (cuuint64_t)cs.sb * 4};
    // a dimension of extent 1 is never stepped along: give it a harmless legal stride
    if (heads == 1 && strides[2] == 0) strides[2] = 16;
    if (batch == 1 && strides[3] == 0) strides[3] = 16;
    cuuint32_t box[5] = {32, 16, (cuuint32_t)(D / 32), 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<float *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int GH>
static cudaError_t launch_grouped_cfg(const CUtensorMap &mk, const CUtensorMap &mv, const CUtensorMap &mkt,
                                      const CUtensorMap &mvt, const GroupedArgs &ga, int grid, cudaStream_t st)
{
    using C = GroupedCfg<GH>;
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(grouped_decode_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    {
        TimedLaunch t(st);
        grouped_decode_kernel<C><<<grid, C::THREADS, C::SMEM_BYTES, st>>>(mk, mv, mkt, mvt, ga);
    }
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const long long warps = (long long)ga.batch * ga.h_q;
    grouped_combine_kernel<GH><<<(int)warps, 128, 0, st>>>(ga);
    count_launch();
    return cudaGetLastError();
}


// Groups of 64 heads with Q and P in tensor memory; same arguments and partial format as
// the shared-memory-operand kernel, so the combine kernel is shared.
static cudaError_t launch_grouped64_cfg(const CUtensorMap &mk, const CUtensorMap &mv, const CUtensorMap &mkt,
                                        const CUtensorMap &mvt, const GroupedArgs &ga, int grid, cudaStream_t st,
                                        bool combine = true)
{
    using C = Grouped64Cfg;
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(grouped64_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    {
        // programmatic stream serialisation: the kernel's set-up overlaps the tail-copy kernel
        // before it, the combine kernel's launch overlaps this kernel's end
        TimedLaunch t(st);
        launch_dependent(grouped64_decode_kernel, grid, C::THREADS, C::SMEM_BYTES, st, mk, mv, mkt, mvt, ga);
    }
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || !combine) return e;
    const long long warps = (long long)ga.batch * ga.h_q;
    launch_dependent(grouped_combine_kernel<64>, (int)warps, 128, 0, st, ga);
    count_launch();
    return cudaGetLastError();
}

template <int GH>
static cudaError_t launch_grouped_cfg(const CUtensorMap &mk, const CUtensorMap &mv, const CUtensorMap &mkt,
                                      const CUtensorMap &mvt, const GroupedArgs &ga, int grid, cudaStream_t st);

// Groups of 17 to 64 heads on 64 head lanes (missing heads are zero lanes): the kernel with Q
// and P in tensor memory, in the variant that keeps the two score chains apart.  Same arguments
// and partial format as the shared-memory-operand kernel, so the combine kernel is shared.
static cudaError_t launch_grouped64(const CUtensorMap &mk, const CUtensorMap &mv, const CUtensorMap &mkt,
                                    const CUtensorMap &mvt, const GroupedArgs &ga, int grid, cudaStream_t st)
{
    return launch_grouped64_cfg(mk, mv, mkt, mvt, ga, grid, st);
}

static cudaError_t launch_generic(const DecodeArgs &a, cudaStream_t st)
{
    const size_t smem = sizeof(float) * ((size_t)a.d_k + (size_t)kGenericWarps * a.d_v + 2 * kGenericWarps);
    if (a.seq_lens != nullptr) {
        check_lens_kernel<<<(a.batch + 127) / 128, 128, 0, st>>>(a.seq_lens, a.len_bias, a.batch, a.n_max);
        count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    {
        TimedLaunch t(st);
        generic_decode_kernel<<<a.batch * a.h_q, kGenericWarps * 32, smem, st>>>(a);
    }
    count_launch();
    return cudaGetLastError();
}

// Groups of 17..32 or of exactly 64 heads at d = 64 on a dense cache with an even number of rows:
// the 64-lane tensor-core kernel in pair mode.  Two consecutive cached rows of 64 features are
// read as one row of 128; every head takes two pseudo-heads whose query is zero in one half, so
// one of them sees the even and the other the odd cached rows; a combine kernel of its own puts
// the halves together.  64 heads run as two virtual kv heads of 32 (the K/V tiles are read twice,
// the second time from L2).
struct PairPlan {
    bool ok = false;
    int share = 1, gs = 0, splits = 1, tiles_per_split = 1;
    size_t ws_bytes = 0;                 // dense: units x splits partial slots
    size_t flat_bytes = 0, tail_bytes = 0;   // ragged: one partial slot per CTA, the tail copies
    size_t ws_ragged() const { return (flat_bytes + 255) / 256 * 256 + tail_bytes; }
};
static PairPlan plan_grouped_pair(const DeviceState &s, int batch, int h_q, int h_kv, int n, int d_k, int d_v)
{
    PairPlan p;
    const int g_s = h_q / h_kv;
    if (d_k != 64 || d_v != 64 || (n & 1) || n < 2) return p;
    if (g_s <= 16 || g_s > 64) return p;
    if (g_grouped_operands != 0 || (g_force_path != 0 && g_force_path != MOA_PATH_GROUPED)) return p;
    p.share = g_s > 32 ? 2 : 1;                   // 33..64 heads: two virtual heads per stored one, the second possibly smaller
    p.gs = g_s > 32 ? (g_s + 1) / 2 : g_s;
    const long long vunits = (long long)batch * h_kv * p.share;
    if (vunits > 0x7fffffffLL / 256) return p;
    const int tiles = (n / 2 + 127) / 128;
    long long splits = vunits >= s.sm_count ? 1 : s.sm_count / vunits;
    if (splits > tiles) splits = tiles;
    p.splits = (int)splits;
    p.tiles_per_split = (tiles + p.splits - 1) / p.splits;
    p.ws_bytes = (size_t)vunits * p.splits * 64 * 132 * sizeof(float);
    // ragged caches (one virtual head per stored one only): one partial per CTA, CTAs dealt by length
    const size_t flat_slots = (size_t)(vunits > s.sm_count ? vunits : s.sm_count);
    p.flat_bytes = flat_slots * 64 * 132 * sizeof(float);
    p.tail_bytes = (size_t)batch * h_kv * 2 * 128 * 128 * sizeof(float);
    p.ok = true;
    return p;
}

struct FusedStep {                 // extra work folded into the decode launch(es)
    float *Kw = nullptr, *Vw = nullptr;
    const float *k_new = nullptr, *v_new = nullptr;
    int32_t *lens_rw = nullptr;
};

// Rows of 64 features on the 64-lane kernel.  Dense caches: `seq_lens` null, one grid of
// units x splits.  Ragged caches and the fused step (one virtual head per stored one): the
// zero-padded copy of every unit's last tile first (which also stores the appended row), CTAs
// dealt to the units by their lengths, then the merge and, for the step, the length advance.
static cudaError_t launch_grouped_pair(const PairPlan &pp, const float *q, const float *K, const float *V, float *out,
                                       float *ws, int batch, int h_q, int h_kv, int n, float scale, cudaStream_t st,
                                       const int32_t *seq_lens = nullptr, int len_bias = 0, const FusedStep *fused = nullptr,
                                       int sm_count = 0)
{
    const long long units = (long long)batch * h_kv;
    CUtensorMap mk, mv;
    if (!make_cache_map(&mk, K, units, n / 2, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_cache_map(&mv, V, units, n / 2, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B))
        return cudaErrorInvalidValue;
    GroupedArgs ga;
    ga.q = q; ga.out = out; ga.ws = ws;
    ga.batch = batch; ga.h_q = h_q; ga.h_kv = h_kv * pp.share; ga.n = n / 2;
    ga.g_s = pp.gs; ga.h_kv_stored = h_kv; ga.share = pp.share;
    ga.splits = pp.splits; ga.tiles_per_split = pp.tiles_per_split;
    ga.qscale = scale * kLog2e;
    ga.partial_out = nullptr; ga.seq_lens = seq_lens; ga.len_bias = len_bias;
    ga.tailK = nullptr; ga.tailV = nullptr; ga.flat = 0;
    ga.pair = 1;
    ga.g_total = h_q / h_kv;
    using C = Grouped64Cfg;
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(grouped64_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    CUtensorMap mkt = mk, mvt = mv;
    int grid = (int)(units * pp.share * pp.splits);
    if (seq_lens != nullptr) {
        ga.tailK = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(ws) + (pp.flat_bytes + 255) / 256 * 256);
        ga.tailV = ga.tailK + (size_t)units * 128 * 128;
        if (!make_cache_map(&mkt, ga.tailK, units, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_cache_map(&mvt, ga.tailV, units, 128, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B))
            return cudaErrorInvalidValue;
        grouped_tail_kernel<<<(int)units * 8, 256, 0, st>>>(ga, K, V, fused ? fused->Kw : nullptr, fused ? fused->Vw : nullptr,
                                                            fused ? fused->k_new : nullptr, fused ? fused->v_new : nullptr);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return cudaErrorLaunchFailure;
        grid = (int)(units > sm_count ? units : sm_count);
        ga.flat = grid;
    }
    {
        TimedLaunch t(st);
        launch_dependent(grouped64_decode_kernel, grid, C::THREADS, C::SMEM_BYTES, st, mk, mv, mkt, mvt, ga);
    }
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const long long rows = (long long)batch * h_q;
    launch_dependent(grouped_pair_combine_kernel, (int)rows, 128, 0, st, ga);
    count_launch();
    e = cudaGetLastError();
    if (e == cudaSuccess && fused != nullptr && fused->lens_rw != nullptr) {
        lens_add_kernel<<<(batch + 127) / 128, 128, 0, st>>>(fused->lens_rw, batch, 1, n);
        count_launch();
        e = cudaGetLastError();
    }
    return e;
}

// Shared implementation of the decode entry points.  `ws` may be null when the chosen
// path needs none.
static int decode_impl(const float *q, const float *K, const float *V, float *out, int batch,
                       int h_q, int h_kv, const int32_t *seq_lens, int len_bias, int n_max,
                       int d_k, int d_v, float scale, void *ws, size_t ws_bytes,
                       bool library_ws, cudaStream_t st, const FusedStep *fused = nullptr,
                       bool allow_grouped = true, float *partial_out = nullptr, const Layout *layp = nullptr)
{
    if (!q || !K || !V || (!out && !partial_out)) return MOA_ERR_INVALID;
    if (partial_out != nullptr) out = partial_out;      // (alignment checks below apply to it)
    int rc = validate_dims(batch, h_q, h_kv, n_max, d_k, d_v);
    if (rc != MOA_OK) return rc;
    if (!isfinite(scale)) return MOA_ERR_INVALID;
    if (!aligned(q, 4) || !aligned(K, 4) || !aligned(V, 4) || !aligned(out, 4)) return MOA_ERR_ALIGN;
    if (seq_lens && !aligned(seq_lens, 4)) return MOA_ERR_ALIGN;
    if ((long long)batch * h_q > 0x7fffffffLL) return MOA_ERR_CAPACITY;

    DeviceState *dev = nullptr;
    rc = current_device(&dev);
    if (rc != MOA_OK) return rc;

    const int g_s = h_q / h_kv;
    const Layout lay = layp ? *layp : dense_layout(h_kv, n_max, d_k, d_v);
    StreamPlan plan = plan_stream(g_s, d_k, d_v, lay.rows_contig);
    bool fast_ok = plan.ok && lay.vec4 && aligned(q, 16) && aligned(K, 16) && aligned(V, 16) && aligned(out, 16);
    if (fast_ok && plan.mma && !lay.dense) {
        // strides a tensor map cannot express (zero, or beyond its range): catch-all kernel
        CUtensorMap probe;
        if (!make_rows_map(&probe, K, plan.Dk, n_max, h_kv, batch, lay.k) ||
            !make_rows_map(&probe, V, plan.D, n_max, h_kv, batch, lay.v))
            fast_ok = false;
    }
    // (ragged caches and the fused step: lengths on the device, scratch from the caller, one virtual head per stored one)
    const bool pair_ragged = (seq_lens != nullptr) || (fused != nullptr);
    if (fast_ok && allow_grouped && lay.dense && partial_out == nullptr &&
        (!pair_ragged || (seq_lens != nullptr && !library_ws &&
                          (fused == nullptr || (aligned(fused->k_new, 16) && aligned(fused->v_new, 16)))))) {
        PairPlan pp = plan_grouped_pair(*dev, batch, h_q, h_kv, n_max, d_k, d_v);
        if (pair_ragged && pp.share != 1) pp.ok = false;
        if (pp.ok && pair_ragged) {
            if (ws && ws_bytes >= pp.ws_ragged()) {
                if (!aligned(ws, 256)) return MOA_ERR_ALIGN;
                if (launch_grouped_pair(pp, q, K, V, out, static_cast<float *>(ws), batch, h_q, h_kv, n_max, scale, st,
                                        seq_lens, len_bias, fused, dev->sm_count) != cudaSuccess)
                    return MOA_ERR_CUDA;
                g_last_path = MOA_PATH_GROUPED;
                return MOA_OK;
            }
        } else if (pp.ok && (library_ws || (ws && ws_bytes >= pp.ws_bytes))) {
            if (library_ws) {
                if (dev->ws_bytes < pp.ws_bytes) {
                    if (dev->ws) { cudaDeviceSynchronize(); cudaFree(dev->ws); dev->ws = nullptr; dev->ws_bytes = 0; }
                    if (cudaMalloc(&dev->ws, pp.ws_bytes) != cudaSuccess) { cudaGetLastError(); return MOA_ERR_CUDA; }
                    dev->ws_bytes = pp.ws_bytes;
                }
                ws = dev->ws;
            } else if (!aligned(ws, 256)) return MOA_ERR_ALIGN;
            if (launch_grouped_pair(pp, q, K, V, out, static_cast<float *>(ws), batch, h_q, h_kv, n_max, scale, st) != cudaSuccess)
                return MOA_ERR_CUDA;
            g_last_path = MOA_PATH_GROUPED;
            return MOA_OK;
        }
    }
    int path = fast_ok ? (plan.mma ? MOA_PATH_MMA : MOA_PATH_STREAM) : MOA_PATH_GENERIC;
    // Large head groups go to the tcgen05 kernel; ragged caches and the fused step need scratch
    // for the zero-padded copy of every unit's last tile on top of the partial slots.
    GroupedPlan gplan;
    const bool ragged = (seq_lens != nullptr) || (fused != nullptr);
    if (fast_ok && allow_grouped && lay.dense && (fused == nullptr || (aligned(fused->k_new, 16) && aligned(fused->v_new, 16))))
        gplan = plan_grouped(*dev, batch, h_q, h_kv, n_max, d_k, d_v);
    if (gplan.ok && ragged && (library_ws || seq_lens == nullptr)) gplan.ok = false;

    if (gplan.ok && (library_ws || (ws && ws_bytes >= (ragged ? gplan.ws_ragged() : gplan.ws_bytes)))) path = MOA_PATH_GROUPED;
    if (g_force_path == MOA_PATH_GENERIC) path = MOA_PATH_GENERIC;
    else if (g_force_path == MOA_PATH_STREAM) {
        if (!fast_ok) return MOA_ERR_UNSUPPORTED;
        path = MOA_PATH_STREAM;
    } else if (g_force_path == MOA_PATH_MMA) {
        if (!fast_ok || !plan.mma) return MOA_ERR_UNSUPPORTED;
        path = MOA_PATH_MMA;
    } else if (g_force_path == MOA_PATH_GROUPED) {
        if (path != MOA_PATH_GROUPED) return MOA_ERR_UNSUPPORTED;
    } else if (g_force_path != 0) return MOA_ERR_UNSUPPORTED;

    DecodeArgs a;
    a.q = q; a.K = K; a.V = V; a.out = out; a.ws = nullptr;
    a.seq_lens = seq_lens; a.len_bias = len_bias;
    a.batch = batch; a.h_q = h_q; a.h_kv = h_kv; a.g_s = g_s; a.kv_share = 1; a.g_total = g_s;
    a.n_max = n_max; a.d_k = d_k; a.d_v = d_v;
    a.k_sb = lay.k.sb; a.k_sh = lay.k.sh; a.k_sr = lay.k.sr;
    a.v_sb = lay.v.sb; a.v_sh = lay.v.sh; a.v_sr = lay.v.sr;
    a.qscale = scale * kLog2e;
    a.Kw = nullptr; a.Vw = nullptr; a.k_new = nullptr; a.v_new = nullptr; a.lens_rw = nullptr;
    a.tickets = nullptr; a.ticket_tag = 0;
    a.wait_limit = g_wait_limit > 0 ? (uint32_t)g_wait_limit : kWaitLimit;
    a.skip_copy_block = g_skip_copy_block;
    a.partial_out = partial_out;
    if (fused != nullptr && path == MOA_PATH_GENERIC) return MOA_ERR_UNSUPPORTED;

    cudaError_t e;
    if (path == MOA_PATH_GROUPED) {
        if (library_ws) {
            if (dev->ws_bytes < gplan.ws_bytes) {
                if (dev->ws) { cudaDeviceSynchronize(); cudaFree(dev->ws); dev->ws = nullptr; dev->ws_bytes = 0; }
                if (cudaMalloc(&dev->ws, gplan.ws_bytes) != cudaSuccess) { cudaGetLastError(); return MOA_ERR_CUDA; }
                dev->ws_bytes = gplan.ws_bytes;
            }
            ws = dev->ws;
        } else if (!aligned(ws, 256)) return MOA_ERR_ALIGN;
        CUtensorMap mk, mv;
        const long long units = (long long)batch * h_kv;
        if (!make_cache_map(&mk, K, units, n_max, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_cache_map(&mv, V, units, n_max, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B))
            return MOA_ERR_CUDA;
        GroupedArgs ga;
        ga.q = q; ga.out = out; ga.ws = static_cast<float *>(ws);
        ga.batch = batch; ga.h_q = h_q; ga.h_kv = h_kv * gplan.share; ga.n = n_max;
        ga.h_kv_stored = h_kv; ga.share = gplan.share;
        ga.g_s = (gplan.share == 1) ? g_s : gplan.GH;
        ga.splits = gplan.splits; ga.tiles_per_split = gplan.tiles_per_split;
        ga.qscale = scale * kLog2e;
        ga.partial_out = partial_out;
        ga.seq_lens = seq_lens; ga.len_bias = len_bias;
        ga.tailK = nullptr; ga.tailV = nullptr;
        ga.flat = 0;
            ga.pair = 0;
        ga.g_total = 0;
        CUtensorMap mkt = mk, mvt = mv;
        if (ragged) {
            // the last, partly filled tile of every unit, zero-padded (and the appended row of
            // the fused step, which this kernel also stores into the cache)
            ga.tailK = reinterpret_cast<float *>(static_cast<unsigned char *>(ws) + (gplan.ws_bytes + 255) / 256 * 256);
            ga.tailV = ga.tailK + (size_t)units * 128 * 128;
            if (!make_cache_map(&mkt, ga.tailK, units, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
                !make_cache_map(&mvt, ga.tailV, units, 128, 32, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B))
                return MOA_ERR_CUDA;
            grouped_tail_kernel<<<(int)units * 8, 256, 0, st>>>(ga, K, V, fused ? fused->Kw : nullptr,
                                                            fused ? fused->Vw : nullptr, fused ? fused->k_new : nullptr,
                                                            fused ? fused->v_new : nullptr);
            count_launch();
            if (cudaGetLastError() != cudaSuccess) return MOA_ERR_CUDA;
        }
        int grid = (int)(units * gplan.share * gplan.splits);
        if (ragged && gplan.share == 1) {          // CTAs follow the lengths, read on the device
            grid = (int)(units > dev->sm_count ? units : dev->sm_count);
            ga.flat = grid;
        }
        if (gplan.GH == 16) e = launch_grouped_cfg<16>(mk, mv, mkt, mvt, ga, grid, st);
        else if (gplan.GH == 32) e = launch_grouped_cfg<32>(mk, mv, mkt, mvt, ga, grid, st);
        else if (gplan.share == 1 && g_grouped_operands == 0) e = launch_grouped64(mk, mv, mkt, mvt, ga, grid, st);
        else e = launch_grouped_cfg<64>(mk, mv, mkt, mvt, ga, grid, st);
        if (e == cudaSuccess && fused != nullptr && fused->lens_rw != nullptr) {
            lens_add_kernel<<<(batch + 127) / 128, 128, 0, st>>>(fused->lens_rw, batch, 1, n_max);
            count_launch();
            e = cudaGetLastError();
        }
    } else if (path == MOA_PATH_STREAM || path == MOA_PATH_MMA) {
        const int num_ctas = stream_grid(*dev, plan, batch, h_kv, n_max);
        const size_t need = stream_ws_bytes(plan, num_ctas);
        if (library_ws) {
            if (dev->ws_bytes < need) {
                if (dev->ws) { cudaDeviceSynchronize(); cudaFree(dev->ws); dev->ws = nullptr; dev->ws_bytes = 0; }
                if (cudaMalloc(&dev->ws, need) != cudaSuccess) { cudaGetLastError(); return MOA_ERR_CUDA; }
                dev->ws_bytes = need;
            }
            ws = dev->ws;
        } else {
            if (!ws || ws_bytes < need) return MOA_ERR_WORKSPACE;
            if (!aligned(ws, 256)) return MOA_ERR_ALIGN;
        }
        a.ws = static_cast<float *>(ws);
        if (num_ctas <= kTicketCtas) {      // merge partials inside the streaming launch
            a.tickets = reinterpret_cast<unsigned long long *>(static_cast<unsigned char *>(ws) + stream_slot_bytes(plan, num_ctas));
            unsigned long long tag = g_launch_tag.fetch_add(1) & ((1ull << 44) - 1ull);
            if (tag == 0) tag = g_launch_tag.fetch_add(1) & ((1ull << 44) - 1ull);
            a.ticket_tag = (tag << 20) | 1ull;
        }
        if (fused != nullptr) {
            if (a.tickets == nullptr && fused->lens_rw != nullptr) return MOA_ERR_UNSUPPORTED;
            a.Kw = fused->Kw; a.Vw = fused->Vw; a.k_new = fused->k_new; a.v_new = fused->v_new;
            a.lens_rw = fused->lens_rw;
        }
        a.h_kv = h_kv * plan.share;        // virtual kv heads of plan.G query heads each
        a.g_s = (plan.share > 1) ? plan.G : g_s;
        a.kv_share = plan.share;
        e = launch_stream(plan, a, num_ctas, st);
    } else {
        e = launch_generic(a, st);
    }
    if (e != cudaSuccess) return MOA_ERR_CUDA;
    g_last_path = path;
    return MOA_OK;
}

// ---- fixed scratch for the allocation-free entry point ---------------------------------
// Lives in the library image; the host-side name below is only a handle for
// cudaGetSymbolAddress, never a pointer a kernel may be given.
static __device__ __align__(256) unsigned char g_noalloc_scratch[MOA_NOALLOC_SCRATCH_BYTES];
static void *g_noalloc_scratch_dev[kMaxDevices] = {};   // resolved device address, per device

}  // namespace moa

using namespace moa;

extern "C" {

int moa_decode_attn(const float *q, const float *K, const float *V, float *out, int batch,
                    int h_q, int h_kv, int n, int d_k, int d_v, float scale, void *stream)
{
    Lock lock(g_mu);
    return decode_impl(q, K, V, out, batch, h_q, h_kv, nullptr, 0, n, d_k, d_v, scale, nullptr, 0,
                       true, static_cast<cudaStream_t>(stream));
}

int moa_decode_attn_noalloc(const float *q, const float *K, const float *V, float *out, int batch,
                            int h_q, int h_kv, int n, int d_k, int d_v, float scale, void *stream)
{
    Lock lock(g_mu);
    // Argument errors first, exactly as the allocating entry point reports them.
    if (!q || !K || !V || !out) return MOA_ERR_INVALID;
    int rc = validate_dims(batch, h_q, h_kv, n, d_k, d_v);
    if (rc != MOA_OK) return rc;
    DeviceState *dev = nullptr;
    rc = current_device(&dev);
    if (rc != MOA_OK) return rc;
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return MOA_ERR_CUDA; }
    // One-time set-up on this device (it is the current one): turn the array's host-side
    // handle into the address kernels can use.
    if (g_noalloc_scratch_dev[device] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return MOA_ERR_CUDA;
        }
        g_noalloc_scratch_dev[device] = p;
    }
    // Refuse problems whose partial-result slots and counters would not fit the fixed array
    // (the same plan and grid the launch below will use).
    const StreamPlan plan = plan_stream(h_q / h_kv, d_k, d_v);
    if (plan.ok && stream_ws_bytes(plan, stream_grid(*dev, plan, batch, h_kv, n)) > (size_t)MOA_NOALLOC_SCRATCH_BYTES)
        return MOA_ERR_CAPACITY;
    // No CUDA events are created for this call (the launch accounting creates them lazily,
    // which allocates driver objects); its launches are still counted.
    const bool events_saved = g_prof_events;
    if (g_prof_ev == nullptr) g_prof_events = false;
    rc = decode_impl(q, K, V, out, batch, h_q, h_kv, nullptr, 0, n, d_k, d_v, scale,
                     g_noalloc_scratch_dev[device], (size_t)MOA_NOALLOC_SCRATCH_BYTES, false,
                     static_cast<cudaStream_t>(stream), nullptr, false);
    g_prof_events = events_saved;
    return rc;
}

int moa_decode_attn_layers(const float *const *q, const float *const *K, const float *const *V, float *const *out,
                           int layers, int batch, int h_q, int h_kv, int n, int d_k, int d_v, float scale,
                           void *stream)
{
    Lock lock(g_mu);
    if (!q || !K || !V || !out || layers < 1) return MOA_ERR_INVALID;
    for (int l = 0; l < layers; ++l) {
        const int rc = decode_impl(q[l], K[l], V[l], out[l], batch, h_q, h_kv, nullptr, 0, n, d_k, d_v, scale,
                                   nullptr, 0, true, static_cast<cudaStream_t>(stream));
        if (rc != MOA_OK) return rc;
    }
    return MOA_OK;
}

int moa_decode_attn_partial(const float *q, const float *K, const float *V, float *partial, int batch,
                            int h_q, int h_kv, int n, int d_k, int d_v, float scale, void *stream)
{
    Lock lock(g_mu);
    return decode_impl(q, K, V, nullptr, batch, h_q, h_kv, nullptr, 0, n, d_k, d_v, scale, nullptr, 0,
                       true, static_cast<cudaStream_t>(stream), nullptr, true, partial);
}

int moa_combine_partials(const float *partials, int nparts, float *out, int batch, int h_q, int d_v,
                         void *stream)
{
    Lock lock(g_mu);
    if (!partials || !out || nparts < 1 || batch < 1 || h_q < 1 || d_v < 1) return MOA_ERR_INVALID;
    if (d_v > MOA_MAX_DV) return MOA_ERR_UNSUPPORTED;
    if (!aligned(partials, 4) || !aligned(out, 4)) return MOA_ERR_ALIGN;
    const long long rows = (long long)batch * h_q;
    if (rows > 0x7fffffffLL) return MOA_ERR_CAPACITY;
    DeviceState *dev = nullptr;
    int rc = current_device(&dev);
    if (rc != MOA_OK) return rc;
    combine_partials_kernel<<<(int)rows, 128, 0, static_cast<cudaStream_t>(stream)>>>(partials, nparts, out, rows, d_v);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? MOA_OK : MOA_ERR_CUDA;
}

int moa_decode_attn_varlen(const float *q, const float *K, const float *V, float *out, int batch,
                           int h_q, int h_kv, const int32_t *seq_lens, int n_max, int d_k,
                           int d_v, float scale, void *workspace, size_t workspace_bytes,
                           void *stream)
{
    Lock lock(g_mu);
    return decode_impl(q, K, V, out, batch, h_q, h_kv, seq_lens, 0, n_max, d_k, d_v, scale,
                       workspace, workspace_bytes, false, static_cast<cudaStream_t>(stream));
}

size_t moa_workspace_bytes(int batch, int h_q, int h_kv, int n_max, int d_k, int d_v)
{
    Lock lock(g_mu);
    if (validate_dims(batch, h_q, h_kv, n_max, d_k, d_v) != MOA_OK) return 0;
    StreamPlan plan = plan_stream(h_q / h_kv, d_k, d_v);
    if (!plan.ok) return 256;              // generic path: no scratch; keep the result non-zero
    DeviceState *dev = nullptr;
    int ctas = g_num_ctas;
    if (ctas <= 0) ctas = (current_device(&dev) == MOA_OK) ? dev->sm_count : 256;
    size_t need = stream_ws_bytes(plan, ctas);
    const StreamPlan tiled = plan_stream(h_q / h_kv, d_k, d_v, false);   // caches with a row stride
    if (tiled.ok && stream_ws_bytes(tiled, ctas) > need) need = stream_ws_bytes(tiled, ctas);
    if (dev != nullptr || current_device(&dev) == MOA_OK) {
        const GroupedPlan gp = plan_grouped(*dev, batch, h_q, h_kv, n_max, d_k, d_v);
        if (gp.ok && gp.ws_ragged() > need) need = gp.ws_ragged();
        const PairPlan pp = plan_grouped_pair(*dev, batch, h_q, h_kv, n_max, d_k, d_v);
        if (pp.ok && pp.ws_bytes > need) need = pp.ws_bytes;
        if (pp.ok && pp.share == 1 && pp.ws_ragged() > need) need = pp.ws_ragged();
    }
    return (need + 255) / 256 * 256;
}

static int kv_append_impl(float *K, float *V, const float *k_new, const float *v_new, const int32_t *pos,
                          int batch, int h_kv, int n_max, int d_k, int d_v, const Layout &lay, void *stream)
{
    if (!K || !V || !k_new || !v_new || !pos) return MOA_ERR_INVALID;
    if (batch < 1 || h_kv < 1 || n_max < 1 || d_k < 1 || d_v < 1) return MOA_ERR_INVALID;
    if (!aligned(K, 4) || !aligned(V, 4) || !aligned(k_new, 4) || !aligned(v_new, 4) || !aligned(pos, 4))
        return MOA_ERR_ALIGN;
    DeviceState *dev = nullptr;
    int rc = current_device(&dev);
    if (rc != MOA_OK) return rc;
    const long long words = (long long)batch * h_kv * ((long long)d_k + d_v);
    const long long blocks = (words + 255) / 256;
    if (blocks > 0x7fffffffLL) return MOA_ERR_CAPACITY;
    kv_append_kernel<<<(int)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<uint32_t *>(K), reinterpret_cast<uint32_t *>(V),
        reinterpret_cast<const uint32_t *>(k_new), reinterpret_cast<const uint32_t *>(v_new), pos,
        batch, h_kv, n_max, d_k, d_v, lay.k, lay.v);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? MOA_OK : MOA_ERR_CUDA;
}

int moa_kv_append(float *K, float *V, const float *k_new, const float *v_new, const int32_t *pos,
                  int batch, int h_kv, int n_max, int d_k, int d_v, void *stream)
{
    Lock lock(g_mu);
    if (batch < 1 || h_kv < 1 || n_max < 1 || d_k < 1 || d_v < 1) return MOA_ERR_INVALID;
    return kv_append_impl(K, V, k_new, v_new, pos, batch, h_kv, n_max, d_k, d_v,
                          dense_layout(h_kv, n_max, d_k, d_v), stream);
}

// A cache that is written must not alias itself: strides of zero are refused here.
static bool writable_layout(const Layout &l, int batch, int h_kv)
{
    return (batch == 1 || (l.k.sb > 0 && l.v.sb > 0)) && (h_kv == 1 || (l.k.sh > 0 && l.v.sh > 0));
}

int moa_kv_append_strided(float *K, float *V, const float *k_new, const float *v_new, const int32_t *pos,
                          int batch, int h_kv, int n_max, int d_k, int d_v, const long long *k_strides,
                          const long long *v_strides, void *stream)
{
    Lock lock(g_mu);
    if (batch < 1 || h_kv < 1 || n_max < 1 || d_k < 1 || d_v < 1) return MOA_ERR_INVALID;
    Layout lay;
    if (!strided_layout(k_strides, v_strides, h_kv, n_max, d_k, d_v, &lay) || !writable_layout(lay, batch, h_kv))
        return MOA_ERR_INVALID;
    return kv_append_impl(K, V, k_new, v_new, pos, batch, h_kv, n_max, d_k, d_v, lay, stream);
}

int moa_lens_add(int32_t *lens, int batch, int delta, void *stream)
{
    Lock lock(g_mu);
    if (!lens || batch < 1) return MOA_ERR_INVALID;
    if (!aligned(lens, 4)) return MOA_ERR_ALIGN;
    DeviceState *dev = nullptr;
    int rc = current_device(&dev);
    if (rc != MOA_OK) return rc;
    lens_add_kernel<<<(batch + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(lens, batch, delta, 0);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? MOA_OK : MOA_ERR_CUDA;
}

// Shared body of moa_append_decode (advance == false) and moa_decode_step (advance == true).
static int step_impl(const float *q, float *K, float *V, const float *k_new, const float *v_new,
                     float *out, int32_t *lens_rw, const int32_t *lens, int batch, int h_q, int h_kv,
                     int n_max, int d_k, int d_v, float scale, void *workspace, size_t workspace_bytes,
                     void *stream, bool advance, const Layout *layp = nullptr)
{
    if (!q || !K || !V || !k_new || !v_new || !out || !lens) return MOA_ERR_INVALID;
    int rc = validate_dims(batch, h_q, h_kv, n_max, d_k, d_v);
    if (rc != MOA_OK) return rc;
    if (!isfinite(scale)) return MOA_ERR_INVALID;
    if (!aligned(q, 4) || !aligned(K, 4) || !aligned(V, 4) || !aligned(out, 4) || !aligned(lens, 4) ||
        !aligned(k_new, 4) || !aligned(v_new, 4))
        return MOA_ERR_ALIGN;
    DeviceState *dev = nullptr;
    rc = current_device(&dev);
    if (rc != MOA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Layout lay = layp ? *layp : dense_layout(h_kv, n_max, d_k, d_v);
    const StreamPlan plan = plan_stream(h_q / h_kv, d_k, d_v, lay.rows_contig);
    bool fast_ok = plan.ok && lay.vec4 && aligned(q, 16) && aligned(K, 16) && aligned(V, 16) && aligned(out, 16);
    if (fast_ok && plan.mma && !lay.dense) {
        CUtensorMap probe;
        if (!make_rows_map(&probe, K, plan.Dk, n_max, h_kv, batch, lay.k) ||
            !make_rows_map(&probe, V, plan.D, n_max, h_kv, batch, lay.v))
            fast_ok = false;
    }
    const bool stream_path = fast_ok && g_force_path != MOA_PATH_GENERIC;
    if ((g_force_path == MOA_PATH_STREAM || g_force_path == MOA_PATH_MMA) && !fast_ok) return MOA_ERR_UNSUPPORTED;
    if (stream_path) {          // validate the scratch before anything is written
        if (!workspace || workspace_bytes < stream_ws_bytes(plan, stream_num_ctas(*dev))) return MOA_ERR_WORKSPACE;
        if (!aligned(workspace, 256)) return MOA_ERR_ALIGN;
    }
    // One launch: the streaming kernel appends the new rows, attends over len+1 rows and
    // (for the step) advances the lengths when the whole grid is done.
    if (stream_path && aligned(k_new, 16) && aligned(v_new, 16) && stream_num_ctas(*dev) <= kTicketCtas) {
        FusedStep f;
        f.Kw = K; f.Vw = V; f.k_new = k_new; f.v_new = v_new; f.lens_rw = advance ? lens_rw : nullptr;
        return decode_impl(q, K, V, out, batch, h_q, h_kv, lens, 1, n_max, d_k, d_v, scale, workspace,
                           workspace_bytes, false, st, &f, true, nullptr, &lay);
    }
    // Otherwise the same thing as three launches.
    rc = kv_append_impl(K, V, k_new, v_new, lens, batch, h_kv, n_max, d_k, d_v, lay, stream);
    if (rc != MOA_OK) return rc;
    rc = decode_impl(q, K, V, out, batch, h_q, h_kv, lens, 1, n_max, d_k, d_v, scale, workspace,
                     workspace_bytes, false, st, nullptr, true, nullptr, &lay);
    if (rc != MOA_OK || !advance) return rc;
    lens_add_kernel<<<(batch + 127) / 128, 128, 0, st>>>(lens_rw, batch, 1, n_max);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? MOA_OK : MOA_ERR_CUDA;
}

int moa_decode_step(const float *q, float *K, float *V, const float *k_new, const float *v_new,
                    float *out, int32_t *lens, int batch, int h_q, int h_kv, int n_max, int d_k,
                    int d_v, float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    Lock lock(g_mu);
    return step_impl(q, K, V, k_new, v_new, out, lens, lens, batch, h_q, h_kv, n_max, d_k, d_v, scale,
                     workspace, workspace_bytes, stream, true);
}

int moa_append_decode(const float *q, float *K, float *V, const float *k_new, const float *v_new,
                      float *out, const int32_t *pos, int batch, int h_q, int h_kv, int n_max, int d_k,
                      int d_v, float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    Lock lock(g_mu);
    return step_impl(q, K, V, k_new, v_new, out, nullptr, pos, batch, h_q, h_kv, n_max, d_k, d_v, scale,
                     workspace, workspace_bytes, stream, false);
}

int moa_decode_attn_strided(const float *q, const float *K, const float *V, float *out, const int32_t *seq_lens,
                            int batch, int h_q, int h_kv, int n_max, int d_k, int d_v, float scale,
                            const long long *k_strides, const long long *v_strides, void *workspace,
                            size_t workspace_bytes, void *stream)
{
    Lock lock(g_mu);
    if (validate_dims(batch, h_q, h_kv, n_max, d_k, d_v) == MOA_ERR_INVALID) return MOA_ERR_INVALID;
    Layout lay;
    if (!strided_layout(k_strides, v_strides, h_kv, n_max, d_k, d_v, &lay)) return MOA_ERR_INVALID;
    return decode_impl(q, K, V, out, batch, h_q, h_kv, seq_lens, 0, n_max, d_k, d_v, scale, workspace,
                       workspace_bytes, workspace == nullptr, static_cast<cudaStream_t>(stream), nullptr, true,
                       nullptr, &lay);
}

int moa_decode_step_strided(const float *q, float *K, float *V, const float *k_new, const float *v_new, float *out,
                            int32_t *lens, int batch, int h_q, int h_kv, int n_max, int d_k, int d_v, float scale,
                            const long long *k_strides, const long long *v_strides, void *workspace,
                            size_t workspace_bytes, void *stream)
{
    Lock lock(g_mu);
    if (validate_dims(batch, h_q, h_kv, n_max, d_k, d_v) == MOA_ERR_INVALID) return MOA_ERR_INVALID;
    Layout lay;
    if (!strided_layout(k_strides, v_strides, h_kv, n_max, d_k, d_v, &lay) || !writable_layout(lay, batch, h_kv))
        return MOA_ERR_INVALID;
    return step_impl(q, K, V, k_new, v_new, out, lens, lens, batch, h_q, h_kv, n_max, d_k, d_v, scale,
                     workspace, workspace_bytes, stream, true, &lay);
}

int moa_decode_attn_host(const float *q, const float *K, const float *V, float *out, int batch,
                         int h_q, int h_kv, int n, int d_k, int d_v, float scale)
{
    Lock lock(g_mu);
    if (!q || !K || !V || !out) return MOA_ERR_INVALID;
    int rc = validate_dims(batch, h_q, h_kv, n, d_k, d_v);
    if (rc != MOA_OK) return rc;
    if (!isfinite(scale)) return MOA_ERR_INVALID;
    DeviceState *dev = nullptr;
    rc = current_device(&dev);
    if (rc != MOA_OK) return rc;
    if (!dev->host_stream &&
        cudaStreamCreateWithFlags(&dev->host_stream, cudaStreamNonBlocking) != cudaSuccess) {
        cudaGetLastError();
        return MOA_ERR_CUDA;
    }
    const size_t bytes[4] = {sizeof(float) * (size_t)batch * h_q * d_k,
                             sizeof(float) * (size_t)batch * h_kv * n * d_k,
                             sizeof(float) * (size_t)batch * h_kv * n * d_v,
                             sizeof(float) * (size_t)batch * h_q * d_v};
    for (int i = 0; i < 4; ++i) {
        if (dev->stage_bytes[i] < bytes[i]) {
            if (dev->stage[i]) { cudaDeviceSynchronize(); cudaFree(dev->stage[i]); dev->stage[i] = nullptr; dev->stage_bytes[i] = 0; }
            if (cudaMalloc(&dev->stage[i], bytes[i]) != cudaSuccess) { cudaGetLastError(); return MOA_ERR_CUDA; }
            dev->stage_bytes[i] = bytes[i];
        }
    }
    cudaStream_t st = dev->host_stream;
    const void *src[3] = {q, K, V};
    for (int i = 0; i < 3; ++i)
        if (cudaMemcpyAsync(dev->stage[i], src[i], bytes[i], cudaMemcpyHostToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return MOA_ERR_CUDA;
        }
    rc = decode_impl(static_cast<float *>(dev->stage[0]), static_cast<float *>(dev->stage[1]),
                     static_cast<float *>(dev->stage[2]), static_cast<float *>(dev->stage[3]), batch,
                     h_q, h_kv, nullptr, 0, n, d_k, d_v, scale, nullptr, 0, true, st);
    if (rc != MOA_OK) return rc;
    if (cudaMemcpyAsync(out, dev->stage[3], bytes[3], cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return MOA_ERR_CUDA;
    }
    return MOA_OK;
}

int moa_device_status(void *stream, int *status_out)
{
    Lock lock(g_mu);
    if (!status_out) return MOA_ERR_INVALID;
    DeviceState *dev = nullptr;
    int rc = current_device(&dev);
    if (rc != MOA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int v = 0;
    const int zero = 0;
    if (cudaMemcpyFromSymbolAsync(&v, g_status_word, sizeof(int), 0, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyToSymbolAsync(g_status_word, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return MOA_ERR_CUDA;
    }
    *status_out = v;
    return MOA_OK;
}

long long moa_min_bytes(int batch, int h_q, int h_kv, long long n, int d_k, int d_v)
{
    const long long row_pair = (long long)d_k + (long long)d_v;
    return 4LL * batch * (h_kv * n * row_pair + h_q * row_pair);
}

int moa_release(void)
{
    Lock lock(g_mu);
    DeviceState *dev = nullptr;
    int rc = current_device(&dev);
    if (rc != MOA_OK) return rc;
    cudaDeviceSynchronize();
    if (dev->ws) cudaFree(dev->ws);
    dev->ws = nullptr; dev->ws_bytes = 0;
    for (int i = 0; i < 4; ++i) {
        if (dev->stage[i]) cudaFree(dev->stage[i]);
        dev->stage[i] = nullptr; dev->stage_bytes[i] = 0;
    }
    if (dev->host_stream) { cudaStreamDestroy(dev->host_stream); dev->host_stream = nullptr; }
    return cudaGetLastError() == cudaSuccess ? MOA_OK : MOA_ERR_CUDA;
}

const char *moa_strerror(int code)
{
    switch (code) {
    case MOA_OK: return "ok";
    case MOA_ERR_INVALID: return "invalid argument";
    case MOA_ERR_UNSUPPORTED: return "unsupported dimensions or forced path";
    case MOA_ERR_ALIGN: return "misaligned pointer";
    case MOA_ERR_CAPACITY: return "size beyond a fixed capacity";
    case MOA_ERR_WORKSPACE: return "workspace missing or too small";
    case MOA_ERR_CUDA: return "CUDA runtime error";
    default: return "unknown error code";
    }
}

int moa_set_option(int option, int value)
{
    Lock lock(g_mu);
    if (option == MOA_OPT_FORCE_PATH) {
        if (value < 0 || value > MOA_PATH_MMA) return MOA_ERR_INVALID;
        g_force_path = value;
        return MOA_OK;
    }
    if (option == MOA_OPT_GROUPED_HEADS) {
        if (value != 0 && value != 16 && value != 32 && value != 64) return MOA_ERR_INVALID;
        g_grouped_heads = value;
        return MOA_OK;
    }
    if (option == MOA_OPT_GROUPED_OPERANDS) {
        if (value != 0 && value != 1) return MOA_ERR_INVALID;
        g_grouped_operands = value;
        return MOA_OK;
    }
    if (option == MOA_OPT_DEPENDENT_LAUNCH) {
        if (value != 0 && value != 1) return MOA_ERR_INVALID;
        g_dependent_launch = value;
        return MOA_OK;
    }
    if (option == MOA_OPT_WAIT_LIMIT) {
        if (value < 0) return MOA_ERR_INVALID;
        g_wait_limit = value;
        return MOA_OK;
    }
    if (option == MOA_OPT_TEST_SKIP_COPY) {
        if (value < -1) return MOA_ERR_INVALID;
        g_skip_copy_block = value;
        return MOA_OK;
    }
    if (option == MOA_OPT_NUM_CTAS) {
        if (value < 0 || value > 65535) return MOA_ERR_INVALID;
        g_num_ctas = value;
        return MOA_OK;
    }
    return MOA_ERR_INVALID;
}

int moa_last_path(void) { Lock lock(g_mu); return g_last_path; }

int moa_profile(int enable)
{
    Lock lock(g_mu);
    g_prof_on = enable != 0;
    g_prof_events = enable == 2;
    if (g_prof_on) { g_prof_all = 0; g_prof_timed = 0; }
    return MOA_OK;
}

int moa_profile_read(double *decode_kernel_ms, long long *decode_kernel_launches,
                     long long *all_kernel_launches)
{
    Lock lock(g_mu);
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return MOA_ERR_CUDA; }
    double ms = 0.0;
    long long timed = 0;
    for (long long i = 0; i < g_prof_timed; ++i) {
        float t = 0.f;
        if (g_prof_ev && g_prof_ev[2 * i] && g_prof_ev[2 * i + 1] &&
            cudaEventElapsedTime(&t, g_prof_ev[2 * i], g_prof_ev[2 * i + 1]) == cudaSuccess) {
            ms += t;
            ++timed;
        } else {
            cudaGetLastError();
        }
    }
    if (decode_kernel_ms) *decode_kernel_ms = ms;
    if (decode_kernel_launches) *decode_kernel_launches = timed;
    if (all_kernel_launches) *all_kernel_launches = g_prof_all;
    return MOA_OK;
}

int moa_profile_launch_ms(long long index, double *ms)
{
    Lock lock(g_mu);
    if (!ms || index < 0 || index >= g_prof_timed) return MOA_ERR_INVALID;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return MOA_ERR_CUDA; }
    float t = 0.f;
    if (!g_prof_ev || !g_prof_ev[2 * index] || !g_prof_ev[2 * index + 1] ||
        cudaEventElapsedTime(&t, g_prof_ev[2 * index], g_prof_ev[2 * index + 1]) != cudaSuccess) {
        cudaGetLastError();
        return MOA_ERR_CUDA;
    }
    *ms = t;
    return MOA_OK;
}

}  // extern "C"
