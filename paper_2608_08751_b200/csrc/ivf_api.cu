// Host side of the C-ABI library: argument checks, the per-device workspace, the persistent
// schedule, kernel launches, and the chunk pipeline for point sets that live in page-locked host
// memory (Table 3: assignment proceeds in batches; Table 1: the host link is the scarce resource,
// so every chunk crosses it exactly once and the copy of chunk i+1 overlaps the kernels of chunk i).
#include "../../include/ivf_b200.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <string>
#include <type_traits>
#include <utility>
#include <vector>

#include "fused_topk.cuh"
#include "merge.cuh"
#include "candidates.cuh"
#include "pq.cuh"
#include "prep.cuh"
#include "update.cuh"

namespace {

using namespace ivf;

thread_local std::string g_err;
std::atomic<int64_t> g_launches{0};
std::atomic<uint64_t> g_wait_limit_ns{2000000000ull};  // 2 s per device-side wait
std::mutex g_mu;

int fail(int code, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_err = buf;
    return code;
}

#define CUDA_TRY(expr)                                                                         \
    do {                                                                                       \
        cudaError_t e__ = (expr);                                                              \
        if (e__ != cudaSuccess)                                                                \
            return fail(IVF_ERR_CUDA, "%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), \
                        __FILE__, __LINE__);                                                   \
    } while (0)

#define LAUNCH_CHECK()                    \
    do {                                  \
        g_launches.fetch_add(1);          \
        CUDA_TRY(cudaGetLastError());     \
    } while (0)

// ------------------------------------------------------------------ launches that may overlap their predecessor's tail
// Kernels of the routing path begin with griddepcontrol.wait, so they may be launched with the
// programmatic-serialization attribute: the launch latency and the kernel's own set-up then overlap
// the end of the kernel before it.  g_pdl = 0 falls back to ordinary launches (test hook).
// Bit per kernel family: 1 prep, 2 fused, 4 threshold merge, 8 merge, 16 tail kernel (passed-on rows
// and recomputation; 32 unused), 64 centroid update, 128 residual-PQ search.  Measured per family on whole calls: every family gains except the
// threshold merge (its waiting warps sit next to the running threshold pass: 256-query batches lose
// 13 us), so that one is launched normally.  The fused kernel's set-up (TMEM allocation, barrier
// initialisation, tensor-map prefetch) overlaps the end of its predecessor: 5-10 us per call.
int g_pdl = 59 | 64 | 128;  // 64: the centroid-update family, 128: the residual-PQ search
template <typename... KArgs, typename... Args>
cudaError_t launch_dep(int cls, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = (g_pdl & cls) ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#define LAUNCH_DEP(cls, kernel, grid, block, smem, stream, ...)                                \
    do {                                                                                    \
        g_launches.fetch_add(1);                                                            \
        CUDA_TRY(launch_dep(cls, kernel, dim3(grid), dim3(block), smem, stream, __VA_ARGS__));   \
    } while (0)

// ------------------------------------------------------------------ optional per-kernel timing
// When enabled, launches of each kernel family are bracketed by CUDA events on the caller's stream.
enum TimedKind { TK_PREP = 0, TK_FUSED_ARGMIN, TK_FUSED_TOPK, TK_MERGE, TK_UPDATE, TK_THRESH, TK_PQ_ENCODE, TK_PQ_SCAN, TK_PQ_MERGE, TK_NUM };
struct TimedLaunch {
    cudaEvent_t a, b;
    int kind;
};
std::vector<TimedLaunch> g_timed;
std::vector<cudaEvent_t> g_event_pool;  // events are recycled: creating one per launch would make the host the bottleneck
bool g_timing = false;

cudaEvent_t pooled_event() {
    if (!g_event_pool.empty()) {
        cudaEvent_t e = g_event_pool.back();
        g_event_pool.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    return e;
}

int timing_begin(int kind, cudaStream_t stream) {
    if (!g_timing) return -1;
    std::lock_guard<std::mutex> lk(g_mu);
    TimedLaunch t;
    t.kind = kind;
    t.a = pooled_event();
    t.b = pooled_event();
    if (!t.a || !t.b) return -1;
    cudaEventRecord(t.a, stream);
    g_timed.push_back(t);
    return static_cast<int>(g_timed.size()) - 1;
}
void timing_end(int idx, cudaStream_t stream) {
    if (idx < 0) return;
    std::lock_guard<std::mutex> lk(g_mu);
    cudaEventRecord(g_timed[idx].b, stream);
}

// ------------------------------------------------------------------ workspace
enum WsSlot {
    WS_X16, WS_C16, WS_XN, WS_SCAL, WS_BITS, WS_PART, WS_PARTMETA, WS_FAIL, WS_FBKEYS, WS_TAU, WS_SKETCH, WS_OUT_IDS0, WS_OUT_IDS1, WS_OUT_DISTS0, WS_OUT_DISTS1,
    WS_UCNT, WS_UOFF, WS_UCUR, WS_UPERM, WS_IDS, WS_CHUNK0, WS_CHUNK1, WS_PQ_CHUNKS, WS_PQ_GCAND, WS_PQ_GCOUNT, WS_PQ_CBT, WS_UPARTS, WS_NUM
};
struct Buf {
    void* p = nullptr;
    size_t cap = 0;
};
struct DeviceCtx {
    bool init = false;
    int num_sms = 0;
    int* status = nullptr;
    unsigned long long* stats = nullptr;  // 4 counters, only written while g_stats is on
    Buf bufs[WS_NUM];
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_copied[2] = {nullptr, nullptr};
    cudaEvent_t ev_free[2] = {nullptr, nullptr};
    cudaEvent_t ev_ready = nullptr;
    // results read back to page-locked host memory: a stream of its own (the host link carries both
    // directions at once), two staging buffer pairs used in turn
    cudaStream_t out_stream = nullptr;
    cudaEvent_t ev_out_ready[2] = {nullptr, nullptr};  // the kernels that fill staging pair i are done
    cudaEvent_t ev_out_done[2] = {nullptr, nullptr};   // the read-back of staging pair i is done
    bool out_used[2] = {false, false};
    unsigned out_seq = 0;
    bool defer_outputs = false;  // ivf_set_deferred_host_outputs
    bool smem_attr_set = false;
    bool merge_attr_set = false;
    bool pq_attr_set = false;
};
constexpr int kMaxDevices = 64;
DeviceCtx g_ctx[kMaxDevices];

int get_ctx(DeviceCtx** out) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(IVF_ERR_CUDA, "device index %d out of range", dev);
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx& c = g_ctx[dev];
    if (!c.init) {
        cudaDeviceProp prop;
        CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
        if (prop.major != 10)
            return fail(IVF_ERR_UNSUPPORTED, "this library runs on sm_100 devices only (found sm_%d%d)", prop.major,
                        prop.minor);
        c.num_sms = prop.multiProcessorCount;
        CUDA_TRY(cudaMalloc(&c.status, 4 * sizeof(int)));
        CUDA_TRY(cudaMemset(c.status, 0, 4 * sizeof(int)));
        CUDA_TRY(cudaMalloc(&c.stats, 4 * sizeof(unsigned long long)));
        CUDA_TRY(cudaMemset(c.stats, 0, 4 * sizeof(unsigned long long)));
        CUDA_TRY(cudaStreamCreateWithFlags(&c.copy_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            CUDA_TRY(cudaEventCreateWithFlags(&c.ev_copied[i], cudaEventDisableTiming));
            CUDA_TRY(cudaEventCreateWithFlags(&c.ev_free[i], cudaEventDisableTiming));
        }
        CUDA_TRY(cudaEventCreateWithFlags(&c.ev_ready, cudaEventDisableTiming));
        CUDA_TRY(cudaStreamCreateWithFlags(&c.out_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            CUDA_TRY(cudaEventCreateWithFlags(&c.ev_out_ready[i], cudaEventDisableTiming));
            CUDA_TRY(cudaEventCreateWithFlags(&c.ev_out_done[i], cudaEventDisableTiming));
        }
#ifdef IVF_CHECK_BOUNDS
        // checked build: the kernels' index checks report into this device's status word
        CUDA_TRY(cudaMemcpyToSymbol(g_check_status, &c.status, sizeof(int*)));
#endif
        c.init = true;
    }
    *out = &c;
    return IVF_OK;
}

// Grow-only, stream-ordered.
std::atomic<int> g_fail_allocs{0};  // test hook (ivf_debug_fail_next_alloc): workspace allocations to refuse

int ws_get(DeviceCtx& c, WsSlot slot, size_t bytes, cudaStream_t stream, void** out) {
    Buf& b = c.bufs[slot];
    if (bytes > b.cap) {
        if (g_fail_allocs.load() > 0) {
            // refused before anything is freed: the workspace stays as it was
            g_fail_allocs.fetch_sub(1);
            return fail(IVF_ERR_ALLOC, "workspace allocation of %zu bytes refused by the test hook", bytes);
        }
        if (b.p) CUDA_TRY(cudaFreeAsync(b.p, stream));
        b.p = nullptr;
        b.cap = 0;
        size_t want = bytes + bytes / 8;
        want = (want + 255) & ~size_t(255);
        void* p = nullptr;
        cudaError_t e = cudaMallocAsync(&p, want, stream);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return fail(IVF_ERR_ALLOC, "workspace allocation of %zu bytes failed: %s", want, cudaGetErrorString(e));
        }
        b.p = p;
        b.cap = want;
    }
    *out = b.p;
    return IVF_OK;
}
#define WS(slot, bytes, ptrvar)                                                              \
    do {                                                                                     \
        void* p__ = nullptr;                                                                 \
        int rc__ = ws_get(ctx, slot, bytes, stream, &p__);                                   \
        if (rc__ != IVF_OK) return rc__;                                                     \
        ptrvar = reinterpret_cast<typename std::remove_reference<decltype(ptrvar)>::type>(p__);                                    \
    } while (0)

// ------------------------------------------------------------------ schedule
struct Plan {
    int kd, kp, kslices, ksteps, block_n, nstage;
    int mtiles;         // row tiles of 128 points per CTA unit (1 or 2)
    int64_t row_tiles;  // row groups of mtiles * 128 points
    int col_tiles;
    int64_t total_units;
    int cross;  // crossing cost of the span partition, in units
    int ctas;
    int partials;    // slots per row: CTAs that can share a row tile x epilogue halves
    int cap;
    size_t smem;
};

constexpr size_t kSmemLimit = 227 * 1024;
inline int fallback_slices(int nlist) { return (nlist + kFallbackSlice - 1) / kFallbackSlice; }

int log_capacity(int k) { return (k == 1) ? 1 : (4 * k > 512 ? 4 * k : 512); }

// Threshold rule of a k > 1 call, and the centroid stride of the sample that the threshold pass
// looks at (every S-th centroid, S = k / 4: the 16th smallest key of a 4/k sample lets about 4k
// candidates through; P(fewer than k) is about 1e-3 and those rows are recomputed exactly).
constexpr int kMinSampleRows = 512;
int choose_rule(int k, int nlist, int* stride) {
    *stride = 1;
    // k <= 16: the 16 sample keys that define tau are themselves candidates, so the given rule can
    // never come up short; a sample of every 16th centroid lets about 256 candidates through
    const int S = k <= kSampleM ? 16 : k / 4;
    if ((nlist + S - 1) / S >= kMinSampleRows) {
        *stride = S;
        return TAU_GIVEN;
    }
    return k <= kSampleM ? TAU_RUNNING : TAU_BOUNDED;
}

int g_sketch_whole = 1;  // test hook (ivf_debug_set_threshold_pass): 0 = the threshold pass always as sketch kernel + merge
int g_tau_fold = 1;      // same hook: 0 = thresholds of tiny batches by the merge kernel, not inside the main pass
int g_rotate = 1;  // test hook (ivf_debug_set_rotation): 0 = every position of a sweep stands for its own tile index
int g_cross = -1;  // crossing cost used by the span partition; -1 = by kernel variant (test hook: ivf_debug_set_crossing_cost)

int make_plan(int64_t n, int nlist, int d, int k, int num_sms, Plan* pl, bool one_row_tile = false) {
    pl->kd = (d + 63) / 64 * 64;
    pl->kp = pl->kd + kAugK;
    pl->kslices = pl->kd / 64;
    pl->ksteps = (d + 15) / 16;
    pl->block_n = pl->kslices <= 2 ? 256 : 128;
    // two row tiles per unit when they fit next to a two-stage ring (d <= 128) and there are at
    // least two row tiles; the epilogues that keep a candidate log stay with one (they are bound by
    // their own instruction count, not by the centroid traffic, and their per-row state is larger)
    pl->mtiles = (!one_row_tile && n > kBlockM && fused_smem_bytes(pl->kslices, pl->block_n, 2, 2) <= kSmemLimit) ? 2 : 1;
    int nstage = kMaxStages;
    while (nstage > 1 && fused_smem_bytes(pl->kslices, pl->block_n, nstage, pl->mtiles) > kSmemLimit) --nstage;
    if (nstage < 2) return fail(IVF_ERR_UNSUPPORTED, "d = %d does not fit the shared-memory ring", d);
    pl->nstage = nstage;
    pl->smem = fused_smem_bytes(pl->kslices, pl->block_n, nstage, pl->mtiles);
    const int group_rows = kBlockM * pl->mtiles;
    pl->row_tiles = (n + group_rows - 1) / group_rows;
    pl->col_tiles = (nlist + pl->block_n - 1) / pl->block_n;
    pl->total_units = pl->row_tiles * pl->col_tiles;
    pl->ctas = static_cast<int>(pl->total_units < num_sms ? pl->total_units : num_sms);
    // a CTA that changes row group in mid-span loses about g_cross units of time; charge it in the
    // partition when spans are long enough for that to be a correction (and there is more than one
    // row group to cross into)
    // measured: 8 units for the k = 1 kernel (10,240 rows: 163 -> 153 us), about 4 for the others
    int cross = pl->row_tiles > 1 ? (g_cross >= 0 ? g_cross : (k == 1 ? 8 : 4)) : 0;
    const int64_t per_cta = pl->total_units / pl->ctas;
    if (cross > per_cta / 4) cross = static_cast<int>(per_cta / 4);
    if (cross > pl->col_tiles / 2) cross = pl->col_tiles / 2;
    pl->cross = cross;
    int64_t lmin = (pl->row_tiles * static_cast<int64_t>(pl->col_tiles + cross)) / pl->ctas - cross;  // shortest span
    if (lmin < 1) lmin = 1;
    int64_t parts = (pl->col_tiles + lmin - 1) / lmin + 1;
    if (parts > pl->ctas) parts = pl->ctas;
    pl->partials = static_cast<int>(parts) * kEpiHalves;
    pl->cap = log_capacity(k);
    return IVF_OK;
}

// rows per launch so that the per-launch scratch stays bounded
int64_t rows_per_launch(int d, int k) {
    const int kp = (d + 63) / 64 * 64 + kAugK;
    const int64_t per_row = static_cast<int64_t>(kp) * 2 +
                            (k > 1 ? 6ll * (4 * (k < 96 ? 96 : k) + kGroupLogMargin) * kRecordBytes + 6ll * 512 * 8 : 6ll * 8);
    int64_t rows = (int64_t(3) << 30) / per_row;
    rows = rows / (2 * kBlockM) * (2 * kBlockM);
    if (rows < 2 * kBlockM) rows = 2 * kBlockM;
    if (rows > (int64_t(4) << 20)) rows = int64_t(4) << 20;
    return rows;
}

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int get_encode() {
    if (g_encode) return IVF_OK;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (qres != cudaDriverEntryPointSuccess || !fn)
        return fail(IVF_ERR_CUDA, "cuTensorMapEncodeTiled is not available in this driver");
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    return IVF_OK;
}

// fp16 matrix [rows][kp] row-major.  Data map: box = 64 columns x box_rows, 128-byte swizzle.
// Norm-column map: box = 16 columns x box_rows, 32-byte swizzle (read at column kd).
// row_step > 1 maps every row_step-th row (rows = number of rows of that strided view).
int make_tmap(CUtensorMap* map, const void* base, int64_t rows, int kp, int box_rows, bool aug, int row_step = 1) {
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(kp), static_cast<cuuint64_t>(rows)};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(kp) * 2 * row_step};
    cuuint32_t box[2] = {static_cast<cuuint32_t>(aug ? kAugK : kSliceK), static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE,
                          aug ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(IVF_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return IVF_OK;
}

// ------------------------------------------------------------------ argument checks (no CUDA calls)
inline bool valid_dtype(int t) { return t == IVF_F32 || t == IVF_U8 || t == IVF_I8; }
inline size_t dtype_size(int t) { return t == IVF_F32 ? 4 : 1; }
int check_d(int d) {
    if (d < 4 || d > 256 || d % 4 != 0)
        return fail(IVF_ERR_UNSUPPORTED, "d = %d: must be a multiple of 4 in [4, 256]", d);
    return IVF_OK;
}

int check_common(const void* points, int64_t n, int d, int ptype, const float* centroids, int nlist, int k,
                 const int32_t* out_ids) {
    if (n < 0) return fail(IVF_ERR_INVALID_ARG, "negative row count %lld", (long long)n);
    if (!valid_dtype(ptype)) return fail(IVF_ERR_INVALID_ARG, "unknown element type %d", ptype);
    if (check_d(d) != IVF_OK) return IVF_ERR_UNSUPPORTED;
    if (nlist < 1) return fail(IVF_ERR_INVALID_ARG, "nlist = %d", nlist);
    if (k < 1 || k > nlist || k > 512)
        return fail(IVF_ERR_UNSUPPORTED, "nprobe = %d: must be in [1, min(nlist, 512)] (nlist = %d)", k, nlist);
    if (n == 0) return IVF_OK;
    if (!points || !centroids || !out_ids) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    if ((reinterpret_cast<uintptr_t>(points) & 15) || (reinterpret_cast<uintptr_t>(centroids) & 15))
        return fail(IVF_ERR_INVALID_ARG, "points and centroids must be 16-byte aligned");
    return IVF_OK;
}

// 0 = device (or managed), 1 = page-locked host, <0 = error
int classify_pointer(const void* p) {
    cudaPointerAttributes attr;
    cudaError_t e = cudaPointerGetAttributes(&attr, p);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return fail(IVF_ERR_CUDA, "cudaPointerGetAttributes failed: %s", cudaGetErrorString(e));
    }
    if (attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged) return 0;
    if (attr.type == cudaMemoryTypeHost) return 1;
    return fail(IVF_ERR_INVALID_ARG, "pageable host memory is not accepted: pass device or page-locked host memory");
}

// ------------------------------------------------------------------ device-resident building blocks
struct CentroidPrep {
    __half* c16;
    float* scal;
    unsigned int* bits;
    CUtensorMap tmap_c, tmap_ca;    // all centroids
    CUtensorMap tmap_cs, tmap_csa;  // every `stride`-th centroid (threshold pass), if rule == TAU_GIVEN
    int rule, stride, sample_rows;
};

int g_force_fallback = 0;
int g_pq_kernel = 0;  // test hook: 1 forces the scan kernel that reads the codebook through L1
int g_pq_groups = 0;  // test hook: groups per query of ivf_pq_search (0 = chosen from the sizes)
bool g_stats = false;
std::atomic<int64_t> g_row_chunk_override{0};  // test hook: rows per fused launch

// Converts the centroids into cp->c16 (already allocated) and computes their scale; cp->scal and
// cp->bits must point to 4 floats / 2 uints of device memory.
int convert_centroids(DeviceCtx& ctx, const float* centroids, int nlist, int d, const Plan& pl, cudaStream_t stream,
                      CentroidPrep* cp) {
    const int tk = timing_begin(TK_PREP, stream);
    CUDA_TRY(cudaMemsetAsync(cp->bits, 0, 2 * sizeof(unsigned int), stream));
    const int64_t count = static_cast<int64_t>(nlist) * d;
    int blocks = static_cast<int>((count + 256 * 8 - 1) / (256 * 8));
    if (blocks > ctx.num_sms * 8) blocks = ctx.num_sms * 8;
    LAUNCH_DEP(1, maxabs_kernel, blocks, 256, 0, stream, centroids, count, cp->bits + 1);
    // the conversion derives the centroid scale from the magnitude word itself and publishes the scale
    // vector (with the byte-type point scale as a placeholder until the points are known)
    const int rows_per_warp = pl.kd <= 64 ? 4 : (pl.kd <= 128 ? 2 : 1);  // the kernel's lane groups
    const int64_t threads = (static_cast<int64_t>(nlist) + rows_per_warp - 1) / rows_per_warp * 32;
    LAUNCH_DEP(1, (convert_rows_kernel<float, true>), static_cast<unsigned>((threads + 255) / 256), 256, 0, stream,
               centroids, nlist, d, pl.kd, cp->scal, cp->c16, nullptr, cp->bits, 1);
    timing_end(tk, stream);
    return IVF_OK;
}

// Tensor maps over cp->c16 and the threshold rule for nprobe = k.
int map_centroids(int nlist, int k, const Plan& pl, CentroidPrep* cp) {
    int rc = make_tmap(&cp->tmap_c, cp->c16, nlist, pl.kp, pl.block_n, false);
    if (rc != IVF_OK) return rc;
    rc = make_tmap(&cp->tmap_ca, cp->c16, nlist, pl.kp, pl.block_n, true);
    if (rc != IVF_OK) return rc;
    cp->rule = (k == 1) ? TAU_RUNNING : choose_rule(k, nlist, &cp->stride);
    cp->sample_rows = 0;
    if (k > 1 && cp->rule == TAU_GIVEN) {
        cp->sample_rows = (nlist + cp->stride - 1) / cp->stride;
        rc = make_tmap(&cp->tmap_cs, cp->c16, cp->sample_rows, pl.kp, pl.block_n, false, cp->stride);
        if (rc != IVF_OK) return rc;
        rc = make_tmap(&cp->tmap_csa, cp->c16, cp->sample_rows, pl.kp, pl.block_n, true, cp->stride);
        if (rc != IVF_OK) return rc;
    }
    return IVF_OK;
}

int prepare_centroids(DeviceCtx& ctx, const float* centroids, int nlist, int d, int k, const Plan& pl,
                      cudaStream_t stream, CentroidPrep* cp) {
    WS(WS_C16, static_cast<size_t>(nlist) * pl.kp * sizeof(__half), cp->c16);
    WS(WS_SCAL, 4 * sizeof(float), cp->scal);
    WS(WS_BITS, 2 * sizeof(unsigned int), cp->bits);
    int rc = convert_centroids(ctx, centroids, nlist, d, pl, stream, cp);
    if (rc != IVF_OK) return rc;
    return map_centroids(nlist, k, pl, cp);
}

struct PointPrep {
    __half* x16;           // fp16 operand copy (float points), or nullptr
    const uint8_t* x_raw;  // raw uint8 points, widened inside the fused kernel
    int d;
    float* xn;
    CUtensorMap tmap_x, tmap_xa;
};

int launch_fused(DeviceCtx& ctx, const Plan& pl, int64_t n, int nlist, int k, int rule, const float* tau_in,
                 const PointPrep& pp, const CUtensorMap& tmap_c, const CUtensorMap& tmap_ca, Entry* part,
                 int2* part_meta, int kind, cudaStream_t stream, const unsigned int* bits, float* scal,
                 int* clear0 = nullptr, int* clear1 = nullptr, int* clear32 = nullptr, float* tau_out = nullptr,
                 float* sketch_t = nullptr, int sketch_pitch = 0, int sketch_slots = 0) {
    FusedParams fp;
    fp.sketch_t = sketch_t;
    fp.sketch_pitch = sketch_pitch;
    fp.sketch_slots = sketch_slots;
    fp.clear0 = clear0;
    fp.clear1 = clear1;
    fp.clear32 = clear32;
    fp.x_raw = pp.x_raw;
    fp.d = pp.d;
    fp.bits = bits;
    fp.scal_out = scal;
    fp.xn_out = pp.xn;
    fp.n = n;
    fp.nlist = nlist;
    fp.k = k;
    fp.ksteps = pl.ksteps;
    fp.kslices = pl.kslices;
    fp.block_n = pl.block_n;
    fp.nstage = pl.nstage;
    fp.col_tiles = pl.col_tiles;
    fp.total_units = pl.total_units;
    fp.cross = pl.cross;
    fp.rotate = g_rotate;
    fp.partials = pl.partials;
    fp.cap = pl.cap;
    fp.rule = rule;
    fp.tau_in = tau_in;
    fp.tau_out = tau_out;
    fp.whole_rows = tau_out != nullptr ? 1 : 0;
    fp.part = part;
    fp.part_meta = part_meta;
    fp.status = ctx.status;
    fp.stats = g_stats ? ctx.stats : nullptr;
    fp.wait_limit_ns = g_wait_limit_ns.load();
    if (!ctx.smem_attr_set) {
        const int lim = static_cast<int>(kSmemLimit);
        const auto attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
        CUDA_TRY(cudaFuncSetAttribute(fused_topk_kernel<EPI_ARGMIN, 1>, attr, lim));
        CUDA_TRY(cudaFuncSetAttribute(fused_topk_kernel<EPI_ARGMIN, 2>, attr, lim));
        CUDA_TRY(cudaFuncSetAttribute(fused_topk_kernel<EPI_RUNNING, 1>, attr, lim));
        CUDA_TRY(cudaFuncSetAttribute(fused_topk_kernel<EPI_FILTER, 1>, attr, lim));
        CUDA_TRY(cudaFuncSetAttribute(fused_topk_kernel<EPI_GROUPS, 1>, attr, lim));
        CUDA_TRY(cudaFuncSetAttribute(fused_topk_kernel<EPI_GROUPS, 2>, attr, lim));
        CUDA_TRY(cudaFuncSetAttribute(fused_topk_kernel<EPI_SKETCH, 1>, attr, lim));
        CUDA_TRY(cudaFuncSetAttribute(fused_topk_kernel<EPI_SKETCH, 2>, attr, lim));
        ctx.smem_attr_set = true;
    }
    const int tk = timing_begin(kind, stream);
    const dim3 grid(pl.ctas), block(kFusedThreads);
#define IVF_LAUNCH(EPI, MT) \
    LAUNCH_DEP(2, (fused_topk_kernel<EPI, MT>), grid, block, pl.smem, stream, pp.tmap_x, pp.tmap_xa, tmap_c, tmap_ca, fp)
    const bool two = pl.mtiles == 2;
    if (k == 1) {
        if (two) IVF_LAUNCH(EPI_ARGMIN, 2); else IVF_LAUNCH(EPI_ARGMIN, 1);
    } else if (rule == TAU_RUNNING) {
        IVF_LAUNCH(EPI_RUNNING, 1);
    } else if (rule == TAU_SKETCH) {
        if (two) IVF_LAUNCH(EPI_SKETCH, 2); else IVF_LAUNCH(EPI_SKETCH, 1);
    } else if (rule == TAU_GIVEN) {
        if (two) IVF_LAUNCH(EPI_GROUPS, 2); else IVF_LAUNCH(EPI_GROUPS, 1);
    } else {
        IVF_LAUNCH(EPI_FILTER, 1);
    }
#undef IVF_LAUNCH
    timing_end(tk, stream);
    return IVF_OK;
}

MergeParams merge_params(const Plan& pl, int64_t n, int k, const Entry* part, const int2* part_meta,
                         const PointPrep& pp, const float* scal) {
    MergeParams mp;
    mp.n = n;
    mp.k = k;
    mp.partials = pl.partials;
    mp.cap = pl.cap;
    mp.col_tiles = pl.col_tiles;
    mp.total_units = pl.total_units;
    mp.cross = pl.cross;
    mp.ctas = pl.ctas;
    mp.group_rows = kBlockM * pl.mtiles;
    mp.part = part;
    mp.part_meta = part_meta;
    mp.xn = pp.xn;
    mp.scal = scal;
    mp.out_ids = nullptr;
    mp.out_dists = nullptr;
    mp.fail = nullptr;
    mp.force_fail = 0;
    mp.tau_out = nullptr;
    mp.records = 0;
    mp.big = nullptr;
    mp.stats = nullptr;
    return mp;
}

// Routes `n` device-resident rows against prepared centroids.
int route_rows_device(DeviceCtx& ctx, const void* points, int64_t n, int d, int ptype, int nlist, int k,
                      const CentroidPrep& cp, int32_t* out_ids, float* out_dists, cudaStream_t stream) {
    Plan pl, pls;
    int rc = make_plan(n, nlist, d, k, ctx.num_sms, &pl, k > 1 && cp.rule != TAU_GIVEN);
    if (rc != IVF_OK) return rc;
    const bool given = k > 1 && cp.rule == TAU_GIVEN;
    // given rule: the logs hold 48-byte group records, at most 4k + 4 per (row, slot)
    if (given) pl.cap = (k <= kSampleM ? 384 : 4 * k) + kGroupLogMargin;
    size_t part_bytes = static_cast<size_t>(n) * pl.partials * pl.cap * (given ? kRecordBytes : sizeof(Entry));
    size_t meta_bytes = static_cast<size_t>(n) * pl.partials * sizeof(int2);
    // Threshold pass in one kernel: with enough row tiles to occupy the GPU every CTA takes whole row tiles
    // of 128 points across the entire centroid sample and finishes the rows' thresholds itself -- no
    // partial sketches in global memory and no merge launch after it (C1: 36 + 17 us -> one kernel).
    // Small batches keep the split schedule: a few CTAs walking the whole sample would take longer.
    bool sketch_whole = false;
    if (given) {
        const int64_t row_tiles128 = (n + kBlockM - 1) / kBlockM;
        const int sample_tiles = (cp.sample_rows + 255) / 256;
        sketch_whole = g_sketch_whole && row_tiles128 >= 48 && sample_tiles <= 48;
        rc = make_plan(n, cp.sample_rows, d, kSampleM, ctx.num_sms, &pls, sketch_whole);
        if (rc != IVF_OK) return rc;
        if (sketch_whole) {
            pls.ctas = static_cast<int>(pls.row_tiles < ctx.num_sms ? pls.row_tiles : ctx.num_sms);
            pls.partials = kEpiHalves;
        }
        const size_t pb = static_cast<size_t>(n) * pls.partials * pls.cap * sizeof(Entry);
        const size_t mb = static_cast<size_t>(n) * pls.partials * sizeof(int2);
        part_bytes = pb > part_bytes ? pb : part_bytes;
        meta_bytes = mb > meta_bytes ? mb : meta_bytes;
    }
    // Batches of a few rows: the main pass finishes the thresholds from the partial sketches itself (one
    // epilogue warp per row, while the first tiles load), so no merge kernel runs between the two passes.
    // (up to two rows per epilogue warp always; up to four when every CTA has enough tiles to compute
    // meanwhile -- 524,288 lists, B = 32: 77.0 -> 72.6 us, but 65,536 lists: 45.5 -> 47.1)
    const bool tau_fold = given && !sketch_whole && g_tau_fold &&
                          (n <= kFoldRows / 2 || (n <= kFoldRows && pl.col_tiles >= 4 * ctx.num_sms));
    PointPrep pp;
    Entry* part;
    int2* part_meta = nullptr;
    int* failbuf = nullptr;
    uint64_t* fbkeys = nullptr;
    float* tau = nullptr;
    // uint8 rows whose length is a multiple of 16 are widened inside the fused kernel (no copy in HBM);
    // every other input goes through an fp16 operand copy
    const bool u8 = ptype == IVF_U8 && d % 16 == 0;
    pp.x16 = nullptr;
    pp.x_raw = u8 ? static_cast<const uint8_t*>(points) : nullptr;
    pp.d = d;
    if (!u8) WS(WS_X16, static_cast<size_t>(n) * pl.kp * sizeof(__half), pp.x16);
    WS(WS_XN, static_cast<size_t>(n) * sizeof(float), pp.xn);
    WS(WS_PART, part_bytes, part);
    if (k > 1) {
        WS(WS_PARTMETA, meta_bytes, part_meta);
        // failed rows, passed-on rows, and the work counters of the tail kernel
        WS(WS_FAIL, (2 * (static_cast<size_t>(n) + 2) + kTailSyncWords) * sizeof(int), failbuf);
        if (given || g_force_fallback) WS(WS_FBKEYS, static_cast<size_t>(kFallbackFastRows + kFallbackCtas) * fallback_slices(nlist) * k * sizeof(uint64_t), fbkeys);
        if (given) WS(WS_TAU, static_cast<size_t>(n) * sizeof(float), tau);
    }

    int tk = -1;
    if (!u8) {
        // magnitude (float points only: byte types have a fixed bound), scales and the fp16 operand
        // copy with |x|^2
        tk = timing_begin(TK_PREP, stream);
        const int rows_per_warp = pl.kd <= 64 ? 4 : (pl.kd <= 128 ? 2 : 1);
        const int64_t threads = (n + rows_per_warp - 1) / rows_per_warp * 32;
        const unsigned cblocks = static_cast<unsigned>((threads + 255) / 256);
        if (ptype == IVF_F32) {
            CUDA_TRY(cudaMemsetAsync(cp.bits, 0, sizeof(unsigned int), stream));
            const int64_t count = n * d;
            int blocks = static_cast<int>((count + 256 * 8 - 1) / (256 * 8));
            if (blocks > ctx.num_sms * 8) blocks = ctx.num_sms * 8;
            LAUNCH_DEP(1, maxabs_kernel, blocks, 256, 0, stream, static_cast<const float*>(points), count, cp.bits);
            LAUNCH_DEP(1, (convert_rows_kernel<float, false>), cblocks, 256, 0, stream, static_cast<const float*>(points), n, d, pl.kd,
                                                                           cp.scal, pp.x16, pp.xn, cp.bits, 0);
        } else if (ptype == IVF_U8) {
            LAUNCH_DEP(1, (convert_rows_kernel<uint8_t, false>), cblocks, 256, 0, stream, static_cast<const uint8_t*>(points), n, d,
                                                                             pl.kd, cp.scal, pp.x16, pp.xn, cp.bits, 1);
        } else {
            LAUNCH_DEP(1, (convert_rows_kernel<int8_t, false>), cblocks, 256, 0, stream, static_cast<const int8_t*>(points), n, d,
                                                                            pl.kd, cp.scal, pp.x16, pp.xn, cp.bits, 1);
        }
        LAUNCH_CHECK();
        timing_end(tk, stream);
        rc = make_tmap(&pp.tmap_x, pp.x16, n, pl.kp, kBlockM, false);
        if (rc != IVF_OK) return rc;
        rc = make_tmap(&pp.tmap_xa, pp.x16, n, pl.kp, kBlockM, true);
        if (rc != IVF_OK) return rc;
    } else {
        pp.tmap_x = cp.tmap_c;  // unused in this mode; the kernel parameters must still be valid maps
        pp.tmap_xa = cp.tmap_ca;
    }

    float* fold_sketch = nullptr;
    int fold_slots = 0;
    if (given) {
        // threshold pass over every S-th centroid: the 16th smallest group minimum becomes the row's tau
        // (batches of at most kFoldRows rows: the sketches go to a buffer of their own, slot-minor, because
        // the main pass, which finishes the thresholds itself, reads them while it fills `part`)
        float* sketch_t = nullptr;
        if (tau_fold) WS(WS_SKETCH, static_cast<size_t>(n) * kSampleM * pls.partials * sizeof(float), sketch_t);
        rc = launch_fused(ctx, pls, n, cp.sample_rows, kSampleM, TAU_SKETCH, nullptr, pp, cp.tmap_cs, cp.tmap_csa, part,
                          part_meta, TK_THRESH, stream, cp.bits, cp.scal, nullptr, nullptr, nullptr,
                          sketch_whole ? tau : nullptr, sketch_t, pls.partials, 0);
        if (rc != IVF_OK) return rc;
        MergeParams ms = merge_params(pls, n, kSampleM, part, part_meta, pp, cp.scal);
        ms.tau_out = tau;
        tk = timing_begin(TK_THRESH, stream);
        if (sketch_whole) {
            // the kernel wrote the thresholds itself
        } else if (tau_fold) {
            // the main pass finishes them
            fold_sketch = sketch_t;
            // (one sketch per CTA that took part of the row group's sample -- its two epilogue halves merge
            // theirs in shared memory -- or one per half with two row tiles per unit)
            fold_slots = (cta_of_unit(pls.total_units, pls.ctas, pls.col_tiles, pls.cross, pls.col_tiles - 1) -
                          cta_of_unit(pls.total_units, pls.ctas, pls.col_tiles, pls.cross, 0) + 1) *
                         (pls.mtiles == 1 ? 1 : kEpiHalves);
        } else if (pls.partials <= 32)
            LAUNCH_DEP(4, merge_tau_warp_kernel, static_cast<unsigned>((n * 32 + 255) / 256), 256, 0, stream, ms);
        else {
            const int threads = pls.partials >= kTauThreads ? kTauThreads : (pls.partials + 31) / 32 * 32;
            // (a handful of rows: the few waiting CTAs of an early start do not disturb the threshold
            // pass, B = 8: -2 us; hundreds of rows: they do, B = 256: +13 us)
            LAUNCH_DEP(n <= 32 ? 1 : 4, merge_tau_kernel, static_cast<unsigned>(n), threads, 0, stream, ms);
        }
        LAUNCH_CHECK();
        timing_end(tk, stream);
    }
    rc = launch_fused(ctx, pl, n, nlist, k, cp.rule, tau, pp, cp.tmap_c, cp.tmap_ca, part, part_meta,
                      k == 1 ? TK_FUSED_ARGMIN : TK_FUSED_TOPK, stream, cp.bits, cp.scal, failbuf,
                      failbuf ? failbuf + n + 2 : nullptr, failbuf ? failbuf + 2 * (n + 2) : nullptr, nullptr,
                      fold_sketch, pls.partials, fold_slots);
    if (rc != IVF_OK) return rc;

    MergeParams mp = merge_params(pl, n, k, part, part_meta, pp, cp.scal);
    mp.out_ids = out_ids;
    mp.out_dists = out_dists;
    mp.fail = failbuf;
    mp.force_fail = g_force_fallback;
    mp.records = given ? 1 : 0;
    mp.stats = g_stats ? ctx.stats : nullptr;
    tk = timing_begin(TK_MERGE, stream);
    if (k == 1) {
        LAUNCH_DEP(8, merge_argmin_kernel, static_cast<unsigned>((n + 255) / 256), 256, 0, stream, mp);
    } else {
        // warp-per-row fast path first; rows it passes on (many partial logs, many candidates or
        // ties) are listed in `big` and merged by the general CTA-per-row kernel
        // (both list counters were cleared by the fused kernel that just ran)
        mp.big = failbuf + n + 2;
        // three sizes of the warp-level kernel (the smaller the key buffer, the more warps per SM): up to
        // 512 candidates in the buffer / 256 sorted (k <= 68 under the given rule; six CTAs of six warps
        // per SM at 56 registers: a row is one serial chain of about 26 us, so the kernel's time is
        // that chain times the number of rounds the rows need -- 10,000 rows: 3 rounds with 32 warps
        // per SM, 2 with 36: 0.084 -> 0.073 ms), 1024 / 512 (k <= 280;
        // a row with more candidates than fit is cut down to its k smallest in mid-gather, which for
        // k = 256 costs less than the lower occupancy of the next size: C4 chunk 0.52 -> 0.40 ms),
        // 2048 / 1024 (k <= 340); beyond that everything goes to the general path of the tail kernel
        const int expect = given ? 5 * k : 2 * k;
        if (!ctx.merge_attr_set) {
            CUDA_TRY(cudaFuncSetAttribute(merge_warp_kernel<512, 256, 6>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(6 * sizeof(MergeWarpSmem<512>))));
            CUDA_TRY(cudaFuncSetAttribute(merge_warp_kernel<1024, 512, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(8 * sizeof(MergeWarpSmem<1024>))));
            CUDA_TRY(cudaFuncSetAttribute(merge_warp_kernel<2048, 1024, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(4 * sizeof(MergeWarpSmem<2048>))));
            ctx.merge_attr_set = true;
        }
        if (pl.partials > kWarpSlots) {
            // (small batches: every CTA of the fused kernel shared the one row group, so every row has
            // more partial logs than the warp-level kernel takes -- all rows go to the tail kernel)
            mp.big = nullptr;
        } else if (expect <= 340) {
            LAUNCH_DEP(8, (merge_warp_kernel<512, 256, 6>), static_cast<unsigned>((n + 5) / 6), 192, 6 * sizeof(MergeWarpSmem<512>), stream, mp);
        } else if (expect <= 1400) {
            LAUNCH_DEP(8, (merge_warp_kernel<1024, 512, 8>), static_cast<unsigned>((n + 7) / 8), 256, 8 * sizeof(MergeWarpSmem<1024>), stream, mp);
        } else if (expect <= 1700) {
            LAUNCH_DEP(8, (merge_warp_kernel<2048, 1024, 4>), static_cast<unsigned>((n + 3) / 4), 128, 4 * sizeof(MergeWarpSmem<2048>), stream, mp);
        } else {
            mp.big = nullptr;
        }
        {
            // one launch for everything that is rarely needed: rows the warp-level kernel passed on,
            // then the brute-force recomputation of rows whose threshold admitted too few candidates
            TailParams tp;
            tp.mp = mp;
            tp.sync = failbuf + 2 * (n + 2);
            tp.status = ctx.status;
            tp.fallback = (given || g_force_fallback) ? 1 : 0;
            FallbackParams& fb = tp.fb;
            fb.nlist = nlist;
            fb.k = k;
            fb.kp = pl.kp;
            fb.x16 = pp.x16;
            fb.x_raw = pp.x_raw;
            fb.d = d;
            fb.kd = pl.kd;
            fb.c16 = cp.c16;
            fb.xn = pp.xn;
            fb.scal = cp.scal;
            fb.fail = failbuf;
            fb.cand = fbkeys;
            fb.slices = fallback_slices(nlist);
            fb.out_ids = out_ids;
            fb.out_dists = out_dists;
            const int64_t most = (mp.big ? 2 : 8) * static_cast<int64_t>(ctx.num_sms);
            int64_t grid = mp.big ? most : (n < most ? n : most);
            if (grid < kFallbackCtas) grid = kFallbackCtas;
            LAUNCH_DEP(16, route_tail_kernel, static_cast<unsigned>(grid), kMergeThreads, 0, stream, tp);
        }
    }
    timing_end(tk, stream);
    return IVF_OK;
}

int update_device(DeviceCtx& ctx, const void* points, int ptype, const int32_t* ids, int64_t n, int d, int nlist,
                  float* sums, int64_t* counts, cudaStream_t stream) {
    int *cnt, *off, *cur, *perm;
    WS(WS_UCNT, static_cast<size_t>(nlist) * sizeof(int), cnt);
    const int scan_blocks = (nlist + kScanBlock - 1) / kScanBlock;
    WS(WS_UOFF, (static_cast<size_t>(nlist) + 1 + scan_blocks) * sizeof(int), off);
    int* block_sums = off + nlist + 1;
    WS(WS_UCUR, static_cast<size_t>(nlist) * sizeof(int), cur);
    WS(WS_UPERM, static_cast<size_t>(n) * sizeof(int), perm);
    const int tk = timing_begin(TK_UPDATE, stream);
    CUDA_TRY(cudaMemsetAsync(cnt, 0, static_cast<size_t>(nlist) * sizeof(int), stream));
    const unsigned rb = static_cast<unsigned>((n + 255) / 256);
    // (the kernels of this family start with griddepcontrol.wait and are launched as programmatic
    // dependents of one another, family bit 64: their launch latencies overlap -- 0.123 -> 0.112 ms at
    // 65,536 lists; with a few hundred lists the histogram's atomics are the bottleneck and early
    // starters only get in its way (0.93 -> 1.01 ms at 256 lists), so those stay ordinary launches)
    const int fam = (n / nlist >= 4096) ? 0 : 64;
    LAUNCH_DEP(fam, update_hist_kernel, rb, 256, 0, stream, ids, n, nlist, cnt, ctx.status);
    LAUNCH_DEP(fam, update_scan_local_kernel, scan_blocks, 1024, 0, stream, static_cast<const int*>(cnt), nlist, off, block_sums);
    LAUNCH_DEP(fam, update_scan_fix_kernel, scan_blocks, 1024, 0, stream, nlist, off, static_cast<const int*>(block_sums), cur);
    LAUNCH_DEP(fam, update_fill_kernel, rb, 256, 0, stream, ids, n, nlist, static_cast<const int*>(off), cur, perm);
    // few long lists: cut every list into pieces, one warp each, and add the pieces up in order
    const int64_t avg = n / nlist;
    int parts = avg >= 4096 ? static_cast<int>((avg + 2047) / 2048) : 1;
    if (parts > 1024) parts = 1024;
    if (parts > 1) {
        float* scratch;
        WS(WS_UPARTS, static_cast<size_t>(nlist) * parts * d * sizeof(float), scratch);
        const unsigned pb = static_cast<unsigned>((static_cast<int64_t>(nlist) * parts * 32 + 255) / 256);
        const int* cperm = perm;
        const int* coff = off;
        if (ptype == IVF_U8)
            LAUNCH_DEP(fam, update_reduce_parts_kernel<uint8_t>, pb, 256, 0, stream, static_cast<const uint8_t*>(points), cperm, coff, nlist, d, parts, scratch);
        else if (ptype == IVF_I8)
            LAUNCH_DEP(fam, update_reduce_parts_kernel<int8_t>, pb, 256, 0, stream, static_cast<const int8_t*>(points), cperm, coff, nlist, d, parts, scratch);
        else
            LAUNCH_DEP(fam, update_reduce_parts_kernel<float>, pb, 256, 0, stream, static_cast<const float*>(points), cperm, coff, nlist, d, parts, scratch);
        const int64_t cells = static_cast<int64_t>(nlist) * d;
        LAUNCH_DEP(fam, update_combine_parts_kernel, static_cast<unsigned>((cells + 255) / 256), 256, 0, stream,
                   static_cast<const float*>(scratch), coff, nlist, d, parts, sums, reinterpret_cast<long long*>(counts));
        timing_end(tk, stream);
        return IVF_OK;
    }
    const unsigned lb = static_cast<unsigned>((static_cast<int64_t>(nlist) * 32 + 255) / 256);
    {
        const int* cperm = perm;
        const int* coff = off;
        long long* lcounts = reinterpret_cast<long long*>(counts);
        if (ptype == IVF_U8)
            LAUNCH_DEP(fam, update_reduce_kernel<uint8_t>, lb, 256, 0, stream, static_cast<const uint8_t*>(points), cperm, coff, nlist, d, sums, lcounts);
        else if (ptype == IVF_I8)
            LAUNCH_DEP(fam, update_reduce_kernel<int8_t>, lb, 256, 0, stream, static_cast<const int8_t*>(points), cperm, coff, nlist, d, sums, lcounts);
        else
            LAUNCH_DEP(fam, update_reduce_kernel<float>, lb, 256, 0, stream, static_cast<const float*>(points), cperm, coff, nlist, d, sums, lcounts);
    }
    timing_end(tk, stream);
    return IVF_OK;
}

// ------------------------------------------------------------------ the chunk pipeline
// Walks the rows in chunks; a host-resident chunk is staged through one of two device buffers on
// the copy stream.  `with_update` adds the Lloyd accumulation of each chunk.
struct ivf_centroids_impl {
    int device;
    int nlist, d;
    __half* c16;     // fp16 operand copy with the norm columns
    float* scal;     // 4 floats: point scale, centroid scale, 1 / product, A
    unsigned* bits;  // 2 uints: max |x| of the current chunk, max |c|
};

int run_chunks(const void* points, int64_t n, int d, int ptype, const float* centroids, int nlist, int k,
               int32_t* out_ids, float* out_dists, bool with_update, float* sums, int64_t* counts,
               int64_t chunk_rows, cudaStream_t stream, const ivf_centroids_impl* prepared = nullptr) {
    DeviceCtx* pctx = nullptr;
    int rc = get_ctx(&pctx);
    if (rc != IVF_OK) return rc;
    DeviceCtx& ctx = *pctx;
    rc = get_encode();
    if (rc != IVF_OK) return rc;
    const int where = classify_pointer(points);
    if (where < 0) return where;
    const bool host = where == 1;
    const size_t esize = dtype_size(ptype);
    // results: device memory, or page-locked host memory (both arrays of the same kind)
    bool out_host = false;
    if (out_ids) {
        const int ow = classify_pointer(out_ids);
        if (ow < 0) return ow;
        out_host = ow == 1;
        if (out_dists) {
            const int dw = classify_pointer(out_dists);
            if (dw < 0) return dw;
            if ((dw == 1) != out_host)
                return fail(IVF_ERR_INVALID_ARG, "out_ids and out_dists must both be device memory or both page-locked host memory");
        }
    } else if (out_dists) {
        const int dw = classify_pointer(out_dists);
        if (dw < 0) return dw;
        if (dw == 1) return fail(IVF_ERR_INVALID_ARG, "out_dists in host memory needs out_ids in host memory as well");
    }

    int64_t rows = rows_per_launch(d, k);
    if (g_row_chunk_override.load() > 0) rows = g_row_chunk_override.load();
    if (chunk_rows <= 0) chunk_rows = int64_t(1) << 20;
    if ((host || with_update) && rows > chunk_rows) rows = chunk_rows;
    if (rows > n) rows = n;
    // host-resident input in fewer than four chunks: cut it in four, so that only a quarter of the
    // copy is exposed before the first kernel can start (the rest runs under the kernels)
    if (host && g_row_chunk_override.load() <= 0 && (n + rows - 1) / rows < 4 && n >= 4 * 65536) {
        const int64_t quarter = ((n + 3) / 4 + 255) / 256 * 256;
        if (quarter < rows) rows = quarter;
    }
    const int64_t nchunks = (n + rows - 1) / rows;

    Plan pl0;
    rc = make_plan(rows, nlist, d, k, ctx.num_sms, &pl0);
    if (rc != IVF_OK) return rc;
    uint8_t* stage[2] = {nullptr, nullptr};
    int32_t* tmp_ids = nullptr;
    if (host) {
        WS(WS_CHUNK0, static_cast<size_t>(rows) * d * esize, stage[0]);
        if (nchunks > 1) WS(WS_CHUNK1, static_cast<size_t>(rows) * d * esize, stage[1]);
        // the copy stream may touch the staging buffers only after their allocation on `stream`
        CUDA_TRY(cudaEventRecord(ctx.ev_ready, stream));
        CUDA_TRY(cudaStreamWaitEvent(ctx.copy_stream, ctx.ev_ready, 0));
    }
    if (with_update && !out_ids) WS(WS_IDS, static_cast<size_t>(rows) * sizeof(int32_t), tmp_ids);
    int32_t* ostage_ids[2] = {nullptr, nullptr};
    float* ostage_dists[2] = {nullptr, nullptr};
    if (out_host) {
        const size_t ob = static_cast<size_t>(rows) * k * sizeof(int32_t);
        // a staging buffer about to grow is freed in `stream` order: no read-back may still be reading it
        if (ctx.bufs[WS_OUT_IDS0].cap < ob || ctx.bufs[WS_OUT_IDS1].cap < ob ||
            (out_dists && (ctx.bufs[WS_OUT_DISTS0].cap < ob || ctx.bufs[WS_OUT_DISTS1].cap < ob))) {
            for (int i = 0; i < 2; ++i)
                if (ctx.out_used[i]) CUDA_TRY(cudaStreamWaitEvent(stream, ctx.ev_out_done[i], 0));
        }
        WS(WS_OUT_IDS0, ob, ostage_ids[0]);
        WS(WS_OUT_IDS1, ob, ostage_ids[1]);
        if (out_dists) {
            WS(WS_OUT_DISTS0, ob, ostage_dists[0]);
            WS(WS_OUT_DISTS1, ob, ostage_dists[1]);
        }
    }
    int last_out = -1;

    auto issue_copy = [&](int64_t c) -> int {
        const int64_t r0 = c * rows;
        const int64_t nr = (n - r0 < rows) ? (n - r0) : rows;
        const int sb = static_cast<int>(c & 1);
        CUDA_TRY(cudaStreamWaitEvent(ctx.copy_stream, ctx.ev_free[sb], 0));
        CUDA_TRY(cudaMemcpyAsync(stage[sb], static_cast<const uint8_t*>(points) + static_cast<size_t>(r0) * d * esize,
                                 static_cast<size_t>(nr) * d * esize, cudaMemcpyHostToDevice, ctx.copy_stream));
        CUDA_TRY(cudaEventRecord(ctx.ev_copied[sb], ctx.copy_stream));
        return IVF_OK;
    };

    if (host) {
        rc = issue_copy(0);
        if (rc != IVF_OK) return rc;
    }
    // the centroid preparation is enqueued after the first copy was issued, so the two overlap
    CentroidPrep cp;
    if (prepared) {
        cp.c16 = prepared->c16;
        cp.scal = prepared->scal;
        cp.bits = prepared->bits;
        rc = map_centroids(nlist, k, pl0, &cp);
    } else {
        rc = prepare_centroids(ctx, centroids, nlist, d, k, pl0, stream, &cp);
    }
    if (rc != IVF_OK) return rc;
    for (int64_t c = 0; c < nchunks; ++c) {
        const int64_t r0 = c * rows;
        const int64_t nr = (n - r0 < rows) ? (n - r0) : rows;
        const int sb = static_cast<int>(c & 1);
        const void* chunk;
        if (host) {
            if (c + 1 < nchunks) {
                rc = issue_copy(c + 1);
                if (rc != IVF_OK) return rc;
            }
            CUDA_TRY(cudaStreamWaitEvent(stream, ctx.ev_copied[sb], 0));
            chunk = stage[sb];
        } else {
            chunk = static_cast<const uint8_t*>(points) + static_cast<size_t>(r0) * d * esize;
        }
        int32_t* ids_c = out_ids ? out_ids + r0 * k : tmp_ids;
        float* dists_c = out_dists ? out_dists + r0 * k : nullptr;
        int so = 0;
        if (out_host) {
            // this chunk's results go to a staging pair; the pair's previous read-back must be over
            so = static_cast<int>(ctx.out_seq++ & 1u);
            if (ctx.out_used[so]) CUDA_TRY(cudaStreamWaitEvent(stream, ctx.ev_out_done[so], 0));
            ids_c = ostage_ids[so];
            dists_c = out_dists ? ostage_dists[so] : nullptr;
        }
        rc = route_rows_device(ctx, chunk, nr, d, ptype, nlist, k, cp, ids_c, dists_c, stream);
        if (rc != IVF_OK) return rc;
        if (out_host) {
            // read-back on its own stream, under the next chunk's (or the next call's) kernels
            const size_t nb = static_cast<size_t>(nr) * k * sizeof(int32_t);
            CUDA_TRY(cudaEventRecord(ctx.ev_out_ready[so], stream));
            CUDA_TRY(cudaStreamWaitEvent(ctx.out_stream, ctx.ev_out_ready[so], 0));
            CUDA_TRY(cudaMemcpyAsync(out_ids + r0 * k, ids_c, nb, cudaMemcpyDeviceToHost, ctx.out_stream));
            if (out_dists) CUDA_TRY(cudaMemcpyAsync(out_dists + r0 * k, dists_c, nb, cudaMemcpyDeviceToHost, ctx.out_stream));
            CUDA_TRY(cudaEventRecord(ctx.ev_out_done[so], ctx.out_stream));
            ctx.out_used[so] = true;
            last_out = so;
        }
        if (with_update) {
            rc = update_device(ctx, chunk, ptype, ids_c, nr, d, nlist, sums, counts, stream);
            if (rc != IVF_OK) return rc;
        }
        if (host) CUDA_TRY(cudaEventRecord(ctx.ev_free[sb], stream));
    }
    // plain stream semantics unless the caller asked otherwise: the call is complete in `stream` only
    // when its results are in host memory (the read-back stream is in order, so the last event covers all)
    if (last_out >= 0 && !ctx.defer_outputs) CUDA_TRY(cudaStreamWaitEvent(stream, ctx.ev_out_done[last_out], 0));
    return IVF_OK;
}

}  // namespace

// ====================================================================== exported C functions
extern "C" {

int ivf_route(const void* queries, int64_t nq, int d, ivf_dtype qtype, const float* centroids, int nlist, int nprobe,
              int32_t* out_ids, float* out_dists, void* stream) {
    int rc = check_common(queries, nq, d, qtype, centroids, nlist, nprobe, out_ids);
    if (rc != IVF_OK || nq == 0) return rc;
    return run_chunks(queries, nq, d, qtype, centroids, nlist, nprobe, out_ids, out_dists, false, nullptr, nullptr, 0,
                      static_cast<cudaStream_t>(stream));
}

int ivf_centroids_create(const float* centroids, int nlist, int d, ivf_centroids** out, void* stream_) {
    if (!out) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    *out = nullptr;
    if (check_d(d) != IVF_OK) return IVF_ERR_UNSUPPORTED;
    if (nlist < 1) return fail(IVF_ERR_INVALID_ARG, "nlist = %d", nlist);
    if (!centroids) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    if (reinterpret_cast<uintptr_t>(centroids) & 15) return fail(IVF_ERR_INVALID_ARG, "centroids must be 16-byte aligned");
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != IVF_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Plan pl;
    rc = make_plan(kBlockM, nlist, d, 1, ctx->num_sms, &pl);
    if (rc != IVF_OK) return rc;
    ivf_centroids_impl* h = new ivf_centroids_impl();
    CUDA_TRY(cudaGetDevice(&h->device));
    h->nlist = nlist;
    h->d = d;
    void* mem = nullptr;
    const size_t c16_bytes = (static_cast<size_t>(nlist) * pl.kp * sizeof(__half) + 255) & ~size_t(255);
    cudaError_t e = cudaMallocAsync(&mem, c16_bytes + 256, stream);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        delete h;
        return fail(IVF_ERR_ALLOC, "allocation of %zu bytes for the prepared centroids failed: %s", c16_bytes + 256,
                    cudaGetErrorString(e));
    }
    h->c16 = static_cast<__half*>(mem);
    h->scal = reinterpret_cast<float*>(static_cast<uint8_t*>(mem) + c16_bytes);
    h->bits = reinterpret_cast<unsigned*>(h->scal + 4);
    CentroidPrep cp;
    cp.c16 = h->c16;
    cp.scal = h->scal;
    cp.bits = h->bits;
    rc = convert_centroids(*ctx, centroids, nlist, d, pl, stream, &cp);
    if (rc != IVF_OK) {
        cudaFreeAsync(mem, stream);
        delete h;
        return rc;
    }
    *out = reinterpret_cast<ivf_centroids*>(h);
    return IVF_OK;
}

int ivf_centroids_destroy(ivf_centroids* handle, void* stream) {
    if (!handle) return IVF_OK;
    ivf_centroids_impl* h = reinterpret_cast<ivf_centroids_impl*>(handle);
    CUDA_TRY(cudaFreeAsync(h->c16, static_cast<cudaStream_t>(stream)));
    delete h;
    return IVF_OK;
}

int ivf_route_prepared(const ivf_centroids* handle, const void* queries, int64_t nq, ivf_dtype qtype, int nprobe,
                       int32_t* out_ids, float* out_dists, void* stream) {
    if (!handle) return fail(IVF_ERR_INVALID_ARG, "null centroid handle");
    const ivf_centroids_impl* h = reinterpret_cast<const ivf_centroids_impl*>(handle);
    int rc = check_common(queries, nq, h->d, qtype, reinterpret_cast<const float*>(h->c16), h->nlist, nprobe, out_ids);
    if (rc != IVF_OK || nq == 0) return rc;
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev != h->device) return fail(IVF_ERR_INVALID_ARG, "the centroid handle belongs to device %d, current is %d", h->device, dev);
    return run_chunks(queries, nq, h->d, qtype, nullptr, h->nlist, nprobe, out_ids, out_dists, false, nullptr, nullptr, 0,
                      static_cast<cudaStream_t>(stream), h);
}

int ivf_assign(const void* points, int64_t n, int d, ivf_dtype ptype, const float* centroids, int nlist,
               int32_t* out_ids, float* out_dists, void* stream) {
    int rc = check_common(points, n, d, ptype, centroids, nlist, 1, out_ids);
    if (rc != IVF_OK || n == 0) return rc;
    return run_chunks(points, n, d, ptype, centroids, nlist, 1, out_ids, out_dists, false, nullptr, nullptr, 0,
                      static_cast<cudaStream_t>(stream));
}

int ivf_centroid_update(const void* points, ivf_dtype ptype, const int32_t* ids, int64_t n, int d, int nlist,
                        float* sums, int64_t* counts, void* stream) {
    if (n < 0) return fail(IVF_ERR_INVALID_ARG, "negative row count %lld", (long long)n);
    if (!valid_dtype(ptype)) return fail(IVF_ERR_INVALID_ARG, "unknown element type %d", (int)ptype);
    if (check_d(d) != IVF_OK) return IVF_ERR_UNSUPPORTED;
    if (nlist < 1) return fail(IVF_ERR_INVALID_ARG, "nlist = %d", nlist);
    if (n >= (int64_t(1) << 31)) return fail(IVF_ERR_UNSUPPORTED, "n = %lld: at most 2^31 - 1 rows per call", (long long)n);
    if (n == 0) return IVF_OK;
    if (!points || !ids || !sums || !counts) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    if ((reinterpret_cast<uintptr_t>(points) & 15) || (reinterpret_cast<uintptr_t>(sums) & 15))
        return fail(IVF_ERR_INVALID_ARG, "points and sums must be 16-byte aligned");
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != IVF_OK) return rc;
    return update_device(*ctx, points, ptype, ids, n, d, nlist, sums, counts, static_cast<cudaStream_t>(stream));
}

int ivf_cluster_major_reorder(const void* points, ivf_dtype ptype, const int32_t* ids, int64_t n, int d, int nlist,
                              void* out_points, int64_t* out_offsets, int32_t* out_order, void* stream_) {
    if (n < 0) return fail(IVF_ERR_INVALID_ARG, "negative row count %lld", (long long)n);
    if (!valid_dtype(ptype)) return fail(IVF_ERR_INVALID_ARG, "unknown element type %d", (int)ptype);
    if (check_d(d) != IVF_OK) return IVF_ERR_UNSUPPORTED;
    if (nlist < 1) return fail(IVF_ERR_INVALID_ARG, "nlist = %d", nlist);
    if (n >= (int64_t(1) << 31)) return fail(IVF_ERR_UNSUPPORTED, "n = %lld: at most 2^31 - 1 rows per call", (long long)n);
    if (!out_offsets || !out_order) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    if (n > 0 && (!points || !ids || !out_points)) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    if ((reinterpret_cast<uintptr_t>(points) & 15) || (reinterpret_cast<uintptr_t>(out_points) & 15))
        return fail(IVF_ERR_INVALID_ARG, "points and out_points must be 16-byte aligned");
    DeviceCtx* pctx = nullptr;
    int rc = get_ctx(&pctx);
    if (rc != IVF_OK) return rc;
    DeviceCtx& ctx = *pctx;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int *cnt, *off, *cur;
    const int scan_blocks = (nlist + kScanBlock - 1) / kScanBlock;
    WS(WS_UCNT, static_cast<size_t>(nlist) * sizeof(int), cnt);
    WS(WS_UOFF, (static_cast<size_t>(nlist) + 1 + scan_blocks) * sizeof(int), off);
    WS(WS_UCUR, static_cast<size_t>(nlist) * sizeof(int), cur);
    int* block_sums = off + nlist + 1;
    const int tk = timing_begin(TK_UPDATE, stream);
    CUDA_TRY(cudaMemsetAsync(cnt, 0, static_cast<size_t>(nlist) * sizeof(int), stream));
    const unsigned rb = static_cast<unsigned>((n + 255) / 256);
    if (n > 0) {
        update_hist_kernel<<<rb, 256, 0, stream>>>(ids, n, nlist, cnt, ctx.status);
        LAUNCH_CHECK();
    }
    update_scan_local_kernel<<<scan_blocks, 1024, 0, stream>>>(cnt, nlist, off, block_sums);
    LAUNCH_CHECK();
    update_scan_fix_kernel<<<scan_blocks, 1024, 0, stream>>>(nlist, off, block_sums, cur);
    LAUNCH_CHECK();
    widen_offsets_kernel<<<(nlist + 256) / 256, 256, 0, stream>>>(off, nlist, reinterpret_cast<long long*>(out_offsets));
    LAUNCH_CHECK();
    if (n > 0) {
        update_fill_kernel<<<rb, 256, 0, stream>>>(ids, n, nlist, off, cur, out_order);
        LAUNCH_CHECK();
        const int row_bytes = d * static_cast<int>(dtype_size(ptype));
        if (row_bytes % 16 == 0) {
            const int row_chunks = row_bytes / 16;
            const int64_t pieces = n * row_chunks;
            reorder_gather_kernel<uint4><<<static_cast<unsigned>((pieces + 255) / 256), 256, 0, stream>>>(
                static_cast<const uint4*>(points), out_order, n, row_chunks, off + nlist, static_cast<uint4*>(out_points));
        } else {
            const int row_chunks = row_bytes / 4;
            const int64_t pieces = n * row_chunks;
            reorder_gather_kernel<uint32_t><<<static_cast<unsigned>((pieces + 255) / 256), 256, 0, stream>>>(
                static_cast<const uint32_t*>(points), out_order, n, row_chunks, off + nlist, static_cast<uint32_t*>(out_points));
        }
        LAUNCH_CHECK();
    }
    timing_end(tk, stream);
    return IVF_OK;
}

int ivf_centroid_finalize(const float* sums, const int64_t* counts, int nlist, int d, float* centroids_inout,
                          void* stream) {
    if (nlist < 1 || d < 1) return fail(IVF_ERR_INVALID_ARG, "nlist = %d, d = %d", nlist, d);
    if (!sums || !counts || !centroids_inout) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    const int64_t total = static_cast<int64_t>(nlist) * d;
    finalize_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        sums, reinterpret_cast<const long long*>(counts), nlist, d, centroids_inout);
    LAUNCH_CHECK();
    return IVF_OK;
}

int ivf_assign_update(const void* points, int64_t n, int d, ivf_dtype ptype, const float* centroids, int nlist,
                      int32_t* out_ids, float* out_dists, float* sums, int64_t* counts, int64_t chunk_rows,
                      void* stream) {
    int32_t dummy = 0;
    int rc = check_common(points, n, d, ptype, centroids, nlist, 1, out_ids ? out_ids : &dummy);
    if (rc != IVF_OK || n == 0) return rc;
    if (!sums || !counts) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    if (reinterpret_cast<uintptr_t>(sums) & 15) return fail(IVF_ERR_INVALID_ARG, "sums must be 16-byte aligned");
    return run_chunks(points, n, d, ptype, centroids, nlist, 1, out_ids, out_dists, true, sums, counts, chunk_rows,
                      static_cast<cudaStream_t>(stream));
}

int ivf_merge_shards(const int32_t* shard_ids, const float* shard_dists, int parts, int64_t nq, int k,
                     int32_t* out_ids, float* out_dists, void* stream_) {
    if (nq < 0) return fail(IVF_ERR_INVALID_ARG, "negative query count %lld", (long long)nq);
    if (parts < 1) return fail(IVF_ERR_INVALID_ARG, "parts = %d", parts);
    if (k < 1 || k > kFallbackMaxK) return fail(IVF_ERR_UNSUPPORTED, "k = %d: must be in [1, %d]", k, kFallbackMaxK);
    if (nq >= (int64_t(1) << 31)) return fail(IVF_ERR_UNSUPPORTED, "nq = %lld: at most 2^31 - 1 queries per call", (long long)nq);
    if (nq == 0) return IVF_OK;
    if (!shard_ids || !shard_dists || !out_ids) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    ShardMergeParams sp;
    sp.nq = nq;
    sp.k = k;
    sp.parts = parts;
    sp.ids = shard_ids;
    sp.dists = shard_dists;
    sp.out_ids = out_ids;
    sp.out_dists = out_dists;
    merge_shards_kernel<<<static_cast<unsigned>(nq), kMergeThreads, 0, static_cast<cudaStream_t>(stream_)>>>(sp);
    LAUNCH_CHECK();
    return IVF_OK;
}

int ivf_assign_candidates(const void* points, int64_t n, int d, ivf_dtype ptype, const float* centroids, int nlist,
                          const int32_t* cand_ids, int m, int32_t* out_ids, float* out_dists, void* stream_) {
    if (n < 0) return fail(IVF_ERR_INVALID_ARG, "negative row count %lld", (long long)n);
    if (!valid_dtype(ptype)) return fail(IVF_ERR_INVALID_ARG, "unknown element type %d", (int)ptype);
    if (d < 4 || d > kCandMaxD || d % 4 != 0)
        return fail(IVF_ERR_UNSUPPORTED, "d = %d: must be a multiple of 4 in [4, %d]", d, kCandMaxD);
    if (nlist < 1 || m < 1) return fail(IVF_ERR_INVALID_ARG, "nlist = %d, candidates per row = %d", nlist, m);
    if (n == 0) return IVF_OK;
    if (!points || !centroids || !cand_ids || !out_ids) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    if ((reinterpret_cast<uintptr_t>(points) & 15) || (reinterpret_cast<uintptr_t>(centroids) & 15))
        return fail(IVF_ERR_INVALID_ARG, "points and centroids must be 16-byte aligned");
    DeviceCtx* pctx = nullptr;
    int rc = get_ctx(&pctx);
    if (rc != IVF_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int tk = timing_begin(TK_FUSED_ARGMIN, stream);
    const unsigned grid = static_cast<unsigned>((n * 32 + 255) / 256);
    if (ptype == IVF_U8)
        assign_candidates_kernel<uint8_t><<<grid, 256, 0, stream>>>(static_cast<const uint8_t*>(points), n, d, centroids, nlist,
                                                                    cand_ids, m, out_ids, out_dists, pctx->status);
    else if (ptype == IVF_I8)
        assign_candidates_kernel<int8_t><<<grid, 256, 0, stream>>>(static_cast<const int8_t*>(points), n, d, centroids, nlist,
                                                                   cand_ids, m, out_ids, out_dists, pctx->status);
    else
        assign_candidates_kernel<float><<<grid, 256, 0, stream>>>(static_cast<const float*>(points), n, d, centroids, nlist,
                                                                  cand_ids, m, out_ids, out_dists, pctx->status);
    LAUNCH_CHECK();
    timing_end(tk, stream);
    return IVF_OK;
}

// ------------------------------------------------------------------ residual-PQ candidate reduction
namespace {
int pq_check_shape(int d, int pq_m, const float* codebooks, bool encode) {
    if (d < 1 || pq_m < 1 || d % pq_m != 0)
        return fail(IVF_ERR_INVALID_ARG, "d = %d, pq_m = %d: pq_m must divide d", d, pq_m);
    if (!codebooks) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    size_t need = encode ? pq_smem_bytes(d, pq_m) : pq_scan_smem_bytes(d, pq_m);
    if (encode && pq_encode_smem_bytes(d) > need) need = pq_encode_smem_bytes(d);
    if (need > kSmemLimit || d > 256)
        return fail(IVF_ERR_UNSUPPORTED, "d = %d, pq_m = %d: %zu bytes of shared memory needed (limit %zu), d at most 256", d,
                    pq_m, need, static_cast<size_t>(kSmemLimit));
    return IVF_OK;
}
int pq_set_attrs(DeviceCtx& ctx) {
    if (!ctx.pq_attr_set) {
        CUDA_TRY(cudaFuncSetAttribute(pq_encode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      static_cast<int>(kSmemLimit)));
        CUDA_TRY(cudaFuncSetAttribute(pq_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      static_cast<int>(kSmemLimit)));
        CUDA_TRY(cudaFuncSetAttribute(pq_scan_teams_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      static_cast<int>(kSmemLimit)));
        ctx.pq_attr_set = true;
    }
    return IVF_OK;
}
}  // namespace

int ivf_pq_residuals(const void* points, int64_t n, int d, ivf_dtype ptype, const int32_t* ids, const float* centroids,
                     int nlist, float* out_residuals, void* stream_) {
    if (n < 0) return fail(IVF_ERR_INVALID_ARG, "negative row count %lld", (long long)n);
    if (!valid_dtype(ptype)) return fail(IVF_ERR_INVALID_ARG, "unknown element type %d", (int)ptype);
    if (d < 1 || nlist < 1) return fail(IVF_ERR_INVALID_ARG, "d = %d, nlist = %d", d, nlist);
    if (n == 0) return IVF_OK;
    if (!points || !ids || !centroids || !out_residuals) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    DeviceCtx* pctx = nullptr;
    int rc = get_ctx(&pctx);
    if (rc != IVF_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int64_t total = n * d;
    pq_residuals_kernel<<<static_cast<unsigned>((total + 255) / 256), 256, 0, stream>>>(points, static_cast<int>(ptype), n, d, ids,
                                                                                     centroids, nlist, out_residuals,
                                                                                     pctx->status);
    LAUNCH_CHECK();
    return IVF_OK;
}

int ivf_pq_encode(const void* points, int64_t n, int d, ivf_dtype ptype, const int32_t* ids, const float* centroids,
                  int nlist, const float* codebooks, int pq_m, uint8_t* out_codes, void* stream_) {
    if (n < 0) return fail(IVF_ERR_INVALID_ARG, "negative row count %lld", (long long)n);
    if (!valid_dtype(ptype)) return fail(IVF_ERR_INVALID_ARG, "unknown element type %d", (int)ptype);
    if (nlist < 1) return fail(IVF_ERR_INVALID_ARG, "nlist = %d", nlist);
    int rc = pq_check_shape(d, pq_m, codebooks, true);
    if (rc != IVF_OK) return rc;
    if (n == 0) return IVF_OK;
    if (!points || !ids || !centroids || !out_codes) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    DeviceCtx* pctx = nullptr;
    rc = get_ctx(&pctx);
    if (rc != IVF_OK) return rc;
    DeviceCtx& ctx = *pctx;
    rc = pq_set_attrs(ctx);
    if (rc != IVF_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    PqEncodeParams p;
    p.x = points;
    p.x_type = ptype;
    p.n = n;
    p.d = d;
    p.pq_m = pq_m;
    p.nlist = nlist;
    p.ids = ids;
    p.centroids = centroids;
    p.codebooks = codebooks;
    p.codes = out_codes;
    p.status = ctx.status;
    const int tk = timing_begin(TK_PQ_ENCODE, stream);
    const unsigned grid = static_cast<unsigned>(n < ctx.num_sms ? n : ctx.num_sms);
    pq_encode_kernel<<<grid, kPqThreads, pq_encode_smem_bytes(d), stream>>>(p);
    LAUNCH_CHECK();
    timing_end(tk, stream);
    return IVF_OK;
}

int ivf_pq_search(const void* queries, int64_t nq, int d, ivf_dtype qtype, const float* centroids, int nlist,
                  const int32_t* probe_ids, int nprobe, const int64_t* list_offsets, const uint8_t* codes,
                  int64_t n_codes, const float* codebooks, int pq_m, int n_rerank, const int64_t* vec_ids,
                  int64_t* out_ids, float* out_est, int64_t* out_counts, void* stream_) {
    if (nq < 0) return fail(IVF_ERR_INVALID_ARG, "negative query count %lld", (long long)nq);
    if (!valid_dtype(qtype)) return fail(IVF_ERR_INVALID_ARG, "unknown element type %d", (int)qtype);
    if (nlist < 1) return fail(IVF_ERR_INVALID_ARG, "nlist = %d", nlist);
    if (nprobe < 1 || nprobe > nlist) return fail(IVF_ERR_INVALID_ARG, "nprobe = %d with nlist = %d", nprobe, nlist);
    if (nprobe > kPqMaxProbes) return fail(IVF_ERR_UNSUPPORTED, "nprobe = %d: at most %d", nprobe, kPqMaxProbes);
    if (n_rerank < 1 || n_rerank > kPqMaxRerank)
        return fail(IVF_ERR_UNSUPPORTED, "n_rerank = %d: must be in [1, %d]", n_rerank, kPqMaxRerank);
    if (n_codes < 0 || n_codes >= (int64_t(1) << 32))
        return fail(IVF_ERR_UNSUPPORTED, "n_codes = %lld: positions must fit 32 bits", (long long)n_codes);
    if (nq >= (int64_t(1) << 24)) return fail(IVF_ERR_UNSUPPORTED, "nq = %lld: at most 2^24 - 1 queries per call", (long long)nq);
    int rc = pq_check_shape(d, pq_m, codebooks, false);
    if (rc != IVF_OK) return rc;
    if (nq == 0) return IVF_OK;
    if (!queries || !centroids || !probe_ids || !list_offsets || !out_ids || !out_est || (n_codes > 0 && !codes))
        return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    if (reinterpret_cast<uintptr_t>(codes) & 15) return fail(IVF_ERR_INVALID_ARG, "codes must be 16-byte aligned");
    DeviceCtx* pctx = nullptr;
    rc = get_ctx(&pctx);
    if (rc != IVF_OK) return rc;
    DeviceCtx& ctx = *pctx;
    rc = pq_set_attrs(ctx);
    if (rc != IVF_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    // groups per query: enough CTAs of work for every SM even at serving-size batches
    // (but no more than one per ~4 chunks of the codes a query is expected to scan: a group hands
    // on up to n_rerank candidates however little it scanned)
    int ngroups = static_cast<int>((8 * static_cast<int64_t>(ctx.num_sms) + nq - 1) / nq);
    const int64_t expect_codes = static_cast<int64_t>(nprobe) * (n_codes / nlist + 1);
    const int64_t by_work = expect_codes / (4 * kPqChunk);
    if (ngroups > by_work) ngroups = static_cast<int>(by_work);
    if (g_pq_groups > 0) ngroups = g_pq_groups;
    if (ngroups < 1) ngroups = 1;
    if (ngroups > 256) ngroups = 256;
    const int64_t total_groups = nq * ngroups;
    int* chunk_start;
    uint64_t* gcand;
    int* gcount;
    WS(WS_PQ_CHUNKS, static_cast<size_t>(nq) * (nprobe + 1) * sizeof(int), chunk_start);
    WS(WS_PQ_GCAND, static_cast<size_t>(total_groups) * n_rerank * sizeof(uint64_t), gcand);
    WS(WS_PQ_GCOUNT, static_cast<size_t>(total_groups) * sizeof(int), gcount);
    float* cbt;
    WS(WS_PQ_CBT, static_cast<size_t>(d) * kPqK * sizeof(float), cbt);
    int tk = timing_begin(TK_PQ_SCAN, stream);
    // (family bit 128 of the dependent-launch mask: the four kernels of a search overlap their launch
    // latencies, which is a tenth of a small batch)
    // the scan reads the codebook as given where one codeword is one aligned vector load
    const bool cb_rows = pq_codebook_by_rows(d / pq_m) && (reinterpret_cast<uintptr_t>(codebooks) & 15) == 0;
    if (!cb_rows)
        LAUNCH_DEP(128, pq_transpose_codebooks_kernel, (d * kPqK + 255) / 256, 256, 0, stream, codebooks, d, d / pq_m, cbt);
    LAUNCH_DEP(128, pq_setup_query_kernel, static_cast<unsigned>(nq), 128, 0, stream, probe_ids, nprobe, nlist,
               reinterpret_cast<const long long*>(list_offsets), chunk_start, reinterpret_cast<long long*>(out_counts),
               ctx.status);
    PqScanParams sp;
    sp.q = queries;
    sp.q_type = qtype;
    sp.nq = nq;
    sp.d = d;
    sp.pq_m = pq_m;
    sp.nlist = nlist;
    sp.nprobe = nprobe;
    sp.n_rerank = n_rerank;
    sp.ngroups = ngroups;
    sp.centroids = centroids;
    sp.cbt = cb_rows ? codebooks : cbt;
    sp.cb_rows = cb_rows ? 1 : 0;
    sp.probes = probe_ids;
    sp.offsets = reinterpret_cast<const long long*>(list_offsets);
    sp.codes = codes;
    sp.chunk_start = chunk_start;
    sp.gcand = gcand;
    sp.gcand_count = gcount;
    sp.status = ctx.status;
    // two teams per CTA around one shared-memory codebook when that fits; otherwise (or when asked by
    // the test hook) two single-team CTAs per SM that read the codebook through L1
    const bool teams = g_pq_kernel != 1 && nprobe <= kPqTeamProbes && pq_teams_smem_bytes(d, pq_m) <= kSmemLimit;
    if (teams) {
        const int64_t pairs = (total_groups + 1) / 2;
        const unsigned grid = static_cast<unsigned>(pairs < ctx.num_sms ? pairs : ctx.num_sms);
        LAUNCH_DEP(128, pq_scan_teams_kernel, grid, 2 * kPqScanThreads, pq_teams_smem_bytes(d, pq_m), stream, sp);
    } else {
        const int64_t resident = 2 * static_cast<int64_t>(ctx.num_sms);
        const unsigned grid = static_cast<unsigned>(total_groups < resident ? total_groups : resident);
        LAUNCH_DEP(128, pq_scan_kernel, grid, kPqScanThreads, pq_scan_smem_bytes(d, pq_m), stream, sp);
    }
    timing_end(tk, stream);
    tk = timing_begin(TK_PQ_MERGE, stream);
    PqMergeParams mp;
    mp.nq = nq;
    mp.n_rerank = n_rerank;
    mp.ngroups = ngroups;
    mp.gcand = gcand;
    mp.gcand_count = gcount;
    mp.vec_ids = reinterpret_cast<const long long*>(vec_ids);
    mp.out_pos = reinterpret_cast<long long*>(out_ids);
    mp.out_est = out_est;
    const int64_t slots = static_cast<int64_t>(ngroups) * n_rerank;
    if (slots > kPqBufKeys && slots <= static_cast<int64_t>(kPqMergeRegKeys) * kPqThreads)
        LAUNCH_DEP(128, pq_merge_kernel<true>, static_cast<unsigned>(nq), kPqThreads, 0, stream, mp);
    else
        LAUNCH_DEP(128, pq_merge_kernel<false>, static_cast<unsigned>(nq), kPqThreads, 0, stream, mp);
    timing_end(tk, stream);
    return IVF_OK;
}

int ivf_check(void* stream) {
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != IVF_OK) return rc;
    CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    if (ctx->out_used[0] || ctx->out_used[1]) CUDA_TRY(cudaStreamSynchronize(ctx->out_stream));  // deferred read-backs
    int h[4] = {0, 0, 0, 0};
    CUDA_TRY(cudaMemcpy(h, ctx->status, sizeof h, cudaMemcpyDeviceToHost));
    if (h[0] != 0) {
        CUDA_TRY(cudaMemset(ctx->status, 0, sizeof h));
        if (h[0] == IVF_ERR_DEVICE_TIMEOUT)
            return fail(IVF_ERR_DEVICE_TIMEOUT, "a device-side wait expired (wait site %d, block %d)", h[1], h[2]);
        if (h[0] == IVF_ERR_BAD_ID) return fail(IVF_ERR_BAD_ID, "ivf_centroid_update skipped ids outside [0, nlist)");
        if (h[0] == IVF_ERR_BOUNDS)
            return fail(IVF_ERR_BOUNDS, "an index check of the checked build failed (site %d, block %d, index %d)", h[1], h[2], h[3]);
        return fail(h[0], "device status %d", h[0]);
    }
    return IVF_OK;
}

int ivf_set_deferred_host_outputs(int on) {
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != IVF_OK) return rc;
    ctx->defer_outputs = on != 0;
    return IVF_OK;
}

int ivf_wait_host_outputs(void* stream) {
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != IVF_OK) return rc;
    // the read-back stream is in order: the younger of the two events covers every read-back issued
    for (int i = 0; i < 2; ++i)
        if (ctx->out_used[i]) CUDA_TRY(cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), ctx->ev_out_done[i], 0));
    return IVF_OK;
}

const char* ivf_last_error(void) { return g_err.c_str(); }

int ivf_release_workspace(void) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceSynchronize());
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceCtx& c = g_ctx[dev];
    for (Buf& b : c.bufs) {
        if (b.p) CUDA_TRY(cudaFree(b.p));
        b.p = nullptr;
        b.cap = 0;
    }
    return IVF_OK;
}

int64_t ivf_launch_count(void) { return g_launches.load(); }

int ivf_debug_plan(int64_t n, int nlist, int d, int k, int num_sms, int64_t out[9]) {
    if (n < 1 || nlist < 1 || num_sms < 1 || !out) return fail(IVF_ERR_INVALID_ARG, "bad plan arguments");
    if (check_d(d) != IVF_OK) return IVF_ERR_UNSUPPORTED;
    Plan pl;
    int stride = 1;
    int rc = make_plan(n, nlist, d, k, num_sms, &pl, k > 1 && choose_rule(k, nlist, &stride) != TAU_GIVEN);
    if (rc != IVF_OK) return rc;
    out[0] = pl.row_tiles;
    out[1] = pl.col_tiles;
    out[2] = pl.ctas;
    out[3] = pl.partials;
    out[4] = pl.block_n;
    out[5] = pl.kslices;
    out[6] = pl.nstage;
    out[7] = static_cast<int64_t>(pl.smem);
    out[8] = pl.mtiles;
    return IVF_OK;
}

int ivf_debug_span(int64_t n, int nlist, int d, int k, int num_sms, int cta, int64_t out[4]) {
    if (n < 1 || nlist < 1 || num_sms < 1 || !out) return fail(IVF_ERR_INVALID_ARG, "bad plan arguments");
    Plan pl;
    int stride = 1;
    int rc = make_plan(n, nlist, d, k, num_sms, &pl, k > 1 && choose_rule(k, nlist, &stride) != TAU_GIVEN);
    if (rc != IVF_OK) return rc;
    if (cta < 0 || cta >= pl.ctas) return fail(IVF_ERR_INVALID_ARG, "cta %d outside [0, %d)", cta, pl.ctas);
    out[0] = span_begin(pl.total_units, pl.ctas, pl.col_tiles, pl.cross, cta);
    out[1] = span_begin(pl.total_units, pl.ctas, pl.col_tiles, pl.cross, cta + 1);
    // the inverse mapping the kernels use to number a row group's partial slots
    out[2] = cta_of_unit(pl.total_units, pl.ctas, pl.col_tiles, pl.cross, out[0]);
    out[3] = cta_of_unit(pl.total_units, pl.ctas, pl.col_tiles, pl.cross, out[1] - 1);
    return IVF_OK;
}

int ivf_debug_rotation(int64_t n, int nlist, int d, int k, int num_sms, int64_t row_group) {
    if (n < 1 || nlist < 1 || num_sms < 1) return fail(IVF_ERR_INVALID_ARG, "bad plan arguments");
    Plan pl;
    int stride = 1;
    int rc = make_plan(n, nlist, d, k, num_sms, &pl, k > 1 && choose_rule(k, nlist, &stride) != TAU_GIVEN);
    if (rc != IVF_OK) return rc;
    if (row_group < 0 || row_group >= pl.row_tiles) return fail(IVF_ERR_INVALID_ARG, "row group outside the plan");
    return col_rotation(pl.total_units, pl.ctas, pl.col_tiles, pl.cross, row_group);
}

int ivf_debug_timing(int enable) {
    std::lock_guard<std::mutex> lk(g_mu);
    for (TimedLaunch& t : g_timed) {
        g_event_pool.push_back(t.a);
        g_event_pool.push_back(t.b);
    }
    g_timed.clear();
    g_timing = enable != 0;
    return IVF_OK;
}

int ivf_debug_timing_read(double ms[9], int64_t launches[9]) {
    if (!ms || !launches) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    CUDA_TRY(cudaDeviceSynchronize());
    std::lock_guard<std::mutex> lk(g_mu);
    for (int i = 0; i < TK_NUM; ++i) {
        ms[i] = 0.0;
        launches[i] = 0;
    }
    for (TimedLaunch& t : g_timed) {
        float e = 0.f;
        if (cudaEventElapsedTime(&e, t.a, t.b) == cudaSuccess) {
            ms[t.kind] += e;
            launches[t.kind] += 1;
        }
        g_event_pool.push_back(t.a);
        g_event_pool.push_back(t.b);
    }
    g_timed.clear();
    return IVF_OK;
}

int ivf_debug_stats(int enable, int64_t out[3]) {
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != IVF_OK) return rc;
    CUDA_TRY(cudaDeviceSynchronize());
    if (out) {
        unsigned long long h[4];
        CUDA_TRY(cudaMemcpy(h, ctx->stats, sizeof h, cudaMemcpyDeviceToHost));
        for (int i = 0; i < 3; ++i) out[i] = static_cast<int64_t>(h[i]);
    }
    CUDA_TRY(cudaMemset(ctx->stats, 0, 4 * sizeof(unsigned long long)));
    g_stats = enable != 0;
    return IVF_OK;
}

int ivf_debug_rule(int k, int nlist, int out[2]) {
    if (k < 1 || nlist < 1 || !out) return fail(IVF_ERR_INVALID_ARG, "bad arguments");
    out[1] = 1;
    out[0] = (k == 1) ? -1 : choose_rule(k, nlist, &out[1]);
    return IVF_OK;
}

int ivf_debug_set_row_chunk(int64_t rows) {
    g_row_chunk_override.store(rows > 0 ? rows : 0);
    return IVF_OK;
}

int ivf_debug_set_dependent_launch(int on) {
    g_pdl = on;
    return IVF_OK;
}

int ivf_debug_set_threshold_pass(int split) {
    g_sketch_whole = split ? 0 : 1;
    g_tau_fold = split ? 0 : 1;
    return IVF_OK;
}

int ivf_debug_set_rotation(int on) {
    g_rotate = on != 0;
    return IVF_OK;
}

int ivf_debug_set_crossing_cost(int units) {
    g_cross = units;  // negative: chosen by kernel variant
    return IVF_OK;
}

int ivf_debug_set_pq_groups(int groups) {
    g_pq_kernel = groups < 0 ? 1 : 0;  // a negative count also selects the single-team kernel
    if (groups < 0) groups = -groups - 1;
    g_pq_groups = groups < 0 ? 0 : groups;
    return IVF_OK;
}

int ivf_debug_fail_next_alloc(int count) {
    g_fail_allocs.store(count > 0 ? count : 0);
    return IVF_OK;
}

int ivf_debug_bounds_checked(void) { return kBoundsChecked ? 1 : 0; }

int ivf_debug_bounds_probe(void* stream) {
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != IVF_OK) return rc;
    bounds_probe_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(5, 3, nullptr);  // 5 is not below 3
    LAUNCH_CHECK();
    return IVF_OK;
}

int ivf_debug_force_fallback(int on) {
    g_force_fallback = on != 0;
    return IVF_OK;
}

int ivf_debug_wait_probe(void* stream) {
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc != IVF_OK) return rc;
    wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->status, g_wait_limit_ns.load());
    LAUNCH_CHECK();
    return IVF_OK;
}

int ivf_debug_set_wait_limit_ns(int64_t ns) {
    g_wait_limit_ns.store(ns > 0 ? static_cast<uint64_t>(ns) : 2000000000ull);
    return IVF_OK;
}

}  // extern "C"

// ====================================================================== allocation-free update
// Scratch of ivf_centroid_update_noalloc: lives in the module image, so every device that loads
// the library holds these ~4.8 MB until the process exits.  Layout (ints):
//   [0, 8)                         header: [0] = "an id was out of range" flag of the last call (written by
//                                  the histogram kernel, read by nobody yet: reserved), [1..7] unused
//   [8, 8 + L)                     per-list member counts of the call        (L = kNoAllocMaxLists)
//   [8 + L, 8 + 2L + 1)            exclusive offsets of the list segments
//   [8 + 2L + 8, 8 + 2L + 40)      partial totals of the offset scan (one per 4096 lists)
//   [8 + 2L + 40, 8 + 3L + 40)     per-list fill cursors
//   [8 + 3L + 40, ... + R)         row permutation sorted by list             (R = kNoAllocMaxRows)
namespace {
constexpr int kNoAllocMaxLists = 65536;
constexpr int kNoAllocMaxRows = 1 << 20;
constexpr size_t kNoAllocInts = 8 + 3 * static_cast<size_t>(kNoAllocMaxLists) + 40 + kNoAllocMaxRows;
static_assert(kNoAllocMaxLists / kScanBlock <= 32, "scan totals must fit their slot");
static __device__ __align__(256) int g_noalloc_scratch[kNoAllocInts];
// device address of the array above, per device (the host-side symbol is not a device pointer)
int* g_noalloc_ptr[kMaxDevices] = {};
}  // namespace

extern "C" int ivf_centroid_update_noalloc(const void* points, ivf_dtype ptype, const int32_t* ids, int64_t n, int d,
                                           int nlist, float* sums, int64_t* counts, void* stream_) {
    if (n < 0) return fail(IVF_ERR_INVALID_ARG, "negative row count %lld", (long long)n);
    if (!valid_dtype(ptype)) return fail(IVF_ERR_INVALID_ARG, "unknown element type %d", (int)ptype);
    if (check_d(d) != IVF_OK) return IVF_ERR_UNSUPPORTED;
    if (nlist < 1) return fail(IVF_ERR_INVALID_ARG, "nlist = %d", nlist);
    if (n > kNoAllocMaxRows)
        return fail(IVF_ERR_UNSUPPORTED,
                    "ivf_centroid_update_noalloc: n = %lld exceeds the built-in scratch (at most %d rows per call); "
                    "split the rows or use ivf_centroid_update",
                    (long long)n, kNoAllocMaxRows);
    if (nlist > kNoAllocMaxLists)
        return fail(IVF_ERR_UNSUPPORTED,
                    "ivf_centroid_update_noalloc: nlist = %d exceeds the built-in scratch (at most %d lists); "
                    "use ivf_centroid_update",
                    nlist, kNoAllocMaxLists);
    if (n == 0) return IVF_OK;
    if (!points || !ids || !sums || !counts) return fail(IVF_ERR_INVALID_ARG, "null pointer argument");
    if ((reinterpret_cast<uintptr_t>(points) & 15) || (reinterpret_cast<uintptr_t>(sums) & 15))
        return fail(IVF_ERR_INVALID_ARG, "points and sums must be 16-byte aligned");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(IVF_ERR_CUDA, "device index %d out of range", dev);
    int* base = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        if (!g_noalloc_ptr[dev]) {
            // first call on this device: look the array's device address up (no allocation involved)
            void* p = nullptr;
            CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
            g_noalloc_ptr[dev] = static_cast<int*>(p);
        }
        base = g_noalloc_ptr[dev];
    }
    int* flag = base;
    int* cnt = base + 8;
    int* off = cnt + kNoAllocMaxLists;
    int* block_sums = off + kNoAllocMaxLists + 8;
    int* cur = block_sums + 32;
    int* perm = cur + kNoAllocMaxLists;

    // the array keeps the previous call's contents: the counts and the flag must start at zero
    // (offsets, cursors and the permutation are fully rewritten by the kernels below)
    CUDA_TRY(cudaMemsetAsync(flag, 0, 8 * sizeof(int), stream));
    CUDA_TRY(cudaMemsetAsync(cnt, 0, static_cast<size_t>(nlist) * sizeof(int), stream));
    const unsigned rb = static_cast<unsigned>((n + 255) / 256);
    update_hist_kernel<<<rb, 256, 0, stream>>>(ids, n, nlist, cnt, flag);
    LAUNCH_CHECK();
    const int scan_blocks = (nlist + kScanBlock - 1) / kScanBlock;
    update_scan_local_kernel<<<scan_blocks, 1024, 0, stream>>>(cnt, nlist, off, block_sums);
    LAUNCH_CHECK();
    update_scan_fix_kernel<<<scan_blocks, 1024, 0, stream>>>(nlist, off, block_sums, cur);
    LAUNCH_CHECK();
    update_fill_kernel<<<rb, 256, 0, stream>>>(ids, n, nlist, off, cur, perm);
    LAUNCH_CHECK();
    const unsigned lb = static_cast<unsigned>((static_cast<int64_t>(nlist) * 32 + 255) / 256);
    if (ptype == IVF_U8)
        update_reduce_kernel<uint8_t><<<lb, 256, 0, stream>>>(static_cast<const uint8_t*>(points), perm, off, nlist, d,
                                                              sums, reinterpret_cast<long long*>(counts));
    else if (ptype == IVF_I8)
        update_reduce_kernel<int8_t><<<lb, 256, 0, stream>>>(static_cast<const int8_t*>(points), perm, off, nlist, d,
                                                             sums, reinterpret_cast<long long*>(counts));
    else
        update_reduce_kernel<float><<<lb, 256, 0, stream>>>(static_cast<const float*>(points), perm, off, nlist, d,
                                                            sums, reinterpret_cast<long long*>(counts));
    LAUNCH_CHECK();
    return IVF_OK;
}
