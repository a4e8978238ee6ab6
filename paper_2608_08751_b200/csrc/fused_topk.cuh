// Fused distance + per-row top-k kernel (Sec. 4.1: dense centroid evaluation by Eq. 6 and
// on-device list selection; Sec. 3.1 / 5.5: assignment is the k = 1 case).
//
// The whole ranking key of Eq. 6 comes out of the tensor core: the operand copies carry 16 extra
// K columns, so that  acc = sum_t x'_t c''_t + A (w_hi + w_mid + w_lo) = sx sc (|c|^2 - 2 x.c)
// with x' = sx x, c'' = -2 sc c, w = sc^2 |c|^2 / 2^15 split into three fp16 parts and
// A = 2^15 sx / sc (sx, sc exact powers of two).  The epilogue only compares.
//
// One persistent CTA per SM walks a contiguous span of (row group, centroid tile) units.  A row
// group is MT = 1 or 2 row tiles of 128 points that stay in shared memory; with MT = 2 every centroid
// tile brought from L2 feeds two MMA sweeps (one TMEM accumulator buffer each), which halves the
// L2 -> shared-memory traffic per FLOP.
//   warp 0      producer: TMA loads of the stationary 128-row point tile(s) and of a ring of centroid
//               tiles.  uint8 points need no fp16 copy in HBM: at the start of a row group every
//               epilogue thread reads its own raw row, widens it to fp16 (exact) and writes it into
//               the swizzled operand tile in shared memory, along with |x|^2.
//   warp 1      single-thread tcgen05.mma issuer; accumulators live in TMEM (fp32), two buffers,
//               so the next tile's MMAs overlap this tile's epilogue
//   warps 2..9  epilogue: TMEM lane = point row; the two warps that share a lane quadrant split
//               each tile's columns in 64-column groups.  Nothing of the n x nlist matrix is
//               written to memory.
// k = 1 keeps (best key, id) in registers.  k > 1 appends every key <= the row's threshold tau to
// a candidate log in global memory.  tau comes from one of three rules, fixed per launch:
//   running   (k <= 16) tau = the 16th smallest group-of-8 minimum seen so far, kept in a sorted
//             register network: at least 16 keys are <= tau, so the result is exact;
//   given     tau is read per row from memory, and the log holds whole groups of 8 keys: if the
//             minimum of a group passes, the 8 raw keys are appended (two 16-byte stores, ~1.4
//             instructions per key, no branch) and the merge kernel compares key by key.  The host computes it with a first, small launch of
//             this same kernel (sketch rule) over every S-th centroid, S = k / 4: the 16th smallest
//             32-key-chunk minimum of that sample lets about 4k candidates through.  Whether tau was loose
//             enough is checked exactly by the merge kernel (at least k candidates <= tau); a row
//             that fails is recomputed by brute force;
//   sketch    the threshold pass itself: nothing is appended; each thread only keeps its 16
//             smallest chunk minima (one per 32 keys) and leaves them as its partial result;
//   bounded   (small problems) tau = +inf until the log fills, then the warp selects the k
//             smallest in place (radix select on the key bits, ties to the lower id) and tau
//             becomes the k-th.  The same in-place selection catches any log that fills up.
#pragma once
#include <cuda_fp16.h>

#include "ptx.cuh"
#include "scales.cuh"

namespace ivf {

constexpr int kBlockM = 128;         // point rows per tile = TMEM lanes
constexpr int kTmemCols = 512;       // whole TMEM: two accumulator buffers of 256 columns
constexpr int kAccStride = 256;      // TMEM columns between the two accumulator buffers
constexpr int kEpiHalves = 2;        // epilogue warps per TMEM lane quadrant
constexpr int kNumEpiWarps = 4 * kEpiHalves;
constexpr int kFusedThreads = 32 * (2 + kNumEpiWarps);
constexpr int kSliceK = 64;          // fp16 elements per 128-byte swizzled row
constexpr int kSliceRowBytes = 128;
constexpr int kAugK = 16;            // extra K columns that carry |c|^2
constexpr int kAugRowBytes = 32;
constexpr int kMaxStages = 8;
constexpr int kSampleM = 16;         // order statistic of the sample that becomes tau

struct Entry {
    float v;  // ranking key  sx sc (|c|^2 - 2 x.c)
    int j;    // centroid id
};

enum { TAU_RUNNING = 0, TAU_GIVEN = 1, TAU_BOUNDED = 2, TAU_SKETCH = 3 };

struct FusedParams {
    int64_t n;            // point rows
    int nlist;
    int k;
    int ksteps;           // data MMA instructions per tile = ceil(d / 16); one more for the norm columns
    int kslices;          // 64-wide K slices of the operand copies
    int block_n;          // centroids per tile: 256 or 128
    int nstage;           // centroid-tile ring depth
    int col_tiles;        // centroid tiles per sweep
    int64_t total_units;  // row groups * col_tiles
    int cross;            // cost of a mid-span row-group crossing in units (span partition)
    int rotate;           // 1: centroid tiles of a row group are swept in the rotated order (col_rotation)
    int partials;         // partial-result slots per row (CTAs sharing a row tile x kEpiHalves)
    int cap;              // candidate-log capacity per (row, slot), k > 1 only
    int rule;             // k > 1: TAU_RUNNING, TAU_GIVEN or TAU_BOUNDED
    const float* tau_in;  // given rule: threshold per row, in key units
    float* sketch_t;      // batches of at most kFoldRows rows, if set: the partial sketches of the threshold
                          // pass as [n][16][sketch_pitch] floats (value i of slot s of row r at
                          // (r * 16 + i) * sketch_pitch + s; ascending in i).  The sketch rule writes them
                          // there instead of `part`; the given rule reads them: its epilogue warps finish
                          // the thresholds themselves and tau_in is not read
    int sketch_pitch;     // >= the slots of a row
    int sketch_slots;     // slots that hold a sketch (given rule)
    float* tau_out;       // sketch rule with whole_rows: the row's threshold is finished inside the kernel
    int whole_rows;       // 1: every CTA owns whole row groups (no row group is shared between CTAs)
    Entry* part;          // k = 1: [n][partials]; k > 1: [n][partials][cap] entries, or 48-byte group
                          // records for the given rule
    int2* part_meta;      // k > 1: [n][partials] {entries (records) in the log or -1 if it overflowed,
                          // bits of the final tau}
    const uint8_t* x_raw; // uint8 points [n][d], widened in shared memory (nullptr: fp16 copy via TMA)
    int d;                // columns of x_raw
    const unsigned int* bits;  // x_raw mode: magnitude words the scales are derived from
    float* scal_out;      // x_raw mode: the four scale factors, published by block 0
    float* xn_out;        // x_raw mode: |x|^2 per row
    int* clear0;          // two optional words that block 0 sets to zero (list counters of the merge)
    int* clear1;
    int* clear32;         // optional: 32 more words for block 0 to clear (work counters of the call's tail kernel)
    int* status;          // sticky device status word
    unsigned long long* stats;  // optional counters: [0] in-kernel selections, [1] log entries written
    uint64_t wait_limit_ns;
};

// ---- persistent schedule: CTA b of G owns units [T*b/G, T*(b+1)/G) of the row-major unit grid
// The T = R * NT units are dealt to G CTAs by cost, not by count: a CTA that crosses from one row
// group to the next in mid-span idles its tensor core while the last accumulators are read and the
// next point tile is fetched, which costs about as much as `cross` units.  In cost space every row
// group is a block of `cross` cost units followed by its NT unit slots; CTA b starts at cost
// C * b / G (C = R * (NT + cross)), and a start that falls inside a crossing block is moved to the row
// group's first unit.  cross = 0 is the plain equal-count split.
__host__ __device__ inline int64_t span_begin(int64_t T, int G, int NT, int cross, int b) {
    const int64_t w = NT + cross;
    const int64_t C = (T / NT) * w;
    const int64_t c = (C * b) / G;
    const int64_t r = c / w, o = c - r * w;
    return r * NT + (o > cross ? o - cross : 0);
}
// the CTA whose span holds unit u: the largest b with span_begin(b) <= u
__host__ __device__ inline int cta_of_unit(int64_t T, int G, int NT, int cross, int64_t u) {
    const int64_t w = NT + cross;
    const int64_t C = (T / NT) * w;
    const int64_t r = u / NT;
    const int64_t cu = r * w + cross + (u - r * NT);  // cost coordinate of the unit's slot
    return static_cast<int>(((cu + 1) * G - 1) / C);
}

// Order of the centroid tiles inside a row group.  A CTA sweeps the positions of its span in order,
// but position p of row group r stands for centroid tile (p + rot_r) mod NT, with rot_r = the time (in
// cost units since the launch) at which position 0 of the row group is reached by the CTA that owns
// it.  Every CTA therefore works on centroid tile (time + i * span length) mod NT for a small integer
// i: the ~G CTAs sweep the table as a handful of fronts, each shared by the CTAs of many row groups,
// instead of G different phases.  A centroid tile is then fetched from HBM once per front passage and
// served to the other CTAs of the front from L2, however large the table is.  (With the positions
// standing for their own tile index, a table larger than L2 was re-read from HBM once per row group.)
__host__ __device__ inline int col_rotation(int64_t T, int G, int NT, int cross, int64_t r) {
    const int64_t w = NT + cross;
    const int first = cta_of_unit(T, G, NT, cross, r * NT);
    const int64_t ub = span_begin(T, G, NT, cross, first);
    const int64_t rb = ub / NT;
    const int64_t arrive = (r * w + cross) - (rb * w + cross + (ub - rb * NT));
    return static_cast<int>(arrive % NT);
}

// (the radix histograms are used by the epilogues that keep a bounded candidate log, which always run
// with one row tile per unit)
__host__ __device__ inline size_t fused_smem_bytes(int kslices, int block_n, int nstage, int mtiles) {
    return 1024                                                                        // alignment slack
           + static_cast<size_t>(mtiles) * kBlockM * (kslices * kSliceRowBytes + kAugRowBytes)  // point tiles
           + static_cast<size_t>(nstage) * block_n * (kslices * kSliceRowBytes + kAugRowBytes)
           + 256                                                                       // barriers etc.
           + (mtiles == 1 ? kNumEpiWarps * 256 * sizeof(int) : 0);                     // radix histograms
}

__device__ __forceinline__ uint32_t orderable(float v) {
    uint32_t b = __float_as_uint(v);
    return b ^ ((static_cast<uint32_t>(static_cast<int32_t>(b) >> 31)) | 0x80000000u);
}
__device__ __forceinline__ float from_orderable(uint32_t u) {
    uint32_t b = (u & 0x80000000u) ? (u ^ 0x80000000u) : ~u;
    return __uint_as_float(b);
}

// One 8-bit step of a warp-cooperative radix select.  hist[256] holds the digit counts of the items
// that match the prefix so far; r is the 1-based rank wanted among them.  Returns the digit that
// contains rank r and rewrites r as the rank inside that digit; eq_out = items in that digit.
__device__ __forceinline__ int radix_pick_digit(const int* hist, int lane, int& r, int& eq_out) {
    int local[8];
    int sum = 0;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        local[b] = hist[8 * lane + b];
        sum += local[b];
    }
    int incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        int t = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += t;
    }
    const int excl = incl - sum;
    const bool mine = (r > excl) && (r <= incl);
    int digit = 0, newr = 0, eq = 0;
    if (mine) {
        int acc = excl;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            if (newr == 0 && r <= acc + local[b]) {
                digit = 8 * lane + b;
                newr = r - acc;
                eq = local[b];
            }
            acc += local[b];
        }
    }
    const uint32_t bal = __ballot_sync(0xFFFFFFFFu, mine);
    const int src = bal ? (__ffs(bal) - 1) : 0;
    digit = __shfl_sync(0xFFFFFFFFu, digit, src);
    r = __shfl_sync(0xFFFFFFFFu, newr, src);
    eq_out = __shfl_sync(0xFFFFFFFFu, eq, src);
    return digit;
}

// The warp keeps the k smallest of log[0..c) (c > k) in log[0..k), compared by (key, id), and
// returns the k-th smallest key.  The log lives in global memory; reads bypass L1.
__device__ __noinline__ float warp_select_k(Entry* log, int c, int k, int* hist, int lane) {
    uint32_t prefix = 0, mask = 0;
    int r = k, eq = 0;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = lane; i < 256; i += 32) hist[i] = 0;
        __syncwarp();
        for (int i = lane; i < c; i += 32) {
            const uint32_t u = orderable(__ldcg(&log[i].v));
            if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1);
        }
        __syncwarp();
        const int digit = radix_pick_digit(hist, lane, r, eq);
        prefix |= static_cast<uint32_t>(digit) << shift;
        mask |= 255u << shift;
        __syncwarp();
    }
    const uint32_t T = prefix;  // k-th smallest key; r of the eq items equal to it are wanted
    uint32_t J = 0xFFFFFFFFu;   // largest id admitted among the items equal to T
    if (eq > r) {
        uint32_t jprefix = 0, jmask = 0;
        int rr = r, dummy = 0;
#pragma unroll 1
        for (int shift = 24; shift >= 0; shift -= 8) {
            for (int i = lane; i < 256; i += 32) hist[i] = 0;
            __syncwarp();
            for (int i = lane; i < c; i += 32) {
                const uint2 e = __ldcg(reinterpret_cast<const uint2*>(&log[i]));
                if (orderable(__uint_as_float(e.x)) == T && (e.y & jmask) == jprefix)
                    atomicAdd(&hist[(e.y >> shift) & 255u], 1);
            }
            __syncwarp();
            const int digit = radix_pick_digit(hist, lane, rr, dummy);
            jprefix |= static_cast<uint32_t>(digit) << shift;
            jmask |= 255u << shift;
            __syncwarp();
        }
        J = jprefix;
    }
    int base = 0;
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int i0 = 0; i0 < c; i0 += 32) {
        const int i = i0 + lane;
        bool keep = false;
        uint2 e = make_uint2(0u, 0u);
        if (i < c) {
            e = __ldcg(reinterpret_cast<const uint2*>(&log[i]));
            const uint32_t u = orderable(__uint_as_float(e.x));
            keep = (u < T) || (u == T && e.y <= J);
        }
        const uint32_t bal = __ballot_sync(0xFFFFFFFFu, keep);
        if (keep && IVF_IN_BOUNDS(101, base + __popc(bal & lt_mask), c)) *reinterpret_cast<uint2*>(&log[base + __popc(bal & lt_mask)]) = e;
        base += __popc(bal);
    }
    __syncwarp();
    return from_orderable(T);
}

// A wait on a barrier that nothing ever completes: exercises the bounded wait and the status word
// without any copy or MMA in flight.
__global__ void wait_probe_kernel(int* status, uint64_t limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    WaitCtl ctl;
    ctl.abort_flag = &abort_flag;
    ctl.status = status;
    ctl.limit_ns = limit_ns;
    (void)mbar_wait(&bar, 0, ctl, 99);
}

// Evaluates one failing index check and touches no memory: shows, in the checked build, that a
// violation reaches the status word and that the context stays usable (a no-op in the regular build).
__global__ void bounds_probe_kernel(int index, int limit, int* sink) {
    if (IVF_IN_BOUNDS(999, index, limit) && sink != nullptr) *sink = index;
}

__device__ __forceinline__ float min3f(float a, float b, float c) {
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// smallest of 32 keys (NaN entries are ignored by min)
__device__ __forceinline__ float min32(const uint32_t (&a)[32]) {
    float m[11];
#pragma unroll
    for (int i = 0; i < 10; ++i)
        m[i] = min3f(__uint_as_float(a[3 * i]), __uint_as_float(a[3 * i + 1]), __uint_as_float(a[3 * i + 2]));
    m[10] = fminf(__uint_as_float(a[30]), __uint_as_float(a[31]));
    m[0] = min3f(m[0], m[1], m[2]);
    m[1] = min3f(m[3], m[4], m[5]);
    m[2] = min3f(m[6], m[7], m[8]);
    m[3] = fminf(m[9], m[10]);
    return fminf(min3f(m[0], m[1], m[2]), m[3]);
}

// sorted insertion of v into a[0] <= a[1] <= ... <= a[15] (the largest falls out); branch-free
__device__ __forceinline__ void network_insert(float (&a)[kSampleM], float v) {
#pragma unroll
    for (int i = kSampleM - 1; i >= 1; --i) a[i] = fminf(a[i], fmaxf(a[i - 1], v));
    a[0] = fminf(a[0], v);
}

// Compile-time variants of the epilogue.
enum { EPI_ARGMIN = 0, EPI_RUNNING = 1, EPI_FILTER = 2, EPI_SKETCH = 3, EPI_GROUPS = 4 };

// A record of the group log (EPI_GROUPS): 8 consecutive keys and the id of the first.
constexpr int kRecordBytes = 48;
// Records one thread can append between two checks of its log's fill level (one tile: 4 chunks of 4 groups).
constexpr int kGroupLogMargin = 16;

template <int EPI>
struct RowState;
template <>
struct RowState<EPI_ARGMIN> {
    float tau;  // best key so far
    int bestj;
};
template <>
struct RowState<EPI_FILTER> {
    float tau;  // threshold (given per row, or +inf until the first in-place selection)
    int cnt;    // entries in the log
    Entry* log;
};
template <>
struct RowState<EPI_RUNNING> {
    float tau;
    int cnt;
    Entry* log;
    float net[kSampleM];  // the 16 smallest group-of-8 minima seen
};
template <>
struct RowState<EPI_GROUPS> {
    float tau;       // threshold, given per row
    char* wp;        // next record of the group log
    char* base;      // first record
    char* limit;     // wp beyond this after a chunk = the log is full
    int overflow;
};
template <>
struct RowState<EPI_SKETCH> {
    float tau;
    float net[kSampleM];
};

__device__ __forceinline__ void mask_ragged(uint32_t (&acc)[32], int jbase, int nlist) {
#pragma unroll
    for (int c = 0; c < 32; ++c)
        if (jbase + c >= nlist) acc[c] = 0x7fc00000u;  // NaN: never below any threshold, ignored by min
}

__device__ __forceinline__ float min8(const uint32_t (&acc)[32], int g) {
    float m = min3f(__uint_as_float(acc[8 * g]), __uint_as_float(acc[8 * g + 1]), __uint_as_float(acc[8 * g + 2]));
    m = min3f(m, __uint_as_float(acc[8 * g + 3]), __uint_as_float(acc[8 * g + 4]));
    m = min3f(m, __uint_as_float(acc[8 * g + 5]), __uint_as_float(acc[8 * g + 6]));
    return fminf(m, __uint_as_float(acc[8 * g + 7]));
}

// 32 accumulator columns of one row.
template <int EPI>
__device__ __forceinline__ void consume(uint32_t (&acc)[32], int jbase, RowState<EPI>& st) {
    if constexpr (EPI == EPI_ARGMIN) {
        // The chunk's minimum first; only a thread whose minimum beats its best looks for the column.
        // That search is kept short (the threads of a warp wait for each other on this branch): the
        // first group of 8 that holds the minimum, then the first column of that group that equals it,
        // which is the lowest id among equal keys.
        const float m0 = min8(acc, 0), m1 = min8(acc, 1), m2 = min8(acc, 2), m3 = min8(acc, 3);
        const float m = fminf(fminf(m0, m1), fminf(m2, m3));
        if (m <= st.tau) {
            const bool in0 = (m0 == m), in1 = (m1 == m), in2 = (m2 == m);
            const int g = in0 ? 0 : (in1 ? 1 : (in2 ? 2 : 3));
            int idx = 7;
#pragma unroll
            for (int i = 6; i >= 0; --i) {
                const float v = __uint_as_float(in0 ? acc[i] : (in1 ? acc[8 + i] : (in2 ? acc[16 + i] : acc[24 + i])));
                if (v == m) idx = i;
            }
            // (a sweep may wrap around to the low centroid ids, so an equal key with a lower id can
            // come later: ties are settled by id)
            const int j = jbase + 8 * g + idx;
            if (m < st.tau || j < st.bestj) st.bestj = j;
            st.tau = m;
        }
    } else if constexpr (EPI == EPI_GROUPS) {
        // One decision per group of 8 columns: if the group's minimum passes the threshold, the
        // whole group (8 raw keys + the id of the first) is appended with two 16-byte stores; the
        // merge kernel does the per-key comparison.  About 1.2 instructions per key, no branch.  The
        // four groups of a chunk are one block: their minimum chains are interleaved and every group
        // stores through its own pointer (w1..w3 = the write pointer advanced by the groups before).
        asm volatile(
            "{\n\t"
            ".reg .pred p0, p1, p2, p3;\n\t.reg .f32 m0, m1, m2, m3;\n\t.reg .b64 w1, w2, w3;\n\t"
            "min.f32 m0, %2, %3, %4;\n\t"
            "min.f32 m1, %10, %11, %12;\n\t"
            "min.f32 m2, %18, %19, %20;\n\t"
            "min.f32 m3, %26, %27, %28;\n\t"
            "min.f32 m0, m0, %5, %6;\n\t"
            "min.f32 m1, m1, %13, %14;\n\t"
            "min.f32 m2, m2, %21, %22;\n\t"
            "min.f32 m3, m3, %29, %30;\n\t"
            "min.f32 m0, m0, %7, %8;\n\t"
            "min.f32 m1, m1, %15, %16;\n\t"
            "min.f32 m2, m2, %23, %24;\n\t"
            "min.f32 m3, m3, %31, %32;\n\t"
            "min.f32 m0, m0, %9;\n\t"
            "min.f32 m1, m1, %17;\n\t"
            "min.f32 m2, m2, %25;\n\t"
            "min.f32 m3, m3, %33;\n\t"
            "setp.le.f32 p0, m0, %1;\n\t"
            "setp.le.f32 p1, m1, %1;\n\t"
            "setp.le.f32 p2, m2, %1;\n\t"
            "setp.le.f32 p3, m3, %1;\n\t"
            "mov.b64 w1, %0;\n\t@p0 add.s64 w1, %0, 48;\n\t"
            "mov.b64 w2, w1;\n\t@p1 add.s64 w2, w1, 48;\n\t"
            "mov.b64 w3, w2;\n\t@p2 add.s64 w3, w2, 48;\n\t"
            "@p0 st.global.cs.v4.f32 [%0], {%2, %3, %4, %5};\n\t"
            "@p0 st.global.cs.v4.f32 [%0+16], {%6, %7, %8, %9};\n\t"
            "@p0 st.global.cs.b32 [%0+32], %34;\n\t"
            "@p1 st.global.cs.v4.f32 [w1], {%10, %11, %12, %13};\n\t"
            "@p1 st.global.cs.v4.f32 [w1+16], {%14, %15, %16, %17};\n\t"
            "@p1 st.global.cs.b32 [w1+32], %35;\n\t"
            "@p2 st.global.cs.v4.f32 [w2], {%18, %19, %20, %21};\n\t"
            "@p2 st.global.cs.v4.f32 [w2+16], {%22, %23, %24, %25};\n\t"
            "@p2 st.global.cs.b32 [w2+32], %36;\n\t"
            "@p3 st.global.cs.v4.f32 [w3], {%26, %27, %28, %29};\n\t"
            "@p3 st.global.cs.v4.f32 [w3+16], {%30, %31, %32, %33};\n\t"
            "@p3 st.global.cs.b32 [w3+32], %37;\n\t"
            "mov.b64 %0, w3;\n\t@p3 add.s64 %0, w3, 48;\n\t}"
            : "+l"(st.wp)
            : "f"(st.tau),
              "f"(__uint_as_float(acc[0])), "f"(__uint_as_float(acc[1])), "f"(__uint_as_float(acc[2])), "f"(__uint_as_float(acc[3])),
              "f"(__uint_as_float(acc[4])), "f"(__uint_as_float(acc[5])), "f"(__uint_as_float(acc[6])), "f"(__uint_as_float(acc[7])),
              "f"(__uint_as_float(acc[8])), "f"(__uint_as_float(acc[9])), "f"(__uint_as_float(acc[10])), "f"(__uint_as_float(acc[11])),
              "f"(__uint_as_float(acc[12])), "f"(__uint_as_float(acc[13])), "f"(__uint_as_float(acc[14])), "f"(__uint_as_float(acc[15])),
              "f"(__uint_as_float(acc[16])), "f"(__uint_as_float(acc[17])), "f"(__uint_as_float(acc[18])), "f"(__uint_as_float(acc[19])),
              "f"(__uint_as_float(acc[20])), "f"(__uint_as_float(acc[21])), "f"(__uint_as_float(acc[22])), "f"(__uint_as_float(acc[23])),
              "f"(__uint_as_float(acc[24])), "f"(__uint_as_float(acc[25])), "f"(__uint_as_float(acc[26])), "f"(__uint_as_float(acc[27])),
              "f"(__uint_as_float(acc[28])), "f"(__uint_as_float(acc[29])), "f"(__uint_as_float(acc[30])), "f"(__uint_as_float(acc[31])),
              "r"(jbase), "r"(jbase + 8), "r"(jbase + 16), "r"(jbase + 24)
            : "memory");
    } else if constexpr (EPI == EPI_FILTER) {
        // Straight-line predicated code on purpose: hits are rare, but 32 rows share every branch,
        // so a branch per column costs more in divergence than the predicated store it would skip.
        Entry* wp = st.log + st.cnt;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "setp.le.f32 p, %1, %2;\n\t"
                "@p st.global.v2.b32 [%0], {%3, %4};\n\t"
                "@p add.s64 %0, %0, 8;\n\t}"
                : "+l"(wp)
                : "f"(__uint_as_float(acc[c])), "f"(st.tau), "r"(acc[c]), "r"(jbase + c)
                : "memory");
        }
        st.cnt = static_cast<int>(wp - st.log);
    } else if constexpr (EPI == EPI_SKETCH) {
        // Threshold pass: the statistic is the minimum of each chunk of 32 keys, one network
        // insertion per chunk; tau will be the 16th smallest chunk minimum of the row, so at least 16
        // sampled keys are <= tau.  (With one insertion per group of 8 this epilogue cost four times
        // the group-record one, because some row of the warp needs nearly every insertion.)
        const float m = fminf(fminf(min8(acc, 0), min8(acc, 1)), fminf(min8(acc, 2), min8(acc, 3)));
        if (__any_sync(0xFFFFFFFFu, m < st.net[kSampleM - 1])) network_insert(st.net, m);
    } else {
        // the sample statistic is the minimum of each group of 8 keys: one network insertion per
        // group.  tau = the 16th smallest group minimum, so at least 16 keys are <= tau.
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const float m = min8(acc, g);
            if (__any_sync(0xFFFFFFFFu, m <= st.tau)) {
                if constexpr (EPI == EPI_RUNNING) {
#pragma unroll
                    for (int c = 8 * g; c < 8 * g + 8; ++c) {
                        if (__uint_as_float(acc[c]) <= st.tau) {
                            *reinterpret_cast<uint2*>(&st.log[st.cnt]) =
                                make_uint2(acc[c], static_cast<uint32_t>(jbase + c));
                            ++st.cnt;
                        }
                    }
                }
                if (m < st.net[kSampleM - 1]) {
                    network_insert(st.net, m);
                    st.tau = fminf(st.tau, st.net[kSampleM - 1]);
                }
            }
        }
    }
}

// One warp widens the 32 consecutive uint8 point rows of one TMEM lane quadrant into the fp16 operand
// tile in shared memory, with coalesced loads: 16-byte chunks of 8 values go to the positions the
// 128-byte swizzle (data) and the 32-byte swizzle (norm columns) give them, exactly as a TMA load of
// an fp16 copy would have placed them.  The rows are contiguous in memory, so lane l of step s takes
// the 16-byte chunk number 32 s + l of the quadrant's 32 * d bytes (four steps in flight).  A chunk of 16 values becomes two 16-byte chunks of
// the operand row, written where the swizzles put them.  The squares are summed per chunk and brought
// to the lane that owns the row (lane = row within the quadrant), which also writes the norm columns
// and |x|^2.  Rows at or beyond `n` become zero rows.
__device__ __forceinline__ void widen_rows_u8_warp(const uint8_t* __restrict__ x_raw, int64_t grow0, int64_t n, int d, int kd,
                                                   uint8_t* tile, int a_data_bytes, int row0, int lane, float sx, float A,
                                                   float* __restrict__ xn_out) {
    const __half2 k1024 = __floats2half2_rn(1024.0f, 1024.0f);
    const __half2 sx2 = __floats2half2_rn(sx, sx);
    auto cvt2 = [&](uint32_t w, uint32_t sel) {  // two bytes -> two fp16 (0x6400 | b is the half 1024 + b; all exact)
        uint32_t q = __byte_perm(w, 0x64646464u, sel);
        const __half2 t2 = __hmul2(__hsub2(*reinterpret_cast<__half2*>(&q), k1024), sx2);
        return *reinterpret_cast<const uint32_t*>(&t2);
    };
    const int cpr = d >> 4;        // 16-byte chunks per row
    const int total = 32 * cpr;    // chunks of the quadrant
    const int64_t left = n - grow0;
    const int rows_valid = left <= 0 ? 0 : (left < 32 ? static_cast<int>(left) : 32);
    const uint4* src = reinterpret_cast<const uint4*>(x_raw + (rows_valid > 0 ? grow0 : 0) * d);
    unsigned int sumsq = 0;        // of row `lane`
    constexpr int U = 8;
#pragma unroll 1
    for (int g0 = 0; g0 < total; g0 += 32 * U) {
        uint4 w[U];
        int rr[U], cc[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int g = g0 + u * 32 + lane;
            rr[u] = g / cpr;
            cc[u] = g - rr[u] * cpr;
            w[u] = make_uint4(0u, 0u, 0u, 0u);
            if (g < total && rr[u] < rows_valid) w[u] = src[g];
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int gb = g0 + u * 32;  // first chunk of this step
            if (gb < total) {            // uniform over the warp
                unsigned int part = __dp4a(w[u].x, w[u].x, 0u);
                part = __dp4a(w[u].y, w[u].y, part);
                part = __dp4a(w[u].z, w[u].z, part);
                part = __dp4a(w[u].w, w[u].w, part);
                if (gb + lane < total) {
                    const int row = row0 + rr[u];
                    uint4 o0, o1;
                    o0.x = cvt2(w[u].x, 0x5140u); o0.y = cvt2(w[u].x, 0x5342u); o0.z = cvt2(w[u].y, 0x5140u); o0.w = cvt2(w[u].y, 0x5342u);
                    o1.x = cvt2(w[u].z, 0x5140u); o1.y = cvt2(w[u].z, 0x5342u); o1.z = cvt2(w[u].w, 0x5140u); o1.w = cvt2(w[u].w, 0x5342u);
                    const int c = 2 * cc[u];  // 8-value chunk index inside the row; c and c + 1 lie in the same 64-wide slice
                    const int slice = c >> 3, j = c & 7;
                    uint8_t* rowp = tile + slice * kBlockM * kSliceRowBytes + row * kSliceRowBytes;
                    if (IVF_IN_BOUNDS(112, slice * kBlockM * kSliceRowBytes + row * kSliceRowBytes + (((j + 1) ^ (row & 7)) << 4),
                                      a_data_bytes - 15)) {
                        *reinterpret_cast<uint4*>(rowp + ((j ^ (row & 7)) << 4)) = o0;
                        *reinterpret_cast<uint4*>(rowp + (((j + 1) ^ (row & 7)) << 4)) = o1;
                    }
                }
                // the chunks of one row are neighbours: add them up towards the row's first lane ...
                int rid = gb + lane < total ? rr[u] : -1;
#pragma unroll
                for (int off = 1; off < 16; off <<= 1) {
                    const unsigned int t = __shfl_down_sync(0xFFFFFFFFu, part, off);
                    const int tr = __shfl_down_sync(0xFFFFFFFFu, rid, off);
                    if (lane + off < 32 && tr == rid) part += t;
                }
                // ... and hand the sum to the lane that owns the row (a row may continue from the step before)
                const int first = lane * cpr - gb;  // step-relative chunk where row `lane` starts
                const bool in_step = first < 32 && first + cpr > 0;
                const unsigned int got = __shfl_sync(0xFFFFFFFFu, part, in_step ? (first > 0 ? first : 0) : 0);
                if (in_step) sumsq += got;
            }
        }
    }
    // zero padding up to kd (rows whose length is not a multiple of 64)
    const int pad = (kd - d) >> 3;  // 8-value chunks per row
    for (int i = lane; i < 32 * pad; i += 32) {
        const int rrow = i / pad, c = (d >> 3) + (i - rrow * pad);
        const int row = row0 + rrow;
        const int slice = c >> 3, j = c & 7;
        *reinterpret_cast<uint4*>(tile + slice * kBlockM * kSliceRowBytes + row * kSliceRowBytes + ((j ^ (row & 7)) << 4)) =
            make_uint4(0u, 0u, 0u, 0u);
    }
    // norm columns of the lane's own row: A A A 0 ... 0; chunk j of the row goes to position j ^ ((row / 4) % 2)
    const int row = row0 + lane;
    const bool valid = lane < rows_valid;
    const uint32_t a16 = static_cast<uint32_t>(__half_as_ushort(__float2half_rn(A)));
    const uint4 aug0 = valid ? make_uint4(a16 | (a16 << 16), a16, 0u, 0u) : make_uint4(0u, 0u, 0u, 0u);
    const int sw = (row >> 2) & 1;
    *reinterpret_cast<uint4*>(tile + a_data_bytes + row * kAugRowBytes + ((0 ^ sw) << 4)) = aug0;
    *reinterpret_cast<uint4*>(tile + a_data_bytes + row * kAugRowBytes + ((1 ^ sw) << 4)) = make_uint4(0u, 0u, 0u, 0u);
    if (valid && IVF_IN_BOUNDS(141, grow0 + lane, n)) xn_out[grow0 + lane] = static_cast<float>(sumsq);
}

// ---------------------------------------------------------------- thresholds finished by the main pass
// Serving-size batches (at most kFoldRows rows): every CTA of the main pass derives the rows'
// thresholds from the partial sketches of the threshold pass itself, one epilogue warp per row
// (four rows per warp at most), while its first tiles are computed -- no launch in between.
constexpr int kFoldRows = 4 * kNumEpiWarps;

// a, b ascending: a becomes the 16 smallest of the 32 values, ascending.  min(a[i], b[15 - i]) are
// those 16 values as a bitonic sequence, which four half-cleaner stages sort.
__device__ __forceinline__ void merge16_sorted(float (&a)[kSampleM], const float (&b)[kSampleM]) {
    static_assert(kSampleM == 16, "network below is written for 16");
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = fminf(a[i], b[15 - i]);
#pragma unroll
    for (int stride = 8; stride > 0; stride >>= 1) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            if ((i & stride) == 0) {
                const float lo = fminf(a[i], a[i + stride]), hi = fmaxf(a[i], a[i + stride]);
                a[i] = lo;
                a[i + stride] = hi;
            }
        }
    }
}

// The 16th smallest of the values in `slots` ascending 16-entry lists (value i of list s at
// base[i * pitch + s], so that a warp's loads are contiguous), computed by one warp; every lane
// returns it.
__device__ __forceinline__ float warp_threshold_of_sketches(const float* base, int slots, int pitch, int lane) {
    const float INF = __int_as_float(0x7f800000);
    float a[kSampleM];
#pragma unroll
    for (int i = 0; i < kSampleM; ++i) a[i] = INF;
    // five lists per lane and memory round trip (the warp is alone on its scheduler half the time and
    // the loads' latency, not their number, is what the batch waits for)
    constexpr int kLists = 5;
    for (int s0 = lane; s0 < slots; s0 += 32 * kLists) {
        float v[kLists][kSampleM];
#pragma unroll
        for (int u = 0; u < kLists; ++u) {
            const int s = s0 + 32 * u;
#pragma unroll
            for (int i = 0; i < kSampleM; ++i) v[u][i] = s < slots ? base[static_cast<size_t>(i) * pitch + s] : INF;
        }
#pragma unroll
        for (int u = 0; u < kLists; ++u) merge16_sorted(a, v[u]);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        float b[kSampleM];
#pragma unroll
        for (int i = 0; i < kSampleM; ++i) b[i] = __shfl_xor_sync(0xFFFFFFFFu, a[i], off);
        merge16_sorted(a, b);
    }
    return a[kSampleM - 1];
}

template <int EPI, int MT>
__global__ void __launch_bounds__(kFusedThreads, 1)
fused_topk_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_xa,
                  const __grid_constant__ CUtensorMap tmap_c, const __grid_constant__ CUtensorMap tmap_ca,
                  const FusedParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int a_data_bytes = p.kslices * kBlockM * kSliceRowBytes;
    const int a_bytes = a_data_bytes + kBlockM * kAugRowBytes;
    const int b_data_bytes = p.kslices * p.block_n * kSliceRowBytes;
    const int stage_bytes = b_data_bytes + p.block_n * kAugRowBytes;
    uint8_t* smem_a = smem;
    uint8_t* smem_b = smem + MT * a_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_b + static_cast<size_t>(p.nstage) * stage_bytes);
    uint64_t* a_full = bars + 0;
    uint64_t* a_empty = bars + 1;
    uint64_t* t_full = bars + 2;    // [2]
    uint64_t* t_empty = bars + 4;   // [2]
    uint64_t* b_full = bars + 6;    // [kMaxStages]
    uint64_t* b_empty = bars + 6 + kMaxStages;
    uint64_t* drain = bars + 6 + 2 * kMaxStages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 7 + 2 * kMaxStages);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* hist_all = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(bars) + 256);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int G = gridDim.x;
    const int b = blockIdx.x;
    const int64_t T = p.total_units;
    const int NT = p.col_tiles;
    int64_t u0 = span_begin(T, G, NT, p.cross, b);
    int64_t u1 = span_begin(T, G, NT, p.cross, b + 1);
    if (p.whole_rows) {  // row groups dealt out whole: CTA b takes row groups [R b / G, R (b + 1) / G)
        const int64_t R = T / NT;
        u0 = (R * b / G) * NT;
        u1 = (R * (b + 1) / G) * NT;
    }
    // hand-over of the two epilogue warps of a lane quadrant (sketch rule with whole row groups)
    uint64_t* x_full = bars + 24;   // [4]
    uint64_t* x_empty = bars + 28;  // [4]

    if (threadIdx.x == 0) {
        mbar_init(a_full, p.x_raw != nullptr ? 4 * MT : 1);  // TMA bytes, or one arrival per widening warp
        mbar_init(a_empty, 1);
        mbar_init(drain, 1);
        for (int i = 0; i < 4; ++i) {
            mbar_init(&x_full[i], 1);
            mbar_init(&x_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&t_full[i], 1);
            mbar_init(&t_empty[i], kNumEpiWarps);
        }
        for (int i = 0; i < p.nstage; ++i) {
            mbar_init(&b_full[i], 1);
            mbar_init(&b_empty[i], 1);
        }
        *abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmap_x);
        tma_prefetch_desc(&tmap_xa);
        tma_prefetch_desc(&tmap_c);
        tma_prefetch_desc(&tmap_ca);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // the set-up above touched no global memory; from here on the predecessor's results are needed
    pdl_wait();
    pdl_trigger();
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        if (p.clear0) *p.clear0 = 0;
        if (p.clear1) *p.clear1 = 0;
    }
    if (threadIdx.x < 32 && blockIdx.x == 0 && p.clear32) p.clear32[threadIdx.x] = 0;

    WaitCtl ctl;
    ctl.abort_flag = abort_flag;
    ctl.status = p.status;
    ctl.limit_ns = p.wait_limit_ns;
    const int kd = p.kslices * kSliceK;  // K column where the norm columns start

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        // (uint8 points: the epilogue warps build the point tiles themselves, see below)
        const bool raw = p.x_raw != nullptr;
        int it = 0, seg = 0, a_armed = 0;
        int st = 0;        // ring stage of tile `it` and the parity of its use, stepped instead of
        uint32_t ph = 0;   // divided out of `it` (the stage count is a run-time value)
        bool ok = true;
        auto load_b = [&](int t) -> bool {  // lane 0: one centroid tile into the next ring stage
            if (!IVF_IN_BOUNDS(120, st, p.nstage) || !IVF_IN_BOUNDS(121, t, NT)) return false;
            if (!mbar_wait(&b_empty[st], ph ^ 1u, ctl, 2)) return false;
            mbar_arrive_expect_tx(&b_full[st], stage_bytes);
            uint8_t* dst = smem_b + static_cast<size_t>(st) * stage_bytes;
            for (int s = 0; s < p.kslices; ++s)
                tma_load_2d(dst + s * p.block_n * kSliceRowBytes, &tmap_c, &b_full[st], s * kSliceK, t * p.block_n);
            tma_load_2d(dst + b_data_bytes, &tmap_ca, &b_full[st], kd, t * p.block_n);
            ++it;
            if (++st == p.nstage) {
                st = 0;
                ph ^= 1u;
            }
            return true;
        };
        for (int64_t u = u0; u < u1 && ok;) {
            const int64_t r = u / NT;
            const int t0 = static_cast<int>(u - r * NT);
            const int t1 = static_cast<int>((u1 - r * NT < NT) ? (u1 - r * NT) : NT);
            if (raw && u1 > (r + 1) * NT) {
                // this CTA will move on to the next row group: pull its raw rows into L2 now, so that
                // the widening at the crossing does not wait for HBM
                const int64_t first_row = (r + 1) * MT * kBlockM;
                const int64_t last_row = (first_row + MT * kBlockM < p.n) ? first_row + MT * kBlockM : p.n;
                const char* base = reinterpret_cast<const char*>(p.x_raw) + first_row * p.d;
                const int64_t bytes = (last_row - first_row) * p.d;
                for (int64_t off = static_cast<int64_t>(lane) * 128; off < bytes; off += 32 * 128)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off));
            }
            if (lane == 0 && seg > 0) ok = mbar_wait(a_empty, (seg - 1) & 1, ctl, 1);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            int t = t0;
            if (!raw && lane == 0) {
                mbar_arrive_expect_tx(a_full, MT * a_bytes);
                ++a_armed;
                for (int h = 0; h < MT; ++h) {
                    const int y = static_cast<int>((r * MT + h) * kBlockM);
                    uint8_t* dst = smem_a + h * a_bytes;
                    for (int s = 0; s < p.kslices; ++s)
                        tma_load_2d(dst + s * kBlockM * kSliceRowBytes, &tmap_x, a_full, s * kSliceK, y);
                    tma_load_2d(dst + a_data_bytes, &tmap_xa, a_full, kd, y);
                }
            }
            if (lane == 0) {
                int col = (t0 + ((p.rotate && !p.whole_rows) ? col_rotation(T, G, NT, p.cross, r) : 0)) % NT;  // centroid tile of position t
                for (; t < t1 && ok; ++t) {
                    ok = load_b(col);
                    if (++col == NT) col = 0;
                }
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            ++seg;
            u = r * NT + t1;
        }
        if (lane == 0 && !ok) {
            // gave up: let the copies already issued land before the CTA goes away (bounded)
            const uint64_t t_start = global_timer_ns();
            const int first = it > p.nstage ? it - p.nstage : 0;
            for (int i = first; i < it; ++i) {
                const int st = i % p.nstage;
                const uint32_t ph = (i / p.nstage) & 1;
                while (!mbar_try_wait(&b_full[st], ph) && global_timer_ns() - t_start < 2000000000ull) {
                }
            }
            if (a_armed > 0) {
                while (!mbar_try_wait(a_full, (a_armed - 1) & 1) && global_timer_ns() - t_start < 2000000000ull) {
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f16(kBlockM, p.block_n);
            const uint32_t a_addr = smem_u32(smem_a);
            const uint32_t b_addr = smem_u32(smem_b);
            const uint32_t a_slice_step = (kBlockM * kSliceRowBytes) >> 4;
            const uint32_t b_slice_step = static_cast<uint32_t>(p.block_n * kSliceRowBytes) >> 4;
            // descriptor low words that never change: the point tiles (data and norm columns) and stage 0
            // of the ring; a stage's words follow by adding its offset in 16-byte units
            uint32_t a_lo_data[MT], a_lo_norm[MT];
#pragma unroll
            for (int h = 0; h < MT; ++h) {
                a_lo_data[h] = umma_desc_lo(a_addr + h * a_bytes);
                a_lo_norm[h] = umma_desc_lo(a_addr + h * a_bytes + a_data_bytes);
            }
            const uint32_t b_lo_data0 = umma_desc_lo(b_addr), b_lo_norm0 = umma_desc_lo(b_addr + b_data_bytes);
            const uint32_t stage_step = static_cast<uint32_t>(stage_bytes) >> 4;
            int it = 0, seg = 0;
            int st = 0;       // ring stage and use parity of tile `it`, stepped
            uint32_t ph = 0;
            bool acc_ready = false, b_ready = false;  // barriers of the next tile already seen complete
            bool ok = true;
            for (int64_t u = u0; u < u1 && ok;) {
                const int64_t r = u / NT;
                const int t0 = static_cast<int>(u - r * NT);
                const int t1 = static_cast<int>((u1 - r * NT < NT) ? (u1 - r * NT) : NT);
                ok = mbar_wait(a_full, seg & 1, ctl, 3);
                if (!ok) break;
                for (int t = t0; t < t1 && ok; ++t) {
                    if (!b_ready) ok = mbar_wait(&b_full[st], ph, ctl, 4);
                    if (!ok) break;
                    b_ready = false;
                    const uint32_t b_lo_data = b_lo_data0 + st * stage_step, b_lo_norm = b_lo_norm0 + st * stage_step;
#pragma unroll
                    for (int h = 0; h < MT; ++h) {
                        const int su = it * MT + h;  // accumulator buffers alternate per (tile, row tile)
                        const int buf = su & 1;
                        const uint32_t aph = (su >> 1) & 1;
                        if (!acc_ready) ok = mbar_wait(&t_empty[buf], aph ^ 1u, ctl, 5);
                        if (!ok) break;
                        acc_ready = false;
                        tc_fence_after_sync();
                        const uint32_t d_tmem = tmem_base + buf * kAccStride;
                        (void)IVF_IN_BOUNDS(130, buf * kAccStride + p.block_n, kTmemCols + 1);
                        (void)IVF_IN_BOUNDS(131, st, p.nstage);
                        // The descriptors of consecutive K steps differ only in the start-address field
                        // (16-byte units, low word): +2 inside a 64-column slice, then on to the next
                        // slice.  Stepping the low words keeps this thread's work per MMA to a few
                        // instructions; building each descriptor from scratch took about as long as the
                        // tensor core needs for the MMA itself.
                        uint32_t a_lo = a_lo_data[h], b_lo = b_lo_data;
                        for (int kk = 0; kk < p.ksteps; ++kk) {
                            umma_f16(d_tmem, umma_desc_join(a_lo, kDescHiSw128), umma_desc_join(b_lo, kDescHiSw128), idesc,
                                     kk > 0 ? 1u : 0u);
                            const bool last_of_slice = (kk & 3) == 3;
                            a_lo += last_of_slice ? a_slice_step - 6u : 2u;
                            b_lo += last_of_slice ? b_slice_step - 6u : 2u;
                        }
                        // While the tensor core works through those, look at the barriers the next tile
                        // will need: a wait costs this thread 50-100 cycles even when the phase has long
                        // completed, and the tensor core's queue runs dry meanwhile.
                        {
                            const int nsu = su + 1;
                            acc_ready = mbar_test_wait(&t_empty[nsu & 1], ((nsu >> 1) & 1u) ^ 1u);
                            if (h == MT - 1) {
                                const bool wrap = st + 1 == p.nstage;
                                b_ready = mbar_test_wait(&b_full[wrap ? 0 : st + 1], wrap ? ph ^ 1u : ph);
                            }
                        }
                        umma_f16(d_tmem, umma_desc_join(a_lo_norm[h], kDescHiSw32), umma_desc_join(b_lo_norm, kDescHiSw32), idesc,
                                 1u);
                        umma_commit(&t_full[buf]);
                    }
                    if (!ok) break;
                    umma_commit(&b_empty[st]);
                    ++it;
                    if (++st == p.nstage) {
                        st = 0;
                        ph ^= 1u;
                    }
                }
                if (ok) umma_commit(a_empty);
                ++seg;
                u = r * NT + t1;
            }
            if (!ok && it > 0) {
                // gave up: wait (bounded) until the MMAs already issued have retired before TMEM is freed
                umma_commit(drain);
                const uint64_t t_start = global_timer_ns();
                while (!mbar_try_wait(drain, 0) && global_timer_ns() - t_start < 2000000000ull) {
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int quad = warp & 3;               // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
        const int half = (warp - 2) >> 2;        // which 64-column groups of a tile this warp takes
        const int row_in_tile = quad * 32 + lane;
        [[maybe_unused]] int* hist = hist_all + (warp - 2) * 256;
        const float INF = __int_as_float(0x7f800000);
        const int nq = p.block_n / 64;  // 32-column chunks per warp and tile: 4 or 2
        constexpr bool kHasLog = (EPI == EPI_RUNNING || EPI == EPI_FILTER);
        constexpr bool kWideLoads = (EPI == EPI_ARGMIN);
        float raw_scales[4] = {1.f, 1.f, 1.f, 1.f};
        if (p.x_raw != nullptr) {
            compute_scales(p.bits, 1, raw_scales);
            if (b == 0 && warp == 2 && lane == 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i) p.scal_out[i] = raw_scales[i];
            }
        }
        int it = 0;
        [[maybe_unused]] int xseg = 0;  // row groups whose threshold this CTA has finished
        bool ok = true;
        [[maybe_unused]] const float* tau_fold = nullptr;
        for (int64_t u = u0; u < u1 && ok;) {
            const int64_t r = u / NT;  // row group
            const int t0 = static_cast<int>(u - r * NT);
            const int t1 = static_cast<int>((u1 - r * NT < NT) ? (u1 - r * NT) : NT);
            const int slot = p.whole_rows ? half : (b - cta_of_unit(T, G, NT, p.cross, r * NT)) * kEpiHalves + half;
            if (!IVF_IN_BOUNDS(140, slot, p.partials)) break;  // (checked build only: a slot outside the row's partials)

            if (p.x_raw != nullptr && half < MT) {
                // uint8 points: this warp widens its 32 rows of point tile `half`.  The tile is free:
                // the last accumulator of the previous row group could only be read after every MMA
                // that used the old tile had completed.
                widen_rows_u8_warp(p.x_raw, (r * MT + half) * kBlockM + quad * 32, p.n, p.d, kd, smem_a + half * a_bytes,
                                   a_data_bytes, quad * 32, lane, raw_scales[0], raw_scales[3], p.xn_out);
                fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(a_full);
            }
            if constexpr (EPI == EPI_GROUPS) {
                if (p.sketch_t != nullptr && tau_fold == nullptr) {
                    // (after the point tile is handed to the MMA warp, so that the first tiles are
                    // computed meanwhile.)  Epilogue warp w finishes the thresholds of rows w, w + 8, ...:
                    // the batch has at most kFoldRows rows
                    float* ts = reinterpret_cast<float*>(hist_all);
                    for (int e = warp - 2; e < p.n; e += kNumEpiWarps) {
                        const float t = warp_threshold_of_sketches(p.sketch_t + static_cast<size_t>(e) * kSampleM * p.sketch_pitch,
                                                                   p.sketch_slots, p.sketch_pitch, lane);
                        if (lane == 0) ts[e] = t;
                    }
                    asm volatile("bar.sync 2, %0;" ::"n"(kNumEpiWarps * 32) : "memory");  // the epilogue warps only
                    tau_fold = ts;
                }
            }

            RowState<EPI> st[MT];
            int64_t row[MT];
            bool valid[MT];
#pragma unroll
            for (int h = 0; h < MT; ++h) {
                row[h] = (r * MT + h) * kBlockM + row_in_tile;
                valid[h] = row[h] < p.n;
                st[h].tau = valid[h] ? INF : -INF;  // invalid rows: a threshold nothing passes
                if constexpr (EPI == EPI_ARGMIN) st[h].bestj = 0x7fffffff;
                if constexpr (EPI == EPI_RUNNING || EPI == EPI_SKETCH) {
#pragma unroll
                    for (int i = 0; i < kSampleM; ++i) st[h].net[i] = INF;
                }
                if constexpr (kHasLog) {
                    st[h].cnt = 0;
                    st[h].log = p.part + (static_cast<size_t>(valid[h] ? row[h] : 0) * p.partials + slot) * p.cap;
                    if (EPI == EPI_FILTER && p.rule == TAU_GIVEN && valid[h]) st[h].tau = p.tau_in[row[h]];
                }
                if constexpr (EPI == EPI_GROUPS) {
                    st[h].base = reinterpret_cast<char*>(p.part) +
                                 (static_cast<size_t>(valid[h] ? row[h] : 0) * p.partials + slot) * p.cap * kRecordBytes;
                    st[h].wp = st[h].base;
                    st[h].limit = st[h].base + static_cast<size_t>(p.cap - kGroupLogMargin) * kRecordBytes;
                    st[h].overflow = 0;
                    if (valid[h]) st[h].tau = tau_fold != nullptr ? tau_fold[row[h]] : p.tau_in[row[h]];
                }
            }

            int col = (t0 + ((p.rotate && !p.whole_rows) ? col_rotation(T, G, NT, p.cross, r) : 0)) % NT;  // centroid tile of position t
            for (int t = t0; t < t1 && ok; ++t) {
                const bool ragged = (col + 1) * p.block_n > p.nlist;
                const int tile_j0 = col * p.block_n;
                if (++col == NT) col = 0;
#pragma unroll
                for (int h = 0; h < MT; ++h) {
                    const int su = it * MT + h;
                    const int buf = su & 1;
                    const uint32_t aph = (su >> 1) & 1;
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(&t_full[buf], aph, ctl, 6));
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * kAccStride;
                    [[maybe_unused]] const int64_t warp_row0 = (r * MT + h) * kBlockM + quad * 32;

                    // chunk q of this warp starts at column ((q/2) * halves + half) * 64 + (q%2) * 32
                    auto col_of = [&](int q) { return ((q >> 1) * kEpiHalves + half) * 64 + (q & 1) * 32; };
                    (void)IVF_IN_BOUNDS(142, buf * kAccStride + col_of(nq - 1) + 32, kTmemCols + 1);
                    auto after_chunk = [&]() {
                        if constexpr (kHasLog) {
                            (void)IVF_IN_BOUNDS(145, st[h].cnt, p.cap + 1);
                            if (__any_sync(0xFFFFFFFFu, st[h].cnt > p.cap - 32)) {
                                __syncwarp();
                                for (int rr = 0; rr < 32; ++rr) {
                                    const int c_r = __shfl_sync(0xFFFFFFFFu, st[h].cnt, rr);
                                    if (c_r > p.cap - 32) {
                                        Entry* lr = p.part +
                                                    (static_cast<size_t>(warp_row0 + rr) * p.partials + slot) * p.cap;
                                        const float tk = warp_select_k(lr, c_r, p.k, hist, lane);
                                        if (p.stats && lane == 0) atomicAdd(&p.stats[0], 1ull);
                                        if (lane == rr) {
                                            st[h].cnt = p.k;
                                            st[h].tau = fminf(st[h].tau, tk);
                                        }
                                    }
                                }
                            }
                        }
                    };
                    // TMEM -> register loads have a long latency and only one wait primitive
                    // (it waits for all of the thread's loads), so each round trip fetches 64 columns
                    // as two 32-column loads issued back to back; the other epilogue warp of the
                    // scheduler computes meanwhile.
                    uint32_t accA[32], accB[32];
                    if (kWideLoads && nq == 4) {
                        // All 128 columns of this warp in one round trip, so that the accumulator goes
                        // back to the MMA warp one load latency after it was filled: the MMA-issuing
                        // thread cannot run far ahead of the tensor core, and every cycle it waits for a
                        // free accumulator is a cycle the tensor core idles.
                        uint32_t accC[32], accD[32];
                        tmem_ld_32x32b_x32(taddr + col_of(0), accA);
                        tmem_ld_32x32b_x32(taddr + col_of(1), accB);
                        tmem_ld_32x32b_x32(taddr + col_of(2), accC);
                        tmem_ld_32x32b_x32(taddr + col_of(3), accD);
                        tmem_wait_ld_regs(accA);
                        tmem_wait_ld_regs(accB);
                        tmem_wait_ld_regs(accC);
                        tmem_wait_ld_regs(accD);
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&t_empty[buf]);
                        if (ragged) {
                            mask_ragged(accA, tile_j0 + col_of(0), p.nlist);
                            mask_ragged(accB, tile_j0 + col_of(1), p.nlist);
                            mask_ragged(accC, tile_j0 + col_of(2), p.nlist);
                            mask_ragged(accD, tile_j0 + col_of(3), p.nlist);
                        }
                        consume<EPI>(accA, tile_j0 + col_of(0), st[h]);
                        after_chunk();
                        consume<EPI>(accB, tile_j0 + col_of(1), st[h]);
                        after_chunk();
                        consume<EPI>(accC, tile_j0 + col_of(2), st[h]);
                        after_chunk();
                        consume<EPI>(accD, tile_j0 + col_of(3), st[h]);
                        after_chunk();
                    } else {
#pragma unroll
                    for (int q = 0; q < 4; q += 2) {
                        if (q < nq) {
                            tmem_ld_32x32b_x32(taddr + col_of(q), accA);
                            tmem_ld_32x32b_x32(taddr + col_of(q + 1), accB);
                            tmem_wait_ld_regs(accA);
                            tmem_wait_ld_regs(accB);
                            if (q + 2 >= nq) {
                                // the warp's last columns of this accumulator are in registers: hand the
                                // buffer back to the MMA warp before working on them
                                tc_fence_before_sync();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(&t_empty[buf]);
                            }
                            if (ragged) {
                                mask_ragged(accA, tile_j0 + col_of(q), p.nlist);
                                mask_ragged(accB, tile_j0 + col_of(q + 1), p.nlist);
                            }
                            consume<EPI>(accA, tile_j0 + col_of(q), st[h]);
                            after_chunk();
                            consume<EPI>(accB, tile_j0 + col_of(q + 1), st[h]);
                            after_chunk();
                        }
                    }
                    }
                    if constexpr (EPI == EPI_GROUPS) {
                        // checked once per tile (a tile appends at most 16 records per thread).  A full
                        // log cannot be compacted here (it holds raw groups): the row is flagged and
                        // recomputed by brute force after the merge
                        (void)IVF_IN_BOUNDS(143, st[h].wp - st[h].base, static_cast<long long>(p.cap) * kRecordBytes + 1);
                        if (st[h].wp > st[h].limit) {
                            st[h].overflow = 1;
                            st[h].wp = st[h].base;
                        }
                    }
                }
                ++it;
            }
            if constexpr (EPI == EPI_SKETCH && MT == 1) {
                if (ok && (p.tau_out != nullptr || p.sketch_t != nullptr)) {
                    // The two warps of every lane quadrant split the tiles' columns between them: the
                    // upper-half warp passes its 16 sorted minima through shared memory to the lower-half
                    // warp.  tau_out: this CTA saw the row group's whole sample and the lower-half warp
                    // finishes the threshold -- with a and b ascending, min(a[i], b[15 - i]) over i are the
                    // 16 smallest of the 32 values, so their maximum is the 16th smallest.  sketch_t: the
                    // lower-half warp merges the two lists into the CTA's one partial sketch.
                    float* xch = reinterpret_cast<float*>(hist_all) + row_in_tile * kSampleM;
                    if (half == 1) {
                        if (xseg > 0) ok = __all_sync(0xFFFFFFFFu, mbar_wait(&x_empty[quad], (xseg - 1) & 1, ctl, 7));
                        if (ok) {
#pragma unroll
                            for (int i = 0; i < kSampleM; i += 4)
                                *reinterpret_cast<float4*>(xch + i) = make_float4(st[0].net[i], st[0].net[i + 1], st[0].net[i + 2], st[0].net[i + 3]);
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&x_full[quad]);
                        }
                    } else {
                        ok = __all_sync(0xFFFFFFFFu, mbar_wait(&x_full[quad], xseg & 1, ctl, 8));
                        if (ok) {
                            float other[kSampleM];
#pragma unroll
                            for (int i = 0; i < kSampleM; i += 4) {
                                const float4 v = *reinterpret_cast<const float4*>(xch + i);
                                other[i] = v.x; other[i + 1] = v.y; other[i + 2] = v.z; other[i + 3] = v.w;
                            }
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&x_empty[quad]);
                            if (p.tau_out != nullptr) {
                                float t16 = -INF;
#pragma unroll
                                for (int i = 0; i < kSampleM; ++i) t16 = fmaxf(t16, fminf(st[0].net[i], other[kSampleM - 1 - i]));
                                if (valid[0]) p.tau_out[row[0]] = t16;
                            } else {
                                merge16_sorted(st[0].net, other);
                            }
                        }
                    }
                    ++xseg;
                }
            }
            if (ok && !(EPI == EPI_SKETCH && p.tau_out != nullptr)) {
#pragma unroll
                for (int h = 0; h < MT; ++h) {
                    if (!valid[h]) continue;
                    const size_t at = static_cast<size_t>(row[h]) * p.partials + slot;
                    if (!IVF_IN_BOUNDS(144, at, p.n * p.partials)) continue;
                    if constexpr (EPI == EPI_ARGMIN) {
                        Entry e;
                        e.v = st[h].tau;
                        e.j = st[h].bestj;
                        p.part[at] = e;
                    } else if constexpr (EPI == EPI_SKETCH) {
                        // the partial result of the threshold pass: the thread's 16 smallest group minima
                        if (p.sketch_t != nullptr) {
                            // (a batch of a few rows, read back by the main pass with slot = lane; with one
                            // row tile per unit the lower-half warp holds the CTA's merged sketch)
                            const int slot_out = MT == 1 ? slot >> 1 : slot;
                            if ((MT != 1 || half == 0) && IVF_IN_BOUNDS(146, slot_out, p.sketch_pitch)) {
                                float* out = p.sketch_t + static_cast<size_t>(row[h]) * kSampleM * p.sketch_pitch + slot_out;
#pragma unroll
                                for (int i = 0; i < kSampleM; ++i) out[static_cast<size_t>(i) * p.sketch_pitch] = st[h].net[i];
                            }
                        } else {
                            Entry* log = p.part + at * p.cap;
#pragma unroll
                            for (int i = 0; i < kSampleM; ++i)
                                *reinterpret_cast<uint2*>(&log[i]) = make_uint2(__float_as_uint(st[h].net[i]), 0u);
                        }
                        p.part_meta[at] = make_int2(kSampleM, __float_as_int(INF));
                    } else if constexpr (EPI == EPI_GROUPS) {
                        const int recs = static_cast<int>((st[h].wp - st[h].base) / kRecordBytes);
                        p.part_meta[at] = make_int2(st[h].overflow ? -1 : recs, __float_as_int(st[h].tau));
                        if (p.stats) atomicAdd(&p.stats[1], static_cast<unsigned long long>(recs));
                    } else {
                        p.part_meta[at] = make_int2(st[h].cnt, __float_as_int(st[h].tau));
                        if (p.stats) atomicAdd(&p.stats[1], static_cast<unsigned long long>(st[h].cnt));
                    }
                }
            }
            u = r * NT + t1;
        }
    }

    // ------------------------------------------------------------ teardown (also the abort path)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace ivf
