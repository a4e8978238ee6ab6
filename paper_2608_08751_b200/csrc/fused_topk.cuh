// Fused distance + per-row top-k kernel (Sec. 4.1: dense centroid evaluation by Eq. 3 and
// on-device list selection; Sec. 3.1 / 5.5: assignment is the k = 1 case).
//
// One persistent CTA per SM walks a contiguous span of (row tile, centroid tile) units.
//   warp 0      TMA producer: the stationary 128-row point tile and a ring of centroid tiles
//   warp 1      single-thread tcgen05.mma issuer; S = X * C^T accumulates in TMEM (fp32), two
//               accumulator buffers so the next tile's MMAs overlap this tile's epilogue
//   warps 2..5  epilogue: each thread owns one point row (= one TMEM lane), reads its 256
//               accumulator columns with tcgen05.ld, forms the ranking key
//               v = |c|^2 - 2 x.c  and keeps the row's candidates.  Nothing of the n x nlist
//               matrix is written to memory.
// k = 1 keeps (best key, id) in registers.  k > 1 appends every key below the row's threshold tau
// to the row's candidate log; when a log fills up, its warp selects the k smallest in place (radix
// select on the key bits, ties to the lower id) and tightens tau to the k-th.  A row tile whose
// centroid sweep is shared by several CTAs yields one partial result per CTA; a second kernel
// merges them (merge.cuh).
#pragma once
#include "ptx.cuh"

namespace ivf {

constexpr int kBlockM = 128;         // point rows per tile = TMEM lanes
constexpr int kTmemCols = 512;       // whole TMEM: two accumulator buffers of 256 columns
constexpr int kAccStride = 256;      // TMEM columns between the two accumulator buffers
constexpr int kNumEpiWarps = 4;
constexpr int kFusedThreads = 32 * (2 + kNumEpiWarps);
constexpr int kSliceK = 64;          // fp16 elements per 128-byte swizzled row
constexpr int kSliceRowBytes = 128;
constexpr int kMaxStages = 8;

struct Entry {
    float v;  // ranking key  |c|^2 - 2 x.c
    int j;    // centroid id
};

enum { MODE_ARGMIN = 0, MODE_APPEND = 1 };

struct FusedParams {
    int64_t n;            // point rows
    int nlist;
    int k;
    int mode;
    int ksteps;           // MMA instructions per tile = ceil(d / 16)
    int kslices;          // 64-wide K slices of the operand copies
    int block_n;          // centroids per tile: 256 or 128
    int nstage;           // centroid-tile ring depth
    int col_tiles;        // centroid tiles per sweep
    int64_t total_units;  // row tiles * col_tiles
    int partials;         // partial-result slots per row
    int cap;              // candidate-log capacity per (row, slot), k > 1 only
    const float* cn;      // |c|^2, padded with +inf to col_tiles * block_n
    const float* scal;    // device scalars: scal[2] = -2 / (point scale * centroid scale)
    Entry* part;          // k = 1: [n][partials]; k > 1: [n][partials][cap]
    int* part_cnt;        // k > 1: [n][partials] entries in each log
    int* status;          // sticky device status word
    uint64_t wait_limit_ns;
};

// ---- persistent schedule: CTA b of G owns units [T*b/G, T*(b+1)/G) of the row-major unit grid
__host__ __device__ inline int64_t span_begin(int64_t T, int G, int b) { return (T * b) / G; }
__host__ __device__ inline int cta_of_unit(int64_t T, int G, int64_t u) {
    return static_cast<int>(((u + 1) * G - 1) / T);
}

__host__ __device__ inline size_t fused_smem_bytes(int kslices, int block_n, int nstage) {
    return 1024                                                    // alignment slack
           + static_cast<size_t>(kslices) * kBlockM * kSliceRowBytes  // point tile
           + static_cast<size_t>(nstage) * kslices * block_n * kSliceRowBytes
           + 256                                                   // barriers, TMEM slot, abort flag
           + kNumEpiWarps * 256 * sizeof(int);                     // radix histograms
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
        if (keep) *reinterpret_cast<uint2*>(&log[base + __popc(bal & lt_mask)]) = e;
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

__device__ __forceinline__ float min3f(float a, float b, float c) { return fminf(fminf(a, b), c); }

__global__ void __launch_bounds__(kFusedThreads, 1)
fused_topk_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_c,
                  const FusedParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int a_bytes = p.kslices * kBlockM * kSliceRowBytes;
    const int stage_bytes = p.kslices * p.block_n * kSliceRowBytes;
    uint8_t* smem_a = smem;
    uint8_t* smem_b = smem + a_bytes;
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
    const int64_t u0 = span_begin(T, G, b);
    const int64_t u1 = span_begin(T, G, b + 1);

    if (threadIdx.x == 0) {
        mbar_init(a_full, 1);
        mbar_init(a_empty, 1);
        mbar_init(drain, 1);
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
        tma_prefetch_desc(&tmap_c);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    WaitCtl ctl;
    ctl.abort_flag = abort_flag;
    ctl.status = p.status;
    ctl.limit_ns = p.wait_limit_ns;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int it = 0, seg = 0, a_armed = 0;
            bool ok = true;
            for (int64_t u = u0; u < u1 && ok;) {
                const int64_t r = u / NT;
                const int t0 = static_cast<int>(u - r * NT);
                const int t1 = static_cast<int>((u1 - r * NT < NT) ? (u1 - r * NT) : NT);
                if (seg > 0) ok = mbar_wait(a_empty, (seg - 1) & 1, ctl, 1);
                if (!ok) break;
                mbar_arrive_expect_tx(a_full, a_bytes);
                ++a_armed;
                for (int s = 0; s < p.kslices; ++s)
                    tma_load_2d(smem_a + s * kBlockM * kSliceRowBytes, &tmap_x, a_full, s * kSliceK,
                                static_cast<int>(r * kBlockM));
                for (int t = t0; t < t1; ++t) {
                    const int st = it % p.nstage;
                    const uint32_t ph = (it / p.nstage) & 1;
                    ok = mbar_wait(&b_empty[st], ph ^ 1u, ctl, 2);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&b_full[st], stage_bytes);
                    uint8_t* dst = smem_b + static_cast<size_t>(st) * stage_bytes;
                    for (int s = 0; s < p.kslices; ++s)
                        tma_load_2d(dst + s * p.block_n * kSliceRowBytes, &tmap_c, &b_full[st], s * kSliceK,
                                    t * p.block_n);
                    ++it;
                }
                ++seg;
                u = r * NT + t1;
            }
            if (!ok) {
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
                    while (!mbar_try_wait(a_full, (a_armed - 1) & 1) &&
                           global_timer_ns() - t_start < 2000000000ull) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f16(kBlockM, p.block_n);
            const uint32_t a_addr = smem_u32(smem_a);
            const uint32_t b_addr = smem_u32(smem_b);
            int it = 0, seg = 0;
            bool ok = true;
            for (int64_t u = u0; u < u1 && ok;) {
                const int64_t r = u / NT;
                const int t0 = static_cast<int>(u - r * NT);
                const int t1 = static_cast<int>((u1 - r * NT < NT) ? (u1 - r * NT) : NT);
                ok = mbar_wait(a_full, seg & 1, ctl, 3);
                if (!ok) break;
                for (int t = t0; t < t1; ++t) {
                    const int st = it % p.nstage;
                    const uint32_t ph = (it / p.nstage) & 1;
                    const int buf = it & 1;
                    const uint32_t aph = (it >> 1) & 1;
                    ok = mbar_wait(&b_full[st], ph, ctl, 4);
                    if (ok) ok = mbar_wait(&t_empty[buf], aph ^ 1u, ctl, 5);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + buf * kAccStride;
                    for (int kk = 0; kk < p.ksteps; ++kk) {
                        const int slice = kk >> 2;
                        const uint32_t off = (kk & 3) * 32;  // 16 fp16 = 32 bytes inside the swizzled row
                        const uint64_t adesc = umma_desc_sw128(a_addr + slice * kBlockM * kSliceRowBytes + off);
                        const uint64_t bdesc =
                            umma_desc_sw128(b_addr + st * stage_bytes + slice * p.block_n * kSliceRowBytes + off);
                        umma_f16(d_tmem, adesc, bdesc, idesc, kk > 0 ? 1u : 0u);
                    }
                    umma_commit(&b_empty[st]);
                    umma_commit(&t_full[buf]);
                    ++it;
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
        const int quad = warp & 3;  // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
        const int row_in_tile = quad * 32 + lane;
        int* hist = hist_all + (warp - 2) * 256;
        const float mult = p.scal[2];
        const float INF = __int_as_float(0x7f800000);
        int it = 0;
        bool ok = true;
        for (int64_t u = u0; u < u1 && ok;) {
            const int64_t r = u / NT;
            const int t0 = static_cast<int>(u - r * NT);
            const int t1 = static_cast<int>((u1 - r * NT < NT) ? (u1 - r * NT) : NT);
            const int64_t row = r * kBlockM + row_in_tile;
            const bool valid = row < p.n;
            const int slot = b - cta_of_unit(T, G, r * NT);
            const int64_t warp_row0 = r * kBlockM + quad * 32;

            float best = valid ? INF : -INF;  // k = 1: best key; k > 1: threshold tau
            int bestj = 0x7fffffff;
            int cnt = 0;
            Entry* log = nullptr;
            if (p.mode == MODE_APPEND && valid)
                log = p.part + (static_cast<size_t>(row) * p.partials + slot) * p.cap;

            for (int t = t0; t < t1; ++t) {
                const int buf = it & 1;
                const uint32_t aph = (it >> 1) & 1;
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(&t_full[buf], aph, ctl, 6));
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + buf * kAccStride;
                const int nchunks = p.block_n / 32;
#pragma unroll 1
                for (int ch = 0; ch < nchunks; ++ch) {
                    uint32_t acc[32];
                    tmem_ld_32x32b_x32(taddr + ch * 32, acc);
                    const int jbase = t * p.block_n + ch * 32;
                    const float4* cn4 = reinterpret_cast<const float4*>(p.cn + jbase);
                    float key[32];
                    float4 cnv[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) cnv[q] = __ldg(cn4 + q);
                    tmem_wait_ld();
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        key[4 * q + 0] = fmaf(__uint_as_float(acc[4 * q + 0]), mult, cnv[q].x);
                        key[4 * q + 1] = fmaf(__uint_as_float(acc[4 * q + 1]), mult, cnv[q].y);
                        key[4 * q + 2] = fmaf(__uint_as_float(acc[4 * q + 2]), mult, cnv[q].z);
                        key[4 * q + 3] = fmaf(__uint_as_float(acc[4 * q + 3]), mult, cnv[q].w);
                    }
                    if (p.mode == MODE_ARGMIN) {
                        float m = key[0];
#pragma unroll
                        for (int c = 1; c < 31; c += 2) m = min3f(m, key[c], key[c + 1]);
                        m = fminf(m, key[31]);
                        if (m < best) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) {
                                if (key[c] < best) {
                                    best = key[c];
                                    bestj = jbase + c;
                                }
                            }
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            if (key[c] < best) {
                                *reinterpret_cast<uint2*>(&log[cnt]) =
                                    make_uint2(__float_as_uint(key[c]), static_cast<uint32_t>(jbase + c));
                                ++cnt;
                            }
                        }
                        if (__any_sync(0xFFFFFFFFu, cnt > p.cap - 32)) {
                            __syncwarp();
                            for (int rr = 0; rr < 32; ++rr) {
                                const int c_r = __shfl_sync(0xFFFFFFFFu, cnt, rr);
                                if (c_r > p.cap - 32) {
                                    Entry* lr = p.part +
                                                (static_cast<size_t>(warp_row0 + rr) * p.partials + slot) * p.cap;
                                    const float tau = warp_select_k(lr, c_r, p.k, hist, lane);
                                    if (lane == rr) {
                                        cnt = p.k;
                                        best = tau;
                                    }
                                }
                            }
                        }
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&t_empty[buf]);
                ++it;
            }
            if (ok && valid) {
                if (p.mode == MODE_ARGMIN) {
                    Entry e;
                    e.v = best;
                    e.j = bestj;
                    p.part[static_cast<size_t>(row) * p.partials + slot] = e;
                } else {
                    p.part_cnt[static_cast<size_t>(row) * p.partials + slot] = cnt;
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
