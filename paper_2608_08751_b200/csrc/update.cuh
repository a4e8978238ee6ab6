// Lloyd centroid update (Sec. 5.5 "Lloyd iterations"): per-list sum and count of the member rows,
// as a segmented reduction.  The ids are turned into list segments by a counting sort (histogram,
// exclusive scan, fill), then one warp per list gathers and adds its member rows and is the only
// writer of that list's sums and count, so no floating-point atomics are involved.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "ptx.cuh"

namespace ivf {

constexpr int kStatusBadId = -6;

__global__ void update_hist_kernel(const int32_t* __restrict__ ids, int64_t n, int nlist, int* __restrict__ cnt,
                                   int* status) {
    pdl_wait();
    pdl_trigger();
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int l = ids[i];
    if (l < 0 || l >= nlist) {
        atomicCAS(status, 0, kStatusBadId);
        return;
    }
    atomicAdd(&cnt[l], 1);
}

// Exclusive scan of cnt[0..nlist) into off[0..nlist] in two small kernels.  First every CTA scans
// its own 4096 counts and publishes their total; then every CTA adds the totals of the CTAs before
// it (at most a few hundred values) to its slice, and clears the fill cursors.
constexpr int kScanBlock = 4096;

__global__ void __launch_bounds__(1024) update_scan_local_kernel(const int* __restrict__ cnt, int nlist,
                                                                 int* __restrict__ off, int* __restrict__ block_sums) {
    pdl_wait();
    pdl_trigger();
    __shared__ int warp_sums[32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int i0 = blockIdx.x * kScanBlock + threadIdx.x * 4;
    int v[4];
    int tsum = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        v[q] = (i0 + q < nlist) ? cnt[i0 + q] : 0;
        tsum += v[q];
    }
    int incl = tsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_sums[w] = incl;
    __syncthreads();
    if (w == 0) {
        const int ws = warp_sums[lane];
        int wi = ws;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
            if (lane >= o) wi += t;
        }
        warp_sums[lane] = wi - ws;  // exclusive prefix of the warp sums
        if (lane == 31) block_sums[blockIdx.x] = wi;
    }
    __syncthreads();
    int run = warp_sums[w] + (incl - tsum);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        if (i0 + q < nlist) off[i0 + q] = run;
        run += v[q];
    }
}

__global__ void __launch_bounds__(1024) update_scan_fix_kernel(int nlist, int* __restrict__ off,
                                                               const int* __restrict__ block_sums,
                                                               int* __restrict__ cursor) {
    pdl_wait();
    pdl_trigger();
    __shared__ int s_part[32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int acc = 0;
    for (int b = threadIdx.x; b < static_cast<int>(blockIdx.x); b += blockDim.x) acc += block_sums[b];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (lane == 0) s_part[w] = acc;
    __syncthreads();
    int before = 0;
#pragma unroll
    for (int i = 0; i < 32; ++i) before += s_part[i];
    const int i0 = blockIdx.x * kScanBlock + threadIdx.x * 4;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        if (i0 + q < nlist) {
            off[i0 + q] += before;
            cursor[i0 + q] = 0;
        }
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) off[nlist] = before + block_sums[blockIdx.x];
}

__global__ void update_fill_kernel(const int32_t* __restrict__ ids, int64_t n, int nlist,
                                   const int* __restrict__ off, int* __restrict__ cursor, int* __restrict__ perm) {
    pdl_wait();
    pdl_trigger();
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int l = ids[i];
    if (l < 0 || l >= nlist) return;
    const int pos = off[l] + atomicAdd(&cursor[l], 1);
    if (IVF_IN_BOUNDS(301, pos, n)) perm[pos] = static_cast<int>(i);
}

// Sum of the member rows perm[beg .. end) for one warp: lane q owns columns [128*blk + 4*q, +4) for
// blk = 0, 1 (d <= 256), four member rows in flight.
template <typename T>
__device__ __forceinline__ void reduce_members(const T* __restrict__ x, const int* __restrict__ perm, int beg, int end, int d,
                                               int lane, float (&acc)[2][4]) {
    for (int m0 = beg; m0 < end; m0 += 32) {
        const int mine = (m0 + lane < end) ? perm[m0 + lane] : -1;
        const int cntm = min(32, end - m0);
        for (int m = 0; m < cntm; m += 4) {  // four member rows in flight
            int64_t rows[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) rows[u] = __shfl_sync(0xFFFFFFFFu, mine, (m + u) & 31);
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) {
                const int c0 = 128 * blk + 4 * lane;
                if (c0 < d) {
                    if constexpr (sizeof(T) == 1) {
                        uint32_t wv[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            wv[u] = (m + u < cntm) ? *reinterpret_cast<const uint32_t*>(x + rows[u] * d + c0) : 0u;
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if constexpr (std::is_signed<T>::value) {
                                const int sv = static_cast<int>(wv[u]);  // arithmetic shifts sign-extend each byte
                                acc[blk][0] += static_cast<float>((sv << 24) >> 24);
                                acc[blk][1] += static_cast<float>((sv << 16) >> 24);
                                acc[blk][2] += static_cast<float>((sv << 8) >> 24);
                                acc[blk][3] += static_cast<float>(sv >> 24);
                            } else {
                                acc[blk][0] += static_cast<float>(wv[u] & 0xFFu);
                                acc[blk][1] += static_cast<float>((wv[u] >> 8) & 0xFFu);
                                acc[blk][2] += static_cast<float>((wv[u] >> 16) & 0xFFu);
                                acc[blk][3] += static_cast<float>(wv[u] >> 24);
                            }
                        }
                    } else {
                        float4 fv[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            fv[u] = (m + u < cntm) ? *reinterpret_cast<const float4*>(x + rows[u] * d + c0)
                                                   : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            acc[blk][0] += fv[u].x;
                            acc[blk][1] += fv[u].y;
                            acc[blk][2] += fv[u].z;
                            acc[blk][3] += fv[u].w;
                        }
                    }
                }
            }
        }
    }
}

// One warp per list.
template <typename T>
__global__ void update_reduce_kernel(const T* __restrict__ x, const int* __restrict__ perm,
                                     const int* __restrict__ off, int nlist, int d, float* __restrict__ sums,
                                     long long* __restrict__ counts) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const int l = static_cast<int>((static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5);
    if (l >= nlist) return;
    const int beg = off[l], end = off[l + 1];
    if (beg == end) return;
    if (!IVF_IN_BOUNDS(302, end - beg, off[nlist] + 1) || !IVF_IN_BOUNDS(303, end, off[nlist] + 1)) return;
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    reduce_members(x, perm, beg, end, d, lane, acc);
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
        const int c0 = 128 * blk + 4 * lane;
        if (c0 < d) {
            float4* dst = reinterpret_cast<float4*>(sums + static_cast<int64_t>(l) * d + c0);
            float4 s = *dst;
            s.x += acc[blk][0];
            s.y += acc[blk][1];
            s.z += acc[blk][2];
            s.w += acc[blk][3];
            *dst = s;
        }
    }
    if (lane == 0) counts[l] += static_cast<long long>(end - beg);
}

// Few long lists (k-means with a handful of clusters, PQ codebook training with 256): every list is
// cut into `parts` equal pieces, one warp per piece writes its partial sum to scratch[l][part][d],
// and update_combine_parts_kernel adds a list's partial sums in piece order.
// Reproducibility: the fill places a list's members with an atomic cursor, so their order inside the
// list depends on scheduling.  Byte-typed rows are summed exactly (integers below 2^24), so their sums
// and all counts are bit-identical from run to run; float sums are reproducible only within the
// rounding of a different summation order (inside the 1e-5 bound the tests use).
template <typename T>
__global__ void update_reduce_parts_kernel(const T* __restrict__ x, const int* __restrict__ perm,
                                           const int* __restrict__ off, int nlist, int d, int parts,
                                           float* __restrict__ scratch) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const int64_t w = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    if (w >= static_cast<int64_t>(nlist) * parts) return;
    const int l = static_cast<int>(w / parts), j = static_cast<int>(w - static_cast<int64_t>(l) * parts);
    const int beg = off[l], len = off[l + 1] - beg;
    const int b0 = beg + static_cast<int>(static_cast<int64_t>(len) * j / parts);
    const int b1 = beg + static_cast<int>(static_cast<int64_t>(len) * (j + 1) / parts);
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    reduce_members(x, perm, b0, b1, d, lane, acc);
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
        const int c0 = 128 * blk + 4 * lane;
        if (c0 < d)
            *reinterpret_cast<float4*>(scratch + w * d + c0) = make_float4(acc[blk][0], acc[blk][1], acc[blk][2], acc[blk][3]);
    }
}

__global__ void update_combine_parts_kernel(const float* __restrict__ scratch, const int* __restrict__ off, int nlist, int d,
                                            int parts, float* __restrict__ sums, long long* __restrict__ counts) {
    pdl_wait();
    pdl_trigger();
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= static_cast<int64_t>(nlist) * d) return;
    const int l = static_cast<int>(i / d), t = static_cast<int>(i - static_cast<int64_t>(l) * d);
    float partial = 0.0f;
    for (int j = 0; j < parts; ++j) partial += scratch[(static_cast<int64_t>(l) * parts + j) * d + t];
    sums[i] += partial;
    if (t == 0) counts[l] += static_cast<long long>(off[l + 1] - off[l]);
}

// Cluster-major copy (Sec. 3.1 index layout): destination row p receives source row order[p];
// one thread per 16-byte piece of a row (4-byte pieces when a row is not a multiple of 16 bytes).
// Rows whose id was outside [0, nlist) were left out by the fill, so only the first *kept positions
// of `order` hold a source row: the positions after them get order = -1 and a zeroed row.
template <typename Piece>
__global__ void reorder_gather_kernel(const Piece* __restrict__ src, int* __restrict__ order, int64_t n,
                                      int row_chunks, const int* __restrict__ kept, Piece* __restrict__ dst) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n * row_chunks) return;
    const int64_t p = i / row_chunks;
    const int c = static_cast<int>(i - p * row_chunks);
    if (p >= *kept) {
        if (c == 0) order[p] = -1;
        dst[i] = Piece{};
        return;
    }
    dst[i] = src[static_cast<int64_t>(order[p]) * row_chunks + c];
}

__global__ void widen_offsets_kernel(const int* __restrict__ off, int nlist, long long* __restrict__ out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i <= nlist) out[i] = off[i];
}

__global__ void finalize_kernel(const float* __restrict__ sums, const long long* __restrict__ counts, int nlist,
                                int d, float* __restrict__ centroids) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= static_cast<int64_t>(nlist) * d) return;
    const long long c = counts[i / d];
    if (c > 0) centroids[i] = sums[i] / static_cast<float>(c);
}

}  // namespace ivf
