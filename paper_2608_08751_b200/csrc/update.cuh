// Lloyd centroid update (Sec. 5.5 "Lloyd iterations"): per-list sum and count of the member rows,
// as a segmented reduction.  The ids are turned into list segments by a counting sort (histogram,
// exclusive scan, fill), then one warp per list gathers and adds its member rows and is the only
// writer of that list's sums and count, so no floating-point atomics are involved.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ivf {

constexpr int kStatusBadId = -6;

__global__ void update_hist_kernel(const int32_t* __restrict__ ids, int64_t n, int nlist, int* __restrict__ cnt,
                                   int* status) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int l = ids[i];
    if (l < 0 || l >= nlist) {
        atomicCAS(status, 0, kStatusBadId);
        return;
    }
    atomicAdd(&cnt[l], 1);
}

// Exclusive scan of cnt[0..nlist) into off[0..nlist]; single CTA of 1024 threads walking the array
// in blocks of 4096 with a running carry.  Also clears cursor[].
__global__ void __launch_bounds__(1024) update_scan_kernel(const int* __restrict__ cnt, int nlist,
                                                           int* __restrict__ off, int* __restrict__ cursor) {
    __shared__ int warp_sums[32];
    __shared__ int carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int base = 0; base < nlist; base += 4096) {
        const int i0 = base + threadIdx.x * 4;
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
            int ws = warp_sums[lane];
            int wi = ws;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
                if (lane >= o) wi += t;
            }
            warp_sums[lane] = wi - ws;  // exclusive prefix of the warp sums
        }
        __syncthreads();
        const int carry = carry_s;
        int run = carry + warp_sums[w] + (incl - tsum);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (i0 + q < nlist) {
                off[i0 + q] = run;
                cursor[i0 + q] = 0;
            }
            run += v[q];
        }
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = run;  // last thread's running total = carry for the next block
        __syncthreads();
    }
    if (threadIdx.x == 0) off[nlist] = carry_s;
}

__global__ void update_fill_kernel(const int32_t* __restrict__ ids, int64_t n, int nlist,
                                   const int* __restrict__ off, int* __restrict__ cursor, int* __restrict__ perm) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int l = ids[i];
    if (l < 0 || l >= nlist) return;
    const int pos = off[l] + atomicAdd(&cursor[l], 1);
    perm[pos] = static_cast<int>(i);
}

// One warp per list.  Lane q owns columns [128*blk + 4*q, +4) for blk = 0, 1 (d <= 256).
template <typename T>
__global__ void update_reduce_kernel(const T* __restrict__ x, const int* __restrict__ perm,
                                     const int* __restrict__ off, int nlist, int d, float* __restrict__ sums,
                                     long long* __restrict__ counts) {
    const int lane = threadIdx.x & 31;
    const int l = static_cast<int>((static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5);
    if (l >= nlist) return;
    const int beg = off[l], end = off[l + 1];
    if (beg == end) return;
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    for (int m0 = beg; m0 < end; m0 += 32) {
        const int mine = (m0 + lane < end) ? perm[m0 + lane] : -1;
        const int cntm = min(32, end - m0);
        for (int m = 0; m < cntm; ++m) {
            const int64_t row = __shfl_sync(0xFFFFFFFFu, mine, m);
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) {
                const int c0 = 128 * blk + 4 * lane;
                if (c0 < d) {
                    if constexpr (sizeof(T) == 1) {
                        const uint32_t w = *reinterpret_cast<const uint32_t*>(x + row * d + c0);
                        acc[blk][0] += static_cast<float>(w & 0xFFu);
                        acc[blk][1] += static_cast<float>((w >> 8) & 0xFFu);
                        acc[blk][2] += static_cast<float>((w >> 16) & 0xFFu);
                        acc[blk][3] += static_cast<float>(w >> 24);
                    } else {
                        const float4 v = *reinterpret_cast<const float4*>(x + row * d + c0);
                        acc[blk][0] += v.x;
                        acc[blk][1] += v.y;
                        acc[blk][2] += v.z;
                        acc[blk][3] += v.w;
                    }
                }
            }
        }
    }
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

__global__ void finalize_kernel(const float* __restrict__ sums, const long long* __restrict__ counts, int nlist,
                                int d, float* __restrict__ centroids) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= static_cast<int64_t>(nlist) * d) return;
    const long long c = counts[i / d];
    if (c > 0) centroids[i] = sums[i] / static_cast<float>(c);
}

}  // namespace ivf
