// Assignment within given candidate centroids (appendix on fast index building: a graph search
// proposes 2 or 8 candidate centroids per vector, Table 3, and the exact distance is evaluated within
// that set only).  The candidate generator is not part of this path; candidates are an input.
//
// HBM-bound gather: per row one point row and m centroid rows of d floats.  One warp per row; the
// squared distance is the direct difference form in fp32 (each lane sums its coordinates in order,
// then a butterfly over the lanes), so no norm expansion and no cancellation.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

namespace ivf {

constexpr int kCandStatusBadId = -6;
constexpr int kCandMaxD = 256;  // two 4-float pieces per lane

template <typename T>
__device__ __forceinline__ void cand_load_piece(const T* row, int t, float (&v)[4]) {
    if constexpr (sizeof(T) == 1) {
        const uint32_t w = *reinterpret_cast<const uint32_t*>(row + t);
        if constexpr (std::is_signed<T>::value) {
            const int sv = static_cast<int>(w);
            v[0] = static_cast<float>((sv << 24) >> 24);
            v[1] = static_cast<float>((sv << 16) >> 24);
            v[2] = static_cast<float>((sv << 8) >> 24);
            v[3] = static_cast<float>(sv >> 24);
        } else {
            v[0] = static_cast<float>(w & 255u);
            v[1] = static_cast<float>((w >> 8) & 255u);
            v[2] = static_cast<float>((w >> 16) & 255u);
            v[3] = static_cast<float>(w >> 24);
        }
    } else {
        const float4 f = *reinterpret_cast<const float4*>(row + t);
        v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
    }
}

// d is a multiple of 4 and at most 256.  Candidates are taken four at a time so that four centroid
// rows are in flight per warp.
template <typename T>
__global__ void __launch_bounds__(256) assign_candidates_kernel(const T* __restrict__ x, int64_t n, int d,
                                                                const float* __restrict__ c, int nlist,
                                                                const int32_t* __restrict__ cand, int m,
                                                                int32_t* __restrict__ out_ids,
                                                                float* __restrict__ out_dists, int* status) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    if (row >= n) return;
    const int t0 = lane * 4, t1 = 128 + lane * 4;
    const bool has0 = t0 < d, has1 = t1 < d;
    float xv0[4] = {0.f, 0.f, 0.f, 0.f}, xv1[4] = {0.f, 0.f, 0.f, 0.f};
    if (has0) cand_load_piece(x + row * d, t0, xv0);
    if (has1) cand_load_piece(x + row * d, t1, xv1);
    float best = __int_as_float(0x7f800000);
    int best_id = -1;
    bool bad = false;
    for (int p0 = 0; p0 < m; p0 += 4) {
        int id[4];
        float acc[4];
        float4 c0[4], c1[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            id[u] = p0 + u < m ? cand[row * m + p0 + u] : -1;
            const bool ok = id[u] >= 0 && id[u] < nlist;
            if (p0 + u < m && !ok) bad = true;
            if (!ok) id[u] = -1;
            c0[u] = c1[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (ok) {
                const float* cr = c + static_cast<int64_t>(id[u]) * d;
                if (has0) c0[u] = *reinterpret_cast<const float4*>(cr + t0);
                if (has1) c1[u] = *reinterpret_cast<const float4*>(cr + t1);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            float a = 0.0f, df;
            df = xv0[0] - c0[u].x; a = fmaf(df, df, a);
            df = xv0[1] - c0[u].y; a = fmaf(df, df, a);
            df = xv0[2] - c0[u].z; a = fmaf(df, df, a);
            df = xv0[3] - c0[u].w; a = fmaf(df, df, a);
            df = xv1[0] - c1[u].x; a = fmaf(df, df, a);
            df = xv1[1] - c1[u].y; a = fmaf(df, df, a);
            df = xv1[2] - c1[u].z; a = fmaf(df, df, a);
            df = xv1[3] - c1[u].w; a = fmaf(df, df, a);
            acc[u] = a;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
            for (int u = 0; u < 4; ++u) acc[u] += __shfl_xor_sync(0xFFFFFFFFu, acc[u], off);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (id[u] >= 0 && (acc[u] < best || (acc[u] == best && id[u] < best_id))) {
                best = acc[u];
                best_id = id[u];
            }
        }
    }
    if (lane == 0) {
        out_ids[row] = best_id;
        if (out_dists) out_dists[row] = best;
        if (bad) atomicCAS(status, 0, kCandStatusBadId);
    }
}

}  // namespace ivf
