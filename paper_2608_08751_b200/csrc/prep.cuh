// Operand preparation for the distance contraction (Sec. 4.1, Eq. 6: the distance is
// assembled from an inner product and norms computed beforehand).  Norms are accumulated in fp32 from the unrounded inputs.  The tensor-core
// operands are fp16 copies scaled by exact powers of two chosen from the largest magnitudes, so
// nothing overflows and small-magnitude data keeps its 11 significant bits; uint8 values are exact.
//
// Row layouts (fp16, pitch kp = kd + 16, kd = d rounded up to 64):
//   point     [ sx * x (d) | zeros to kd | A  A  A  0 ... 0 ]
//   centroid  [ -2 sc * c (d) | zeros to kd | w_hi w_mid w_lo 0 ... 0 ],  w = sc^2 |c|^2 / 2^15
// so that one K sweep of the MMA yields  sx sc (|c|^2 - 2 x.c)  with A = 2^15 sx / sc.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "ptx.cuh"
#include "scales.cuh"

namespace ivf {

// max |x| over a float array, as the bit pattern of a non-negative float (atomicMax on uint).
__global__ void maxabs_kernel(const float* __restrict__ x, int64_t count, unsigned int* out_bits) {
    pdl_wait();
    pdl_trigger();
    float m = 0.0f;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    const int64_t tid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    // 16-byte loads, four in flight per thread (the rows are 16-byte aligned and d is a multiple of 4,
    // so the element count is a multiple of 4)
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const int64_t count4 = count >> 2;
    int64_t i = tid;
    for (; i + 3 * stride < count4; i += 4 * stride) {
        const float4 a = x4[i], b = x4[i + stride], c = x4[i + 2 * stride], e = x4[i + 3 * stride];
        m = fmaxf(m, fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(a.z), fabsf(a.w))));
        m = fmaxf(m, fmaxf(fmaxf(fabsf(b.x), fabsf(b.y)), fmaxf(fabsf(b.z), fabsf(b.w))));
        m = fmaxf(m, fmaxf(fmaxf(fabsf(c.x), fabsf(c.y)), fmaxf(fabsf(c.z), fabsf(c.w))));
        m = fmaxf(m, fmaxf(fmaxf(fabsf(e.x), fabsf(e.y)), fmaxf(fabsf(e.z), fabsf(e.w))));
    }
    for (; i < count4; i += stride) {
        const float4 a = x4[i];
        m = fmaxf(m, fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(a.z), fabsf(a.w))));
    }
    for (int64_t j = (count4 << 2) + tid; j < count; j += stride) m = fmaxf(m, fabsf(x[j]));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
    __shared__ float wmax[32];
    if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = threadIdx.x < (blockDim.x >> 5) ? wmax[threadIdx.x] : 0.0f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
        if (threadIdx.x == 0) atomicMax(out_bits, __float_as_uint(m));
    }
}

// One lane group per row: 8 lanes for kd = 64 (four rows per warp), 16 for kd = 128 (two rows per warp),
// the whole warp beyond.  Lane g of a group converts columns [8g, 8g+8) of the data part; after the norm
// is reduced inside the group its lanes 0 and 1 write the 16 extra columns.  (rows_per_warp = 32 / group)  If `bits` is given (point rows), the scales are derived
// here from the magnitude words instead of being read, and the first thread publishes them in `scal`
// for the kernels that follow.
template <typename T, bool CENTROID>
__global__ void convert_rows_kernel(const T* __restrict__ x, int64_t rows, int d, int kd, float* scal,
                                    __half* __restrict__ out, float* __restrict__ norms,
                                    const unsigned int* __restrict__ bits, int points_are_u8) {
    pdl_wait();
    pdl_trigger();
    const int group = kd <= 64 ? 8 : (kd <= 128 ? 16 : 32);
    const int lane = threadIdx.x & (group - 1);
    const int64_t warp = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int64_t row = warp * (32 / group) + ((threadIdx.x & 31) / group);
    if (row >= rows) return;  // (a whole lane group leaves together: the shuffles below stay inside a group)
    const int kp = kd + 16;
    float sv[4];
    if (bits != nullptr) {
        compute_scales(bits, points_are_u8, sv);
        if (blockIdx.x == 0 && threadIdx.x == 0) {
#pragma unroll
            for (int i = 0; i < 4; ++i) scal[i] = sv[i];
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) sv[i] = scal[i];
    }
    const float sc = sv[1];
    const float s = CENTROID ? -2.0f * sc : sv[0];
    float acc = 0.0f;
    const int c0 = lane * 8;
    if (c0 < kd) {
        // two 4-element pieces per lane, each present or absent as a whole (d is a multiple of 4)
        float v[8];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int t = c0 + 4 * half;
            if (t < d) {
                if constexpr (sizeof(T) == 1) {
                    const uint32_t w = *reinterpret_cast<const uint32_t*>(x + row * d + t);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t b = (w >> (8 * i)) & 0xFFu;
                        if constexpr (std::is_signed<T>::value)
                            v[4 * half + i] = static_cast<float>(static_cast<int>(static_cast<int8_t>(b)));
                        else
                            v[4 * half + i] = static_cast<float>(b);
                    }
                } else {
                    const float4 a = *reinterpret_cast<const float4*>(x + row * d + t);
                    v[4 * half] = a.x; v[4 * half + 1] = a.y; v[4 * half + 2] = a.z; v[4 * half + 3] = a.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) v[4 * half + i] = 0.0f;
            }
        }
        __half2 h[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            acc = fmaf(v[2 * i], v[2 * i], acc);
            acc = fmaf(v[2 * i + 1], v[2 * i + 1], acc);
            h[i] = __floats2half2_rn(v[2 * i] * s, v[2 * i + 1] * s);
        }
        *reinterpret_cast<uint4*>(out + row * kp + c0) = *reinterpret_cast<const uint4*>(h);
    }
    // (the mask names the lanes of this group only: groups whose row is past the end have returned)
    const uint32_t gmask = group == 32 ? 0xFFFFFFFFu : (((1u << group) - 1u) << ((threadIdx.x & 31) / group * group));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
        if (off < group) acc += __shfl_xor_sync(gmask, acc, off);
    if (lane < 2) {
        __half a[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) a[i] = __float2half_rn(0.0f);
        if (lane == 0) {
            if (CENTROID) {
                const float w = sc * sc * acc * 3.0517578125e-05f;  // 2^-15; exact power-of-two scaling
                const __half hi = __float2half_rn(w);
                const float r1 = w - __half2float(hi);
                const __half mid = __float2half_rn(r1);
                const float r2 = r1 - __half2float(mid);
                a[0] = hi;
                a[1] = mid;
                a[2] = __float2half_rn(r2);
            } else {
                const __half av = __float2half_rn(sv[3]);
                a[0] = av;
                a[1] = av;
                a[2] = av;
            }
        }
        *reinterpret_cast<uint4*>(out + row * kp + kd + lane * 8) = *reinterpret_cast<const uint4*>(a);
    }
    if (lane == 0 && norms != nullptr) norms[row] = acc;
}

}  // namespace ivf
