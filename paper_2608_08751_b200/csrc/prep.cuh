// Operand preparation for the distance contraction (Sec. 4.1, Eq. 3: "inner products and
// precomputed norms").  Norms are accumulated in fp32 from the unrounded inputs; the tensor-core
// operands are fp16 copies scaled by an exact power of two chosen from the largest magnitude, so
// nothing overflows and small-magnitude data keeps its 11 significant bits.  uint8 values are exact.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ivf {

// max |x| over a float array, as the bit pattern of a non-negative float (atomicMax on uint).
__global__ void maxabs_kernel(const float* __restrict__ x, int64_t count, unsigned int* out_bits) {
    float m = 0.0f;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < count; i += stride)
        m = fmaxf(m, fabsf(x[i]));
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

__device__ __forceinline__ float pow2_scale_for(float maxabs) {
    // largest power of two s with s * maxabs < 2^14 (fp16 overflows at 65504); exponent clamped so
    // that the product of two scales stays finite in fp32
    if (!(maxabs > 0.0f) || isinf(maxabs)) return 1.0f;
    int e;
    frexpf(maxabs, &e);  // maxabs = f * 2^e, f in [0.5, 1)
    int s = 14 - e;
    s = s < -60 ? -60 : (s > 60 ? 60 : s);
    return ldexpf(1.0f, s);
}

// scal[0] = point scale, scal[1] = centroid scale, scal[2] = -2 / (scal[0] * scal[1]).
// bits[0] = max |x| bits (ignored for uint8 points), bits[1] = max |c| bits.
__global__ void scales_kernel(const unsigned int* bits, int points_are_u8, float* scal) {
    const float sx = points_are_u8 ? 1.0f : pow2_scale_for(__uint_as_float(bits[0]));
    const float sc = pow2_scale_for(__uint_as_float(bits[1]));
    scal[0] = sx;
    scal[1] = sc;
    scal[2] = -2.0f / (sx * sc);
}

// One warp per row: writes the scaled fp16 copy (row pitch kp, zero padded beyond d) and the fp32
// squared norm.  Rows in [rows, rows_padded) only get norm = +inf (their operand rows are never
// read: the TMA zero-fills rows beyond the tensor).  Lane g handles columns [8g, 8g+8).
template <typename T>
__global__ void convert_rows_kernel(const T* __restrict__ x, int64_t rows, int64_t rows_padded, int d, int kp,
                                    const float* __restrict__ scal, int which_scale, __half* __restrict__ out,
                                    float* __restrict__ norms) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    if (row >= rows_padded) return;
    if (row >= rows) {
        if (lane == 0) norms[row] = __int_as_float(0x7f800000);
        return;
    }
    const float s = scal[which_scale];
    float acc = 0.0f;
    const int c0 = lane * 8;
    if (c0 < kp) {
        float v[8];
        if (c0 < d) {
            if constexpr (sizeof(T) == 1) {
                const uint2 raw = *reinterpret_cast<const uint2*>(x + row * d + c0);
                const uint32_t w[2] = {raw.x, raw.y};
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = static_cast<float>((w[i >> 2] >> (8 * (i & 3))) & 0xFFu);
            } else {
                const float4 a = *reinterpret_cast<const float4*>(x + row * d + c0);
                const float4 b = *reinterpret_cast<const float4*>(x + row * d + c0 + 4);
                v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
                v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = 0.0f;
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
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
    if (lane == 0) norms[row] = acc;
}

}  // namespace ivf
