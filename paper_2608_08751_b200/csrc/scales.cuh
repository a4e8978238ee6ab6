// Power-of-two scale factors of the operand copies (shared by the preparation kernels and by the
// fused kernel when it widens uint8 rows itself).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ivf {

__device__ __forceinline__ float pow2_scale_for(float maxabs) {
    // largest power of two s with s * maxabs < 2^11: the scaled squared norm of a row then stays
    // below d * 2^22, and its 2^-15 multiple fits fp16.  Exponent clamped to keep products finite.
    if (!(maxabs > 0.0f) || isinf(maxabs)) return 1.0f;
    int e;
    frexpf(maxabs, &e);  // maxabs = f * 2^e, f in [0.5, 1)
    int s = 11 - e;
    s = s < -40 ? -40 : (s > 40 ? 40 : s);
    return ldexpf(1.0f, s);
}

// out[0] = sx (point scale), out[1] = sc (centroid scale), out[2] = 1 / (sx sc),
// out[3] = A = 2^15 sx / sc.  bits[0] = max |x| bits (unused for uint8 points), bits[1] = max |c|.
// The point scale never exceeds the centroid scale (so A <= 2^15) and is at least sc * 2^-29
// (so A stays a normal fp16 number).
__device__ __forceinline__ void compute_scales(const unsigned int* bits, int points_are_u8, float (&out)[4]) {
    const float sc = pow2_scale_for(__uint_as_float(bits[1]));
    float sx = points_are_u8 ? 8.0f : pow2_scale_for(__uint_as_float(bits[0]));
    sx = fminf(sx, sc);
    sx = fmaxf(sx, sc * 1.862645149230957e-09f);  // 2^-29
    out[0] = sx;
    out[1] = sc;
    out[2] = 1.0f / (sx * sc);
    out[3] = 32768.0f * sx / sc;
}

}  // namespace ivf
