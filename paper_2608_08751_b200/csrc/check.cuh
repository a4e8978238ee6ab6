// Index checks of the checked build (-DIVF_CHECK_BOUNDS): a stand-in for a memory checker on
// machines where none can be run.  IVF_IN_BOUNDS(site, index, limit) is true when 0 <= index < limit.
// In the checked build a false result also records IVF_ERR_BOUNDS, the site number, the block and
// the offending index in the device's status word (first violation wins), and the caller skips the
// access -- nothing traps, the kernel runs to its end and the host reads the status with ivf_check.
// In the regular build the macro is the constant `true` and costs nothing.
//
// Site numbers: 1xx fused kernel, 2xx merges and recomputation, 3xx centroid update and reorder,
// 4xx residual-PQ kernels, 5xx preparation and candidate assignment.
#pragma once
#include <cuda_runtime.h>

namespace ivf {

constexpr int kStatusBounds = -7;

#ifdef IVF_CHECK_BOUNDS
// the current device's status word (4 ints); set by the host when the device context is created
__device__ int* g_check_status = nullptr;

__device__ __noinline__ bool report_bounds(int site, long long index) {
    int* st = g_check_status;
    if (st != nullptr && atomicCAS(st, 0, kStatusBounds) == 0) {
        st[1] = site;
        st[2] = static_cast<int>(blockIdx.x);
        st[3] = static_cast<int>(index);
    }
    return false;
}
#define IVF_IN_BOUNDS(site, index, limit)                                                              \
    ((static_cast<long long>(index) >= 0 && static_cast<long long>(index) < static_cast<long long>(limit)) \
         ? true                                                                                        \
         : ::ivf::report_bounds((site), static_cast<long long>(index)))
constexpr bool kBoundsChecked = true;
#else
#define IVF_IN_BOUNDS(site, index, limit) (true)
constexpr bool kBoundsChecked = false;
#endif

}  // namespace ivf
