// Second stage of the on-device list selection (Sec. 4.1: tile-local candidates are merged on the
// device): the partial results that the CTAs sharing a row tile left behind are merged into the
// final k ids per row, ascending by (distance, id), and the point norm is added back
// (Eq. 3: |x-c|^2 = |x|^2 + (|c|^2 - 2 x.c)).
#pragma once
#include "fused_topk.cuh"

namespace ivf {

struct MergeParams {
    int64_t n;
    int k;
    int partials;
    int cap;
    int col_tiles;
    int64_t total_units;
    int ctas;              // grid size of the fused kernel (defines which slots exist)
    const Entry* part;
    const int* part_cnt;
    const float* xn;       // |x|^2 per row
    int32_t* out_ids;      // [n, k]
    float* out_dists;      // [n, k] or nullptr
};

__device__ __forceinline__ int slots_of_row_tile(const MergeParams& p, int64_t r) {
    const int first = cta_of_unit(p.total_units, p.ctas, r * p.col_tiles);
    const int last = cta_of_unit(p.total_units, p.ctas, (r + 1) * p.col_tiles - 1);
    return last - first + 1;
}

// k = 1: one thread per row takes the lexicographic minimum over the row's partial results.
__global__ void merge_argmin_kernel(const MergeParams p) {
    const int64_t row = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (row >= p.n) return;
    const int ns = slots_of_row_tile(p, row / kBlockM);
    const Entry* e = p.part + static_cast<size_t>(row) * p.partials;
    float bv = e[0].v;
    int bj = e[0].j;
    for (int s = 1; s < ns; ++s) {
        const float v = e[s].v;
        const int j = e[s].j;
        if (v < bv || (v == bv && j < bj)) {
            bv = v;
            bj = j;
        }
    }
    p.out_ids[row] = bj;
    if (p.out_dists) p.out_dists[row] = fmaxf(bv + p.xn[row], 0.0f);
}

constexpr int kSortCap = 4096;
constexpr int kMergeThreads = 256;

__device__ __forceinline__ void bitonic_sort_smem(uint64_t* keys, int m /* power of two */) {
    for (int size = 2; size <= m; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = threadIdx.x; t < (m >> 1); t += blockDim.x) {
                const int lo = 2 * t - (t & (stride - 1));
                const int hi = lo + stride;
                const bool up = (lo & size) == 0;
                const uint64_t a = keys[lo], b = keys[hi];
                if ((a > b) == up) {
                    keys[lo] = b;
                    keys[hi] = a;
                }
            }
        }
    }
    __syncthreads();
}

// k > 1: one CTA per row sorts the row's candidates by the 64-bit key (orderable value, id) in
// shared memory and writes the first k.  More than kSortCap candidates are folded in rounds.
__global__ void __launch_bounds__(kMergeThreads) merge_select_kernel(const MergeParams p) {
    __shared__ uint64_t keys[kSortCap];
    __shared__ int s_fill;
    const int64_t row = blockIdx.x;
    const int ns = slots_of_row_tile(p, row / kBlockM);
    const Entry* base = p.part + static_cast<size_t>(row) * p.partials * p.cap;
    const int* cnts = p.part_cnt + static_cast<size_t>(row) * p.partials;

    int kept = 0;  // sorted keys carried at the front of keys[]
    int slot = 0, pos = 0;
    bool more = ns > 0;
    while (more) {
        // fill keys[kept ..) from the remaining candidates, slot by slot
        int fill = kept;
        while (slot < ns && fill < kSortCap) {
            const int c = min(cnts[slot], p.cap);
            const int take = min(c - pos, kSortCap - fill);
            for (int i = threadIdx.x; i < take; i += blockDim.x) {
                const Entry e = base[static_cast<size_t>(slot) * p.cap + pos + i];
                keys[fill + i] = (static_cast<uint64_t>(orderable(e.v)) << 32) | static_cast<uint32_t>(e.j);
            }
            fill += take;
            pos += take;
            if (pos >= c) {
                ++slot;
                pos = 0;
            }
        }
        more = slot < ns;
        int m = 2;
        while (m < fill) m <<= 1;
        for (int i = fill + threadIdx.x; i < m; i += blockDim.x) keys[i] = ~0ull;
        bitonic_sort_smem(keys, m);
        kept = min(fill, p.k);
        if (kept == kSortCap) more = false;  // cannot happen for k <= 512; guards the loop
    }
    (void)s_fill;
    const float xn = p.xn[row];
    for (int i = threadIdx.x; i < p.k; i += blockDim.x) {
        int32_t id = -1;
        float dist = __int_as_float(0x7f800000);
        if (i < kept) {
            const uint64_t key = keys[i];
            id = static_cast<int32_t>(key & 0xFFFFFFFFull);
            dist = fmaxf(from_orderable(static_cast<uint32_t>(key >> 32)) + xn, 0.0f);
        }
        p.out_ids[row * p.k + i] = id;
        if (p.out_dists) p.out_dists[row * p.k + i] = dist;
    }
}

}  // namespace ivf
