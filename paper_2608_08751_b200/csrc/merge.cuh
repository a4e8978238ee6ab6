// Second stage of the on-device list selection (Sec. 4.1: tile-local candidates are merged on the
// device): the partial results left by the CTAs (and epilogue warps) that shared a row are merged
// into the final k ids per row, ascending by (distance, id); the key is rescaled and the point norm
// added back (Eq. 6: |x-c|^2 = |x|^2 + (|c|^2 - 2 x.c)).
//
// For k > 16 the candidate logs were filled against per-partial thresholds tau_p.  Every element
// with key < tau_p is in log p, and enough of the elements equal to tau_p, so the union of the logs
// holds the true top-k whenever at least k candidates are <= min_p tau_p.  That test is exact; a
// row that fails it is recomputed by fallback_rows_kernel (brute force over all centroids).
#pragma once
#include <cuda_fp16.h>

#include "fused_topk.cuh"

namespace ivf {

struct MergeParams {
    int64_t n;
    int k;
    int partials;
    int cap;
    int col_tiles;
    int64_t total_units;
    int cross;             // crossing cost of the fused kernel's span partition
    int ctas;              // grid size of the fused kernel (defines which slots exist)
    int group_rows;        // point rows per row group of the fused kernel (128 or 256)
    const Entry* part;
    const int2* part_meta;
    const float* xn;       // |x|^2 per row
    const float* scal;     // scal[2] = 1 / (sx sc)
    int32_t* out_ids;      // [n, k]
    float* out_dists;      // [n, k] or nullptr
    int* fail;             // fail[0] = number of failed rows, fail[1..] = their indices
    int force_fail;        // test hook: treat every row as failed
    float* tau_out;        // if set: write only the 16th smallest key of every row here (threshold pass)
    int records;           // the logs hold 48-byte group records (8 keys + first id), not entries
    int* big;              // big[0] = number of rows the warp-level merge passed on, big[1..] = the rows
    unsigned long long* stats;  // optional counters: [2] rows sent to the brute-force recomputation
};

__device__ __forceinline__ int slots_of_row_tile(const MergeParams& p, int64_t r) {
    const int first = cta_of_unit(p.total_units, p.ctas, p.col_tiles, p.cross, r * p.col_tiles);
    const int last = cta_of_unit(p.total_units, p.ctas, p.col_tiles, p.cross, (r + 1) * p.col_tiles - 1);
    return (last - first + 1) * kEpiHalves;
}

// k = 1: one thread per row takes the lexicographic minimum over the row's partial results.
__global__ void merge_argmin_kernel(const MergeParams p) {
    pdl_wait();
    pdl_trigger();
    const int64_t row = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (row >= p.n) return;
    int ns = slots_of_row_tile(p, row / p.group_rows);
    if (!IVF_IN_BOUNDS(201, ns, p.partials + 1)) ns = p.partials;
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
    if (p.out_dists) p.out_dists[row] = fmaxf(fmaf(bv, p.scal[2], p.xn[row]), 0.0f);
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

constexpr int kMaxSlots = 512;  // >= 2 * number of CTAs of the fused kernel

// Writes the first k sorted keys of a row (or hands the row to the brute-force path).
__device__ __forceinline__ void merge_write_row(const MergeParams& p, int64_t row, const uint64_t* keys, int i0,
                                                int istep) {
    const float xn = p.xn[row];
    const float inv = p.scal[2];
    for (int i = i0; i < p.k; i += istep) {
        const uint64_t key = keys[i];
        if (!IVF_IN_BOUNDS(202, row * p.k + i, p.n * p.k)) continue;
        p.out_ids[row * p.k + i] = static_cast<int32_t>(key & 0xFFFFFFFFull);
        if (p.out_dists)
            p.out_dists[row * p.k + i] = fmaxf(fmaf(from_orderable(static_cast<uint32_t>(key >> 32)), inv, xn), 0.0f);
    }
}
__device__ __forceinline__ void merge_fail_row(const MergeParams& p, int64_t row) {
    const int at = atomicAdd(&p.fail[0], 1);
    if (IVF_IN_BOUNDS(203, at, p.n)) p.fail[1 + at] = static_cast<int>(row);
    if (p.stats) atomicAdd(&p.stats[2], 1ull);
}

// k > 1, general path: one CTA per row (a device function of route_tail_kernel).  The row's logs are
// read as one flattened array (all loads in flight together); candidates <= the row's smallest tau
// are sorted by the 64-bit key (orderable value, id) in shared memory; more than kSortCap raw entries
// are folded in rounds.
struct SelectSmem {
    uint64_t keys[kSortCap];
    int pre[kMaxSlots + 1];  // exclusive prefix of the slots' entry counts
    float s_tau[kMergeThreads / 32];
    int hist[256];
    int s_wcnt[kMergeThreads / 32];
    int s_sel[2];
    int s_fill;
};

__device__ __forceinline__ void merge_select_row(const MergeParams& p, int64_t row, SelectSmem& sm) {
    uint64_t* const keys = sm.keys;
    int* const pre = sm.pre;
    float* const s_tau = sm.s_tau;
    int* const hist = sm.hist;
    int* const s_wcnt = sm.s_wcnt;
    int* const s_sel = sm.s_sel;
    int& s_fill = sm.s_fill;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    {
        const int ns = min(slots_of_row_tile(p, row / p.group_rows), kMaxSlots);
        const Entry* base = p.part + static_cast<size_t>(row) * p.partials * p.cap;
        const int2* meta = p.part_meta + static_cast<size_t>(row) * p.partials;
        __syncthreads();  // the previous row of this CTA is finished with the shared arrays

        // ---- per-slot counts, their prefix sums, and the smallest threshold
        float tau = __int_as_float(0x7f800000);
        int overflowed = 0;
        for (int s0 = 0; s0 < ns; s0 += kMergeThreads) {
            const int sidx = s0 + threadIdx.x;
            if (sidx < ns) {
                const int2 m = meta[sidx];
                if (m.x < 0) overflowed = 1;  // a group log filled up: the row goes to the brute-force path
                pre[sidx + 1] = max(0, min(m.x, p.cap));
                tau = fminf(tau, __int_as_float(m.y));
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) tau = fminf(tau, __shfl_xor_sync(0xFFFFFFFFu, tau, off));
        if (lane == 0) s_tau[warp] = tau;
        if (threadIdx.x == 0) {
            pre[0] = 0;
            s_fill = 0;
        }
        __syncthreads();
        if (warp == 0) {  // inclusive scan of pre[1..ns] by one warp, 32 slots at a time
            int carry = 0;
            for (int s0 = 0; s0 < ns; s0 += 32) {
                const int sidx = s0 + lane;
                int v = sidx < ns ? pre[sidx + 1] : 0;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const int t = __shfl_up_sync(0xFFFFFFFFu, v, off);
                    if (lane >= off) v += t;
                }
                if (sidx < ns) pre[sidx + 1] = v + carry;
                carry += __shfl_sync(0xFFFFFFFFu, v, 31);
            }
        }
        overflowed = __syncthreads_or(overflowed);
        float tau_min = s_tau[0];
#pragma unroll
        for (int w = 1; w < kMergeThreads / 32; ++w) tau_min = fminf(tau_min, s_tau[w]);
        const int raw_total = pre[ns];

        int kept = 0;   // sorted keys carried at the front of keys[]
        int total = 0;  // candidates <= tau_min seen so far
        for (int done = 0; done < raw_total || done == 0;) {
            // a record yields 8 candidates at most but about one in practice: take half as many
            // records as there is room for keys; should a round still overflow, the row fails
            const int room = (kSortCap - kept) / (p.records ? 2 : 1);
            const int take = min(raw_total - done, room);
            for (int i0 = 0; i0 < take; i0 += blockDim.x) {  // uniform trip count: ballots inside
                const int i = i0 + threadIdx.x;
                float v[8];
                uint32_t j0 = 0;
                int nv = 0;
                if (i < take) {
                    const int idx = done + i;
                    int lo = 0, hi = ns;  // slot with pre[slot] <= idx < pre[slot + 1]
                    while (hi - lo > 1) {
                        const int mid = (lo + hi) >> 1;
                        if (pre[mid] <= idx) lo = mid; else hi = mid;
                    }
                    if (!IVF_IN_BOUNDS(210, lo, p.partials) || !IVF_IN_BOUNDS(211, idx - pre[lo], p.cap)) {
                        nv = 0;
                    } else if (p.records) {
                        const char* rec = reinterpret_cast<const char*>(p.part) +
                                          ((static_cast<size_t>(row) * p.partials + lo) * p.cap + (idx - pre[lo])) *
                                              kRecordBytes;
                        const float4 a = *reinterpret_cast<const float4*>(rec);
                        const float4 b = *reinterpret_cast<const float4*>(rec + 16);
                        j0 = *reinterpret_cast<const uint32_t*>(rec + 32);
                        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
                        v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
                        nv = 8;
                    } else {
                        const Entry e = base[static_cast<size_t>(lo) * p.cap + (idx - pre[lo])];
                        v[0] = e.v;
                        j0 = static_cast<uint32_t>(e.j);
                        nv = 1;
                    }
                }
                // one shared-memory atomic per warp and column instead of one per candidate
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const bool hit = q < nv && v[q] <= tau_min;
                    const uint32_t bal = __ballot_sync(0xFFFFFFFFu, hit);
                    if (bal) {
                        int at0 = 0;
                        if (lane == 0) at0 = atomicAdd(&s_fill, __popc(bal));
                        at0 = __shfl_sync(0xFFFFFFFFu, at0, 0);
                        const int at = at0 + __popc(bal & ((1u << lane) - 1u));
                        if (hit) {
                            if (at < kSortCap) keys[at] = (static_cast<uint64_t>(orderable(v[q])) << 32) | (j0 + q);
                            else overflowed = 1;
                        }
                    }
                    if (!p.records) break;
                }
            }
            __syncthreads();
            done += take;
            int fill = min(s_fill, kSortCap);
            total += fill - kept;
            if (fill > 2 * p.k) {
                // only the k smallest matter: find the k-th smallest value (8-bit radix select over the
                // keys' upper halves) and keep what is <= it, so that the sort below is short
                uint32_t prefix = 0, mask = 0;
                int rank = p.k;
                for (int shift = 24; shift >= 0; shift -= 8) {
                    for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
                    __syncthreads();
                    for (int i = threadIdx.x; i < fill; i += blockDim.x) {
                        const uint32_t u = static_cast<uint32_t>(keys[i] >> 32);
                        if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1);
                    }
                    __syncthreads();
                    if (warp == 0) {
                        int r = rank, eq = 0;
                        const int digit = radix_pick_digit(hist, lane, r, eq);
                        if (lane == 0) {
                            s_sel[0] = digit;
                            s_sel[1] = r;
                        }
                    }
                    __syncthreads();
                    prefix |= static_cast<uint32_t>(s_sel[0]) << shift;
                    mask |= 255u << shift;
                    rank = s_sel[1];
                }
                // stable in-place compaction, 256 keys at a time
                int outp = 0;
                for (int i0 = 0; i0 < fill; i0 += blockDim.x) {
                    const int i = i0 + threadIdx.x;
                    uint64_t key = 0;
                    bool keep = false;
                    if (i < fill) {
                        key = keys[i];
                        keep = static_cast<uint32_t>(key >> 32) <= prefix;
                    }
                    const uint32_t bal = __ballot_sync(0xFFFFFFFFu, keep);
                    if (lane == 0) s_wcnt[warp] = __popc(bal);
                    __syncthreads();
                    int before = 0, all = 0;
#pragma unroll
                    for (int w = 0; w < kMergeThreads / 32; ++w) {
                        const int c = s_wcnt[w];
                        if (w < warp) before += c;
                        all += c;
                    }
                    if (keep) keys[outp + before + __popc(bal & ((1u << lane) - 1u))] = key;
                    outp += all;
                    __syncthreads();
                }
                fill = outp;
            }
            int m = 2;
            while (m < fill) m <<= 1;
            for (int i = fill + threadIdx.x; i < m; i += blockDim.x) keys[i] = ~0ull;
            bitonic_sort_smem(keys, m);
            kept = min(fill, p.k);
            if (done >= raw_total) break;
            if (threadIdx.x == 0) s_fill = kept;
            __syncthreads();
        }
        overflowed = __syncthreads_or(overflowed);
        if (total < p.k || p.force_fail || overflowed) {
            if (threadIdx.x == 0) merge_fail_row(p, row);
            return;
        }
        merge_write_row(p, row, keys, threadIdx.x, blockDim.x);
    }
}

// k > 1, fast path: one WARP per row, no block-wide barriers.  Serves rows with at most kWarpSlots
// partial logs and at most kWarpKeys candidates <= tau: the candidates go to the warp's slice of
// shared memory, an 8-bit radix select on the key's value finds the k-th smallest, and only the
// keys up to it are sorted.  Other rows are appended to p.big for route_tail_kernel.
constexpr int kWarpSlots = 64;

// Two sizes: KEYS candidates per row at most, SORT keys sorted at most, WARPS rows per CTA.
template <int KEYS>
struct MergeWarpSmem {
    uint64_t keys[KEYS];
    int hist[256];
    int pre[kWarpSlots + 1];
};

__device__ __forceinline__ void warp_bitonic_sort(uint64_t* keys, int m, int lane) {
    for (int size = 2; size <= m; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncwarp();
            for (int t = lane; t < (m >> 1); t += 32) {
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
    __syncwarp();
}

template <int KEYS, int SORT, int WARPS>
__global__ void __launch_bounds__(32 * WARPS, KEYS <= 512 ? 6 : (KEYS <= 1024 ? 3 : 2)) merge_warp_kernel(const MergeParams p) {
    pdl_wait();
    pdl_trigger();
    extern __shared__ __align__(16) uint8_t merge_smem_raw[];
    constexpr int kWarpKeys = KEYS, kWarpSort = SORT;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    MergeWarpSmem<KEYS>& sm = reinterpret_cast<MergeWarpSmem<KEYS>*>(merge_smem_raw)[warp];
    const int64_t row = static_cast<int64_t>(blockIdx.x) * WARPS + warp;
    if (row >= p.n) return;
    const uint32_t FULL = 0xFFFFFFFFu;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const int ns = slots_of_row_tile(p, row / p.group_rows);
    const int2* meta = p.part_meta + static_cast<size_t>(row) * p.partials;
    bool pass_on = ns > kWarpSlots || p.force_fail;

    // ---- slot counts, prefix sums, smallest threshold
    float tau_min = __int_as_float(0x7f800000);
    int raw_total = 0;
    if (!pass_on) {
        int carry = 0;
        for (int s0 = 0; s0 < ns; s0 += 32) {
            const int sidx = s0 + lane;
            int c = 0;
            if (sidx < ns) {
                const int2 m = meta[sidx];
                if (m.x < 0) pass_on = true;
                c = max(0, min(m.x, p.cap));
                tau_min = fminf(tau_min, __int_as_float(m.y));
            }
            int v = c;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(FULL, v, off);
                if (lane >= off) v += t;
            }
            if (sidx < ns && IVF_IN_BOUNDS(220, sidx + 1, kWarpSlots + 1)) sm.pre[sidx + 1] = v + carry;
            carry += __shfl_sync(FULL, v, 31);
        }
        if (lane == 0) sm.pre[0] = 0;
        raw_total = carry;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) tau_min = fminf(tau_min, __shfl_xor_sync(FULL, tau_min, off));
        pass_on = __any_sync(FULL, pass_on);
        __syncwarp();
    }

    // ---- k-th smallest value of keys[0 .. fill) by radix select, then everything up to it moved to
    // the front (ties all stay); returns how many were kept.  Used when the buffer fills up during
    // the gather and once at the end.
    auto keep_k_smallest = [&](int fill) -> int {
        uint32_t prefix = 0, mask = 0;
        int r = p.k, eq = 0;
#pragma unroll 1
        for (int shift = 24; shift >= 0; shift -= 8) {
            for (int i = lane; i < 256; i += 32) sm.hist[i] = 0;
            __syncwarp();
            for (int i = lane; i < fill; i += 32) {
                const uint32_t u = static_cast<uint32_t>(sm.keys[i] >> 32);
                if ((u & mask) == prefix) atomicAdd(&sm.hist[(u >> shift) & 255u], 1);
            }
            __syncwarp();
            const int digit = radix_pick_digit(sm.hist, lane, r, eq);
            prefix |= static_cast<uint32_t>(digit) << shift;
            mask |= 255u << shift;
            __syncwarp();
        }
        int outp = 0;
        for (int i0 = 0; i0 < fill; i0 += 32) {
            const int i = i0 + lane;
            uint64_t key = 0;
            bool keep = false;
            if (i < fill) {
                key = sm.keys[i];
                keep = static_cast<uint32_t>(key >> 32) <= prefix;
            }
            const uint32_t bal = __ballot_sync(FULL, keep);
            __syncwarp();
            if (keep) sm.keys[outp + __popc(bal & lt_mask)] = key;
            outp += __popc(bal);
        }
        __syncwarp();
        return outp;
    };

    // ---- gather the candidates <= tau_min into the warp's key buffer.  The loads of the next 32
    // log entries are issued before the current ones are filtered, so that a row's entries arrive in
    // one memory round trip after another without the filtering in between.  A batch that does not fit
    // (a row with several times the usual number of candidates) is filtered again after the buffer
    // has been cut down to the k smallest so far; only a row whose ties fill the buffer is passed on.
    int fill = 0;    // keys in the buffer
    int total = 0;   // candidates <= tau_min seen (the exactness test needs at least k)
    if (!pass_on) {
        float4 na = make_float4(0.f, 0.f, 0.f, 0.f), nb = na;
        uint32_t nj0 = 0;
        auto fetch = [&](int idx) {
            if (idx >= raw_total) return;
            int lo = 0, hi = ns;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (sm.pre[mid] <= idx) lo = mid; else hi = mid;
            }
            const size_t at = (static_cast<size_t>(row) * p.partials + lo) * p.cap + (idx - sm.pre[lo]);
            if (!IVF_IN_BOUNDS(221, lo, p.partials) || !IVF_IN_BOUNDS(222, idx - sm.pre[lo], p.cap)) return;
            if (p.records) {
                const char* rec = reinterpret_cast<const char*>(p.part) + at * kRecordBytes;
                na = *reinterpret_cast<const float4*>(rec);
                nb = *reinterpret_cast<const float4*>(rec + 16);
                nj0 = *reinterpret_cast<const uint32_t*>(rec + 32);
            } else {
                const Entry e = p.part[at];
                na.x = e.v;
                nj0 = static_cast<uint32_t>(e.j);
            }
        };
        fetch(lane);
        for (int i0 = 0; i0 < raw_total && !pass_on; i0 += 32) {
            const int idx = i0 + lane;
            const float v[8] = {na.x, na.y, na.z, na.w, nb.x, nb.y, nb.z, nb.w};
            const uint32_t j0 = nj0;
            const int nv = (idx < raw_total) ? (p.records ? 8 : 1) : 0;
            fetch(idx + 32);
            for (int attempt = 0; attempt < 2; ++attempt) {
                int f = fill;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const bool hit = q < nv && v[q] <= tau_min;
                    const uint32_t bal = __ballot_sync(FULL, hit);
                    if (bal) {
                        const int at = f + __popc(bal & lt_mask);
                        if (hit && at < kWarpKeys) sm.keys[at] = (static_cast<uint64_t>(orderable(v[q])) << 32) | (j0 + q);
                        f += __popc(bal);
                    }
                    if (!p.records) break;
                }
                if (f <= kWarpKeys) {
                    total += f - fill;
                    fill = f;
                    break;
                }
                // the batch did not fit: cut the buffer down (the batch's keys written so far are
                // dropped with it) and filter the batch once more
                __syncwarp();
                if (attempt == 1 || fill <= p.k) {
                    pass_on = true;
                    break;
                }
                fill = keep_k_smallest(fill);
                if (fill + 256 > kWarpKeys) pass_on = true;  // ties: no room for a worst-case batch
                if (pass_on) break;
            }
        }
        __syncwarp();
    }
    if (!pass_on && total < p.k) {  // too few candidates: the threshold was too tight for this row
        if (lane == 0) merge_fail_row(p, row);
        return;
    }

    int kept = fill;
    if (!pass_on && fill > 2 * p.k) kept = keep_k_smallest(fill);
    if (!pass_on && kept > kWarpSort) pass_on = true;  // very many ties: let the general path sort
    if (pass_on) {
        if (lane == 0) {
            const int at = atomicAdd(&p.big[0], 1);
            if (IVF_IN_BOUNDS(223, at, p.n)) p.big[1 + at] = static_cast<int>(row);
        }
        return;
    }
    int m = 2;
    while (m < kept) m <<= 1;
    for (int i = kept + lane; i < m; i += 32) sm.keys[i] = ~0ull;
    warp_bitonic_sort(sm.keys, m, lane);
    merge_write_row(p, row, sm.keys, lane, 32);
}

// Threshold pass: per row, the 16th smallest of all the sketch values its partial results hold.
// Every partial sketch is 16 values in ascending order, so a lane that holds one sketch only ever
// offers its head: 16 rounds of "take the smallest head, advance that lane" give the 16 smallest of
// up to 32 sketches.  One CTA per row; each warp reduces 32 sketches at a time to a sorted list of
// 16 in shared memory, and warp 0 reduces those lists the same way.
constexpr int kTauThreads = 256;

__device__ __forceinline__ void take16(float (&v)[kSampleM], int lane, float* out /* 16 ascending, may be null */,
                                       float& last) {
    const float INF = __int_as_float(0x7f800000);
#pragma unroll 1
    for (int round = 0; round < kSampleM; ++round) {
        float m = v[0];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m = fminf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
        last = m;
        if (out != nullptr && lane == 0) out[round] = m;
        const uint32_t who = __ballot_sync(0xFFFFFFFFu, v[0] == m);
        if (lane == __ffs(who) - 1) {  // the first lane holding m advances its sorted list
#pragma unroll
            for (int i = 0; i < kSampleM - 1; ++i) v[i] = v[i + 1];
            v[kSampleM - 1] = INF;
        }
    }
}

__global__ void __launch_bounds__(kTauThreads) merge_tau_kernel(const MergeParams p) {
    pdl_wait();
    pdl_trigger();
    __shared__ float lists[kTauThreads / 32 + 1][kSampleM];  // one per warp, plus the running result
    const float INF = __int_as_float(0x7f800000);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = blockIdx.x;
    const int ns = slots_of_row_tile(p, row / p.group_rows);
    const Entry* base = p.part + static_cast<size_t>(row) * p.partials * p.cap;
    if (threadIdx.x < kSampleM) lists[kTauThreads / 32][threadIdx.x] = INF;
    float result = INF;
    const int nw = blockDim.x >> 5;  // the launch sizes the CTA to the number of partial sketches
    for (int s0 = 0; s0 < ns; s0 += blockDim.x) {
        __syncthreads();
        float v[kSampleM];
        const int slot = s0 + threadIdx.x;
#pragma unroll
        for (int i = 0; i < kSampleM; ++i)
            v[i] = (slot < ns && IVF_IN_BOUNDS(240, slot, p.partials)) ? base[static_cast<size_t>(slot) * p.cap + i].v : INF;
        float last;
        take16(v, lane, lists[warp], last);
        __syncthreads();
        if (warp == 0) {
            // lanes 0..8 hold the lists of the 8 warps and the running result
#pragma unroll
            for (int i = 0; i < kSampleM; ++i)
                v[i] = lane < nw ? lists[lane][i] : (lane == nw ? lists[kTauThreads / 32][i] : INF);
            __syncwarp();
            take16(v, lane, lists[kTauThreads / 32], result);
        }
    }
    if (threadIdx.x == 0) p.tau_out[row] = result;
}

// The same with one warp per row, for rows with at most 32 partial sketches (large batches, where
// few CTAs share a row): lane = sketch.
__global__ void __launch_bounds__(256) merge_tau_warp_kernel(const MergeParams p) {
    pdl_wait();
    pdl_trigger();
    const float INF = __int_as_float(0x7f800000);
    const int lane = threadIdx.x & 31;
    const int64_t row = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    if (row >= p.n) return;
    const int ns = slots_of_row_tile(p, row / p.group_rows);
    const Entry* base = p.part + static_cast<size_t>(row) * p.partials * p.cap;
    float v[kSampleM];
#pragma unroll
    for (int i = 0; i < kSampleM; ++i)
        v[i] = (lane < ns && IVF_IN_BOUNDS(241, lane, p.partials)) ? base[static_cast<size_t>(lane) * p.cap + i].v : INF;
    float result;
    take16(v, lane, nullptr, result);
    if (lane == 0) p.tau_out[row] = result;
}

// ------------------------------------------------------------------ brute-force recomputation
// A row whose threshold admitted fewer than k candidates (or that was forced here by a test hook) is
// recomputed exactly: all nlist keys with the MMA's own contraction in fp32 FMA, then the k smallest
// by (key, id).  Two stages so that one failed row still uses many SMs: every CTA takes a slice of
// kFallbackSlice centroids, keeps the slice's keys in shared memory and emits the slice's k smallest
// (key, id) pairs; a second CTA selects the k smallest of those candidates and sorts them.
struct FallbackParams {
    int nlist;
    int k;
    int kp;                // pitch of the fp16 operand copies
    const __half* x16;     // [n][kp], or nullptr when the points are raw uint8 rows
    const uint8_t* x_raw;  // [n][d] uint8 (widened on the fly with the same scales)
    int d, kd;
    const __half* c16;     // [nlist][kp]
    const float* xn;
    const float* scal;
    const int* fail;       // fail[0] = count, fail[1..] = rows
    uint64_t* cand;        // [kFallbackFastRows + slow-path CTAs][slices * k] candidate pairs
    int slices;            // ceil(nlist / kFallbackSlice)
    int32_t* out_ids;
    float* out_dists;
};

constexpr int kFallbackThreads = 256;
constexpr int kFallbackMaxK = 512;
constexpr int kFallbackFastRows = 16;  // failed rows whose slices are spread over the grid
constexpr int kFallbackSlice = 8192;   // centroids per slice

struct FallbackSmem {
    float xs[288];
    float keys[kFallbackSlice];
    uint64_t top[kFallbackMaxK];
    int hist[256];
    int cnt, digit, rank, eq;
};

// fp32 copy of one point's operand row (data columns, zero padding, the three norm columns)
__device__ __forceinline__ void fallback_load_point(const FallbackParams& p, int64_t row, float* xs) {
    for (int t = threadIdx.x; t < p.kp; t += blockDim.x) {
        float v;
        if (p.x16 != nullptr) {
            v = __half2float(p.x16[row * p.kp + t]);
        } else {
            v = 0.0f;
            if (t < p.d) v = p.scal[0] * static_cast<float>(p.x_raw[row * p.d + t]);
            else if (t >= p.kd && t < p.kd + 3) v = __half2float(__float2half_rn(p.scal[3]));
        }
        xs[t] = v;
    }
}

// Keys of centroids [j0, j1) against the point row in xs, into keys[0 .. j1-j0).  One warp per
// centroid, four centroids in flight per warp.
__device__ __forceinline__ void fallback_slice_keys(const FallbackParams& p, const float* xs, int j0, int j1,
                                                    float* keys) {
    constexpr int kInFlight = 4;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nwarps = blockDim.x >> 5;
    for (int jb = j0 + warp * kInFlight; jb < j1; jb += nwarps * kInFlight) {
        float acc[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) acc[u] = 0.0f;
        for (int t = lane * 8; t < p.kp; t += 256) {
            uint4 raw[kInFlight];
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                const int j = min(jb + u, j1 - 1);
                raw[u] = *reinterpret_cast<const uint4*>(p.c16 + static_cast<size_t>(j) * p.kp + t);
            }
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                const __half2* h = reinterpret_cast<const __half2*>(&raw[u]);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float2 f = __half22float2(h[q]);
                    acc[u] = fmaf(xs[t + 2 * q], f.x, acc[u]);
                    acc[u] = fmaf(xs[t + 2 * q + 1], f.y, acc[u]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc[u] += __shfl_xor_sync(0xFFFFFFFFu, acc[u], off);
            if (lane == 0 && jb + u < j1 && IVF_IN_BOUNDS(250, jb + u - j0, kFallbackSlice)) keys[jb + u - j0] = acc[u];
        }
    }
}

// Block-wide selection of the k smallest of `count` distinct 64-bit items (get(i), i < count): radix
// select from the top byte down, stopping as soon as the digit that holds rank k is wanted whole;
// returns the largest admitted item (every item <= it is among the k smallest, and there are
// exactly min(k, count) of those).  Histogram increments are combined per warp, because the keys of
// one row share their leading bytes.
template <typename Get>
__device__ __forceinline__ uint64_t fallback_select_bound(Get get, int count, int k, FallbackSmem& sm) {
    if (count <= k) return ~0ull;
    const int lane = threadIdx.x & 31;
    uint64_t prefix = 0, mask = 0;
    int rank = k;
    const int rounded = (count + 31) & ~31;
    for (int shift = 56; shift >= 0; shift -= 8) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) sm.hist[i] = 0;
        __syncthreads();
        for (int i = threadIdx.x; i < rounded; i += blockDim.x) {
            uint32_t dg = 0xFFFFFFFFu;
            if (i < count) {
                const uint64_t v = get(i);
                if ((v & mask) == prefix) dg = static_cast<uint32_t>(v >> shift) & 255u;
            }
            const uint32_t peers = __match_any_sync(0xFFFFFFFFu, dg);
            if (dg != 0xFFFFFFFFu && lane == __ffs(peers) - 1) atomicAdd(&sm.hist[dg], __popc(peers));
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            int r = rank, eq = 0;
            const int digit = radix_pick_digit(sm.hist, lane, r, eq);
            if (lane == 0) {
                sm.digit = digit;
                sm.rank = r;
                sm.eq = eq;
            }
        }
        __syncthreads();
        prefix |= static_cast<uint64_t>(sm.digit) << shift;
        mask |= 255ull << shift;
        rank = sm.rank;
        const bool whole = sm.eq == rank;
        __syncthreads();
        if (whole) return prefix | ~mask;
    }
    return prefix;
}

__device__ __forceinline__ int fallback_slice_len(const FallbackParams& p, int slice) {
    return min(kFallbackSlice, p.nlist - slice * kFallbackSlice);
}

// Stage 1 for one slice: keys into shared memory, the slice's min(k, len) smallest (key, id) pairs
// into out[0 .. min(k, len)) in no particular order.
__device__ __forceinline__ void fallback_slice(const FallbackParams& p, int slice, uint64_t* out, FallbackSmem& sm) {
    const int j0 = slice * kFallbackSlice, len = fallback_slice_len(p, slice);
    fallback_slice_keys(p, sm.xs, j0, j0 + len, sm.keys);
    if (threadIdx.x == 0) sm.cnt = 0;
    __syncthreads();
    auto get = [&](int i) { return (static_cast<uint64_t>(orderable(sm.keys[i])) << 32) | static_cast<uint32_t>(j0 + i); };
    const uint64_t bound = fallback_select_bound(get, len, p.k, sm);
    for (int i = threadIdx.x; i < len; i += blockDim.x) {
        const uint64_t v = get(i);
        if (v <= bound) {
            const int at = atomicAdd(&sm.cnt, 1);
            if (IVF_IN_BOUNDS(251, at, p.k)) out[at] = v;
        }
    }
    __syncthreads();
}

// Stage 2: the k smallest of a row's candidates (slot s of k per slice, the first min(k, len_s) of
// each filled), sorted, to the row's outputs.
__device__ __forceinline__ void fallback_finish_row(const FallbackParams& p, const uint64_t* cand, int64_t row,
                                                    FallbackSmem& sm) {
    const int total = p.slices * p.k;
    auto get = [&](int i) {
        const int s = i / p.k, r = i - s * p.k;
        return r < fallback_slice_len(p, s) ? __ldcg(cand + i) : ~0ull;
    };
    const uint64_t bound = fallback_select_bound(get, total, p.k, sm);
    if (threadIdx.x == 0) sm.cnt = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        const uint64_t v = get(i);
        if (v <= bound && v != ~0ull) {
            const int at = atomicAdd(&sm.cnt, 1);
            if (at < kFallbackMaxK) sm.top[at] = v;
        }
    }
    __syncthreads();
    const int got = min(sm.cnt, kFallbackMaxK);  // == k
    int m = 2;
    while (m < got) m <<= 1;
    for (int i = got + threadIdx.x; i < m; i += blockDim.x) sm.top[i] = ~0ull;
    bitonic_sort_smem(sm.top, m);
    const float xn = p.xn[row];
    const float inv = p.scal[2];
    for (int i = threadIdx.x; i < p.k; i += blockDim.x) {
        const uint64_t key = sm.top[i];
        if (!IVF_IN_BOUNDS(252, i, got)) continue;
        p.out_ids[row * p.k + i] = static_cast<int32_t>(key & 0xFFFFFFFFull);
        if (p.out_dists)
            p.out_dists[row * p.k + i] = fmaxf(fmaf(from_orderable(static_cast<uint32_t>(key >> 32)), inv, xn), 0.0f);
    }
    __syncthreads();
}

// ------------------------------------------------------------------ tail of a routing call
// Everything that is rarely needed after the warp-level merge, as ONE launch (three launches that
// found nothing to do cost 19 us per call, a quarter of a small serving batch):
//   A. rows the warp-level kernel passed on (many partial logs, many candidates or ties) are merged
//      by one CTA each (merge_select_row); with p.big == nullptr every row goes this way;
//   B. rows whose threshold admitted fewer than k candidates (found by the warp-level kernel or in A)
//      are recomputed by brute force: the first kFallbackFastRows of them slice by slice over the
//      whole grid, the CTA that finishes a row's last slice also finishes the row; any further rows
//      by one CTA each (blocks below kFallbackCtas).
// Work is dealt through counters in global memory (`sync`, cleared by the fused kernel): [0] next
// item of A, [1] items of A done, [2] next (row, slice) item of B, [3] next whole-row item of B,
// [4 + i] slices of fast row i done.  B may only start when every item of A is done (A appends to the
// list of failed rows); a CTA that finds no item of A left waits for that -- for CTAs that are
// running, never for CTAs yet to be scheduled -- with a time limit, after which it records a timeout
// in the status word and returns.  When both lists are empty a CTA reads two words and exits.
constexpr int kTailSyncWords = 32;
constexpr int kFallbackCtas = 32;  // CTAs that take whole rows beyond the fast ones

struct TailParams {
    MergeParams mp;
    FallbackParams fb;
    int* sync;
    int* status;
    int fallback;  // 0: the logs are exact by construction (no recomputation stage)
};

__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__global__ void __launch_bounds__(kMergeThreads) route_tail_kernel(const TailParams t) {
    pdl_wait();
    pdl_trigger();
    static_assert(kMergeThreads == kFallbackThreads, "one block size for both stages");
    constexpr size_t kSmem = sizeof(SelectSmem) > sizeof(FallbackSmem) ? sizeof(SelectSmem) : sizeof(FallbackSmem);
    __shared__ __align__(16) unsigned char raw[kSmem];
    __shared__ int s_item, s_flag;
    auto next_item = [&](int* ctr) {
        __syncthreads();
        if (threadIdx.x == 0) s_item = atomicAdd(ctr, 1);
        __syncthreads();
        return s_item;
    };

    // ---- A
    const MergeParams& p = t.mp;
    const int64_t nbig = p.big ? __ldcg(p.big) : p.n;
    if (nbig > 0) {
        SelectSmem& sel = *reinterpret_cast<SelectSmem*>(raw);
        for (;;) {
            const int64_t item = next_item(&t.sync[0]);
            if (item >= nbig) break;
            merge_select_row(p, p.big ? __ldcg(p.big + 1 + item) : item, sel);
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) atomicAdd(&t.sync[1], 1);
        }
        if (t.fallback) {
            if (threadIdx.x == 0) {
                const uint64_t t_start = global_timer_ns();
                int ok = 1;
                while (ld_acquire_gpu(&t.sync[1]) < nbig) {
                    if (global_timer_ns() - t_start > 4000000000ull) {
                        ok = 0;
                        break;
                    }
                    __nanosleep(200);
                }
                if (!ok && atomicCAS(t.status, 0, kStatusTimeout) == 0) {
                    t.status[1] = 20;
                    t.status[2] = static_cast<int>(blockIdx.x);
                }
                s_flag = ok;
            }
            __syncthreads();
            if (!s_flag) return;
        }
    }
    if (!t.fallback) return;

    // ---- B
    const FallbackParams& f = t.fb;
    const int nfail = ld_acquire_gpu(f.fail);
    if (nfail == 0) return;
    FallbackSmem& sm = *reinterpret_cast<FallbackSmem*>(raw);
    const int nfast = min(nfail, kFallbackFastRows);
    const int items = nfast * f.slices;
    int loaded = -1;
    for (;;) {
        const int item = next_item(&t.sync[2]);
        if (item >= items) break;
        const int idx = item / f.slices, slice = item - idx * f.slices;
        const int64_t row = __ldcg(f.fail + 1 + idx);
        if (idx != loaded) {
            fallback_load_point(f, row, sm.xs);
            loaded = idx;
            __syncthreads();
        }
        if (!IVF_IN_BOUNDS(260, idx, kFallbackFastRows) || !IVF_IN_BOUNDS(261, row, p.n)) break;
        fallback_slice(f, slice, f.cand + (static_cast<size_t>(idx) * f.slices + slice) * f.k, sm);
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) s_flag = atomicAdd(&t.sync[4 + idx], 1) == f.slices - 1;
        __syncthreads();
        if (s_flag) {  // this CTA finished the row's last slice: every slice's candidates are visible now
            __threadfence();
            fallback_finish_row(f, f.cand + static_cast<size_t>(idx) * f.slices * f.k, row, sm);
        }
    }
    if (nfail > kFallbackFastRows && blockIdx.x < kFallbackCtas) {
        uint64_t* cand = f.cand + static_cast<size_t>(kFallbackFastRows + blockIdx.x) * f.slices * f.k;
        for (;;) {
            const int idx = kFallbackFastRows + next_item(&t.sync[3]);
            if (idx >= nfail) break;
            const int64_t row = __ldcg(f.fail + 1 + idx);
            fallback_load_point(f, row, sm.xs);
            __syncthreads();
            for (int s2 = 0; s2 < f.slices; ++s2) fallback_slice(f, s2, cand + static_cast<size_t>(s2) * f.k, sm);
            fallback_finish_row(f, cand, row, sm);
        }
    }
}

// ------------------------------------------------------------------ merge of centroid shards
// When the centroid table is split over several GPUs (tables too large to replicate; Sec. 4.1 sweeps
// N_list up to 4M), every GPU routes the queries against its own shard and the [nq, k] lists of all
// shards are gathered: this kernel merges, per query, `parts` lists of k (distance, global id) pairs
// -- each ascending, unused places holding (+inf, any id) -- into the k smallest by (distance, id).
// One CTA per query; the running result and the next shard's list are sorted together in shared
// memory (at most 2 * 512 keys), shard after shard, so any number of shards is taken.
struct ShardMergeParams {
    int64_t nq;
    int k, parts;
    const int32_t* ids;    // [parts][nq][k]
    const float* dists;    // [parts][nq][k]
    int32_t* out_ids;      // [nq][k]
    float* out_dists;      // [nq][k] or nullptr
};

__global__ void __launch_bounds__(kMergeThreads) merge_shards_kernel(const ShardMergeParams p) {
    __shared__ uint64_t keys[2 * kFallbackMaxK];
    const int64_t q = blockIdx.x;
    int m = 2;
    while (m < 2 * p.k) m <<= 1;
    auto load = [&](int part, int base) {
        const size_t at = (static_cast<size_t>(part) * p.nq + q) * p.k;
        for (int i = threadIdx.x; i < p.k; i += blockDim.x)
            keys[base + i] = (static_cast<uint64_t>(orderable(p.dists[at + i])) << 32) | static_cast<uint32_t>(p.ids[at + i]);
    };
    load(0, 0);
    for (int part = 1; part < p.parts; ++part) {
        load(part, p.k);
        for (int i = 2 * p.k + threadIdx.x; i < m; i += blockDim.x) keys[i] = ~0ull;
        bitonic_sort_smem(keys, m);  // begins and ends with a barrier
    }
    __syncthreads();
    for (int i = threadIdx.x; i < p.k; i += blockDim.x) {
        const uint64_t key = keys[i];
        p.out_ids[q * p.k + i] = static_cast<int32_t>(key & 0xFFFFFFFFull);
        if (p.out_dists) p.out_dists[q * p.k + i] = from_orderable(static_cast<uint32_t>(key >> 32));
    }
}

}  // namespace ivf
