// Residual-PQ candidate reduction on the GPU (Sec. 2.2 Eq. 3-5; Sec. 4.3 residual encoding and
// lookup tables; Sec. 4.4: compact codes resident in GPU memory, task set-up on the device by
// prefix scans, chunked ADC scan with a bounded local candidate set, chunk -> group -> query
// merging, and the scan fused with the first merge level).
//
// Arithmetic, in fp32 with one fixed order so that every byte and every kept candidate is
// reproducible (the paper fixes fp32 lookup tables):
//     r_t = float(x_t) - c_t
//     LUT_m[j] : acc = 0; for t in order: diff = r_t - p_m[j][t]; acc = fma(diff, diff, acc)
//     ADC      : acc = 0; for m in order: acc = acc + LUT_m[a_m]
// Encoding is the arg-min over j of the vector's own table (ties to the lower j).
//
// Design: a persistent CTA keeps the whole codebook (256 * d floats, transposed so that the 256
// codewords of one coordinate are contiguous) in shared memory next to one lookup table, so a
// table costs d/PQ_M fused multiply-adds per entry and no global traffic.  A group of chunks of one
// query is scanned by one CTA; candidates that beat the running bound go to a shared-memory buffer
// that is cut back to the N_rerank smallest by a 64-bit radix select when it fills, and only the
// group's survivors are written out.  A last kernel selects and sorts per query.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "fused_topk.cuh"  // orderable(), radix_pick_digit()

namespace ivf {

constexpr int kPqK = 256;          // codewords per subspace (one byte per sub-code)
constexpr int kPqThreads = 1024;       // encode and query-merge kernels
constexpr int kPqScanThreads = 512;    // scan kernel: two CTAs per SM, so one scores while the other builds a table
constexpr int kPqChunk = kPqScanThreads;  // codes per chunk = one code per thread
constexpr int kPqBufKeys = 2048;       // candidate buffer of the query merge
constexpr int kPqScanBufKeys = 1536;   // candidate buffer of a group: a chunk on top of kPqMaxRerank
constexpr int kPqMaxRerank = 1024;
constexpr int kPqMaxProbes = 512;   // lists per query (the paper sweeps the probe count up to 512)
constexpr int kPqStatusBadId = -6;

// the stated bound on the encoder's shared memory (codebook, one lookup table, one residual); the
// kernel itself asks for pq_encode_smem_bytes
__host__ __device__ inline size_t pq_smem_bytes(int d, int pq_m) {
    return static_cast<size_t>(d) * kPqK * 4 + static_cast<size_t>(pq_m) * kPqK * 4 + static_cast<size_t>(d) * 4;
}

// A thread group: NT threads numbered tid that synchronise on hardware barrier BAR (BAR = 0 with
// NT = the CTA size is __syncthreads).  The scan kernels run one or two such groups per CTA.
template <int BAR, int NT>
__device__ __forceinline__ void pq_group_sync() {
    if constexpr (BAR == 0) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(NT) : "memory");
}

// Lookup-table build.  Thread -> codeword j = tid & 255; the 256-thread slices of the CTA take
// alternate subspaces.
template <bool kGlobal>
__device__ __forceinline__ float pq_cb(const float* p) {
    if constexpr (kGlobal) return __ldg(p);
    else return *p;
}

// One sub-vector width: all strides are compile-time constants, so every load takes an immediate
// offset from three running pointers; four subspaces per trip give four independent chains.
template <bool kGlobal, int DSUB>
__device__ __forceinline__ void pq_build_lut_fixed(const float* __restrict__ r, const float* __restrict__ cbt,
                                                   float* __restrict__ lut, int pq_m, int tid, int nthreads) {
    const int j = tid & (kPqK - 1);
    const int first = tid >> 8;
    const int step = nthreads >> 8;
    const float* col = cbt + first * (DSUB * kPqK) + j;
    const float* rp = r + first * DSUB;
    float* out = lut + first * kPqK + j;
    const int col_step = step * DSUB * kPqK, r_step = step * DSUB, out_step = step * kPqK;
#pragma unroll 4
    for (int m = first; m < pq_m; m += step) {
        float rv[DSUB];
        if constexpr ((DSUB & 3) == 0) {
#pragma unroll
            for (int t4 = 0; t4 < DSUB / 4; ++t4) {
                const float4 v = reinterpret_cast<const float4*>(rp)[t4];
                rv[4 * t4] = v.x; rv[4 * t4 + 1] = v.y; rv[4 * t4 + 2] = v.z; rv[4 * t4 + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int t = 0; t < DSUB; ++t) rv[t] = rp[t];
        }
        float cv[DSUB];
#pragma unroll
        for (int t = 0; t < DSUB; ++t) cv[t] = pq_cb<kGlobal>(col + t * kPqK);
        float acc = 0.0f;
#pragma unroll
        for (int t = 0; t < DSUB; ++t) {
            const float diff = __fsub_rn(rv[t], cv[t]);
            acc = __fmaf_rn(diff, diff, acc);
        }
        *out = acc;
        col += col_step;
        rp += r_step;
        out += out_step;
    }
}

// The same build from the codebook in its given layout [pq_m][256][dsub], for the widths whose
// codeword is one 8- or 16-byte load (a warp's 32 codewords are then contiguous, so the load has as
// many shared-memory wavefronts as the coordinate-major copy needs but a quarter or half of the
// instructions).  Same operations in the same order as pq_build_lut_fixed: bit-identical tables.
template <bool kGlobal, int DSUB>
__device__ __forceinline__ void pq_build_lut_rows(const float* __restrict__ r, const float* __restrict__ cb,
                                                  float* __restrict__ lut, int pq_m, int tid, int nthreads) {
    static_assert(DSUB == 2 || DSUB == 4, "one vector load per codeword");
    const int j = tid & (kPqK - 1);
    const int first = tid >> 8;
    const int step = nthreads >> 8;
    const float* row = cb + (first * kPqK + j) * DSUB;
    const float* rp = r + first * DSUB;
    float* out = lut + first * kPqK + j;
    const int row_step = step * kPqK * DSUB, r_step = step * DSUB, out_step = step * kPqK;
#pragma unroll 4
    for (int m = first; m < pq_m; m += step) {
        float rv[DSUB], cv[DSUB];
        if constexpr (DSUB == 4) {
            const float4 v = *reinterpret_cast<const float4*>(rp);
            rv[0] = v.x; rv[1] = v.y; rv[2] = v.z; rv[3] = v.w;
            float4 c;
            if constexpr (kGlobal) c = __ldg(reinterpret_cast<const float4*>(row));
            else c = *reinterpret_cast<const float4*>(row);
            cv[0] = c.x; cv[1] = c.y; cv[2] = c.z; cv[3] = c.w;
        } else {
            const float2 v = *reinterpret_cast<const float2*>(rp);
            rv[0] = v.x; rv[1] = v.y;
            float2 c;
            if constexpr (kGlobal) c = __ldg(reinterpret_cast<const float2*>(row));
            else c = *reinterpret_cast<const float2*>(row);
            cv[0] = c.x; cv[1] = c.y;
        }
        float acc = 0.0f;
#pragma unroll
        for (int t = 0; t < DSUB; ++t) {
            const float diff = __fsub_rn(rv[t], cv[t]);
            acc = __fmaf_rn(diff, diff, acc);
        }
        *out = acc;
        row += row_step;
        rp += r_step;
        out += out_step;
    }
}

// true: the scan kernels can read the codebook in its given layout (pq_build_lut_rows), if it starts
// on a 16-byte boundary; false: they need the coordinate-major copy
__host__ __device__ inline bool pq_codebook_by_rows(int dsub) { return dsub == 2 || dsub == 4; }

// lut[m * 256 + j] for the residual r.  cbt: the codebook, as given when by_rows, else coordinate-
// major.  kGlobal: it is in global memory (read through L1); otherwise a copy in shared memory.
template <bool kGlobal>
__device__ __forceinline__ void pq_build_lut(const float* r, const float* cbt, float* lut, int pq_m, int dsub, int tid,
                                             int nthreads, bool by_rows) {
    if (by_rows) {
        if (dsub == 4) return pq_build_lut_rows<kGlobal, 4>(r, cbt, lut, pq_m, tid, nthreads);
        return pq_build_lut_rows<kGlobal, 2>(r, cbt, lut, pq_m, tid, nthreads);
    }
    switch (dsub) {
        case 2: return pq_build_lut_fixed<kGlobal, 2>(r, cbt, lut, pq_m, tid, nthreads);
        case 3: return pq_build_lut_fixed<kGlobal, 3>(r, cbt, lut, pq_m, tid, nthreads);
        case 4: return pq_build_lut_fixed<kGlobal, 4>(r, cbt, lut, pq_m, tid, nthreads);
        case 6: return pq_build_lut_fixed<kGlobal, 6>(r, cbt, lut, pq_m, tid, nthreads);
        case 8: return pq_build_lut_fixed<kGlobal, 8>(r, cbt, lut, pq_m, tid, nthreads);
        default: break;
    }
    const int j = tid & (kPqK - 1);
    const int step = nthreads >> 8;
    for (int m = tid >> 8; m < pq_m; m += step) {
        const float* col = cbt + static_cast<size_t>(m) * dsub * kPqK + j;
        const float* rm = r + m * dsub;
        float acc = 0.0f;
        for (int t = 0; t < dsub; ++t) {
            const float diff = __fsub_rn(rm[t], pq_cb<kGlobal>(col + t * kPqK));
            acc = __fmaf_rn(diff, diff, acc);
        }
        lut[m * kPqK + j] = acc;
    }
}

// element idx of a row matrix of the given type code (0 float, 1 uint8, 2 int8), as a float
__device__ __forceinline__ float pq_elem(const void* x, int type, int64_t idx) {
    if (type == 1) return static_cast<float>(static_cast<const uint8_t*>(x)[idx]);
    if (type == 2) return static_cast<float>(static_cast<const int8_t*>(x)[idx]);
    return static_cast<const float*>(x)[idx];
}

// ------------------------------------------------------------------ residual encoding (Eq. 3 on x - c(x))
struct PqEncodeParams {
    const void* x;
    int x_type;  // 0 float, 1 uint8, 2 int8
    int64_t n;
    int d, pq_m, nlist;
    const int32_t* ids;
    const float* centroids;
    const float* codebooks;
    uint8_t* codes;  // [n][pq_m]
    int* status;
};

// Shared memory of the encode kernel: the codebook in its own layout [m][j][dsub] and two buffers of
// kPqEncodeElems residual coordinates (a batch of vectors each).
constexpr int kPqEncodeElems = kPqThreads;  // coordinates per batch = one per thread
__host__ __device__ inline size_t pq_encode_smem_bytes(int d) {
    return static_cast<size_t>(d) * kPqK * 4 + 2 * static_cast<size_t>(kPqEncodeElems) * 4 + 2 * 64 * 4;
}

// Codes of one (vector, subspace) pair by one warp: lane q takes codewords lane, lane + 32, ... (8 of
// them), each table entry is the same chain of rounded operations as in the lookup-table build
// (diff = r_t - p_t, acc = fma(diff, diff, acc), t ascending), the smallest entry wins, ties to the
// lower codeword.  No table is written anywhere: the entries live in registers.  REGS: the lane's 8
// codewords are already in registers (cwr), otherwise they are read from the shared-memory codebook.
template <int DSUB, bool REGS>
__device__ __forceinline__ int pq_encode_subspace(const float* __restrict__ rm, const float* __restrict__ cbm, int dsub,
                                                  int lane, const float (&cwr)[kPqK / 32][DSUB > 0 ? DSUB : 1]) {
    const int ds = DSUB > 0 ? DSUB : dsub;
    float rv[DSUB > 0 ? DSUB : 1];
    if constexpr (DSUB > 0) {
        if constexpr ((DSUB & 3) == 0) {
#pragma unroll
            for (int t4 = 0; t4 < DSUB / 4; ++t4) {
                const float4 v = reinterpret_cast<const float4*>(rm)[t4];
                rv[4 * t4] = v.x; rv[4 * t4 + 1] = v.y; rv[4 * t4 + 2] = v.z; rv[4 * t4 + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int t = 0; t < DSUB; ++t) rv[t] = rm[t];
        }
    }
    float best = __int_as_float(0x7f800000);
    int bj = 0x7fffffff;
#pragma unroll
    for (int q = 0; q < kPqK / 32; ++q) {
        const int j = lane + 32 * q;
        float acc = 0.0f;
        if constexpr (REGS) {
#pragma unroll
            for (int t = 0; t < DSUB; ++t) {
                const float diff = __fsub_rn(rv[t], cwr[q][t]);
                acc = __fmaf_rn(diff, diff, acc);
            }
        } else {
            const float* cw = cbm + j * ds;
            if constexpr (DSUB > 0 && (DSUB & 3) == 0) {
#pragma unroll
                for (int t4 = 0; t4 < DSUB / 4; ++t4) {
                    const float4 c = reinterpret_cast<const float4*>(cw)[t4];
                    float diff = __fsub_rn(rv[4 * t4], c.x);
                    acc = __fmaf_rn(diff, diff, acc);
                    diff = __fsub_rn(rv[4 * t4 + 1], c.y);
                    acc = __fmaf_rn(diff, diff, acc);
                    diff = __fsub_rn(rv[4 * t4 + 2], c.z);
                    acc = __fmaf_rn(diff, diff, acc);
                    diff = __fsub_rn(rv[4 * t4 + 3], c.w);
                    acc = __fmaf_rn(diff, diff, acc);
                }
            } else if constexpr (DSUB > 0) {
#pragma unroll
                for (int t = 0; t < DSUB; ++t) {
                    const float diff = __fsub_rn(rv[t], cw[t]);
                    acc = __fmaf_rn(diff, diff, acc);
                }
            } else {
                for (int t = 0; t < ds; ++t) {
                    const float diff = __fsub_rn(rm[t], cw[t]);
                    acc = __fmaf_rn(diff, diff, acc);
                }
            }
        }
        if (acc < best) {  // codewords ascend within a lane, so an equal entry keeps the lower one
            best = acc;
            bj = j;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(0xFFFFFFFFu, best, off);
        const int oj = __shfl_xor_sync(0xFFFFFFFFu, bj, off);
        if (ov < best || (ov == best && oj < bj)) {
            best = ov;
            bj = oj;
        }
    }
    return bj;
}

// The batch loop of the encode kernel for one sub-vector width.  A CTA walks batches of V = 1024 / d
// (rounded down to a power of two) vectors.  While the warps encode a batch -- one (vector, subspace)
// pair per warp and step -- every thread already holds one residual coordinate of the next batch in a
// register (row, id and centroid fetched from global memory under the arithmetic), so the kernel never
// waits for memory between vectors.  REGS (the number of subspaces divides 32, sub-vectors of at most 4):
// a warp then meets the same subspace at every step and keeps its 8 codewords per lane in registers for
// the whole launch, so the shared-memory pipe carries only the residuals (the codebook reads were what
// bounded the kernel: 1,024 wavefronts per vector).
template <int DSUB, bool REGS>
__device__ __forceinline__ void pq_encode_body(const PqEncodeParams& p, const float* cb, float* rbuf, int* badbuf) {
    const int dsub = p.d / p.pq_m;
    int V = kPqEncodeElems / p.d;
    V = V >= 32 ? 32 : (V >= 16 ? 16 : (V >= 8 ? 8 : (V >= 4 ? 4 : (V >= 2 ? 2 : 1))));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int e = threadIdx.x;                 // this thread's coordinate of a batch
    const int ev = e / p.d, et = e - ev * p.d;  // vector within the batch, coordinate

    // residual coordinate (ev, et) of the batch that starts at vector `base`; bad = the id is out of range
    auto fetch = [&](int64_t base, float& r, int& bad) {
        r = 0.0f;
        bad = 0;
        const int64_t i = base + ev;
        if (ev < V && i < p.n) {
            const int32_t l = p.ids[i];
            if (l >= 0 && l < p.nlist) {
                const float xv = pq_elem(p.x, p.x_type, i * p.d + et);
                r = __fsub_rn(xv, p.centroids[static_cast<int64_t>(l) * p.d + et]);
            } else {
                bad = 1;
            }
        }
    };
    const int64_t stride = static_cast<int64_t>(gridDim.x) * V;
    int64_t base = static_cast<int64_t>(blockIdx.x) * V;
    float r_next;
    int bad_next;
    fetch(base, r_next, bad_next);
    __syncthreads();  // the codebook is in shared memory
    float cwr[kPqK / 32][DSUB > 0 ? DSUB : 1];
    if constexpr (REGS) {
        const int m = warp % p.pq_m;  // the one subspace this warp ever meets
#pragma unroll
        for (int q = 0; q < kPqK / 32; ++q)
#pragma unroll
            for (int t = 0; t < DSUB; ++t) cwr[q][t] = cb[(static_cast<size_t>(m) * kPqK + lane + 32 * q) * DSUB + t];
    }
    int buf = 0;
    for (; base < p.n; base += stride) {
        rbuf[buf * kPqEncodeElems + e] = r_next;
        if (et == 0 && ev < V) badbuf[buf * 64 + ev] = bad_next;
        __syncthreads();  // this batch's residuals are in place
        fetch(base + stride, r_next, bad_next);  // the next batch travels while this one is encoded
        const int nv = static_cast<int>(p.n - base < V ? p.n - base : V);
        const float* rb = rbuf + buf * kPqEncodeElems;
        const int* bb = badbuf + buf * 64;
        for (int item = warp; item < nv * p.pq_m; item += nwarps) {
            const int vi = item / p.pq_m, m = item - vi * p.pq_m;
            const int64_t i = base + vi;
            int code = 0;
            if (bb[vi]) {
                if (lane == 0 && m == 0) atomicCAS(p.status, 0, kPqStatusBadId);
            } else {
                code = pq_encode_subspace<DSUB, REGS>(rb + vi * p.d + m * dsub, cb + static_cast<size_t>(m) * kPqK * dsub, dsub,
                                                      lane, cwr);
            }
            if (lane == 0 && IVF_IN_BOUNDS(430, code, kPqK)) p.codes[i * p.pq_m + m] = static_cast<uint8_t>(code);
        }
        buf ^= 1;  // (the buffer written next was last read two batches ago: one barrier per batch is enough)
    }
}

// Persistent: one CTA per SM keeps the codebook [m][j][dsub] in shared memory.
__global__ void __launch_bounds__(kPqThreads, 1) pq_encode_kernel(const PqEncodeParams p) {
    extern __shared__ __align__(16) uint8_t pq_smem_raw[];
    float* cb = reinterpret_cast<float*>(pq_smem_raw);                       // [pq_m][256][dsub]
    float* rbuf = cb + static_cast<size_t>(p.d) * kPqK;                      // [2][kPqEncodeElems]
    int* badbuf = reinterpret_cast<int*>(rbuf + 2 * kPqEncodeElems);         // [2][64]
    const int dsub = p.d / p.pq_m;
    const int total_cb = p.d * kPqK;
    if ((reinterpret_cast<uintptr_t>(p.codebooks) & 15) == 0) {
        for (int i = threadIdx.x * 4; i < total_cb; i += blockDim.x * 4)    // d * 256 is a multiple of 4
            *reinterpret_cast<float4*>(cb + i) = __ldg(reinterpret_cast<const float4*>(p.codebooks + i));
    } else {
        for (int i = threadIdx.x; i < total_cb; i += blockDim.x) cb[i] = __ldg(p.codebooks + i);
    }
    const bool regs = (32 % p.pq_m) == 0;  // every warp meets one subspace only
    switch (dsub) {
        case 2: return regs ? pq_encode_body<2, true>(p, cb, rbuf, badbuf) : pq_encode_body<2, false>(p, cb, rbuf, badbuf);
        case 3: return regs ? pq_encode_body<3, true>(p, cb, rbuf, badbuf) : pq_encode_body<3, false>(p, cb, rbuf, badbuf);
        case 4: return regs ? pq_encode_body<4, true>(p, cb, rbuf, badbuf) : pq_encode_body<4, false>(p, cb, rbuf, badbuf);
        case 6: return pq_encode_body<6, false>(p, cb, rbuf, badbuf);
        case 8: return pq_encode_body<8, false>(p, cb, rbuf, badbuf);
        default: return pq_encode_body<0, false>(p, cb, rbuf, badbuf);
    }
}

// Residuals x - c(x) as fp32 rows (the training set of the codebooks, Sec. 4.3): one rounded
// subtraction per coordinate, exactly what the encoder and the oracle compute.
__global__ void pq_residuals_kernel(const void* __restrict__ x, int x_type, int64_t n, int d,
                                    const int32_t* __restrict__ ids, const float* __restrict__ centroids, int nlist,
                                    float* __restrict__ out, int* status) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n * d) return;
    const int64_t row = i / d;
    const int t = static_cast<int>(i - row * d);
    const int32_t l = ids[row];
    if (l < 0 || l >= nlist) {
        if (t == 0) atomicCAS(status, 0, kPqStatusBadId);
        out[i] = 0.0f;
        return;
    }
    out[i] = __fsub_rn(pq_elem(x, x_type, i), centroids[static_cast<int64_t>(l) * d + t]);
}

// codebooks [pq_m][256][dsub] -> out[(m * dsub + t) * 256 + j] (coordinate-major), for the scan kernel
__global__ void pq_transpose_codebooks_kernel(const float* __restrict__ codebooks, int d, int dsub, float* __restrict__ out) {
    pdl_wait();
    pdl_trigger();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;  // index in the output
    if (i >= d * kPqK) return;
    const int j = i & (kPqK - 1);
    const int mt = i >> 8;  // m * dsub + t
    const int m = mt / dsub, t = mt - m * dsub;
    out[i] = codebooks[(static_cast<size_t>(m) * kPqK + j) * dsub + t];
}

// ------------------------------------------------------------------ task set-up (prefix scans on the device)
// Per query: chunk_start[b][p] = chunks of the probes before p (a probed list of length L has
// ceil(L / kPqChunk) chunks), chunk_start[b][nprobe] = the query's chunks; cand_count[b] = the codes
// it will scan.  Every query's chunks are then dealt to a fixed number of groups, so the output
// offset of a group follows from its index alone.
__global__ void __launch_bounds__(128) pq_setup_query_kernel(const int32_t* __restrict__ probes, int nprobe, int nlist,
                                                             const long long* __restrict__ offsets,
                                                             int* __restrict__ chunk_start,
                                                             long long* __restrict__ cand_count, int* status) {
    pdl_wait();
    pdl_trigger();
    __shared__ int wsum[4];
    __shared__ long long wlen[4];
    __shared__ int carry_s;
    __shared__ long long total_len_s;
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        carry_s = 0;
        total_len_s = 0;
    }
    __syncthreads();
    int* cs = chunk_start + static_cast<size_t>(b) * (nprobe + 1);
    for (int p0 = 0; p0 < nprobe; p0 += blockDim.x) {
        const int p = p0 + threadIdx.x;
        int nch = 0;
        long long len = 0;
        if (p < nprobe) {
            const int l = probes[static_cast<size_t>(b) * nprobe + p];
            if (l >= 0 && l < nlist) {
                len = offsets[l + 1] - offsets[l];
                if (len < 0) len = 0;
                nch = static_cast<int>((len + kPqChunk - 1) / kPqChunk);
            } else {
                atomicCAS(status, 0, kPqStatusBadId);
            }
        }
        int v = nch;
        long long lv = len;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, v, off);
            if (lane >= off) v += t;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) lv += __shfl_xor_sync(0xFFFFFFFFu, lv, off);
        if (lane == 31) wsum[warp] = v;
        if (lane == 0) wlen[warp] = lv;
        __syncthreads();
        int before = carry_s;
        for (int w = 0; w < warp; ++w) before += wsum[w];
        if (p < nprobe) cs[p] = before + v - nch;
        __syncthreads();
        if (threadIdx.x == 0) {
            carry_s += wsum[0] + wsum[1] + wsum[2] + wsum[3];
            total_len_s += wlen[0] + wlen[1] + wlen[2] + wlen[3];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        cs[nprobe] = carry_s;
        if (cand_count) cand_count[b] = total_len_s;
    }
}

// ------------------------------------------------------------------ selection of the k smallest keys by a thread group
// Largest admitted key among the `count` distinct 64-bit keys get(0 .. count) (count > k; keys that
// read as all-ones are padding and must number fewer than count - k): radix select from the top
// byte down, stopping once the digit that holds rank k is wanted whole.
template <int BAR, int NT, typename Get>
__device__ __forceinline__ uint64_t pq_select_bound(Get get, int count, int k, int* hist, int* misc, int tid) {
    const int lane = tid & 31;
    uint64_t prefix = 0, mask = 0;
    int rank = k;
    const int rounded = (count + 31) & ~31;
    for (int shift = 56; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += NT) hist[i] = 0;
        pq_group_sync<BAR, NT>();
        for (int i = tid; i < rounded; i += NT) {
            uint32_t dg = 0xFFFFFFFFu;
            if (i < count) {
                const uint64_t v = get(i);
                if ((v & mask) == prefix) dg = static_cast<uint32_t>(v >> shift) & 255u;
            }
            const uint32_t peers = __match_any_sync(0xFFFFFFFFu, dg);
            if (dg != 0xFFFFFFFFu && lane == __ffs(peers) - 1) atomicAdd(&hist[dg], __popc(peers));
        }
        pq_group_sync<BAR, NT>();
        if (tid < 32) {
            int r = rank, eq = 0;
            const int digit = radix_pick_digit(hist, lane, r, eq);
            if (lane == 0) {
                misc[1] = digit;
                misc[2] = r;
                misc[3] = eq;
            }
        }
        pq_group_sync<BAR, NT>();
        prefix |= static_cast<uint64_t>(misc[1]) << shift;
        mask |= 255ull << shift;
        rank = misc[2];
        const bool whole = misc[3] == rank;
        pq_group_sync<BAR, NT>();
        if (whole) return prefix | ~mask;
    }
    return prefix;
}

// The same selection over keys that every thread holds in registers (PER per thread; all-ones =
// padding), so that the passes touch no memory but the histogram.
template <int BAR, int NT, int PER>
__device__ __forceinline__ uint64_t pq_select_bound_regs(const uint64_t (&mine)[PER], int k, int* hist, int* misc,
                                                         int tid) {
    const int lane = tid & 31;
    uint64_t prefix = 0, mask = 0;
    int rank = k;
    for (int shift = 56; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += NT) hist[i] = 0;
        pq_group_sync<BAR, NT>();
#pragma unroll
        for (int q = 0; q < PER; ++q) {
            const uint64_t v = mine[q];
            uint32_t dg = 0xFFFFFFFFu;
            if (v != ~0ull && (v & mask) == prefix) dg = static_cast<uint32_t>(v >> shift) & 255u;
            if (__any_sync(0xFFFFFFFFu, dg != 0xFFFFFFFFu)) {
                const uint32_t peers = __match_any_sync(0xFFFFFFFFu, dg);
                if (dg != 0xFFFFFFFFu && lane == __ffs(peers) - 1) atomicAdd(&hist[dg], __popc(peers));
            }
        }
        pq_group_sync<BAR, NT>();
        if (tid < 32) {
            int r = rank, eq = 0;
            const int digit = radix_pick_digit(hist, lane, r, eq);
            if (lane == 0) {
                misc[1] = digit;
                misc[2] = r;
                misc[3] = eq;
            }
        }
        pq_group_sync<BAR, NT>();
        prefix |= static_cast<uint64_t>(misc[1]) << shift;
        mask |= 255ull << shift;
        rank = misc[2];
        const bool whole = misc[3] == rank;
        pq_group_sync<BAR, NT>();
        if (whole) return prefix | ~mask;
    }
    return prefix;
}

// Cuts the buffer (capacity CAP) back to its k smallest keys (in no particular order); returns the
// bound, i.e. the largest key kept.  count > k on entry; on exit misc[0] == k.
template <int BAR, int NT, int CAP>
__device__ __forceinline__ uint64_t pq_cut_buffer(uint64_t* buf, int count, int k, int* hist, int* misc, int tid) {
    const uint64_t bound = pq_select_bound<BAR, NT>([buf](int i) { return buf[i]; }, count, k, hist, misc, tid);
    constexpr int kPer = CAP / NT;
    static_assert(CAP % NT == 0, "buffer capacity must be a multiple of the thread count");
    uint64_t mine[kPer];
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
        const int i = tid + q * NT;
        mine[q] = i < count ? buf[i] : ~0ull;
    }
    if (tid == 0) misc[0] = 0;
    pq_group_sync<BAR, NT>();
#pragma unroll
    for (int q = 0; q < kPer; ++q)
        if (mine[q] <= bound && mine[q] != ~0ull) {
            const int at = atomicAdd(&misc[0], 1);
            if (IVF_IN_BOUNDS(401, at, CAP)) buf[at] = mine[q];
        }
    pq_group_sync<BAR, NT>();
    return bound;
}

// ------------------------------------------------------------------ chunked ADC scan fused with the group merge
struct PqScanParams {
    const void* q;
    int q_type;  // 0 float, 1 uint8, 2 int8
    int64_t nq;
    int d, pq_m, nlist, nprobe, n_rerank;
    int ngroups;             // groups per query
    const float* centroids;
    const float* cbt;        // codebook in global memory (read through L1, or copied to shared memory): as given
                             // ([pq_m][256][dsub]) when cb_rows, else transposed [d][256]
    int cb_rows;
    const int32_t* probes;
    const long long* offsets;
    const uint8_t* codes;
    const int* chunk_start;  // [nq][nprobe + 1]
    uint64_t* gcand;         // [nq * ngroups][n_rerank] keys: (estimate bits << 32) | position
    int* gcand_count;        // [nq * ngroups]
    int* status;
};

// Working set of one scanning team (kPqScanThreads threads) in shared memory.  r and hist share a
// region: the residual is dead once the table is built, the histogram lives only inside a buffer cut.
struct PqTeamSmem {
    float* lut;            // [pq_m][256]
    float* r;              // [d], d <= 256
    uint64_t* buf;         // [kPqScanBufKeys]
    int* hist;             // [256]
    int* misc;             // [16]
    uint32_t* list_begin;  // [maxp] first position of each probed list
    int* list_len;         // [maxp]
    int* list_id;          // [maxp]
    int* cs;               // [maxp + 1] chunk prefix of the query
};
__host__ __device__ inline size_t pq_team_bytes(int pq_m, int maxp) {
    return static_cast<size_t>(pq_m) * kPqK * 4 + static_cast<size_t>(kPqScanBufKeys) * 8 + 1024 + 64 +
           static_cast<size_t>(maxp) * 12 + ((static_cast<size_t>(maxp) + 1) * 4 + 15) / 16 * 16;
}
__device__ __forceinline__ PqTeamSmem pq_team_carve(uint8_t* raw, int pq_m, int maxp) {
    PqTeamSmem s;
    s.buf = reinterpret_cast<uint64_t*>(raw);
    raw += static_cast<size_t>(kPqScanBufKeys) * 8;
    s.lut = reinterpret_cast<float*>(raw);
    raw += static_cast<size_t>(pq_m) * kPqK * 4;
    s.hist = reinterpret_cast<int*>(raw);
    s.r = reinterpret_cast<float*>(raw);
    raw += 1024;
    s.misc = reinterpret_cast<int*>(raw);
    raw += 64;
    s.list_begin = reinterpret_cast<uint32_t*>(raw);
    raw += static_cast<size_t>(maxp) * 4;
    s.list_len = reinterpret_cast<int*>(raw);
    raw += static_cast<size_t>(maxp) * 4;
    s.list_id = reinterpret_cast<int*>(raw);
    raw += static_cast<size_t>(maxp) * 4;
    s.cs = reinterpret_cast<int*>(raw);
    return s;
}
// shared memory of the two scan kernels
__host__ __device__ inline size_t pq_scan_smem_bytes(int d, int pq_m) { return pq_team_bytes(pq_m, kPqMaxProbes); }
constexpr int kPqTeamProbes = 256;  // probes per query that the two-team kernel stages
__host__ __device__ inline size_t pq_teams_smem_bytes(int d, int pq_m) {
    return static_cast<size_t>(d) * kPqK * 4 + 2 * pq_team_bytes(pq_m, kPqTeamProbes);
}

// The code bytes of one stored vector, held in registers so that the next chunk's bytes can be
// fetched while the current chunk is being scored (sub-code counts that are a multiple of 16, up
// to 32, take this path; others are read byte-wise while scoring).
struct PqCodeRegs {
    uint4 w[2];
};
__device__ __forceinline__ bool pq_codes_in_regs(int pq_m) { return pq_m == 16 || pq_m == 32; }
// streamed once: read-only path, not kept in L1 (which holds the codebook)
__device__ __forceinline__ uint4 pq_ld_stream(const uint8_t* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void pq_fetch_code(PqCodeRegs& c, const uint8_t* code, int pq_m) {
    c.w[0] = pq_ld_stream(code);
    if (pq_m == 32) c.w[1] = pq_ld_stream(code + 16);
}
// ADC estimate from code bytes held in registers.  Every table entry is fetched with a
// shared-space load whose row offset is an immediate: per sub-code one shift, one mask, one load,
// one add.  lut_s = shared-space address of the table.
#define PQ_ADC_STEP(WORD, Q, M)                                                                          \
    {                                                                                                    \
        const uint32_t scaled = ((Q) == 0 ? ((WORD) << 2) : ((WORD) >> (8 * (Q) - 2))) & 0x3FCu;       \
        float v;                                                                                         \
        asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(lut_s + scaled), "n"((M) * kPqK * 4)); \
        acc = __fadd_rn(acc, v);                                                                         \
    }
#define PQ_ADC_WORD(WORD, M0) \
    PQ_ADC_STEP(WORD, 0, (M0)) PQ_ADC_STEP(WORD, 1, (M0) + 1) PQ_ADC_STEP(WORD, 2, (M0) + 2) PQ_ADC_STEP(WORD, 3, (M0) + 3)
__device__ __forceinline__ float pq_adc_regs(uint32_t lut_s, const PqCodeRegs& c, int pq_m) {
    float acc = 0.0f;
    PQ_ADC_WORD(c.w[0].x, 0)
    PQ_ADC_WORD(c.w[0].y, 4)
    PQ_ADC_WORD(c.w[0].z, 8)
    PQ_ADC_WORD(c.w[0].w, 12)
    if (pq_m == 32) {
        PQ_ADC_WORD(c.w[1].x, 16)
        PQ_ADC_WORD(c.w[1].y, 20)
        PQ_ADC_WORD(c.w[1].z, 24)
        PQ_ADC_WORD(c.w[1].w, 28)
    }
    return acc;
}
#undef PQ_ADC_WORD
#undef PQ_ADC_STEP

__device__ __forceinline__ float pq_adc_code(const float* lut, const uint8_t* code, int pq_m) {
    float acc = 0.0f;
    if ((pq_m & 15) == 0) {
        for (int m0 = 0; m0 < pq_m; m0 += 16) {
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(code + m0));
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int q = 0; q < 16; ++q)
                acc = __fadd_rn(acc, lut[(m0 + q) * kPqK + ((w[q >> 2] >> (8 * (q & 3))) & 255u)]);
        }
    } else if ((pq_m & 3) == 0) {
        for (int m0 = 0; m0 < pq_m; m0 += 4) {
            const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(code + m0));
#pragma unroll
            for (int q = 0; q < 4; ++q) acc = __fadd_rn(acc, lut[(m0 + q) * kPqK + ((w >> (8 * q)) & 255u)]);
        }
    } else {
        for (int m = 0; m < pq_m; ++m) acc = __fadd_rn(acc, lut[m * kPqK + __ldg(code + m)]);
    }
    return acc;
}

// The groups g_first, g_first + g_step, ... scanned by one team: thread tid of kPqScanThreads,
// synchronising on barrier BAR.  kGlobalCb: cbt is the transposed codebook in global memory (read
// through L1), otherwise the copy in shared memory.
template <bool kGlobalCb, int BAR>
__device__ __forceinline__ void pq_scan_groups(const PqScanParams& p, const PqTeamSmem& s, const float* cbt,
                                               int64_t g_first, int64_t g_step, int tid) {
    constexpr int NT = kPqScanThreads;
    const int dsub = p.d / p.pq_m;
    const int64_t total_groups = p.nq * p.ngroups;
    const int lane = tid & 31;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const bool in_regs = pq_codes_in_regs(p.pq_m);
    const uint32_t lut_s = static_cast<uint32_t>(__cvta_generic_to_shared(s.lut));

    for (int64_t g = g_first; g < total_groups; g += g_step) {
        const int64_t b = g / p.ngroups;
        const int gi = static_cast<int>(g - b * p.ngroups);
        const int* cs_g = p.chunk_start + static_cast<size_t>(b) * (p.nprobe + 1);
        pq_group_sync<BAR, NT>();  // the previous group's descriptors, table and buffer are no longer in use
        // the query's probe descriptors, once per group: chunk prefix, list begin, list length
        for (int pr = tid; pr <= p.nprobe; pr += NT) {
            if (!IVF_IN_BOUNDS(410, pr, kPqMaxProbes + 1)) continue;
            s.cs[pr] = cs_g[pr];
            if (pr < p.nprobe) {
                const int l = p.probes[static_cast<size_t>(b) * p.nprobe + pr];
                long long begin = 0, len = 0;
                if (l >= 0 && l < p.nlist) {
                    begin = p.offsets[l];
                    len = p.offsets[l + 1] - begin;
                }
                s.list_id[pr] = l;
                s.list_begin[pr] = static_cast<uint32_t>(begin);
                s.list_len[pr] = static_cast<int>(len < 0 ? 0 : (len > 0x7fffffffLL ? 0x7fffffffLL : len));
            }
        }
        if (tid == 0) s.misc[0] = 0;
        pq_group_sync<BAR, NT>();
        const int nchunks = s.cs[p.nprobe];
        const int group_chunks = (nchunks + p.ngroups - 1) / p.ngroups;
        const int chunk0 = min(nchunks, gi * group_chunks);
        const int chunk1 = min(nchunks, chunk0 + group_chunks);
        uint64_t bound = ~0ull;  // a candidate must be below this key to matter
        if (chunk0 < chunk1) {
            // owner of chunk0: the last probe pr with cs[pr] <= chunk0 (empty lists own no chunk)
            int pr = 0;
            {
                int hi = p.nprobe;
                while (hi - pr > 1) {
                    const int mid = (pr + hi) >> 1;
                    if (s.cs[mid] <= chunk0) pr = mid; else hi = mid;
                }
            }
            float qv = 0.0f, cnext = 0.0f;  // thread t < d: its query coordinate, the coming list's centroid coordinate
            if (tid < p.d) {
                qv = pq_elem(p.q, p.q_type, b * p.d + tid);
                cnext = p.centroids[static_cast<int64_t>(s.list_id[pr]) * p.d + tid];
            }
            int built = -1;
            // the code of the first chunk
            PqCodeRegs nxt;
            nxt.w[0] = nxt.w[1] = make_uint4(0, 0, 0, 0);
            long long nxt_pos = -1;
            {
                const int in_list = (chunk0 - s.cs[pr]) * kPqChunk + tid;
                if (in_list < s.list_len[pr]) nxt_pos = static_cast<long long>(s.list_begin[pr]) + in_list;
                if (in_regs && nxt_pos >= 0) pq_fetch_code(nxt, p.codes + nxt_pos * p.pq_m, p.pq_m);
            }
            int npr = pr;  // owner of the chunk whose code is in `nxt`
            for (int ch = chunk0; ch < chunk1; ++ch) {
                pr = npr;
                if (pr != built) {
                    pq_group_sync<BAR, NT>();  // the previous table is no longer read (nor the histogram, which r overlays)
                    if (tid < p.d) s.r[tid] = __fsub_rn(qv, cnext);
                    // fetch the centroid of the next list that owns a chunk of this group
                    int later = pr + 1;
                    while (later < p.nprobe && s.cs[later + 1] == s.cs[later]) ++later;
                    if (later < p.nprobe && s.cs[later] < chunk1 && tid < p.d)
                        cnext = p.centroids[static_cast<int64_t>(s.list_id[later]) * p.d + tid];
                    pq_group_sync<BAR, NT>();
                    pq_build_lut<kGlobalCb>(s.r, cbt, s.lut, p.pq_m, dsub, tid, NT, p.cb_rows != 0);
                    pq_group_sync<BAR, NT>();
                    built = pr;
                }
                const long long pos = nxt_pos;
                const PqCodeRegs cur = nxt;
                // fetch the next chunk's code while this one is scored
                nxt_pos = -1;
                if (ch + 1 < chunk1) {
                    while (s.cs[npr + 1] <= ch + 1) ++npr;
                    const int in_list = (ch + 1 - s.cs[npr]) * kPqChunk + tid;
                    if (in_list < s.list_len[npr]) nxt_pos = static_cast<long long>(s.list_begin[npr]) + in_list;
                    if (in_regs && nxt_pos >= 0) pq_fetch_code(nxt, p.codes + nxt_pos * p.pq_m, p.pq_m);
                }
                bool hit = false;
                uint64_t key = 0;
                if (pos >= 0) {
                    const float est = in_regs ? pq_adc_regs(lut_s, cur, p.pq_m)
                                              : pq_adc_code(s.lut, p.codes + pos * p.pq_m, p.pq_m);
                    key = (static_cast<uint64_t>(orderable(est)) << 32) | static_cast<uint32_t>(pos);
                    hit = key < bound;
                }
                const uint32_t bal = __ballot_sync(0xFFFFFFFFu, hit);
                if (bal) {
                    int base = 0;
                    if (lane == 0) base = atomicAdd(&s.misc[0], __popc(bal));
                    base = __shfl_sync(0xFFFFFFFFu, base, 0);
                    if (hit && IVF_IN_BOUNDS(411, base + __popc(bal & lt_mask), kPqScanBufKeys)) s.buf[base + __popc(bal & lt_mask)] = key;
                }
                pq_group_sync<BAR, NT>();
                const int count = s.misc[0];
                if (count > kPqScanBufKeys - kPqChunk)
                    bound = pq_cut_buffer<BAR, NT, kPqScanBufKeys>(s.buf, count, p.n_rerank, s.hist, s.misc, tid);
            }
        }
        pq_group_sync<BAR, NT>();
        int count = s.misc[0];
        if (count > p.n_rerank) {
            pq_cut_buffer<BAR, NT, kPqScanBufKeys>(s.buf, count, p.n_rerank, s.hist, s.misc, tid);
            count = p.n_rerank;
        }
        uint64_t* out = p.gcand + static_cast<size_t>(g) * p.n_rerank;
        for (int i = tid; i < count; i += NT)
            if (IVF_IN_BOUNDS(412, i, p.n_rerank)) out[i] = s.buf[i];
        if (tid == 0) p.gcand_count[g] = count;
    }
}

// One team per CTA, two CTAs per SM; the codebook is read through L1 from its transposed copy.
// Serves every shape (up to kPqMaxProbes probes) with little shared memory.
__global__ void __launch_bounds__(kPqScanThreads, 2) pq_scan_kernel(const PqScanParams p) {
    pdl_wait();
    pdl_trigger();
    extern __shared__ __align__(16) uint8_t pq_smem_raw[];
    if (static_cast<int64_t>(blockIdx.x) >= p.nq * p.ngroups) return;
    const PqTeamSmem s = pq_team_carve(pq_smem_raw, p.pq_m, kPqMaxProbes);
    pq_scan_groups<true, 0>(p, s, p.cbt, blockIdx.x, gridDim.x, threadIdx.x);
}

// Two teams per CTA, one CTA per SM: both teams read the codebook from one transposed copy in shared
// memory and otherwise work on different groups with their own table, buffer and barrier, so one
// team's table build (arithmetic) runs under the other's scan (shared-memory lookups).
__global__ void __launch_bounds__(2 * kPqScanThreads, 1) pq_scan_teams_kernel(const PqScanParams p) {
    pdl_wait();
    pdl_trigger();
    extern __shared__ __align__(16) uint8_t pq_smem_raw[];
    if (2 * static_cast<int64_t>(blockIdx.x) >= p.nq * p.ngroups) return;
    float* cbt = reinterpret_cast<float*>(pq_smem_raw);
    {   // straight copy of the codebook (d * 256 floats, 16-byte pieces)
        const float4* src = reinterpret_cast<const float4*>(p.cbt);
        float4* dst = reinterpret_cast<float4*>(cbt);
        for (int i = threadIdx.x; i < p.d * (kPqK / 4); i += blockDim.x) dst[i] = __ldg(src + i);
    }
    __syncthreads();
    uint8_t* teams = pq_smem_raw + static_cast<size_t>(p.d) * kPqK * 4;
    const int team = threadIdx.x / kPqScanThreads;
    const int tid = threadIdx.x - team * kPqScanThreads;
    const PqTeamSmem s = pq_team_carve(teams + team * pq_team_bytes(p.pq_m, kPqTeamProbes), p.pq_m, kPqTeamProbes);
    if (team == 0) pq_scan_groups<false, 1>(p, s, cbt, 2 * static_cast<int64_t>(blockIdx.x), 2 * static_cast<int64_t>(gridDim.x), tid);
    else pq_scan_groups<false, 2>(p, s, cbt, 2 * static_cast<int64_t>(blockIdx.x) + 1, 2 * static_cast<int64_t>(gridDim.x), tid);
}

// ------------------------------------------------------------------ group -> query merge
struct PqMergeParams {
    int64_t nq;
    int n_rerank;
    int ngroups;
    const uint64_t* gcand;
    const int* gcand_count;
    const long long* vec_ids;  // optional: position -> caller's identifier
    long long* out_pos;        // [nq][n_rerank]
    float* out_est;            // [nq][n_rerank]
};

// One CTA per query.  The n_rerank smallest of the query's group candidates are selected (in shared
// memory when they all fit, else by a radix select over the group outputs in place), sorted, and
// written in ascending (estimate, position) order.
// kRegs: the variant for group outputs of more than kPqBufKeys and at most 16 keys per thread, which
// holds them in registers during the selection (one CTA per SM); the other variant keeps two CTAs
// per SM for large batches.
constexpr int kPqMergeRegKeys = 16;
template <bool kRegs>
__global__ void __launch_bounds__(kPqThreads, kRegs ? 1 : 2) pq_merge_kernel(const PqMergeParams p) {
    pdl_wait();
    pdl_trigger();
    __shared__ uint64_t buf[kPqBufKeys];
    __shared__ int hist[256];
    __shared__ int misc[16];
    const int64_t b = blockIdx.x;
    const uint64_t* cand = p.gcand + static_cast<size_t>(b) * p.ngroups * p.n_rerank;
    const int* cnt = p.gcand_count + b * p.ngroups;
    const int slots = p.ngroups * p.n_rerank;
    auto get = [&](int i) {
        const int g = i / p.n_rerank;
        return (i - g * p.n_rerank) < cnt[g] ? __ldcg(cand + i) : ~0ull;
    };
    if (threadIdx.x == 0) misc[4] = 0;
    __syncthreads();
    int own = 0;
    for (int g = threadIdx.x; g < p.ngroups; g += blockDim.x) own += cnt[g];
    if (own) atomicAdd(&misc[4], own);
    __syncthreads();
    const int total = misc[4];
    if (threadIdx.x == 0) misc[0] = 0;
    __syncthreads();
    constexpr int kRegKeys = kPqMergeRegKeys;
    if constexpr (kRegs) {
        // every slot is read once into registers; selection and gathering work from there
        uint64_t mine[kRegKeys];
#pragma unroll
        for (int q = 0; q < kRegKeys; ++q) {
            const int i = threadIdx.x + q * kPqThreads;
            mine[q] = i < slots ? get(i) : ~0ull;
        }
        uint64_t bound = ~0ull;
        if (total > kPqBufKeys) {
            bound = pq_select_bound_regs<0, kPqThreads, kRegKeys>(mine, p.n_rerank, hist, misc, threadIdx.x);
            if (threadIdx.x == 0) misc[0] = 0;
            __syncthreads();
        }
#pragma unroll
        for (int q = 0; q < kRegKeys; ++q)
            if (mine[q] != ~0ull && mine[q] <= bound) {
                const int at = atomicAdd(&misc[0], 1);
                if (IVF_IN_BOUNDS(420, at, kPqBufKeys)) buf[at] = mine[q];
            }
    } else {
        uint64_t bound = ~0ull;
        if (total > kPqBufKeys) {
            bound = pq_select_bound<0, kPqThreads>(get, slots, p.n_rerank, hist, misc, threadIdx.x);
            if (threadIdx.x == 0) misc[0] = 0;
            __syncthreads();
        }
        for (int i = threadIdx.x; i < slots; i += blockDim.x) {
            const uint64_t v = get(i);
            if (v != ~0ull && v <= bound) {
                const int at = atomicAdd(&misc[0], 1);
                if (IVF_IN_BOUNDS(421, at, kPqBufKeys)) buf[at] = v;
            }
        }
    }
    __syncthreads();
    int count = misc[0];
    if (count > p.n_rerank) {
        __syncthreads();
        pq_cut_buffer<0, kPqThreads, kPqBufKeys>(buf, count, p.n_rerank, hist, misc, threadIdx.x);
        count = p.n_rerank;
    }
    int m = 2;
    while (m < count) m <<= 1;
    for (int i = count + threadIdx.x; i < m; i += blockDim.x) buf[i] = ~0ull;
    // bitonic sort of buf[0 .. m)
    for (int size = 2; size <= m; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = threadIdx.x; t < (m >> 1); t += blockDim.x) {
                const int lo = 2 * t - (t & (stride - 1));
                const int hi = lo + stride;
                const bool up = (lo & size) == 0;
                const uint64_t a = buf[lo], c = buf[hi];
                if ((a > c) == up) {
                    buf[lo] = c;
                    buf[hi] = a;
                }
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < p.n_rerank; i += blockDim.x) {
        long long pos = -1;
        float est = __int_as_float(0x7f800000);
        if (i < count) {
            const uint64_t key = buf[i];
            pos = static_cast<long long>(key & 0xFFFFFFFFull);
            (void)IVF_IN_BOUNDS(422, i, kPqBufKeys);
            if (p.vec_ids) pos = p.vec_ids[pos];
            est = from_orderable(static_cast<uint32_t>(key >> 32));
        }
        p.out_pos[b * p.n_rerank + i] = pos;
        p.out_est[b * p.n_rerank + i] = est;
    }
}

}  // namespace ivf
