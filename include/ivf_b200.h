/*
 * ivf_b200 -- C-ABI of the B200 (sm_100a) IVF coarse-routing / assignment / Lloyd-update library.
 *
 * The one computation behind every call is the batched squared-L2 distance from each row of a
 * point matrix to every centroid, with the k smallest per row kept on the device:
 *   - coarse search (Eq. 1): the P nearest lists of each query, P = nprobe;
 *   - distances come from inner products and precomputed norms,
 *     |x-c|^2 = |x|^2 + |c|^2 - 2 x.c  (Sec. 4.1, Eq. 6), as a dense tensor-core contraction;
 *   - only ids and optional distances, O(B*P), leave the kernel (Sec. 4.1, on-device list
 *     selection); the B x N_list distance matrix is never written to memory;
 *   - index construction assigns every vector to its nearest centroid (Sec. 3.1, Sec. 5.5) -- the
 *     k = 1 case -- and Lloyd iterations recompute each centroid as the mean of its members.
 *
 * Conventions shared by all calls
 *   Layout     every matrix is dense row-major with contiguous rows (leading dimension = d).
 *   Pointers   "device" = memory of the current CUDA device; "host" = page-locked host memory.
 *              The caller owns every buffer; the library keeps none past stream completion.  All work is
 *              asynchronous: a buffer (host buffers above all) must stay allocated and unchanged until
 *              the work the call enqueued has completed.
 *   Streams    work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = legacy default
 *              stream) and the call returns without waiting, except where stated.
 *   Workspace  the library keeps one grow-only device workspace per device; it grows with a
 *              stream-ordered allocation on `stream`.  Calls that share a device must therefore be
 *              issued in stream order with respect to each other (one stream, or streams the
 *              caller has ordered with events).
 *   Graphs     a call whose buffers are all device memory enqueues only kernels and memsets once the
 *              workspace has been sized by an earlier call of the same shape, so it may be captured
 *              in a CUDA graph by the caller (tested for ivf_assign and ivf_route_prepared); calls
 *              with page-locked host buffers wait on internal events and are not meant for capture.
 *   Errors     every call returns IVF_OK or a negative ivf_status.  Argument errors are detected
 *              before anything is enqueued.  Device-side problems (a bounded wait that expired, an
 *              id out of range) set a sticky per-device status word that ivf_check reads.
 *   Limits     d must be a multiple of 4, 4 <= d <= 256 (d = 100 is padded to the next multiple of 16 inside the operand copies;
 *              uint8 rows with d a multiple of 16 take the fastest path: no fp16 copy in HBM).  1 <= nprobe <= min(nlist, 512).
 *              Float inputs are scaled by an exact power of two (exponent clamped to +-40) before they are
 *              rounded to fp16: finite values with magnitude between about 1e-12 and 1e12 keep the stated
 *              tolerance (tested); beyond 2^51 the operands overflow and the results are undefined,
 *              as they are for non-finite inputs (always memory-safe).  The scale is one power of
 *              two per matrix, taken from its largest magnitude M: inside one matrix the tolerance
 *              1e-3 (|x|^2 + |c|^2) holds for every pair whose combined norm sqrt(|x|^2 + |c|^2) is at
 *              least about 2^-9 M_centroids (tested down to 2^-7); for a pair of rows both far
 *              smaller than that, next to much larger rows in the same matrices, the norm term
 *              falls below fp16's smallest step and the error bound becomes the absolute
 *              2^-30 M_centroids^2 instead.
 *              nlist < 2^31.  n == 0 is IVF_OK and enqueues nothing.
 *   Non-finite inputs give unspecified (but memory-safe) results.
 *
 * The problem statement gives neither the element type of the points nor d for the update; both are
 * needed, so the signatures below carry `ptype` and `d` in addition.
 */
#ifndef IVF_B200_H
#define IVF_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { IVF_F32 = 0, IVF_U8 = 1, IVF_I8 = 2 } ivf_dtype;  /* IVF_I8: signed bytes (SPACEV-shaped data, Table 2) */

typedef enum {
    IVF_OK = 0,
    IVF_ERR_INVALID_ARG = -1,    /* null pointer, negative size, pageable host memory ...        */
    IVF_ERR_UNSUPPORTED = -2,    /* d, nprobe or nlist outside the limits above                   */
    IVF_ERR_ALLOC = -3,          /* workspace allocation failed                                   */
    IVF_ERR_CUDA = -4,           /* a CUDA runtime/driver call failed (see ivf_last_error)        */
    IVF_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait expired; results are invalid       */
    IVF_ERR_BAD_ID = -6,         /* ivf_centroid_update met an id outside [0, nlist); row skipped */
    IVF_ERR_BOUNDS = -7          /* checked build only: an index check inside a kernel failed     */
} ivf_status;

/*
 * Coarse routing (Eq. 1; Sec. 4.1 dense centroid evaluation + on-device list selection).
 *   queries    [nq, d] float32 or uint8 (qtype); device, or page-locked host (then the rows are
 *              streamed through the device in chunks, the copies overlapping the kernels)
 *   centroids  [nlist, d] float32, device
 *   out_ids    [nq, nprobe] int32, device: the nprobe nearest centroids of every query, ascending
 *              by (distance, id) -- equal distances are ordered by the lower id
 *   out_dists  [nq, nprobe] float32 squared L2 distances (clamped at 0), device; may be NULL
 * Results in host memory (Sec. 4.1: what leaves the GPU is the O(B * P) list of selected lists, which
 * the CPU-side search consumes): out_ids and out_dists may instead both be page-locked host memory.
 * The kernels then write to staging buffers of the workspace and every row chunk is copied to the
 * host on a stream of the library's own, under the next chunk's kernels; before the call returns it
 * makes `stream` wait for the last copy, so in `stream` the call is complete when its results are in
 * host memory -- ordinary stream semantics.  The same holds for ivf_route_prepared, ivf_assign and
 * ivf_assign_update.  Pageable host memory -> IVF_ERR_INVALID_ARG.
 */
int ivf_route(const void* queries, int64_t nq, int d, ivf_dtype qtype,
              const float* centroids, int nlist, int nprobe,
              int32_t* out_ids, float* out_dists, void* stream);

/*
 * Deferred read-back, for a serving loop that routes batch i + 1 while batch i's results travel to
 * the host.  ivf_set_deferred_host_outputs(1) (per device; default 0): calls with host outputs no
 * longer make `stream` wait for their read-back, so the next call's kernels start at once (two
 * staging buffer pairs are used in turn; a pair is reused only after its read-back).  Read-backs
 * finish in the order of the calls.  The host buffers of a call may be read after
 * ivf_wait_host_outputs(stream) -- it makes `stream` wait for every read-back issued so far on the
 * current device -- followed by whatever the caller uses to wait for `stream`, or after
 * ivf_check(stream), which waits for them on the host.
 */
int ivf_set_deferred_host_outputs(int on);
int ivf_wait_host_outputs(void* stream);

/*
 * Routing against a centroid table that stays resident on the device (Sec. 3.1 / 4.1: the centroid
 * matrix is GPU-resident routing state; only the query batch changes per call).  ivf_route prepares
 * the tensor-core copy of the centroids on every call, which is right while they change (Lloyd
 * iterations) and wasteful when they do not (serving).  ivf_centroids_create does that preparation
 * once -- it enqueues its work on `stream` and allocates the prepared copy (nlist * (d rounded up
 * to 64, + 16) * 2 bytes) stream-ordered; the float32 `centroids` may be freed after that work is
 * done.  ivf_route_prepared is ivf_route without the centroid preparation; outputs are identical.
 * A handle belongs to the device that was current at creation and must be used by one stream at a
 * time (every call updates per-batch scale factors stored with it).  ivf_centroids_destroy frees it
 * stream-ordered.
 */
typedef struct ivf_centroids ivf_centroids;
int ivf_centroids_create(const float* centroids, int nlist, int d, ivf_centroids** out, void* stream);
int ivf_centroids_destroy(ivf_centroids* handle, void* stream);
int ivf_route_prepared(const ivf_centroids* handle, const void* queries, int64_t nq, ivf_dtype qtype,
                       int nprobe, int32_t* out_ids, float* out_dists, void* stream);

/*
 * Assignment to the nearest centroid (Sec. 3.1 index layout; Sec. 5.5 full-mode construction).
 * Same as ivf_route with nprobe = 1: out_ids [n] int32, out_dists [n] float32 (may be NULL).
 * `points` may be device or page-locked host memory as for ivf_route.
 */
int ivf_assign(const void* points, int64_t n, int d, ivf_dtype ptype,
               const float* centroids, int nlist,
               int32_t* out_ids, float* out_dists, void* stream);

/*
 * Lloyd accumulation (Sec. 5.5, "Lloyd iterations"):
 *   sums[l, :] += sum of the rows i with ids[i] == l      [nlist, d] float32, device
 *   counts[l]  += number of such rows                     [nlist]    int64,   device
 * ACCUMULATES into sums/counts so that chunks of one iteration compose; the caller zeroes them
 * at the start of an iteration.  points [n, d] (ptype) and ids [n] int32 are device pointers.
 * A row whose id is outside [0, nlist) is skipped and flags IVF_ERR_BAD_ID in the status word.
 * For uint8 and int8 points the sums are exact while every list sum stays below 2^24, hence
 * bit-identical from run to run, like the counts.  Float points are added in an order that depends
 * on scheduling: their sums are reproducible only up to the rounding of a different summation order
 * (within 1e-5 of the sum of the members' magnitudes).
 */
int ivf_centroid_update(const void* points, ivf_dtype ptype, const int32_t* ids, int64_t n, int d,
                        int nlist, float* sums, int64_t* counts, void* stream);

/*
 * The same accumulation for callers that must not allocate device memory when they call.
 * (This entry point has no counterpart in the paper; it exists for how the library is deployed.)
 * Think of an index-maintenance thread living beside a serving process that has already handed all
 * free device memory to its own pool, where a cudaMalloc would fail or stall; or of a latency-bound
 * loop that cannot afford the device-wide synchronisation a cudaMalloc or cudaFree implies.
 * ivf_centroid_update grows the library workspace on demand; this variant never does.  It calls no
 * cudaMalloc, cudaFree or other allocating routine: its scratch (list counts, offsets, cursors and
 * the row permutation) is a fixed array of about 4.8 MB inside the library image, which every
 * device that loads the library holds until the process exits.
 *   Limits   n <= 1,048,576 rows and nlist <= 65,536 lists per call; anything larger returns
 *            IVF_ERR_UNSUPPORTED with a message (split the rows over several calls: the
 *            accumulation composes).  Other arguments, layouts and results are those of
 *            ivf_centroid_update.
 *   Set-up   the first call on each device looks up the array's device address (with that device
 *            current); make that first call before starting any stream capture.  The array is part
 *            of the library image, and the CUDA runtime places an image on a device when the
 *            library is first used there: so make that first call (or any other call into the
 *            library) on each device before the device's free memory is handed to the serving
 *            pool -- afterwards there may be no room left for the image itself.
 *   Sharing  all calls on a device use the one array, which still holds the previous call's
 *            contents (the call clears what it needs cleared).  Two calls whose kernels overlap on
 *            the GPU -- different streams without an ordering between them -- race on it: keep the
 *            calls of a device in one stream or order them with events.
 *   Bad ids  rows whose id is outside [0, nlist) are skipped; this variant does not report them
 *            through ivf_check.
 */
int ivf_centroid_update_noalloc(const void* points, ivf_dtype ptype, const int32_t* ids, int64_t n, int d,
                                int nlist, float* sums, int64_t* counts, void* stream);

/*
 * Helper: new centroid = sums / counts per list (float32 divide); a list with count 0 keeps its
 * row of centroids_inout (the paper does not say what an empty list does).  All device pointers.
 */
int ivf_centroid_finalize(const float* sums, const int64_t* counts, int nlist, int d,
                          float* centroids_inout, void* stream);

/*
 * Cluster-major layout (Sec. 3.1 index layout: the vectors of a list are stored contiguously, with
 * per-list offset, length and ids), the step right after the final assignment of an index build.
 *   points       [n, d] (ptype), ids [n] int32: device
 *   out_offsets  [nlist + 1] int64, device: list l occupies rows [out_offsets[l], out_offsets[l+1])
 *   out_order    [n] int32, device: out_order[p] = source row stored at position p
 *   out_points   [n, d] (ptype), device: row p = points[out_order[p]]
 * The order of the rows inside a list is unspecified (every order is a valid layout; out_order tells
 * which one was taken).  A row whose id is outside [0, nlist) is dropped from the layout and flags
 * IVF_ERR_BAD_ID in the status word: the kept rows fill positions [0, out_offsets[nlist]); the
 * positions after them get out_order = -1 and an all-zero row in out_points.  At most 2^31 - 1 rows
 * per call.
 */
int ivf_cluster_major_reorder(const void* points, ivf_dtype ptype, const int32_t* ids, int64_t n, int d,
                              int nlist, void* out_points, int64_t* out_offsets, int32_t* out_order,
                              void* stream);

/*
 * Helper: one pass of a Lloyd iteration over a point set that may exceed device memory
 * (Table 3: assignment in batches of 1,048,576 vectors; Table 1: the host link is the scarce
 * resource).  For each chunk of `chunk_rows` rows: copy to the device if `points` is page-locked
 * host memory (double-buffered on an internal copy stream), assign (k = 1), accumulate
 * sums/counts.  Each chunk crosses the host link once.  out_ids [n] int32 and out_dists [n]
 * float32 are device pointers and may be NULL.  chunk_rows <= 0 selects 1,048,576.
 */
int ivf_assign_update(const void* points, int64_t n, int d, ivf_dtype ptype,
                      const float* centroids, int nlist,
                      int32_t* out_ids, float* out_dists,
                      float* sums, int64_t* counts, int64_t chunk_rows, void* stream);

/* Synchronises `stream`, then returns and clears the sticky device status of the current device. */
int ivf_check(void* stream);

/* Message of the last error returned on this host thread ("" if none). */
const char* ivf_last_error(void);

/* Frees the current device's workspace (after synchronising the device). */
int ivf_release_workspace(void);

/* Number of kernels this library has launched on this host process so far (all devices). */
int64_t ivf_launch_count(void);

/*
 * Test hooks (host logic only; no kernel is launched).
 *   ivf_debug_plan   the persistent schedule of the fused kernel for a problem size on a device
 *                    with `num_sms` SMs: writes {row_groups, col_tiles, ctas, max_partials_per_row,
 *                    block_n, k_slices, stages, smem_bytes, row tiles of 128 points per row group}
 *                    to out[9].
 *   ivf_debug_span   out[0], out[1]: first unit and one-past-last unit of CTA `cta` in that schedule;
 *                    out[2], out[3]: the CTA that the kernels' unit-to-CTA mapping gives for the first and
 *                    the last unit of the span (both must equal `cta`).
 *   ivf_debug_set_wait_limit_ns   time limit of every device-side wait (0 restores the default
 *                    of 2 s).
 *   ivf_debug_wait_probe   launches a one-warp kernel that waits, with the library's bounded wait,
 *                    on a barrier nothing ever completes: after the limit it records
 *                    IVF_ERR_DEVICE_TIMEOUT (wait site 99) in the status word and returns normally.
 */
int ivf_debug_plan(int64_t n, int nlist, int d, int k, int num_sms, int64_t out[9]);
int ivf_debug_span(int64_t n, int nlist, int d, int k, int num_sms, int cta, int64_t out[4]);
/* Test hook (host only): the rotation of row group `row_group` in that schedule -- position p of the
 * row group's sweep stands for centroid tile (p + rotation) mod col_tiles, so that the CTAs walk the
 * centroid table as a few shared fronts.  Returns the rotation (>= 0) or a negative status. */
int ivf_debug_rotation(int64_t n, int nlist, int d, int k, int num_sms, int64_t row_group);
/* Measurement hook: 0 switches the rotation off (every position stands for its own tile index), so that
 * the two sweep orders can be timed against each other; results do not depend on it.  Default 1. */
int ivf_debug_set_rotation(int on);
/* Measurement / test hook: 1 makes the threshold pass of k > 16 calls always run as sketch kernel plus
 * merge launch; 0 (default) lets batches of at least 48 row tiles finish their thresholds inside the
 * sketch kernel, and batches of at most 16 rows (32 against tables of at least 4 x 256 centroids per
 * SM) inside the main pass (its epilogue warps merge the partial sketches while the first tiles are
 * computed).  All three give the same thresholds, hence
 * the same results. */
int ivf_debug_set_threshold_pass(int split);
int ivf_debug_set_wait_limit_ns(int64_t ns);
int ivf_debug_wait_probe(void* stream);
/* Test hook: the next `count` workspace allocations are refused (the call returns IVF_ERR_ALLOC
 * before anything is freed or launched for that allocation); 0 switches the hook off. */
int ivf_debug_fail_next_alloc(int count);
/* 1 if this library was built with -DIVF_CHECK_BOUNDS (every kernel checks its shared-memory,
 * tensor-memory and global indices, records the first violation as IVF_ERR_BOUNDS with a site number
 * in the status word and skips the access -- a stand-in for a memory checker), else 0. */
int ivf_debug_bounds_checked(void);
/* Launches a one-thread kernel that evaluates one failing index check (index 5 against limit 3, site
 * 999) and touches no memory: in the checked build ivf_check then reports IVF_ERR_BOUNDS, in the
 * regular build nothing happens. */
int ivf_debug_bounds_probe(void* stream);
/* Test hook: when on, the merge of a k > 1 call declares every row's candidate set insufficient, so
 * that all rows take the exact brute-force recomputation that normally only catches rare rows. */
int ivf_debug_force_fallback(int on);
/* Test hook: rows per fused-kernel launch (0 restores the size derived from the scratch budget), so
 * that the row-chunk loop of large calls can be exercised on small inputs. */
int ivf_debug_set_row_chunk(int64_t rows);
/* Test hook (host only): which threshold rule a call with this nprobe and nlist uses -- out[0] =
 * -1 (k = 1: argmin), 0 running (k <= 16), 1 given (threshold pass over every out[1]-th centroid),
 * 2 bounded (sample too small). */
int ivf_debug_rule(int k, int nlist, int out[2]);

/*
 * Measurement hooks.  ivf_debug_timing(1) makes every later call bracket its kernels with CUDA
 * events on the caller's stream, grouped into nine families: 0 operand preparation (norms,
 * fp16 copies), 1 fused distance+argmin (k = 1), 2 fused distance+top-k (k > 1), 3 merge of
 * partial results (and the brute-force recomputation of failed rows), 4 centroid update,
 * 5 threshold pass of k > 16 calls (fused kernel over the centroid sample + its merge), 6 PQ encoding, 7 PQ set-up + scan, 8 PQ group merge.  ivf_debug_timing_read synchronises the device, writes the
 * summed milliseconds and launch-group counts of each family since the last read, and clears
 * them.  ivf_debug_timing(0) switches the events off (the default).
 */
/*
 * ivf_debug_stats synchronises the device, writes three counters accumulated by k > 1 calls since
 * the last read to out[3] (may be NULL) -- in-kernel log selections, candidate-log entries left for
 * the merge, rows recomputed by brute force -- clears them, and switches the counting on or off.
 */
int ivf_debug_stats(int enable, int64_t out[3]);
/* Test hook: groups per query used by ivf_pq_search (clamped to [1, 256]); 0 = chosen from the sizes.
 * A negative value -(g + 1) asks for g groups and for the scan kernel variant that reads the codebook
 * through L1 (otherwise the two-team shared-memory variant is used whenever it fits). */
int ivf_debug_set_pq_groups(int groups);
/* Test hook: the cost, in units of one (row group, centroid tile) step, that the persistent schedule
 * charges a CTA for changing row group in the middle of its span (0 = equal unit counts; negative =
 * the default: 8 for the k = 1 kernel, 4 otherwise). */
int ivf_debug_set_crossing_cost(int units);
/* Test hook: mask of the kernel families of the routing path that may start while their predecessor
 * drains (programmatic dependent launch): 1 operand preparation, 2 fused kernel, 4 threshold merge,
 * 8 merge, 16 tail kernel (passed-on rows and recomputation; bit 32 is unused), 64 centroid update,
 * 128 residual-PQ search.  0 = ordinary stream launches; default 251. */
int ivf_debug_set_dependent_launch(int mask);
int ivf_debug_timing(int enable);
int ivf_debug_timing_read(double ms[9], int64_t launches[9]);

/*
 * Assignment within given candidates (appendix on fast index building; Table 3 lists 8 and 2
 * candidate centroids per vector).  cand_ids [n][m] int32 (device) holds m candidate centroid ids
 * per row, produced by whatever search the caller runs (the paper uses a graph over the centroid
 * table, which is not part of this library); repeats are allowed.  out_ids[i] = the candidate with
 * the smallest squared L2 distance to row i (ties to the lower id), out_dists[i] (may be NULL) that
 * distance, computed in fp32 from the differences (no norm expansion).  All pointers are device
 * pointers; points and centroids 16-byte aligned; d a multiple of 4, at most 256.  A candidate id
 * outside [0, nlist) is skipped and sets the sticky status IVF_ERR_BAD_ID (a row whose candidates
 * are all invalid gets id -1 and +inf).
 */
int ivf_assign_candidates(const void* points, int64_t n, int d, ivf_dtype ptype, const float* centroids, int nlist,
                          const int32_t* cand_ids, int m, int32_t* out_ids, float* out_dists, void* stream);

/*
 * Merge step of routing against a centroid table that is split over several GPUs (Sec. 4.1: finer
 * partitions, N_list up to millions; Eq. 1: the P nearest centroids overall are the P smallest of
 * the shards' P nearest).  Every GPU routes the queries against its own shard with ivf_route and
 * adds its shard's first global id to the ids; the [nq, k] results of all shards are gathered
 * (an all-gather) into
 *   shard_ids    [parts][nq][k] int32, shard_dists [parts][nq][k] float32: device; each list
 *                ascending by (distance, id); a shard with fewer than k centroids fills the unused
 *                places with +inf;
 * and this call writes the k smallest pairs by (distance, id) per query, ascending, to
 *   out_ids [nq][k] int32, out_dists [nq][k] float32 (may be NULL): device.
 * k <= 512; any number of parts.  Equal distances are settled by the lower global id.
 */
int ivf_merge_shards(const int32_t* shard_ids, const float* shard_dists, int parts, int64_t nq, int k,
                     int32_t* out_ids, float* out_dists, void* stream);

/*
 * Residual-PQ candidate reduction (Sec. 2.2 Eq. 3-5; Sec. 4.3; Sec. 4.4).  K = 256 codewords per
 * subspace, one byte per sub-code, fp32 lookup tables (the paper's setting).  All pointers are
 * DEVICE pointers owned by the caller; calls enqueue on `stream` and return.
 *
 * Arithmetic (fp32, every operation rounded once, in this order, so codes and kept candidates are
 * reproducible bit for bit):
 *     r_t = float(x_t) - c_t;   LUT_m[j]: acc = 0, for t ascending: diff = r_t - p_m[j][t],
 *     acc = fma(diff, diff, acc);   estimate: acc = 0, for m ascending: acc = acc + LUT_m[a_m].
 *
 * codebooks  [pq_m][256][d / pq_m] float32, row-major.  pq_m must divide d.  Encoding keeps the
 *            codebook in shared memory: 1024 * (d + pq_m) + 4 * d bytes (and 1024 * d + 8,704)
 *            must fit one SM's 227 KB (d = 128 with pq_m = 32 does; d = 256 does not); searching needs
 *            1024 * pq_m + 21,584 bytes and d <= 256 -> IVF_ERR_UNSUPPORTED otherwise.
 *
 * ivf_pq_encode: out_codes[i][m] = arg-min over j of the table of x_i - centroids[ids[i]]
 *            (Eq. 3 on the residual; ties to the lower j).  An id outside [0, nlist) writes zero
 *            codes for that row and sets the sticky status IVF_ERR_BAD_ID.
 *
 * ivf_pq_search: for every query the codes of its nprobe (<= 512) probed lists (list l = positions
 *            [list_offsets[l], list_offsets[l+1]) of the list-major `codes` array, n_codes rows in
 *            all, n_codes < 2^32) are scored with the (query, list) table (Eq. 4 on q - c_l, Eq. 5) and
 *            the n_rerank (<= 1024) smallest estimates are kept: out_ids [nq][n_rerank] = position
 *            (or vec_ids[position] when vec_ids is given), out_est [nq][n_rerank] ascending by
 *            (estimate, position); unused slots hold -1 and +inf.  out_counts [nq] (may be NULL) =
 *            codes scanned for the query.  A list must not appear twice among a query's probes;
 *            probe ids outside [0, nlist) are skipped and set IVF_ERR_BAD_ID.  `codes` must be
 *            16-byte aligned.  Chunk and group descriptors are built on the device (no host
 *            synchronisation); the workspace is the library's grow-only one.
 */
/* out_residuals[i][t] = float(points[i][t]) - centroids[ids[i]][t] (fp32 [n][d], device): the vectors
 * the PQ codebooks are trained on (Sec. 4.3).  Training itself is k-means per subspace and is composed
 * from ivf_assign_update / ivf_centroid_finalize on the sub-vector columns (256 lists, d / pq_m wide).
 * An id outside [0, nlist) gives a zero row and sets IVF_ERR_BAD_ID. */
int ivf_pq_residuals(const void* points, int64_t n, int d, ivf_dtype ptype, const int32_t* ids,
                     const float* centroids, int nlist, float* out_residuals, void* stream);
int ivf_pq_encode(const void* points, int64_t n, int d, ivf_dtype ptype, const int32_t* ids,
                  const float* centroids, int nlist, const float* codebooks, int pq_m,
                  uint8_t* out_codes, void* stream);
int ivf_pq_search(const void* queries, int64_t nq, int d, ivf_dtype qtype, const float* centroids, int nlist,
                  const int32_t* probe_ids, int nprobe, const int64_t* list_offsets, const uint8_t* codes,
                  int64_t n_codes, const float* codebooks, int pq_m, int n_rerank, const int64_t* vec_ids,
                  int64_t* out_ids, float* out_est, int64_t* out_counts, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* IVF_B200_H */
