/*
 * CPU oracle for the IVF coarse-routing / assignment / Lloyd-update path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition of what the GPU
 * library must compute.  It shares no code, header, table or helper with the CUDA
 * path and must never be called from it.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may load it.
 *
 * Everything is fp64, written from the definitions:
 *   - coarse search (Eq. 1): the P-subset of lists minimising the summed distance to
 *     the query, i.e. the P nearest centroids;
 *   - the distance is squared L2.  Sec. 4.1 (Eq. 6, the norm expansion) writes it as
 *     |q|^2 + |c|^2 - 2 q.c, an algebraic identity; the oracle deliberately uses the
 *     direct difference form sum_t (x_t - c_t)^2 instead;
 *   - selection is a full sort on (distance, id), ties broken by the lower id;
 *   - assignment is the k = 1 case (index layout, Sec. 3.1: each vector goes to its
 *     nearest centroid);
 *   - the Lloyd update is the naive per-list sum and count, then the mean
 *     (Sec. 5.5 "Lloyd iterations"; the paper gives no formula beyond citing Lloyd).
 *
 * Readings where the paper is silent: outputs are squared distances in ascending
 * (distance, id) order; an empty list keeps its previous centroid; the update
 * accumulates into sums/counts so that chunks compose.
 *
 * Pins (tests/test_oracle_pins.py): hand-computed tiny cases, one-hot closed form,
 * unit-norm identity, scipy cdist, brute force over all k-subsets, lexsort,
 * permutation / translation / scaling invariants, bincount cross-check, Lloyd
 * monotonicity and toy clusters, numpy stable argsort for the reorder; the candidate-restricted
 * assignment against the full assignment, numpy arg-min over the gathered rows and a hand case.
 * No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_U8 = 1, ORACLE_I8 = 2 };

typedef struct {
    double dist;
    int32_t id;
} pair_t;

static int pair_cmp(const void *pa, const void *pb) {
    const pair_t *a = (const pair_t *)pa, *b = (const pair_t *)pb;
    if (a->dist < b->dist) return -1;
    if (a->dist > b->dist) return 1;
    return (a->id > b->id) - (a->id < b->id);
}

static inline double elem(const void *x, int xtype, int64_t idx) {
    if (xtype == ORACLE_U8) return (double)((const uint8_t *)x)[idx];
    if (xtype == ORACLE_I8) return (double)((const int8_t *)x)[idx];
    return (double)((const float *)x)[idx];
}

/* squared L2 distance between row i of x and row j of c, direct difference form */
static double sqdist(const void *x, int xtype, int64_t i, const float *c, int64_t j, int d) {
    double s = 0.0;
    for (int t = 0; t < d; ++t) {
        double diff = elem(x, xtype, i * d + t) - (double)c[j * d + t];
        s += diff * diff;
    }
    return s;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Coarse routing (Eq. 1 with squared L2).  For every row: all nlist distances, a full
 * sort on (distance, id), the first k emitted.
 *   out_ids   [n*k] int32, out_dists [n*k] double, ascending (distance, id)
 *   out_next  [n]   double, the (k+1)-th smallest distance (+inf when k == nlist); may be NULL
 * Returns 0, or -1 on bad arguments / allocation failure.
 */
int oracle_route(const void *x, int xtype, int64_t n, int d, const float *c, int32_t nlist, int32_t k,
                 int32_t *out_ids, double *out_dists, double *out_next) {
    if (n < 0 || d <= 0 || nlist <= 0 || k <= 0 || k > nlist) return -1;
    int failed = 0;
#pragma omp parallel
    {
        pair_t *buf = (pair_t *)malloc(sizeof(pair_t) * (size_t)nlist);
        if (!buf) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t i = 0; i < n; ++i) {
            if (!buf) continue;
            for (int32_t j = 0; j < nlist; ++j) {
                buf[j].dist = sqdist(x, xtype, i, c, j, d);
                buf[j].id = j;
            }
            qsort(buf, (size_t)nlist, sizeof(pair_t), pair_cmp);
            for (int32_t p = 0; p < k; ++p) {
                out_ids[i * k + p] = buf[p].id;
                out_dists[i * k + p] = buf[p].dist;
            }
            if (out_next) out_next[i] = (k < nlist) ? buf[k].dist : INFINITY;
        }
        free(buf);
    }
    return failed ? -1 : 0;
}

/* Assignment: the nearest centroid of every row (k = 1 case of the routing). */
int oracle_assign(const void *x, int xtype, int64_t n, int d, const float *c, int32_t nlist,
                  int32_t *out_ids, double *out_dists) {
    return oracle_route(x, xtype, n, d, c, nlist, 1, out_ids, out_dists, NULL);
}

/* Distances of given (row, centroid) pairs: out[p] = |x_row[p] - c_col[p]|^2. */
int oracle_pair_dists(const void *x, int xtype, int d, const float *c, int64_t npairs,
                      const int64_t *rows, const int32_t *cols, double *out) {
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < npairs; ++p) out[p] = sqdist(x, xtype, rows[p], c, cols[p], d);
    return 0;
}

/* Squared norms of rows in fp64 (used by the tolerance 1e-3 * (|x|^2 + |c|^2)). */
int oracle_sqnorms(const void *x, int xtype, int64_t n, int d, double *out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double s = 0.0;
        for (int t = 0; t < d; ++t) {
            double v = elem(x, xtype, i * d + t);
            s += v * v;
        }
        out[i] = s;
    }
    return 0;
}

/*
 * Naive Lloyd accumulation, serial, in row order:
 *   sums[l, :] += x_i  and  counts[l] += 1  for every row i with ids[i] == l.
 * Accumulates into the caller's arrays.  Returns -1 if an id is out of range
 * (nothing is written for that row).
 */
int oracle_update(const void *x, int xtype, const int32_t *ids, int64_t n, int d, int32_t nlist,
                  double *sums, int64_t *counts) {
    int bad = 0;
    for (int64_t i = 0; i < n; ++i) {
        int32_t l = ids[i];
        if (l < 0 || l >= nlist) {
            bad = 1;
            continue;
        }
        for (int t = 0; t < d; ++t) sums[(int64_t)l * d + t] += elem(x, xtype, i * d + t);
        counts[l] += 1;
    }
    return bad ? -1 : 0;
}

/*
 * Cluster-major layout (Sec. 3.1 index layout: the vectors of one list are stored contiguously,
 * with per-list offset / length / ids).  Stable counting sort written out:
 *   offsets[l]  = number of rows whose id is smaller than l          (offsets[nlist] = n)
 *   order[p]    = source row stored at position p; within a list the rows keep their input order
 * Returns -1 if an id is out of range.
 */
int oracle_reorder(const int32_t *ids, int64_t n, int32_t nlist, int64_t *offsets, int64_t *order) {
    for (int32_t l = 0; l <= nlist; ++l) offsets[l] = 0;
    for (int64_t i = 0; i < n; ++i) {
        if (ids[i] < 0 || ids[i] >= nlist) return -1;
        offsets[ids[i] + 1] += 1;
    }
    for (int32_t l = 0; l < nlist; ++l) offsets[l + 1] += offsets[l];
    int64_t *cursor = (int64_t *)malloc(sizeof(int64_t) * (size_t)(nlist > 0 ? nlist : 1));
    if (!cursor) return -1;
    for (int32_t l = 0; l < nlist; ++l) cursor[l] = offsets[l];
    for (int64_t i = 0; i < n; ++i) order[cursor[ids[i]]++] = i;
    free(cursor);
    return 0;
}

/* Mean per list, rounded once to float; an empty list keeps its previous centroid. */
int oracle_finalize(const double *sums, const int64_t *counts, int32_t nlist, int d, float *centroids) {
    for (int32_t l = 0; l < nlist; ++l) {
        if (counts[l] == 0) continue;
        for (int t = 0; t < d; ++t)
            centroids[(int64_t)l * d + t] = (float)(sums[(int64_t)l * d + t] / (double)counts[l]);
    }
    return 0;
}

/*
 * Lloyd's algorithm.  centroids [nlist*d] holds the initial centroids on entry (the caller
 * picks the seeded sample of input rows) and the final ones on exit.  Each iteration:
 * assign every row, accumulate, finalize.  inertia[it] = sum_i |x_i - c_assign(i)|^2
 * measured with the centroids that iteration started from; ids [n] are the last
 * iteration's assignments.
 */
int oracle_lloyd(const void *x, int xtype, int64_t n, int d, int32_t nlist, int iters,
                 float *centroids, int32_t *ids, double *inertia) {
    double *dist = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    double *sums = (double *)malloc(sizeof(double) * (size_t)nlist * d);
    int64_t *counts = (int64_t *)malloc(sizeof(int64_t) * (size_t)nlist);
    if (!dist || !sums || !counts) {
        free(dist); free(sums); free(counts);
        return -1;
    }
    int rc = 0;
    for (int it = 0; it < iters && rc == 0; ++it) {
        rc = oracle_assign(x, xtype, n, d, centroids, nlist, ids, dist);
        if (rc) break;
        double tot = 0.0;
        for (int64_t i = 0; i < n; ++i) tot += dist[i];
        inertia[it] = tot;
        memset(sums, 0, sizeof(double) * (size_t)nlist * d);
        memset(counts, 0, sizeof(int64_t) * (size_t)nlist);
        rc = oracle_update(x, xtype, ids, n, d, nlist, sums, counts);
        if (rc) break;
        oracle_finalize(sums, counts, nlist, d, centroids);
    }
    free(dist); free(sums); free(counts);
    return rc;
}

/*
 * Assignment within given candidates (Appendix "Fast index building": a graph search proposes a
 * small candidate-centroid set per vector -- 8 in the fast mode, 2 in the ultra-fast one, Table 3 --
 * and the exact distance is evaluated within that set only).  The candidate generator is not part
 * of this path; candidates are an input.
 *   cand [n*m] int32: m candidate centroid ids per row (repeats allowed; every id must be in range)
 *   out_ids [n], out_dists [n]: the candidate with the smallest squared L2 distance, ties to the
 *   lower centroid id.
 * Returns -1 on bad arguments or an id out of range.
 */
int oracle_assign_candidates(const void *x, int xtype, int64_t n, int d, const float *c, int32_t nlist,
                             const int32_t *cand, int m, int32_t *out_ids, double *out_dists) {
    if (n < 0 || d <= 0 || nlist <= 0 || m <= 0) return -1;
    for (int64_t i = 0; i < n * m; ++i)
        if (cand[i] < 0 || cand[i] >= nlist) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double best = INFINITY;
        int32_t best_id = -1;
        for (int p = 0; p < m; ++p) {
            const int32_t j = cand[i * m + p];
            const double dist = sqdist(x, xtype, i, c, j, d);
            if (dist < best || (dist == best && j < best_id)) {
                best = dist;
                best_id = j;
            }
        }
        out_ids[i] = best_id;
        out_dists[i] = best;
    }
    return 0;
}
