/*
 * CPU oracle for the residual-PQ candidate-reduction chain.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow definition of what the GPU library must compute; it shares
 * no code, header, table or helper with the CUDA path and is never called from it.  Only the tests,
 * the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * What is computed (Sec. 2.2 Eq. 3-5, Sec. 4.3 residual-PQ candidate reduction, Sec. 4.4):
 *   - residual encoding: a vector x assigned to centroid c(x) is encoded as, per subspace m, the
 *     index of the codeword nearest to the sub-vector of x - c(x) (Eq. 3; K = 256, one byte each);
 *   - per (query, probed list) lookup table LUT_m[j] = |r_q^(m) - p_m[j]|^2 with r_q = q - c (Eq. 4 on the residual);
 *   - ADC estimate of a stored code: the sum over m of LUT_m[a_m(x)] (Eq. 5);
 *   - candidate reduction: over all codes of the query's probed lists, the N_rerank smallest
 *     estimates, handed on in ascending order.
 *
 * Precision: the paper fixes fp32 lookup tables (Sec. 5, experimental setup), and both the code bytes and the kept
 * candidate set are integer decisions taken on those floats, so the oracle takes them in fp32 with
 * one stated order of operations (each operation rounded once, IEEE-754 binary32):
 *     r_t   = float(x_t) - c_t
 *     LUT   : acc = 0; for t = 0 .. dsub-1 in order: diff = r_t - p_t; acc = fma(diff, diff, acc)
 *     ADC   : acc = 0; for m = 0 .. PQ_M-1 in order: acc = acc + LUT_m[a_m]
 * Encoding uses the same table of the vector's own residual and takes the arg-min per subspace.
 *
 * Readings where the paper is silent: ties go to the lower codeword index (encoding) and to the
 * lower stored position (candidates); candidates are identified by their position in the
 * list-major code array; a query with fewer than N_rerank candidates gets position -1 and +inf in
 * the unused slots; a list appears at most once among a query's probes.
 *
 * Pins (tests/test_pq_oracle_pins.py): hand-computed case, exact-codeword closed form, duplicate
 * codewords, the identity ADC(q, x) = |q - (c + decoded code)|^2 against fp64 numpy, integer data
 * (every operation exact, so the result must equal int64 arithmetic bit for bit), fp64 arg-min and
 * lexsort cross-checks, prefix / padding / translation invariants.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { PQ_F32 = 0, PQ_U8 = 1, PQ_I8 = 2 };
enum { PQ_K = 256 };

static inline float elem_f(const void *x, int xtype, int64_t idx) {
    if (xtype == PQ_U8) return (float)((const uint8_t *)x)[idx];
    if (xtype == PQ_I8) return (float)((const int8_t *)x)[idx];
    return ((const float *)x)[idx];
}

/* lut[m*256 + j] = |r^(m) - p_m[j]|^2 for a residual r of d floats; codebooks [pq_m][256][dsub] */
void oracle_pq_lut(const float *r, int d, int pq_m, const float *codebooks, float *lut) {
    const int dsub = d / pq_m;
    for (int m = 0; m < pq_m; ++m) {
        for (int j = 0; j < PQ_K; ++j) {
            const float *p = codebooks + ((int64_t)m * PQ_K + j) * dsub;
            float acc = 0.0f;
            for (int t = 0; t < dsub; ++t) {
                const float diff = r[m * dsub + t] - p[t];
                acc = fmaf(diff, diff, acc);
            }
            lut[m * PQ_K + j] = acc;
        }
    }
}

static void residual(const void *x, int xtype, int64_t row, const float *c, int64_t list, int d, float *r) {
    for (int t = 0; t < d; ++t) r[t] = elem_f(x, xtype, row * d + t) - c[list * d + t];
}

/*
 * Residual encoding (Eq. 3 on x - c(x)).  ids[i] is the list row i was assigned to.
 * codes [n][pq_m] bytes.  Returns -1 on bad arguments or an id out of range.
 */
int oracle_pq_encode(const void *x, int xtype, int64_t n, int d, const int32_t *ids, const float *c,
                     int32_t nlist, const float *codebooks, int pq_m, uint8_t *codes) {
    if (n < 0 || d <= 0 || pq_m <= 0 || d % pq_m != 0) return -1;
    int rc = 0;
    for (int64_t i = 0; i < n; ++i)
        if (ids[i] < 0 || ids[i] >= nlist) return -1;
#pragma omp parallel
    {
        float *r = (float *)malloc(sizeof(float) * (size_t)d);
        float *lut = (float *)malloc(sizeof(float) * (size_t)pq_m * PQ_K);
        if (!r || !lut) {
#pragma omp atomic write
            rc = -1;
        }
#pragma omp for schedule(static)
        for (int64_t i = 0; i < n; ++i) {
            if (!r || !lut) continue;
            residual(x, xtype, i, c, ids[i], d, r);
            oracle_pq_lut(r, d, pq_m, codebooks, lut);
            for (int m = 0; m < pq_m; ++m) {
                int best = 0;
                for (int j = 1; j < PQ_K; ++j)
                    if (lut[m * PQ_K + j] < lut[m * PQ_K + best]) best = j;  /* strict: ties keep the lower j */
                codes[i * pq_m + m] = (uint8_t)best;
            }
        }
        free(r); free(lut);
    }
    return rc;
}

typedef struct {
    float est;
    int64_t pos;
} cand_t;

static int cand_cmp(const void *pa, const void *pb) {
    const cand_t *a = (const cand_t *)pa, *b = (const cand_t *)pb;
    if (a->est < b->est) return -1;
    if (a->est > b->est) return 1;
    return (a->pos > b->pos) - (a->pos < b->pos);
}

/* ADC estimates of the codes at positions [p0, p1) with the table of one (query, list) pair. */
void oracle_pq_adc(const float *lut, int pq_m, const uint8_t *codes, int64_t p0, int64_t p1, float *est) {
    for (int64_t p = p0; p < p1; ++p) {
        float acc = 0.0f;
        for (int m = 0; m < pq_m; ++m) acc = acc + lut[m * PQ_K + codes[p * pq_m + m]];
        est[p - p0] = acc;
    }
}

static int search_one(const void *q, int qtype, int64_t b, int d, const float *c, int32_t nlist,
                      const int32_t *probes, int nprobe, const int64_t *offsets, const uint8_t *codes,
                      const float *codebooks, int pq_m, int n_rerank, int64_t *out_pos, float *out_est,
                      int64_t *out_count) {
    int64_t total = 0;
    for (int p = 0; p < nprobe; ++p) {
        const int32_t l = probes[b * nprobe + p];
        if (l < 0 || l >= nlist) return -1;
        total += offsets[l + 1] - offsets[l];
    }
    float *r = (float *)malloc(sizeof(float) * (size_t)d);
    float *lut = (float *)malloc(sizeof(float) * (size_t)pq_m * PQ_K);
    cand_t *cand = (cand_t *)malloc(sizeof(cand_t) * (size_t)(total > 0 ? total : 1));
    float *est = (float *)malloc(sizeof(float) * (size_t)(total > 0 ? total : 1));
    if (!r || !lut || !cand || !est) {
        free(r); free(lut); free(cand); free(est);
        return -1;
    }
    int64_t at = 0;
    for (int p = 0; p < nprobe; ++p) {
        const int32_t l = probes[b * nprobe + p];
        residual(q, qtype, b, c, l, d, r);
        oracle_pq_lut(r, d, pq_m, codebooks, lut);
        oracle_pq_adc(lut, pq_m, codes, offsets[l], offsets[l + 1], est);
        for (int64_t i = 0; i < offsets[l + 1] - offsets[l]; ++i) {
            cand[at].est = est[i];
            cand[at].pos = offsets[l] + i;
            ++at;
        }
    }
    qsort(cand, (size_t)total, sizeof(cand_t), cand_cmp);
    for (int s = 0; s < n_rerank; ++s) {
        out_pos[b * n_rerank + s] = s < total ? cand[s].pos : -1;
        out_est[b * n_rerank + s] = s < total ? cand[s].est : INFINITY;
    }
    if (out_count) out_count[b] = total;
    free(r); free(lut); free(cand); free(est);
    return 0;
}

/*
 * Candidate reduction.  For every query: the codes of its nprobe probed lists (list l occupies
 * positions [offsets[l], offsets[l+1]) of the list-major code array) are scored by ADC with that
 * (query, list) pair's table; all (estimate, position) pairs are sorted and the first n_rerank kept.
 *   out_pos   [nq][n_rerank] int64 (-1 in unused slots)
 *   out_est   [nq][n_rerank] float (+inf in unused slots)
 *   out_count [nq] int64: candidates the query had in total; may be NULL
 * Returns -1 on bad arguments.
 */
int oracle_pq_search(const void *q, int qtype, int64_t nq, int d, const float *c, int32_t nlist,
                     const int32_t *probes, int nprobe, const int64_t *offsets, const uint8_t *codes,
                     const float *codebooks, int pq_m, int n_rerank, int64_t *out_pos, float *out_est,
                     int64_t *out_count) {
    if (nq < 0 || d <= 0 || pq_m <= 0 || d % pq_m != 0 || nprobe <= 0 || n_rerank <= 0) return -1;
    int rc = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t b = 0; b < nq; ++b) {
        if (search_one(q, qtype, b, d, c, nlist, probes, nprobe, offsets, codes, codebooks, pq_m, n_rerank, out_pos,
                       out_est, out_count) != 0) {
#pragma omp atomic write
            rc = -1;
        }
    }
    return rc;
}

/*
 * Residuals x - c(x) (Sec. 4.3: the vectors that the PQ codebooks are trained on and that are
 * encoded), in fp32 as one rounded subtraction per coordinate.  out [n][d] float.
 * Returns -1 on an id out of range.
 */
int oracle_residuals(const void *x, int xtype, int64_t n, int d, const int32_t *ids, const float *c, int32_t nlist,
                     float *out) {
    for (int64_t i = 0; i < n; ++i)
        if (ids[i] < 0 || ids[i] >= nlist) return -1;
    for (int64_t i = 0; i < n; ++i) residual(x, xtype, i, c, ids[i], d, out + i * d);
    return 0;
}
