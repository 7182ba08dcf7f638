/*
 * CPU oracle for the best-matching-unit (BMU) search on sparse binary documents.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the arbiter the CUDA library is
 * checked against; it is never a fallback for it.  It shares no code, header,
 * table or helper with the CUDA path and is only ever called from the tests,
 * from the smoke check and from the CPU-baseline leg of the benchmark.
 *
 * What it computes (the exact result the paper's kernel reaches faster;
 * Section 3: the search finds, for each article, the neuron whose weight
 * vector is closest, and an exact-argmin BMU does not depend on how the
 * codebook is stored):
 *
 *     d_ij = |x_i| + ||w_j||^2 - 2 * sum_{f in x_i} W[f][j]
 *
 * for document i (a set x_i of active feature ids, binary values) and neuron j
 * of a feature-major codebook W[f*M + j] (Section 3, "W[v.M+i]").  For binary x
 * this equals the squared Euclidean distance ||x_i - w_j||^2.  The BMU is the
 * lowest j that attains min_j d_ij.
 *
 * All arithmetic is IEEE double on the float inputs, in the plainest order:
 * one accumulator per neuron, features added in the order the row lists them,
 * neurons scanned in ascending order with a strict "<".  No blocking, no
 * fusion, no reordering.  Threads (OpenMP) split the documents only.
 *
 * Parity status: pinned (dense brute force, closed forms, invariants, a
 * library matmul and a hand-worked fixture; see tests/test_oracle_pins.py).
 */
#include <stdint.h>
#include <stdlib.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* n_j = sum_f W[f][j]^2, the "norms" step of the epoch (Table 4). */
void oracle_norms(const float *W, int64_t D, int64_t M, double *norms)
{
    for (int64_t j = 0; j < M; ++j)
        norms[j] = 0.0;
    for (int64_t f = 0; f < D; ++f) {
        const float *row = W + f * M;
        for (int64_t j = 0; j < M; ++j) {
            double w = (double)row[j];
            norms[j] += w * w;
        }
    }
}

/* Distance of one (document, neuron) pair, by the definition above. */
double oracle_eval(const float *W, int64_t D, int64_t M, const double *norms,
                   const int32_t *rowptr, const int32_t *colidx, int64_t i, int64_t j)
{
    (void)D;
    double s = 0.0;
    for (int32_t e = rowptr[i]; e < rowptr[i + 1]; ++e)
        s += (double)W[(int64_t)colidx[e] * M + j];
    double nx = (double)(rowptr[i + 1] - rowptr[i]);
    return nx + norms[j] - 2.0 * s;
}

/*
 * BMU of every document.  Outputs per document i:
 *   bmu[i]  lowest index attaining the minimum distance
 *   d1[i]   the minimum distance
 *   d2[i]   the second-smallest distance (over j != bmu[i]; +inf when M == 1)
 *   bmu2[i] (optional, may be NULL) the lowest index j != bmu[i] attaining d2[i],
 *           -1 when M == 1: the second-best unit the paper's kernel tracks for
 *           topographic error (Table 5, "bmu1-only")
 * d2 also lets a comparison tell a near-tie from a wrong answer.
 * Returns 0, or -1 if scratch memory could not be allocated.
 */
int oracle_bmu2(const float *W, int64_t D, int64_t M, const double *norms,
                const int32_t *rowptr, const int32_t *colidx, int64_t N,
                int32_t *bmu, double *d1, double *d2, int32_t *bmu2, int nthreads);

int oracle_bmu(const float *W, int64_t D, int64_t M, const double *norms,
               const int32_t *rowptr, const int32_t *colidx, int64_t N,
               int32_t *bmu, double *d1, double *d2, int nthreads)
{
    return oracle_bmu2(W, D, M, norms, rowptr, colidx, N, bmu, d1, d2, (int32_t *)0, nthreads);
}

int oracle_bmu2(const float *W, int64_t D, int64_t M, const double *norms,
                const int32_t *rowptr, const int32_t *colidx, int64_t N,
                int32_t *bmu, double *d1, double *d2, int32_t *bmu2, int nthreads)
{
    (void)D;
    int failed = 0;
#ifdef _OPENMP
    if (nthreads > 0)
        omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif
#pragma omp parallel
    {
        double *acc = (double *)malloc((size_t)(M > 0 ? M : 1) * sizeof(double));
        if (!acc) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 16)
        for (int64_t i = 0; i < N; ++i) {
            if (!acc)
                continue;
            for (int64_t j = 0; j < M; ++j)
                acc[j] = 0.0;
            for (int32_t e = rowptr[i]; e < rowptr[i + 1]; ++e) {
                const float *row = W + (int64_t)colidx[e] * M;
                for (int64_t j = 0; j < M; ++j)
                    acc[j] += (double)row[j];
            }
            double nx = (double)(rowptr[i + 1] - rowptr[i]);
            double best = INFINITY, second = INFINITY;
            int32_t arg = -1, arg2 = -1;
            for (int64_t j = 0; j < M; ++j) {
                double d = nx + norms[j] - 2.0 * acc[j];
                if (arg < 0 || d < best) {
                    second = (arg < 0) ? INFINITY : best;
                    arg2 = arg;
                    best = d;
                    arg = (int32_t)j;
                } else if (arg2 < 0 || d < second) {
                    second = d;
                    arg2 = (int32_t)j;
                }
            }
            bmu[i] = arg;
            d1[i] = best;
            d2[i] = second;
            if (bmu2)
                bmu2[i] = arg2;
        }
        free(acc);
    }
    return failed ? -1 : 0;
}

/* Number of threads an oracle_bmu call with nthreads <= 0 would use. */
int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------
 * The rest of a batch epoch (Table 4: "scatter", "blur", "write-back"; Section 6:
 * "the scatter into accumulators is O(N.nnz) ... the blur is the O(M) term").
 * The paper times these steps but does not print their formulas; what follows is
 * the textbook batch self-organizing-map update written out, on a rectangular,
 * non-periodic map of edge_y rows by edge_x columns (neuron j = y * edge_x + x):
 *
 *   scatter     num[f][j] = #{ i : bmu_i = j and f in x_i }   (a repeated id counts
 *               twice), cnt[j] = #{ i : bmu_i = j }           -- exact integers
 *   blur        B[f][j] = sum_k h(j, k) num[f][k],  c[j] = sum_k h(j, k) cnt[k],
 *               h(j, k) = exp(-((xj-xk)^2 + (yj-yk)^2) / (2 sigma^2)) when both
 *               |xj-xk| and |yj-yk| are at most R = ceil(3 sigma), else 0;
 *               sigma == 0 means h = identity
 *   write-back  W[f][j] = B[f][j] / c[j] where c[j] > 0, otherwise W[f][j] stays
 *
 * Parity status: pinned by mathematics only (dense brute force with the explicit
 * h matrix, closed forms, invariants; tests/test_oracle_pins_update.py) -- the
 * paper prints no formula or value for these steps, so against the paper they
 * are "parity unpinned".
 */
void oracle_scatter(const int32_t *rowptr, const int32_t *colidx, int64_t N, const int32_t *bmu,
                    int64_t M, uint64_t *num, uint64_t *cnt)
{
    for (int64_t i = 0; i < N; ++i) {
        const int64_t j = bmu[i];
        cnt[j] += 1;
        for (int32_t e = rowptr[i]; e < rowptr[i + 1]; ++e)
            num[(int64_t)colidx[e] * M + j] += 1;
    }
}

/* One plane (edge_y x edge_x doubles in, doubles out), by the definition: a
 * double loop over the neighbours inside the square of half-width R. */
void oracle_blur_plane(const double *in, int32_t edge_x, int32_t edge_y, double sigma, double *out)
{
    const int R = sigma > 0.0 ? (int)ceil(3.0 * sigma) : 0;
    for (int y = 0; y < edge_y; ++y)
        for (int x = 0; x < edge_x; ++x) {
            double s = 0.0;
            for (int dy = -R; dy <= R; ++dy)
                for (int dx = -R; dx <= R; ++dx) {
                    const int yy = y + dy, xx = x + dx;
                    if (yy < 0 || yy >= edge_y || xx < 0 || xx >= edge_x)
                        continue;
                    const double h = sigma > 0.0
                        ? exp(-((double)(dx * dx + dy * dy)) / (2.0 * sigma * sigma)) : 1.0;
                    s += h * in[(int64_t)yy * edge_x + xx];
                }
            out[(int64_t)y * edge_x + x] = s;
        }
}

void oracle_writeback(const double *B, const double *c, int64_t D, int64_t M, float *W)
{
    for (int64_t f = 0; f < D; ++f)
        for (int64_t j = 0; j < M; ++j)
            if (c[j] > 0.0)
                W[f * M + j] = (float)(B[f * M + j] / c[j]);
}

/* ------------------------------------------------------------------------
 * Stopping metrics of an epoch (Table 4 column "stopping metric"; Section 5: the
 * second-best unit "feeds topographic error", which the stopping rules gate on
 * together with the quantisation error).  The paper names the two measures and
 * prints no formula; these are their textbook definitions over the outputs of a
 * search with second-best units, on the map of edge_y rows by edge_x columns
 * (neuron j = y * edge_x + x):
 *
 *   out[0]  mean of d_i                  (mean squared quantisation error: d is the
 *                                         squared distance to the best unit)
 *   out[1]  mean of sqrt(max(d_i, 0))    (quantisation error; a d_i rounded below
 *                                         zero counts as zero)
 *   out[2]  fraction of documents whose best and second-best units are not
 *           neighbours on the map (topographic error): neighbours share an edge
 *           (adjacency == 4: |dx| + |dy| == 1) or an edge or a corner (adjacency
 *           == 8: max(|dx|, |dy|) == 1); a document without a second unit
 *           (bmu2 < 0, a one-neuron map) is not an error.
 *
 * N == 0 gives zeros.  Parity status: pinned by hand-computed cases and
 * invariants (tests/test_oracle_pins_update.py); against the paper "parity
 * unpinned" (no formula, no value printed).
 */
void oracle_map_errors(const int32_t *bmu, const int32_t *bmu2, const float *dist, int64_t N,
                       int32_t edge_x, int32_t edge_y, int32_t adjacency, double *out)
{
    double sum_d = 0.0, sum_r = 0.0;
    int64_t errors = 0;
    (void)edge_y;
    for (int64_t i = 0; i < N; ++i) {
        const double d = (double)dist[i];
        sum_d += d;
        sum_r += d > 0.0 ? sqrt(d) : 0.0;
        if (bmu2[i] < 0) continue;
        const int32_t x1 = bmu[i] % edge_x, y1 = bmu[i] / edge_x;
        const int32_t x2 = bmu2[i] % edge_x, y2 = bmu2[i] / edge_x;
        const int32_t dx = x1 > x2 ? x1 - x2 : x2 - x1, dy = y1 > y2 ? y1 - y2 : y2 - y1;
        const int near = adjacency == 8 ? ((dx > dy ? dx : dy) == 1) : (dx + dy == 1);
        if (!near) ++errors;
    }
    out[0] = N ? sum_d / (double)N : 0.0;
    out[1] = N ? sum_r / (double)N : 0.0;
    out[2] = N ? (double)errors / (double)N : 0.0;
}
