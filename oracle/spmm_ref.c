/*
 * TEST INFRASTRUCTURE ONLY -- CPU oracle for the normalized sparse aggregation.
 *
 * Plain, slow, double-precision evaluation of the neighbor sum of the GCN layer
 * (Eq. 1 / Eq. 6 of the paper):
 *
 *     out[i, :] = sum_{j in N(v_i)}  x[j, :] / ( sqrt|N(v_i)| * sqrt|N(v_j)| )
 *
 * with N(v) = the stored entries of row v of the adjacency matrix.  Two other aggregators
 * of message-passing layers (the paper's closing section points at "a broader range of GNN
 * methods"; it defines only the one above) share the loops: the mean over the neighbor set,
 * weight 1/|N(v_i)| (norm 1), and the plain sum, weight 1 (norm 2).  No blocking,
 * no reordering: one loop over rows, one over the row's neighbors, one over
 * feature columns, in storage order.  Shares no code with the CUDA library.
 *
 * Build:  gcc -O2 -fopenmp -shared -fPIC spmm_ref.c -o liboracle_spmm.so -lm
 * Threads only split the outer row loop (gather form), so the result does not
 * depend on the thread count.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Weight of stored entry (i, j).  norm 0: 1/c_ij of Eq. 1 (a node with an empty neighbor set
 * contributes / receives 0); norm 1: 1/|N(v_i)| (mean over the neighbors of i); norm 2: 1 (sum). */
static double weight(int norm, int32_t deg_i, int32_t deg_j) {
    if (norm == 2) return 1.0;
    if (norm == 1) return deg_i > 0 ? 1.0 / (double)deg_i : 0.0;
    if (deg_i <= 0 || deg_j <= 0) return 0.0;
    return 1.0 / (sqrt((double)deg_i) * sqrt((double)deg_j));
}

/* Gather form: out = A_hat * x.  x is n x w with leading dimension ldx,
 * out is n x w with leading dimension ldo (both in elements, row-major).
 * rows[] (nullable) restricts the computation to a list of n_rows row ids;
 * then out row r holds the result for node rows[r]. */
void oracle_spmm_gather(int64_t n, const int32_t* rowptr, const int32_t* colidx,
                        const int32_t* deg, const double* x, int64_t ldx,
                        int64_t w, double* out, int64_t ldo,
                        const int64_t* rows, int64_t n_rows, int threads, int norm) {
    int64_t count = rows ? n_rows : n;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t r = 0; r < count; ++r) {
        int64_t i = rows ? rows[r] : r;
        double* o = out + r * ldo;
        for (int64_t c = 0; c < w; ++c) o[c] = 0.0;
        for (int32_t k = rowptr[i]; k < rowptr[i + 1]; ++k) {
            int32_t j = colidx[k];
            double a = weight(norm, deg[i], deg[j]);
            const double* xj = x + (int64_t)j * ldx;
            for (int64_t c = 0; c < w; ++c) o[c] += a * xj[c];
        }
    }
}

/* Scatter form: out = A_hat^T * y, straight from the definition of a transpose:
 * entry (i, j) of A_hat sends y[i, :] to out[j, :].  Single-threaded. */
void oracle_spmm_scatter_t(int64_t n, const int32_t* rowptr, const int32_t* colidx,
                           const int32_t* deg, const double* y, int64_t ldy,
                           int64_t w, double* out, int64_t ldo, int norm) {
    for (int64_t i = 0; i < n; ++i)
        for (int64_t c = 0; c < w; ++c) out[i * ldo + c] = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        const double* yi = y + i * ldy;
        for (int32_t k = rowptr[i]; k < rowptr[i + 1]; ++k) {
            int32_t j = colidx[k];
            double a = weight(norm, deg[i], deg[j]);
            double* o = out + (int64_t)j * ldo;
            for (int64_t c = 0; c < w; ++c) o[c] += a * yi[c];
        }
    }
}

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
