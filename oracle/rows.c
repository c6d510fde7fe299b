/* CPU float64 oracle, row-sampled form.  TEST INFRASTRUCTURE ONLY.
 *
 * Evaluates selected rows of the Gaussian application of Sec. 2.1 straight from
 * its definition (Eq. 1 for the kernel entry, Eq. 3 / Eq. 6 for the product):
 *
 *   Y[r, c] = left[r] * sum_j exp(-beta * |xrow_r - x_j|^2) * right[j] * V[j, c]
 *
 * with the squared distance taken by direct differences.  One pair at a time,
 * no blocking, no Gram trick, libm exp.  OpenMP only spreads the independent
 * rows over cores.  Shares nothing with the CUDA path.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int fd_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Xrow: R x D row-major; X: N x D row-major; V: N x b row-major (may be NULL => b = 1, V = 1);
 * left: R or NULL (= 1); right: N or NULL (= 1); Y: R x b row-major;
 * rowsq: R or NULL, receives sum_j K_rj^2 (= row sum of the kernel at 2 beta). */
void fd_oracle_rows(const double* Xrow, int64_t R, const double* X, int64_t N, int32_t D, double beta,
                    const double* left, const double* right, const double* V, int32_t b,
                    double* Y, double* rowsq) {
    if (V == NULL) b = 1;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t r = 0; r < R; ++r) {
        const double* xr = Xrow + (size_t)r * D;
        double* y = Y + (size_t)r * b;
        for (int32_t c = 0; c < b; ++c) y[c] = 0.0;
        double sq = 0.0;
        for (int64_t j = 0; j < N; ++j) {
            const double* xj = X + (size_t)j * D;
            double h = 0.0;
            for (int32_t k = 0; k < D; ++k) {
                double diff = xr[k] - xj[k];
                h += diff * diff;
            }
            double kij = exp(-beta * h);
            sq += kij * kij;
            double w = right ? kij * right[j] : kij;
            if (V) {
                const double* v = V + (size_t)j * b;
                for (int32_t c = 0; c < b; ++c) y[c] += w * v[c];
            } else {
                y[0] += w;
            }
        }
        if (left)
            for (int32_t c = 0; c < b; ++c) y[c] *= left[r];
        if (rowsq) rowsq[r] = sq;
    }
}
