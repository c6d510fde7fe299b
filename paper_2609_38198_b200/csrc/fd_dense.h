// Tall-skinny dense helpers (fd_dense.cu) and the host symmetric eigensolver (fd_symeig.cpp).
#pragma once
#include <vector>

#include "fd_internal.h"

namespace fd {

// out_dev[m1 x m2] (column-major doubles, device) = A^T B over N rows, fp64 accumulation.
// scratch: device doubles for the per-chunk partials.
fd_status tn_product(fd_ctx* c, const float* A, int64_t lda, int m1, const float* B, int64_t ldb, int m2, int64_t N,
                     double* out_dev, double* scratch, size_t scratch_doubles);
// C[N x p] = alpha * A[N x m] S[m x p] + beta * C; S_dev column-major floats with pitch lds.  C must not alias A.
fd_status nn_product(fd_ctx* c, const float* A, int64_t lda, int m, const float* S_dev, int lds, int p, float* C,
                     int64_t ldc, float alpha, float beta, int64_t N);
// out_dev[c] = |A[:, c]|^2 (fp64) for the first p columns.
fd_status col_sqnorms(fd_ctx* c, const float* A, int64_t lda, int p, int64_t N, double* out_dev);
fd_status d2f(fd_ctx* c, const double* in, float* out, int64_t n, double scale);
fd_status scale_cols(fd_ctx* c, float* A, int64_t lda, int p, const float* f_dev, int64_t N);
// Counter-based uniform(-1, 1) fill of N rows x p columns; row i of A is row row0 + i of the stream, so a row range of
// a larger block gets the values the whole block would.
fd_status random_fill(fd_ctx* c, float* A, int64_t lda, int p, int64_t N, int64_t row0, uint32_t seed);
fd_status sqrt_vec(fd_ctx* c, const float* d, float* out, int64_t N);
fd_status copy_cols(fd_ctx* c, const float* src, int64_t lds, float* dst, int64_t ldd, int p, int64_t N);

// Eigen-decomposition of a dense symmetric n x n matrix (column-major, only read).  On return evals ascending (all n) and
// evecs n x n column-major with orthonormal columns; with 0 <= nvec < n only the columns of the nvec LARGEST eigenvalues
// (columns n - nvec .. n - 1) are computed, the others are zero.  Householder tridiagonalisation followed by implicit
// symmetric QR.  Returns false if the iteration fails to converge.
bool sym_eig(const double* A, int n, std::vector<double>& evals, std::vector<double>& evecs, int nvec = -1);

}  // namespace fd
