// Host fp64 eigen-decomposition of the small projected matrices (m up to a few hundred).
// Textbook method, written out here: reduce to tridiagonal form with Householder reflectors
// (accumulating the orthogonal factor), then implicit-shift QL iterations with Wilkinson-type
// shifts applied as plane rotations to the accumulated factor.
#include <algorithm>
#include <cmath>
#include <numeric>

#include "fd_dense.h"

namespace fd {

namespace {

// z: n x n row-major, symmetric on entry (both triangles); on exit the orthogonal Q with A = Q T Q^T.
// diag / off receive T's diagonal and sub-diagonal (off[0] unused = 0).
//
// Householder reduction from the last row upwards.  Both triangles of the shrinking active block are kept up to
// date, so the matrix-vector product and the rank-two update run along rows (contiguous, vectorisable); that
// costs twice the flops of a lower-triangle-only update and is several times faster at n of a few hundred.
void tridiagonalise(std::vector<double>& z, int n, std::vector<double>& diag, std::vector<double>& off) {
    auto Z = [&](int i, int j) -> double& { return z[(size_t)i * n + j]; };
    std::vector<double> U((size_t)n * n, 0.0), hval(n, 0.0), u(n), pv(n), qv(n);
    for (int i = n - 1; i >= 1; --i) {
        const int l = i - 1;                       // active block: indices 0..l
        if (l == 0) { off[i] = Z(i, 0); diag[i] = Z(i, i); continue; }
        double scale = 0.0;
        for (int k = 0; k <= l; ++k) scale += std::fabs(Z(i, k));
        if (scale == 0.0) { off[i] = 0.0; diag[i] = Z(i, i); continue; }
        double sigma = 0.0;
        for (int k = 0; k <= l; ++k) { u[k] = Z(i, k) / scale; sigma += u[k] * u[k]; }
        const double f = u[l];
        const double g = f >= 0.0 ? -std::sqrt(sigma) : std::sqrt(sigma);
        off[i] = scale * g;
        const double h = sigma - f * g;            // = |u|^2 / 2 after the next line
        u[l] = f - g;
        // p = A u / h on the active block, K = u.p / (2 h), q = p - K u
        double up = 0.0;
        for (int j = 0; j <= l; ++j) {
            const double* row = &z[(size_t)j * n];
            double acc = 0.0;
            for (int k = 0; k <= l; ++k) acc += row[k] * u[k];
            pv[j] = acc / h;
            up += u[j] * pv[j];
        }
        const double K = up / (h + h);
        for (int j = 0; j <= l; ++j) qv[j] = pv[j] - K * u[j];
        // A <- A - u q^T - q u^T (both triangles)
        for (int j = 0; j <= l; ++j) {
            double* row = &z[(size_t)j * n];
            const double uj = u[j], qj = qv[j];
            for (int k = 0; k <= l; ++k) row[k] -= uj * qv[k] + qj * u[k];
        }
        std::copy(u.begin(), u.begin() + l + 1, &U[(size_t)i * n]);
        hval[i] = h;
        diag[i] = Z(i, i);
    }
    diag[0] = Z(0, 0);
    off[0] = 0.0;
    // Q = H_{n-1} ... H_2 H_1 (H_i = I - u_i u_i^T / h_i acts on indices 0..i-1): start from I, multiply from the right
    std::fill(z.begin(), z.end(), 0.0);
    for (int i = 0; i < n; ++i) Z(i, i) = 1.0;
    for (int i = n - 1; i >= 1; --i) {
        if (hval[i] == 0.0) continue;
        const int l = i - 1;
        const double* ui = &U[(size_t)i * n];
        const double hinv = 1.0 / hval[i];
        for (int r = 0; r < n; ++r) {
            double* row = &z[(size_t)r * n];
            double acc = 0.0;
            for (int k = 0; k <= l; ++k) acc += row[k] * ui[k];
            if (acc == 0.0) continue;
            acc *= hinv;
            for (int k = 0; k <= l; ++k) row[k] -= acc * ui[k];
        }
    }
}

// Implicit QL on (diag, off); rotations are applied to the COLUMNS of zt, which holds Q transposed
// (row k of zt = k-th column of Q) so the inner loop runs over contiguous memory.
bool ql_implicit(std::vector<double>& diag, std::vector<double>& off, int n, std::vector<double>& zt) {
    for (int i = 1; i < n; ++i) off[i - 1] = off[i];
    off[n - 1] = 0.0;
    for (int l = 0; l < n; ++l) {
        int iter = 0, m;
        do {
            for (m = l; m < n - 1; ++m) {
                const double dd = std::fabs(diag[m]) + std::fabs(diag[m + 1]);
                if (std::fabs(off[m]) <= 2.3e-16 * dd) break;
            }
            if (m != l) {
                if (iter++ == 60) return false;
                double g = (diag[l + 1] - diag[l]) / (2.0 * off[l]);
                double r = std::hypot(g, 1.0);
                g = diag[m] - diag[l] + off[l] / (g + (g >= 0.0 ? std::fabs(r) : -std::fabs(r)));
                double s = 1.0, c = 1.0, p = 0.0;
                int i;
                for (i = m - 1; i >= l; --i) {
                    double f = s * off[i];
                    const double b = c * off[i];
                    off[i + 1] = (r = std::hypot(f, g));
                    if (r == 0.0) {
                        diag[i + 1] -= p;
                        off[m] = 0.0;
                        break;
                    }
                    s = f / r;
                    c = g / r;
                    g = diag[i + 1] - p;
                    r = (diag[i] - g) * s + 2.0 * c * b;
                    diag[i + 1] = g + (p = s * r);
                    g = c * r - b;
                    double* zi = &zt[(size_t)i * n];
                    double* zi1 = &zt[(size_t)(i + 1) * n];
                    for (int k = 0; k < n; ++k) {
                        f = zi1[k];
                        zi1[k] = s * zi[k] + c * f;
                        zi[k] = c * zi[k] - s * f;
                    }
                }
                if (r == 0.0 && i >= l) continue;
                diag[l] -= p;
                off[l] = g;
                off[m] = 0.0;
            }
        } while (m != l);
    }
    return true;
}

}  // namespace

bool sym_eig(const double* A, int n, std::vector<double>& evals, std::vector<double>& evecs) {
    evals.assign(n, 0.0);
    evecs.assign((size_t)n * n, 0.0);
    if (n == 0) return true;
    if (n == 1) { evals[0] = A[0]; evecs[0] = 1.0; return true; }
    std::vector<double> z((size_t)n * n), diag(n), off(n);
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) z[(size_t)i * n + j] = 0.5 * (A[i + (size_t)j * n] + A[j + (size_t)i * n]);
    tridiagonalise(z, n, diag, off);
    // transpose so that each eigenvector-to-be is a contiguous row during the QL sweeps
    std::vector<double> zt((size_t)n * n);
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) zt[(size_t)j * n + i] = z[(size_t)i * n + j];
    if (!ql_implicit(diag, off, n, zt)) return false;
    std::vector<int> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::sort(order.begin(), order.end(), [&](int a, int b) { return diag[a] < diag[b]; });
    for (int c = 0; c < n; ++c) {
        evals[c] = diag[order[c]];
        const double* src = &zt[(size_t)order[c] * n];
        std::copy(src, src + n, &evecs[(size_t)c * n]);      // column c of evecs (column-major) = row of zt
    }
    return true;
}

}  // namespace fd
