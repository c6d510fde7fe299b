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

// z: n x n row-major, symmetric on entry; on exit the orthogonal Q with A = Q T Q^T.
// diag / off receive T's diagonal and sub-diagonal (off[0] unused = 0).
void tridiagonalise(std::vector<double>& z, int n, std::vector<double>& diag, std::vector<double>& off) {
    auto Z = [&](int i, int j) -> double& { return z[(size_t)i * n + j]; };
    for (int i = n - 1; i >= 1; --i) {
        const int l = i - 1;
        double h = 0.0, scale = 0.0;
        if (l > 0) {
            for (int k = 0; k <= l; ++k) scale += std::fabs(Z(i, k));
            if (scale == 0.0) {
                off[i] = Z(i, l);
            } else {
                for (int k = 0; k <= l; ++k) { Z(i, k) /= scale; h += Z(i, k) * Z(i, k); }
                double f = Z(i, l);
                double g = f >= 0.0 ? -std::sqrt(h) : std::sqrt(h);
                off[i] = scale * g;
                h -= f * g;
                Z(i, l) = f - g;
                f = 0.0;
                for (int j = 0; j <= l; ++j) {
                    Z(j, i) = Z(i, j) / h;
                    g = 0.0;
                    for (int k = 0; k <= j; ++k) g += Z(j, k) * Z(i, k);
                    for (int k = j + 1; k <= l; ++k) g += Z(k, j) * Z(i, k);
                    off[j] = g / h;
                    f += off[j] * Z(i, j);
                }
                const double hh = f / (h + h);
                for (int j = 0; j <= l; ++j) {
                    f = Z(i, j);
                    off[j] = g = off[j] - hh * f;
                    for (int k = 0; k <= j; ++k) Z(j, k) -= f * off[k] + g * Z(i, k);
                }
            }
        } else {
            off[i] = Z(i, l);
        }
        diag[i] = h;
    }
    diag[0] = 0.0;
    off[0] = 0.0;
    for (int i = 0; i < n; ++i) {
        const int l = i - 1;
        if (diag[i] != 0.0) {
            for (int j = 0; j <= l; ++j) {
                double g = 0.0;
                for (int k = 0; k <= l; ++k) g += Z(i, k) * Z(k, j);
                for (int k = 0; k <= l; ++k) Z(k, j) -= g * Z(k, i);
            }
        }
        diag[i] = Z(i, i);
        Z(i, i) = 1.0;
        for (int j = 0; j <= l; ++j) Z(j, i) = Z(i, j) = 0.0;
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
