// Host fp64 eigen-decomposition of the small projected matrices (m up to a few hundred), several times per second
// inside the eigensolver's loop, so it is written for the host's cores:
//
//   1. Householder reduction to tridiagonal form T = Q^T A Q with the reflectors kept (row-contiguous updates of both
//      triangles).
//   2. Implicit symmetric QR iteration on T (Wilkinson shift, bulge chased from the top of the active block to its
//      bottom, deflation at the bottom).  The plane rotations of one sweep are only RECORDED while the tridiagonal is
//      updated (O(n) work); they are applied to the eigenvector matrix afterwards, each thread taking a slice of the
//      vector components and running through the whole list, which is where the O(n^3) work goes.
//   3. Q is formed from the reflectors (parallel over rows) before step 2, so the rotations act on it directly.
//
// The eigenvector matrix is held transposed (row k = k-th eigenvector-to-be) so that a rotation of two eigenvectors
// touches two contiguous rows.
#include <algorithm>
#include <cmath>
#include <numeric>

#include "fd_dense.h"

namespace fd {

namespace {

constexpr int kParallelFrom = 64;      // below this size the thread team costs more than it saves

// z: n x n row-major, symmetric on entry (both triangles); on exit the orthogonal Q with A = Q T Q^T.
// diag / off receive T's diagonal and sub-diagonal (off[i] couples i - 1 and i; off[0] = 0).
//
// Reduction from the last row upwards.  Both triangles of the shrinking active block are kept up to date, so the
// matrix-vector product and the rank-two update run along rows (contiguous, vectorisable).
void tridiagonalise(std::vector<double>& z, int n, std::vector<double>& diag, std::vector<double>& off) {
    auto Z = [&](int i, int j) -> double& { return z[(size_t)i * n + j]; };
    std::vector<double> U((size_t)n * n, 0.0), hval(n, 0.0), u(n), pv(n), qv(n);
    const bool par = n >= kParallelFrom;
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
    // Q = H_{n-1} ... H_2 H_1 (H_i = I - u_i u_i^T / h_i acts on indices 0..i-1): start from I, multiply from the right;
    // every row of Q is transformed independently of the others
    std::fill(z.begin(), z.end(), 0.0);
    for (int i = 0; i < n; ++i) Z(i, i) = 1.0;
#pragma omp parallel for schedule(static) if (par)
    for (int r = 0; r < n; ++r) {
        double* row = &z[(size_t)r * n];
        for (int i = n - 1; i >= 1; --i) {
            if (hval[i] == 0.0) continue;
            const int l = i - 1;
            const double* ui = &U[(size_t)i * n];
            double acc = 0.0;
            for (int k = 0; k <= l; ++k) acc += row[k] * ui[k];
            if (acc == 0.0) continue;
            acc /= hval[i];
            for (int k = 0; k <= l; ++k) row[k] -= acc * ui[k];
        }
    }
}

struct Rotation { int row; double c, s; };      // mixes eigenvector rows `row` and `row + 1`

// One implicit QR sweep with shift mu on the active block [lo, hi] of the tridiagonal (d = diagonal, e[i] couples i and
// i + 1).  The bulge is chased from lo to hi; every rotation is appended to `rots`.
void qr_sweep(std::vector<double>& d, std::vector<double>& e, int lo, int hi, double mu, std::vector<Rotation>& rots) {
    double x = d[lo] - mu;          // first column of T - mu I determines the first rotation
    double zb = e[lo];
    for (int k = lo; k < hi; ++k) {
        // rotation in the (k, k + 1) plane that annihilates zb against x
        const double r = std::hypot(x, zb);
        double c = 1.0, s = 0.0;
        if (r != 0.0) { c = x / r; s = zb / r; }
        // apply G^T T G to the 2 x 2 block and its neighbours; G = [c -s; s c] in the convention  [x zb] G = [r 0]
        if (k > lo) e[k - 1] = r;
        const double dk = d[k], dk1 = d[k + 1], ek = e[k];
        d[k] = c * c * dk + 2.0 * c * s * ek + s * s * dk1;
        d[k + 1] = s * s * dk - 2.0 * c * s * ek + c * c * dk1;
        e[k] = (c * c - s * s) * ek + c * s * (dk1 - dk);
        if (k + 1 < hi) {
            // the rotation creates a bulge at (k, k + 2) out of e[k + 1]
            zb = s * e[k + 1];
            e[k + 1] = c * e[k + 1];
            x = e[k];
        }
        rots.push_back({k, c, s});
    }
}

// Applies the recorded rotations to zt (row k = k-th eigenvector-to-be, n components each): every thread takes a slice
// of the components and runs through the whole list in order.
void apply_rotations(std::vector<double>& zt, int n, const std::vector<Rotation>& rots) {
    if (rots.empty()) return;
    const bool par = n >= kParallelFrom && rots.size() >= 8;
    const int slice = 64;
    const int nslices = (n + slice - 1) / slice;
#pragma omp parallel for schedule(static) if (par)
    for (int sidx = 0; sidx < nslices; ++sidx) {
        const int k0 = sidx * slice, k1 = std::min(n, k0 + slice);
        for (const Rotation& g : rots) {
            double* a = &zt[(size_t)g.row * n];
            double* b = &zt[(size_t)(g.row + 1) * n];
            const double c = g.c, s = g.s;
            for (int k = k0; k < k1; ++k) {
                const double ak = a[k], bk = b[k];
                a[k] = c * ak + s * bk;
                b[k] = c * bk - s * ak;
            }
        }
    }
}

// Implicit symmetric QR iteration on (d, e) with the eigenvectors accumulated in zt.  Returns false if an eigenvalue
// needs more than 60 sweeps.
bool tridiagonal_qr(std::vector<double>& d, std::vector<double>& e, int n, std::vector<double>& zt) {
    std::vector<Rotation> rots;
    rots.reserve((size_t)4 * n);
    int hi = n - 1;
    int sweeps_here = 0;
    while (hi > 0) {
        // deflate at the bottom: negligible coupling between hi - 1 and hi
        if (std::fabs(e[hi - 1]) <= 2.3e-16 * (std::fabs(d[hi - 1]) + std::fabs(d[hi]))) {
            e[hi - 1] = 0.0;
            --hi;
            sweeps_here = 0;
            continue;
        }
        // the active block is the unreduced block that ends at hi
        int lo = hi - 1;
        while (lo > 0 && std::fabs(e[lo - 1]) > 2.3e-16 * (std::fabs(d[lo - 1]) + std::fabs(d[lo]))) --lo;
        if (lo > 0) e[lo - 1] = 0.0;
        if (++sweeps_here > 60) return false;
        // Wilkinson shift: the eigenvalue of the trailing 2 x 2 block that is closer to d[hi]
        const double a = d[hi - 1], b = e[hi - 1], cdiag = d[hi];
        const double delta = 0.5 * (a - cdiag);
        const double denom = std::fabs(delta) + std::hypot(delta, b);
        const double mu = denom == 0.0 ? cdiag : cdiag - (delta >= 0.0 ? 1.0 : -1.0) * b * b / denom;
        qr_sweep(d, e, lo, hi, mu, rots);
        // flush the list from time to time so it stays cache-sized
        if (rots.size() >= (size_t)2 * n) { apply_rotations(zt, n, rots); rots.clear(); }
    }
    apply_rotations(zt, n, rots);
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
    // transpose so that each eigenvector-to-be is a contiguous row during the rotations; e[i] couples i and i + 1
    std::vector<double> zt((size_t)n * n), e(n, 0.0);
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) zt[(size_t)j * n + i] = z[(size_t)i * n + j];
    for (int i = 0; i + 1 < n; ++i) e[i] = off[i + 1];
    if (!tridiagonal_qr(diag, e, n, zt)) return false;
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
