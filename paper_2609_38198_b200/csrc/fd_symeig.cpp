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
//
// When only the eigenvectors of the nvec largest eigenvalues are wanted (the eigensolver needs the leading Ritz vectors on
// most steps and a larger set only at a restart), ALL rotations are recorded, the wanted eigenvalues are identified at
// the end, and the product of the rotations is applied in reverse order to the nvec unit vectors that select them:
// 6 * (number of rotations) * nvec flops instead of * n, followed by one n x n x nvec product with Q.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <numeric>

#ifdef _OPENMP
#include <omp.h>
#endif

#include "fd_dense.h"

namespace fd {

namespace {

constexpr int kParallelFrom = 64;      // below this size the thread team costs more than it saves

// Width of the column slices the independent-column loops hand to the threads: one slice per thread, whole cache lines.
inline int slice_width(int columns) {
#ifdef _OPENMP
    const int threads = std::max(1, omp_get_max_threads());
#else
    const int threads = 1;
#endif
    const int w = (columns + threads - 1) / threads;
    return std::max(8, (w + 7) / 8 * 8);
}

// z: n x n row-major, symmetric on entry (both triangles); on exit the orthogonal Q with A = Q T Q^T.
// diag / off receive T's diagonal and sub-diagonal (off[i] couples i - 1 and i; off[0] = 0).
//
// Reduction from the last row upwards.  Both triangles of the shrinking active block are kept up to date, so the
// matrix-vector product and the rank-two update run along rows (contiguous, vectorisable).
// With form_q false, z is left undefined and the reflectors (U: row i = u_i on indices 0..i-1, hval[i] = |u_i|^2 / 2) are
// returned for back_transform instead.
void tridiagonalise(std::vector<double>& z, int n, std::vector<double>& diag, std::vector<double>& off,
                    std::vector<double>& U, std::vector<double>& hval, bool form_q) {
    auto Z = [&](int i, int j) -> double& { return z[(size_t)i * n + j]; };
    U.assign((size_t)n * n, 0.0);
    hval.assign(n, 0.0);
    std::vector<double> u(n), pv(n);
    // One thread team lives through the whole reduction: per step the scalar work (reflector, K, q) is done by one
    // thread and the two O(l^2) sweeps (matrix-vector product, rank-two update) are shared by rows; the team meets at
    // the barriers that end each `single` / `for`.  A fresh team per step would cost more than the sweeps of a small step.
    double h = 0.0;
    bool skip = false;
#pragma omp parallel if (n >= 2 * kParallelFrom) default(shared)
    {
        std::vector<double> q(n);                  // every thread keeps its own copy of q (O(l) to form, read l^2 / T times)
        for (int i = n - 1; i >= 1; --i) {
            const int l = i - 1;                   // active block: indices 0..l
#pragma omp single
            {
                skip = false;
                diag[i] = Z(i, i);
                if (l == 0) { off[i] = Z(i, 0); skip = true; }
                else {
                    double scale = 0.0;
                    for (int k = 0; k <= l; ++k) scale += std::fabs(Z(i, k));
                    if (scale == 0.0) { off[i] = 0.0; skip = true; }
                    else {
                        double sigma = 0.0;
                        for (int k = 0; k <= l; ++k) { u[k] = Z(i, k) / scale; sigma += u[k] * u[k]; }
                        const double f = u[l];
                        const double g = f >= 0.0 ? -std::sqrt(sigma) : std::sqrt(sigma);
                        off[i] = scale * g;
                        h = sigma - f * g;         // = |u|^2 / 2 after the next line
                        u[l] = f - g;
                        std::copy(u.begin(), u.begin() + l + 1, &U[(size_t)i * n]);
                        hval[i] = h;
                    }
                }
            }
            if (skip) {
                // nobody may start the next step (and rewrite `skip`) before everybody has read it
#pragma omp barrier
                continue;
            }
            // p = A u / h on the active block
#pragma omp for schedule(static)
            for (int j = 0; j <= l; ++j) {
                const double* row = &z[(size_t)j * n];
                double acc = 0.0;
                for (int k = 0; k <= l; ++k) acc += row[k] * u[k];
                pv[j] = acc / h;
            }
            // K = u.p / (2 h), q = p - K u
            double up = 0.0;
            for (int j = 0; j <= l; ++j) up += u[j] * pv[j];
            const double K = up / (h + h);
            for (int j = 0; j <= l; ++j) q[j] = pv[j] - K * u[j];
            // A <- A - u q^T - q u^T (both triangles)
#pragma omp for schedule(static)
            for (int j = 0; j <= l; ++j) {
                double* row = &z[(size_t)j * n];
                const double uj = u[j], qj = q[j];
                for (int k = 0; k <= l; ++k) row[k] -= uj * q[k] + qj * u[k];
            }
        }
    }
    diag[0] = Z(0, 0);
    off[0] = 0.0;
    if (!form_q) return;
    // Q = H_{n-1} ... H_2 H_1 (H_i = I - u_i u_i^T / h_i acts on indices 0..i-1): start from I, multiply from the right;
    // every row of Q is transformed independently of the others
    std::fill(z.begin(), z.end(), 0.0);
    for (int i = 0; i < n; ++i) Z(i, i) = 1.0;
#pragma omp parallel for schedule(static) if (n >= kParallelFrom)
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

// w (n x cw row-major, one thread's private slice of the selected vectors) <- Q w with Q = H_{n-1} ... H_1 given by its
// reflectors: H_1 is applied first.
void back_transform(double* w, int n, int cw, const std::vector<double>& U, const std::vector<double>& hval, double* t) {
    for (int i = 1; i < n; ++i) {
        if (hval[i] == 0.0) continue;
        const double* ui = &U[(size_t)i * n];
        for (int c = 0; c < cw; ++c) t[c] = 0.0;
        for (int k = 0; k < i; ++k) {
            const double uk = ui[k];
            const double* wk = w + (size_t)k * cw;
            for (int c = 0; c < cw; ++c) t[c] += uk * wk[c];
        }
        const double inv = 1.0 / hval[i];
        for (int c = 0; c < cw; ++c) t[c] *= inv;
        for (int k = 0; k < i; ++k) {
            const double uk = ui[k];
            double* wk = w + (size_t)k * cw;
            for (int c = 0; c < cw; ++c) wk[c] -= uk * t[c];
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
        // (entries of the projected matrices are O(1) and couplings below 1e-16 of the diagonal are deflated before a
        // sweep, so the plain square root neither overflows nor loses the rotation to underflow)
        const double r = std::sqrt(x * x + zb * zb);
        double c = 1.0, s = 0.0;
        if (r != 0.0) { const double rinv = 1.0 / r; c = x * rinv; s = zb * rinv; }
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
// zt is 64-byte aligned with a row pitch that is a multiple of eight doubles, and slices are whole cache lines, so no
// line is written by two threads.
void apply_rotations(double* zt, int n, int pitch, const std::vector<Rotation>& rots) {
    if (rots.empty()) return;
    const int slice = slice_width(n);
    const int nslices = (n + slice - 1) / slice;
    const bool par = n >= kParallelFrom && rots.size() >= 8 && nslices > 1;
#pragma omp parallel for schedule(static) if (par)
    for (int sidx = 0; sidx < nslices; ++sidx) {
        const int k0 = sidx * slice, k1 = std::min(n, k0 + slice);
        for (const Rotation& g : rots) {
            double* a = zt + (size_t)g.row * pitch;
            double* b = a + pitch;
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
// keep_all: only record (the caller applies them in reverse to selected unit vectors); otherwise zt is updated as the
// list fills.
bool tridiagonal_qr(std::vector<double>& d, std::vector<double>& e, int n, double* zt, int pitch, std::vector<Rotation>& rots,
                    bool keep_all) {
    rots.clear();
    rots.reserve(keep_all ? (size_t)n * n + 16 : (size_t)4 * n);
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
        if (!keep_all && rots.size() >= (size_t)2 * n) { apply_rotations(zt, n, pitch, rots); rots.clear(); }
    }
    if (!keep_all) { apply_rotations(zt, n, pitch, rots); rots.clear(); }
    return true;
}

// w: n x cw row-major (row i = component i of each of this slice's vectors).  On entry column c is the unit vector
// that selects one eigenvector; on exit it holds that eigenvector's coefficients in the basis of Q's columns.
// Row k of (R_last ... R_1) is e_k^T R_last ... R_1: the rotations are applied from the right, last one first.
void apply_rotations_reversed(double* w, int cw, const std::vector<Rotation>& rots) {
    for (size_t r = rots.size(); r-- > 0;) {
        const Rotation& g = rots[r];
        double* a = w + (size_t)g.row * cw;
        double* b = a + cw;
        const double c = g.c, s = g.s;
        for (int k = 0; k < cw; ++k) {
            const double ak = a[k], bk = b[k];
            a[k] = c * ak - s * bk;
            b[k] = s * ak + c * bk;
        }
    }
}

}  // namespace

bool sym_eig(const double* A, int n, std::vector<double>& evals, std::vector<double>& evecs, int nvec) {
    evals.assign(n, 0.0);
    evecs.assign((size_t)n * n, 0.0);
    if (n == 0) return true;
    if (n == 1) { evals[0] = A[0]; evecs[0] = 1.0; return true; }
    if (nvec < 0 || nvec > n) nvec = n;
    const bool partial = nvec < n - n / 8 && n >= 32;       // close to all of them: the direct accumulation is as cheap
    std::vector<double> z((size_t)n * n), diag(n), off(n);
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) z[(size_t)i * n + j] = 0.5 * (A[i + (size_t)j * n] + A[j + (size_t)i * n]);
    std::vector<double> refl, hval;
    tridiagonalise(z, n, diag, off, refl, hval, !partial);
    std::vector<double> e(n, 0.0);
    for (int i = 0; i + 1 < n; ++i) e[i] = off[i + 1];
    std::vector<Rotation> rots;
    std::vector<int> order(n);
    std::iota(order.begin(), order.end(), 0);
    if (partial) {
        if (!tridiagonal_qr(diag, e, n, nullptr, 0, rots, true)) return false;
        std::sort(order.begin(), order.end(), [&](int a, int b) { return diag[a] < diag[b]; });
        for (int c = 0; c < n; ++c) evals[c] = diag[order[c]];
        // The nvec largest eigenvalues sit at ascending positions n - nvec .. n - 1.  Their vectors are independent of one
        // another from here on: each thread takes a slice of them in a buffer of its own (no cache line is shared between
        // threads), starts from the unit vectors that select them, undoes the rotations and then the reflectors.
        const int slice = slice_width(nvec);
        const int nslices = (nvec + slice - 1) / slice;
#pragma omp parallel for schedule(static) if (nslices > 1 && n >= kParallelFrom)
        for (int sidx = 0; sidx < nslices; ++sidx) {
            const int c0 = sidx * slice, cw = std::min(nvec, c0 + slice) - c0;
            std::vector<double> w((size_t)n * cw + 8, 0.0), t(cw);
            for (int c = 0; c < cw; ++c) w[(size_t)order[n - nvec + c0 + c] * cw + c] = 1.0;
            apply_rotations_reversed(w.data(), cw, rots);
            back_transform(w.data(), n, cw, refl, hval, t.data());
            for (int c = 0; c < cw; ++c) {
                double* dst = &evecs[(size_t)(n - nvec + c0 + c) * n];
                for (int i = 0; i < n; ++i) dst[i] = w[(size_t)i * cw + c];
            }
        }
        return true;
    }
    // transpose so that each eigenvector-to-be is a contiguous row during the rotations; e[i] couples i and i + 1
    const int pitch = (n + 7) / 8 * 8;
    std::vector<double> zt_store((size_t)n * pitch + 8);
    double* zt = reinterpret_cast<double*>((reinterpret_cast<uintptr_t>(zt_store.data()) + 63) & ~(uintptr_t)63);
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) zt[(size_t)j * pitch + i] = z[(size_t)i * n + j];
    if (!tridiagonal_qr(diag, e, n, zt, pitch, rots, false)) return false;
    std::sort(order.begin(), order.end(), [&](int a, int b) { return diag[a] < diag[b]; });
    for (int c = 0; c < n; ++c) {
        evals[c] = diag[order[c]];
        const double* src = zt + (size_t)order[c] * pitch;
        std::copy(src, src + n, &evecs[(size_t)c * n]);      // column c of evecs (column-major) = row of zt
    }
    return true;
}

}  // namespace fd
