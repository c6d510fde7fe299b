// fd_eigs: leading eigenpairs of M = diag(s) K diag(s) (Eq. 2) by block Krylov / Rayleigh-Ritz
// with residual expansion and thick restart.
//
// The paper names "block implicitly restarted Lanczos" (Sec. 2.3) and gives no detail, so the
// scheme is fixed here.  An orthonormal basis Q (N x m) is kept together with its image
// W = M Q.  Each step: projected matrix T = Q^T W (fp64), Ritz pairs, explicit residuals
// R_i = W x_i - theta_i Q x_i for the leading k + 1 + buffer pairs, the b residuals of largest
// norm are orthogonalised against Q (classical Gram-Schmidt twice) and among themselves
// (eigen-based orthogonalisation that drops dependent directions), appended, and M is applied
// to the new block only.  For a cold one-block start this spans the same block Krylov space as
// block Lanczos; unlike the three-term recurrence it accepts an arbitrary warm-start basis.
// When the basis is full it is compressed onto the leading Ritz vectors (thick restart).
// The Perron vector sqrt(d) / |sqrt(d)| is known in closed form and always seeds the basis.
// Vectors are fp32; every inner product and the small eigenproblem are fp64, and the measured
// Gram matrix Q^T Q corrects the projected problem to first order, so fp32 loss of
// orthogonality does not reach the Ritz values.
//
// Row-sharded contexts: every rank keeps rows [r0, r0 + n) of Q, W and the work blocks (pitch N, same addresses as
// the unsharded layout), all tall-skinny products run on those rows, every reduced quantity that reaches the host
// is summed over the ranks there (so all ranks take the same decisions), and the rows of a new block are gathered
// from their owners before M is applied to it.
#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <vector>

#include "fd_dense.h"

namespace fd {

namespace {

using clk = std::chrono::steady_clock;
inline double secs(clk::time_point a, clk::time_point b) { return std::chrono::duration<double>(b - a).count(); }

struct Solver {
    fd_ctx* c;
    int64_t N;                      // pitch of every tall matrix = number of points
    int64_t r0, n;                  // rows this rank owns (0, N unless the context is row-sharded)
    int m_cap, BP;
    float *Q, *W, *X;               // N x m_cap each (X = spare for out-of-place updates)
    float *R, *R2;                  // N x BP each
    double* d_out;                  // device: m_cap x BP doubles (projection results)
    float* d_S;                     // device: m_cap x m_cap floats (small right factors)
    double* d_scr; size_t scr_n;    // device: partials of the projections
    std::vector<double> T, G;       // host, column-major, pitch m_cap
    std::vector<double> h_out;      // host staging
    int stage_next = 0;             // next slot of the context's pinned staging ring
    int m = 0;
    int applies = 0, restarts = 0;
    double t_apply = 0.0;

    fd_status to_host(int cnt) {
        FD_CUDA(c, cudaMemcpyAsync(h_out.data(), d_out, sizeof(double) * (size_t)cnt, cudaMemcpyDeviceToHost, c->stream));
        FD_CUDA(c, cudaStreamSynchronize(c->stream));
        return allreduce_host(c, h_out.data(), cnt);
    }
    // The staging ring lives in the context (pinned HOST memory, allocated once): an upload never waits for the stream
    // unless its slot is still in flight.
    fd_status init_staging(size_t floats) {
        if (c->stage_floats >= floats) return FD_OK;
        for (int i = 0; i < fd_ctx::kStageSlots; ++i) {
            if (c->stage[i]) { FD_CUDA(c, cudaFreeHost(c->stage[i])); c->stage[i] = nullptr; }
            FD_CUDA(c, cudaMallocHost(reinterpret_cast<void**>(&c->stage[i]), sizeof(float) * floats));
            if (!c->stage_ev[i]) FD_CUDA(c, cudaEventCreateWithFlags(&c->stage_ev[i], cudaEventDisableTiming));
        }
        c->stage_floats = floats;
        return FD_OK;
    }
    fd_status upload_S(const std::vector<float>& S) {
        if (S.size() > c->stage_floats) return fail(c, FD_ERR_WORKSPACE, "staging buffer too small for a right factor");
        const int k = stage_next;
        stage_next = (stage_next + 1) % fd_ctx::kStageSlots;
        FD_CUDA(c, cudaEventSynchronize(c->stage_ev[k]));  // the copy that used this slot last (four uploads ago) has finished
        std::copy(S.begin(), S.end(), c->stage[k]);
        FD_CUDA(c, cudaMemcpyAsync(d_S, c->stage[k], sizeof(float) * S.size(), cudaMemcpyHostToDevice, c->stream));
        FD_CUDA(c, cudaEventRecord(c->stage_ev[k], c->stream));
        return FD_OK;
    }

    // W[:, c0 : c0 + n) = M Q[:, c0 : c0 + n), in blocks of at most bw columns
    fd_status apply_cols(int c0, int cnt, int bw) {
        auto t0 = clk::now();
        FD_TRY(gather_rows(c, Q + (int64_t)c0 * N, N, cnt));         // the product needs all rows of the right block
        for (int o = 0; o < cnt; o += bw) {
            int w = std::min(bw, cnt - o);
            FD_TRY(apply_general(c, c->beta, c->s(), c->s(), false, nullptr, N, 0, Q + (int64_t)(c0 + o) * N, N, w,
                                 W + (int64_t)(c0 + o) * N, N, c->eigs_prec, /*gather_out=*/false));
            ++applies;
        }
        FD_TRY(tc_check_status(c));
        t_apply += secs(t0, clk::now());
        return FD_OK;
    }

    // out(m1 x m2) -> host h_out, column-major pitch m1; right factor chunked to BP columns
    fd_status project(const float* A, int m1, const float* B, int m2, std::vector<double>& dst) {
        dst.assign((size_t)m1 * m2, 0.0);
        for (int c0 = 0; c0 < m2; c0 += BP) {
            int w = std::min(BP, m2 - c0);
            FD_TRY(tn_product(c, A + r0, N, m1, B + (int64_t)c0 * N + r0, N, w, n, d_out, d_scr, scr_n));
            FD_TRY(to_host(m1 * w));
            std::copy(h_out.begin(), h_out.begin() + (size_t)m1 * w, dst.begin() + (size_t)c0 * m1);
        }
        return FD_OK;
    }

    // Recompute T = Q^T W and G = Q^T Q for the first m columns.
    fd_status full_projection() {
        std::vector<double> tmp;
        FD_TRY(project(Q, m, W, m, tmp));
        for (int j = 0; j < m; ++j)
            for (int i = 0; i < m; ++i) T[i + (size_t)j * m_cap] = 0.5 * (tmp[i + (size_t)j * m] + tmp[j + (size_t)i * m]);
        FD_TRY(project(Q, m, Q, m, tmp));
        for (int j = 0; j < m; ++j)
            for (int i = 0; i < m; ++i) G[i + (size_t)j * m_cap] = 0.5 * (tmp[i + (size_t)j * m] + tmp[j + (size_t)i * m]);
        return FD_OK;
    }

    // After appending nb columns at position m: fill the new rows / columns of T and G.
    fd_status extend_projection(int nb) {
        const int mt = m + nb;
        std::vector<double> tmp;
        FD_TRY(project(Q, mt, W + (int64_t)m * N, nb, tmp));
        for (int j = 0; j < nb; ++j)
            for (int i = 0; i < mt; ++i) {
                double v = tmp[i + (size_t)j * mt];
                if (i >= m) v = 0.5 * (v + tmp[(m + j) + (size_t)(i - m) * mt]);
                T[i + (size_t)(m + j) * m_cap] = v;
                T[(m + j) + (size_t)i * m_cap] = v;
            }
        FD_TRY(project(Q, mt, Q + (int64_t)m * N, nb, tmp));
        for (int j = 0; j < nb; ++j)
            for (int i = 0; i < mt; ++i) {
                double v = tmp[i + (size_t)j * mt];
                if (i >= m) v = 0.5 * (v + tmp[(m + j) + (size_t)(i - m) * mt]);
                G[i + (size_t)(m + j) * m_cap] = v;
                G[(m + j) + (size_t)i * m_cap] = v;
            }
        m = mt;
        return FD_OK;
    }

    // Orthonormalise the p columns of B (N x p, pitch N) among themselves; dependent directions
    // (eigenvalue of the unit-diagonal Gram matrix below drop_tol) are dropped.  Result in B, p updated.
    fd_status orthonormalise(float*& B, float*& spare, int& p, double drop_tol) {
        if (p == 0) return FD_OK;
        FD_TRY(tn_product(c, B + r0, N, p, B + r0, N, p, n, d_out, d_scr, scr_n));
        FD_TRY(to_host(p * p));
        std::vector<double> g((size_t)p * p), dinv(p);
        for (int j = 0; j < p; ++j) {
            double dj = h_out[j + (size_t)j * p];
            dinv[j] = dj > 1e-60 ? 1.0 / std::sqrt(dj) : 0.0;
        }
        for (int j = 0; j < p; ++j)
            for (int i = 0; i < p; ++i)
                g[i + (size_t)j * p] = 0.5 * (h_out[i + (size_t)j * p] + h_out[j + (size_t)i * p]) * dinv[i] * dinv[j];
        std::vector<double> lam, U;
        if (!sym_eig(g.data(), p, lam, U)) return fail(c, FD_ERR_NOT_CONVERGED, "small eigenproblem (orthonormalise) failed");
        std::vector<int> keep;
        for (int j = p - 1; j >= 0; --j)
            if (lam[j] > drop_tol) keep.push_back(j);
        const int pk = (int)keep.size();
        if (pk == 0) { p = 0; return FD_OK; }
        std::vector<float> S((size_t)p * pk);
        for (int jj = 0; jj < pk; ++jj) {
            const int j = keep[jj];
            const double f = 1.0 / std::sqrt(lam[j]);
            for (int i = 0; i < p; ++i) S[i + (size_t)jj * p] = (float)(dinv[i] * U[i + (size_t)j * p] * f);
        }
        FD_TRY(upload_S(S));
        FD_TRY(nn_product(c, B + r0, N, p, d_S, p, pk, spare + r0, N, 1.f, 0.f, n));
        std::swap(B, spare);
        p = pk;
        return FD_OK;
    }

    // B <- B - Q[:, 0:mq) (Q^T B), once.
    fd_status project_out(float* B, int p, int mq) {
        if (p == 0 || mq == 0) return FD_OK;
        FD_TRY(tn_product(c, Q + r0, N, mq, B + r0, N, p, n, d_out, d_scr, scr_n));
        if (c->sh.on) {
            // the coefficients are sums over the ranks: through the host, like every other projection
            FD_TRY(to_host(mq * p));
            std::vector<float> S((size_t)mq * p);
            for (size_t i = 0; i < S.size(); ++i) S[i] = (float)(-h_out[i]);
            FD_TRY(upload_S(S));
        } else {
            FD_TRY(d2f(c, d_out, d_S, (int64_t)mq * p, -1.0));
        }
        FD_TRY(nn_product(c, Q + r0, N, mq, d_S, mq, p, B + r0, N, 1.f, 1.f, n));
        return FD_OK;
    }
};

}  // namespace
}  // namespace fd

using namespace fd;

extern "C" fd_status fd_eigs(fd_ctx* c, int32_t k, int32_t b, double tol, int32_t max_applies, const float* Q0_dev,
                             int64_t ldq0, int32_t q0_cols, double* evals_host, float* evecs_dev, int64_t ldv,
                             fd_eigs_info* info) {
    if (!c) return FD_ERR_INVALID;
    auto t_start = clk::now();
    const Layout& L = c->L;
    const int64_t N = L.N;
    if (!c->have_s) return fail(c, FD_ERR_INVALID, "fd_eigs before fd_degree");
    if (k < 0 || (int64_t)k + 1 > N) return fail(c, FD_ERR_INVALID, "k + 1 = %d exceeds N or k < 0", k + 1);
    if (b < 1 || b > L.b_max) return fail(c, FD_ERR_INVALID, "b outside 1..b_max");
    if (!(tol > 0) || max_applies < 1 || !evals_host || !evecs_dev || ldv < N) return fail(c, FD_ERR_INVALID, "bad fd_eigs argument");
    if (Q0_dev && (q0_cols < 1 || ldq0 < N)) return fail(c, FD_ERR_INVALID, "bad warm-start basis");
    const int nwant = k + 1;
    if (L.m_max < 2 * nwant + b && L.m_max < N) return fail(c, FD_ERR_WORKSPACE, "m_max = %d < 2 (k + 1) + b = %d", L.m_max, 2 * nwant + b);

    Solver S;
    S.c = c; S.N = N; S.r0 = c->row0(); S.n = c->rows(); S.BP = L.BP;
    const int64_t r0 = S.r0, n = S.n;
    S.m_cap = (int)std::min<int64_t>(L.m_max, N);
    const int m_cap = S.m_cap;
    S.Q = c->at<float>(L.eig_q); S.W = c->at<float>(L.eig_w); S.X = c->at<float>(L.eig_x);
    S.R = c->at<float>(L.eig_r); S.R2 = c->at<float>(L.eig_t);
    double* small = c->at<double>(L.eig_small);
    S.d_out = small;
    S.d_S = reinterpret_cast<float*>(small + (size_t)L.m_max * std::max(L.m_max, L.BP));
    S.d_scr = small + (size_t)2 * L.m_max * std::max(L.m_max, L.BP);
    S.scr_n = L.eig_small_doubles - (size_t)2 * L.m_max * std::max(L.m_max, L.BP);
    S.T.assign((size_t)m_cap * m_cap, 0.0);
    S.G.assign((size_t)m_cap * m_cap, 0.0);
    S.h_out.assign((size_t)L.m_max * std::max(L.m_max, L.BP), 0.0);
    auto t_i0 = clk::now();
    FD_TRY(S.init_staging((size_t)L.m_max * (size_t)std::max(L.m_max, 2 * L.BP)));
    const double t_init = secs(t_i0, clk::now());

    const int buffer = std::min<int>(std::min(b, 8), (int)std::max<int64_t>(0, N - nwant));
    const int nsel_max = nwant + buffer;

    // ---- start basis: Perron vector, then the warm-start columns or a random block ----------
    FD_TRY(sqrt_vec(c, c->d() + r0, S.Q + r0, n));
    int cols = 1;
    const int room = std::max(0, m_cap - b - 1);                 // leave space for one expansion block
    if (Q0_dev) {
        int take = std::min(q0_cols, std::max(room, std::min(m_cap - 1, nwant)));
        take = std::min(take, m_cap - 1);
        FD_TRY(copy_cols(c, Q0_dev + r0, ldq0, S.Q + N + r0, N, take, n));
        cols += take;
    } else {
        int take = std::min(std::max(b, 1), m_cap - 1);
        if (take > 0) FD_TRY(random_fill(c, S.Q + N + r0, N, take, n, r0, 0x5EEDu));
        cols += take;
    }
    {
        // orthonormalise the start block in place (may exceed BP columns: use the spare basis buffer)
        float* B = S.Q; float* spare = S.X; int p = cols;
        // d_S must hold p x p floats: p <= m_cap
        FD_TRY(S.orthonormalise(B, spare, p, 1e-10));
        FD_TRY(S.orthonormalise(B, spare, p, 1e-10));
        S.Q = B; S.X = spare;
        if (p == 0) return fail(c, FD_ERR_NONFINITE, "start basis has no usable column");
        S.m = p;
    }
    FD_TRY(S.apply_cols(0, S.m, b));
    FD_TRY(S.full_projection());

    std::vector<double> theta, Xr;        // Ritz values (descending) and vectors (m x nsel, pitch m)
    std::vector<double> resid;
    int nsel = 0, nconv = 0, nlock = 0;
    fd_status final_status = FD_ERR_NOT_CONVERGED;
    int stagnation = 0;
    // stagnation of the residuals at the accuracy floor of the fp32 operator (noise-smeared spectra): stop early
    double best_res = 1e300;
    int since_best = 0;

    double t_rr = 0, t_eig = 0, t_res = 0, t_restart = 0, t_orth = 0, t_ext = 0;
    for (int iter = 0;; ++iter) {
        const int m = S.m;
        auto tp0 = clk::now();
        // ---- Rayleigh-Ritz with first-order correction for G = Q^T Q = I + E ---------------------
        // Tc = T - (E T + T E) / 2 with E = G - I; T E = (E T)^T because both are symmetric
        std::vector<double> Tc((size_t)m * m), ET((size_t)m * m, 0.0);
#pragma omp parallel for schedule(static) if (m >= 64)
        for (int j = 0; j < m; ++j)
            for (int l = 0; l < m; ++l) {
                const double t = S.T[l + (size_t)j * m_cap];
                const double* Ecol = &S.G[(size_t)l * m_cap];
                double* o = &ET[(size_t)j * m];
                for (int i = 0; i < m; ++i) o[i] += Ecol[i] * t;          // G column l ...
                o[l] -= t;                                                 // ... minus the identity
            }
        for (int j = 0; j < m; ++j)
            for (int i = 0; i < m; ++i)
                Tc[i + (size_t)j * m] = S.T[i + (size_t)j * m_cap] - 0.5 * (ET[i + (size_t)j * m] + ET[j + (size_t)i * m]);
        std::vector<double> lam, U;
        auto tp1 = clk::now();
        // eigenvectors: the leading Ritz vectors on every step; the larger kept set only when this step may restart
        const int nvec_ritz = std::min(nsel_max, m);
        const int nvec = (m + b > m_cap) ? std::max(nvec_ritz, std::min(m - 1, (m_cap * 3) / 5)) : nvec_ritz;
        if (!sym_eig(Tc.data(), m, lam, U, nvec)) return fail(c, FD_ERR_NOT_CONVERGED, "projected eigenproblem failed");
        auto tp2 = clk::now();
        t_rr += secs(tp0, tp1); t_eig += secs(tp1, tp2);
        nsel = std::min(nsel_max, m);
        theta.resize(nsel);
        Xr.assign((size_t)m * nsel, 0.0);
#pragma omp parallel for schedule(static) if (m >= 64)
        for (int jj = 0; jj < nsel; ++jj) {
            const int j = m - 1 - jj;
            theta[jj] = lam[j];
            for (int i = 0; i < m; ++i) {
                double corr = 0.0;
                for (int l = 0; l < m; ++l) corr += (S.G[i + (size_t)l * m_cap] - (i == l ? 1.0 : 0.0)) * U[l + (size_t)j * m];
                Xr[i + (size_t)jj * m] = U[i + (size_t)j * m] - 0.5 * corr;
            }
        }
        // ---- explicit residuals R_i = W x_i - theta_i Q x_i, BP columns at a time -----------------
        // Leading pairs that converged with a margin at an earlier step are not re-evaluated every step (their Ritz
        // vectors only improve as the basis grows); before convergence is declared every pair is evaluated afresh.
        resid.resize(nsel, 1e300);
        const double thr = tol * std::fabs(theta[0]);
        bool all = false;
        for (int pass = 0; pass < 2; ++pass) {
            std::vector<int> act;
            for (int i = std::min(nlock, nsel); i < nsel; ++i) act.push_back(i);
            for (size_t a0 = 0; a0 < act.size(); a0 += (size_t)S.BP) {
                const int w = (int)std::min<size_t>((size_t)S.BP, act.size() - a0);
                std::vector<float> Sx((size_t)m * w * 2);
                for (int jj = 0; jj < w; ++jj) {
                    const int col = act[a0 + jj];
                    for (int i = 0; i < m; ++i) {
                        Sx[i + (size_t)jj * m] = (float)Xr[i + (size_t)col * m];
                        Sx[(size_t)m * w + i + (size_t)jj * m] = (float)(-theta[col] * Xr[i + (size_t)col * m]);
                    }
                }
                FD_TRY(S.upload_S(Sx));
                FD_TRY(nn_product(c, S.W + r0, N, m, S.d_S, m, w, S.R + r0, N, 1.f, 0.f, n));
                FD_TRY(nn_product(c, S.Q + r0, N, m, S.d_S + (size_t)m * w, m, w, S.R + r0, N, 1.f, 1.f, n));
                FD_TRY(col_sqnorms(c, S.R + r0, N, w, n, S.d_out));
                FD_TRY(S.to_host(w));
                for (int jj = 0; jj < w; ++jj) resid[act[a0 + jj]] = std::sqrt(std::max(0.0, S.h_out[jj]));
            }
            nconv = 0;
            while (nconv < std::min(nwant, nsel) && resid[nconv] <= thr) ++nconv;
            all = nsel >= nwant;
            for (int i = 0; i < std::min(nwant, nsel); ++i) all = all && resid[i] <= thr;
            if (all && nlock > 0) { nlock = 0; continue; }       // verify the locked pairs before declaring convergence
            break;
        }
        {
            int lead = 0;
            while (lead < std::min(nwant, nsel) && resid[lead] <= 0.5 * thr) ++lead;
            nlock = lead;
        }
        auto tp3 = clk::now();
        t_res += secs(tp2, tp3);
        if (all) { final_status = FD_OK; break; }
        if (S.applies >= max_applies) break;
        {
            double worst = 0.0;
            for (int i = 0; i < std::min(nwant, nsel); ++i) worst = std::max(worst, resid[i]);
            if (nsel >= nwant && worst < 0.9 * best_res) { best_res = worst; since_best = 0; }
            else if (nsel >= nwant) ++since_best;
            // the largest wanted residual has not improved by 10 % over 25 expansions and is within 2x of the target:
            // the operator's own rounding error is the floor; more applies do not help
            if (since_best >= 25 && best_res <= 2.0 * thr) break;
        }
        if (m >= N) break;                                        // basis spans everything: nothing more to add

        // ---- choose the expansion columns: largest residuals first ------------------------------
        std::vector<int> order(nsel);
        for (int i = 0; i < nsel; ++i) order[i] = i;
        std::sort(order.begin(), order.end(), [&](int a, int bb) { return resid[a] > resid[bb]; });
        int want_new = std::min<int64_t>(b, N - m);
        std::vector<int> pick;
        for (int i = 0; i < nsel && (int)pick.size() < want_new; ++i)
            if (resid[order[i]] > 0.1 * thr) pick.push_back(order[i]);
        if (pick.empty()) { final_status = FD_OK; break; }

        // ---- thick restart when the new block would not fit ----------------------------------------
        if (m + (int)pick.size() > m_cap) {
            int keep = std::max(nsel, std::min(m - 1, (m_cap * 3) / 5));
            keep = std::min(keep, m_cap - (int)pick.size());
            keep = std::min(keep, m);
            // Ritz vectors for the kept block (beyond nsel use the uncorrected eigenvectors)
            std::vector<float> Sk((size_t)m * keep);
            for (int jj = 0; jj < keep; ++jj) {
                const int j = m - 1 - jj;
                for (int i = 0; i < m; ++i)
                    Sk[i + (size_t)jj * m] = jj < nsel ? (float)Xr[i + (size_t)jj * m] : (float)U[i + (size_t)j * m];
            }
            // residual block for the picked columns must be formed BEFORE the basis changes
            std::vector<float> Sx((size_t)m * pick.size() * 2);
            const int w = (int)pick.size();
            for (int jj = 0; jj < w; ++jj)
                for (int i = 0; i < m; ++i) {
                    Sx[i + (size_t)jj * m] = (float)Xr[i + (size_t)pick[jj] * m];
                    Sx[(size_t)m * w + i + (size_t)jj * m] = (float)(-theta[pick[jj]] * Xr[i + (size_t)pick[jj] * m]);
                }
            FD_TRY(S.upload_S(Sx));
            FD_TRY(nn_product(c, S.W + r0, N, m, S.d_S, m, w, S.R + r0, N, 1.f, 0.f, n));
            FD_TRY(nn_product(c, S.Q + r0, N, m, S.d_S + (size_t)m * w, m, w, S.R + r0, N, 1.f, 1.f, n));
            FD_TRY(S.upload_S(Sk));
            FD_TRY(nn_product(c, S.Q + r0, N, m, S.d_S, m, keep, S.X + r0, N, 1.f, 0.f, n));
            std::swap(S.Q, S.X);                                  // X now holds the old basis: reuse it for W
            FD_TRY(nn_product(c, S.W + r0, N, m, S.d_S, m, keep, S.X + r0, N, 1.f, 0.f, n));
            std::swap(S.W, S.X);
            S.m = keep;
            ++S.restarts;
            FD_TRY(S.full_projection());
        } else {
            const int w = (int)pick.size();
            std::vector<float> Sx((size_t)m * w * 2);
            for (int jj = 0; jj < w; ++jj)
                for (int i = 0; i < m; ++i) {
                    Sx[i + (size_t)jj * m] = (float)Xr[i + (size_t)pick[jj] * m];
                    Sx[(size_t)m * w + i + (size_t)jj * m] = (float)(-theta[pick[jj]] * Xr[i + (size_t)pick[jj] * m]);
                }
            FD_TRY(S.upload_S(Sx));
            FD_TRY(nn_product(c, S.W + r0, N, m, S.d_S, m, w, S.R + r0, N, 1.f, 0.f, n));
            FD_TRY(nn_product(c, S.Q + r0, N, m, S.d_S + (size_t)m * w, m, w, S.R + r0, N, 1.f, 1.f, n));
        }
        auto tp4 = clk::now();
        t_restart += secs(tp3, tp4);
        // ---- orthogonalise the new block against the basis and within itself ---------------------
        int p = (int)pick.size();
        FD_TRY(S.project_out(S.R, p, S.m));
        FD_TRY(S.project_out(S.R, p, S.m));
        FD_TRY(S.orthonormalise(S.R, S.R2, p, 1e-5));
        FD_TRY(S.project_out(S.R, p, S.m));
        FD_TRY(S.orthonormalise(S.R, S.R2, p, 1e-3));
        if (p == 0) {
            // the residuals lie (numerically) inside the basis: try a random direction, give up after a few
            if (++stagnation > 3) break;
            p = std::min<int64_t>(b, N - S.m);
            FD_TRY(random_fill(c, S.R + r0, N, p, n, r0, 0xABCD1234u + (uint32_t)iter));
            FD_TRY(S.project_out(S.R, p, S.m));
            FD_TRY(S.project_out(S.R, p, S.m));
            FD_TRY(S.orthonormalise(S.R, S.R2, p, 1e-5));
            FD_TRY(S.project_out(S.R, p, S.m));
            FD_TRY(S.orthonormalise(S.R, S.R2, p, 1e-3));
            if (p == 0) break;
        }
        FD_TRY(copy_cols(c, S.R + r0, N, S.Q + (int64_t)S.m * N + r0, N, p, n));
        auto tp5 = clk::now();
        t_orth += secs(tp4, tp5);
        FD_TRY(S.apply_cols(S.m, p, b));
        auto tp6 = clk::now();
        FD_TRY(S.extend_projection(p));
        t_ext += secs(tp6, clk::now());
    }

    // ---- outputs: evecs = Q X[:, 0 : k + 1) ----------------------------------------------------------
    const int nout = std::min(nwant, nsel);
    {
        const int m = S.m;
        for (int c0 = 0; c0 < nout; c0 += S.BP) {
            const int w = std::min(S.BP, nout - c0);
            std::vector<float> Sx((size_t)m * w);
            for (int jj = 0; jj < w; ++jj)
                for (int i = 0; i < m; ++i) Sx[i + (size_t)jj * m] = (float)Xr[i + (size_t)(c0 + jj) * m];
            FD_TRY(S.upload_S(Sx));
            FD_TRY(nn_product(c, S.Q + r0, N, m, S.d_S, m, w, evecs_dev + (int64_t)c0 * ldv + r0, ldv, 1.f, 0.f, n));
        }
        FD_TRY(gather_rows(c, evecs_dev, ldv, nout));              // complete eigenvectors on every rank
        for (int i = 0; i < nwant; ++i) evals_host[i] = i < nout ? theta[i] : 0.0;
        FD_CUDA(c, cudaStreamSynchronize(c->stream));
    }
#ifdef FD_EIGS_TIMING
    fprintf(stderr, "fd_eigs: staging init %.3f s, total so far %.3f s\n", t_init, secs(t_start, clk::now()));
    fprintf(stderr, "fd_eigs: RR setup %.3f s, small eig %.3f s, residuals %.3f s, select+restart %.3f s, orthogonalise %.3f s, apply %.3f s, extend projection %.3f s\n",
            t_rr, t_eig, t_res, t_restart, t_orth, S.t_apply, t_ext);
#else
    (void)t_init; (void)t_rr; (void)t_eig; (void)t_res; (void)t_restart; (void)t_orth; (void)t_ext;
#endif
    if (info) {
        info->applies = S.applies; info->restarts = S.restarts; info->converged = nconv; info->basis_cols = S.m;
        double mx = 0.0;
        for (int i = 0; i < nout; ++i) mx = std::max(mx, resid[i]);
        info->max_residual = mx;
        info->seconds_apply = S.t_apply;
        info->seconds_total = secs(t_start, clk::now());
    }
    if (final_status != FD_OK) return fail(c, FD_ERR_NOT_CONVERGED, "fd_eigs: %d of %d pairs converged after %d applies", nconv, nwant, S.applies);
    return FD_OK;
}
