// Bandwidth flow (Sec. 2.3, Eqs. 8-14) and the out-of-sample extension the (n, beta) ladder
// uses (Sec. 1).  Host logic around fd_degree / fd_eigs / fd_apply_general; the only kernel
// here is the elementwise division that finishes the extension.
#include <algorithm>
#include <cmath>
#include <vector>

#include "fd_internal.h"

namespace fd {
namespace {

constexpr double kKappaP = 10.0;     // Eq. 11
constexpr int kPExponent = 6;        // Eq. 11

// out[i + j * ldout] /= lambda[j] * den[i]
__global__ void k_nystrom_finish(float* __restrict__ out, int64_t ldout, int m, const float* __restrict__ den,
                                 const double* __restrict__ lambda, int64_t n) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const double dn = (double)den[i];
    for (int j = 0; j < m; ++j) {
        float* o = out + i + (int64_t)j * ldout;
        *o = (float)((double)*o / (lambda[j] * dn));
    }
}

double median_of(std::vector<double> v) {
    std::sort(v.begin(), v.end());
    const size_t n = v.size();
    return n % 2 ? v[n / 2] : 0.5 * (v[n / 2 - 1] + v[n / 2]);
}

// Eqs. 8-14 for one probe.
void fill_potential(fd_probe& p, const double* lam, int k, int64_t N, double eta) {
    std::vector<double> act(k);
    for (int j = 1; j <= k; ++j) act[j - 1] = -std::log(lam[j] / lam[0]);
    p.V_bias = median_of(act);                                             // Eq. 8
    p.n_eff = p.S_off * p.S_off / ((double)N * p.S_off_2beta);             // Eq. 9
    p.V_stat = 1.0 / std::sqrt(p.n_eff * p.V_bias);                        // Eq. 10
    p.g_P = (lam[0] - lam[1]) / std::fabs(lam[0]);
    p.V_mach = p.g_P > 0 ? std::pow(kKappaP * eta / p.g_P, kPExponent) : INFINITY;   // Eq. 11
    p.V = p.V_bias + p.V_stat + p.V_mach;                                  // Eq. 13
    p.d_hat = -2.0 * (std::log(p.S_off_2beta) - std::log(p.S_off)) / std::log(2.0);  // Eq. 14
    p.lambda1 = lam[1];
}

bool brackets(const fd_probe& a, const fd_probe& b, const fd_probe& c) {
    return b.V <= std::min(a.V, c.V) && c.V_bias < a.V_bias && (c.V_stat > a.V_stat || c.V_mach > a.V_mach);
}

double parabola_vertex(const fd_probe& a, const fd_probe& b, const fd_probe& c) {
    const double x0 = std::log(a.beta), x1 = std::log(b.beta), x2 = std::log(c.beta);
    const double d01 = (b.V - a.V) / (x1 - x0), d12 = (c.V - b.V) / (x2 - x1);
    const double c2 = (d12 - d01) / (x2 - x0);
    double xv = x1;
    if (c2 > 0) xv = 0.5 * (x0 + x1) - d01 / (2.0 * c2);
    xv = std::min(std::max(xv, x0), x2);
    return std::exp(xv);
}

}  // namespace
}  // namespace fd

using namespace fd;

namespace fd {
namespace {

// One sweep of the flow in one precision mode: probes beta_start * ratio^j with the stage's eta and tolerance.
// log has room for cap records; *n_out receives the number written.
fd_status flow_stage(fd_ctx* c, const fd_flow_opts* o, fd_precision prec, double eta, double tol, double beta,
                     const float* Q0_dev, int64_t ldq0, int32_t q0_cols, fd_probe* log, int cap, int32_t* n_out,
                     int32_t* outcome, double* beta_x_host, double* evals_host, float* evecs_dev, int64_t ldv) {
    *n_out = 0;
    const int64_t N = c->L.N;
    const int k = o->k;
    std::vector<double> lam(k + 1);
    int n = 0;
    bool have_prev = false;
    struct PrecGuard {                                   // fd_eigs applies M in the stage's mode; restored on every exit
        fd_ctx* c; fd_precision saved;
        ~PrecGuard() { c->eigs_prec = saved; }
    } guard{c, c->eigs_prec};
    c->eigs_prec = prec;

    auto run_probe = [&](double b_, fd_probe& rec, bool warm) -> fd_status {
        rec = fd_probe{};
        rec.beta = b_;
        FD_TRY(fd_degree(c, b_, o->alpha, prec, nullptr, nullptr, nullptr, &rec.S_off, &rec.S_off_2beta));
        fd_eigs_info info{};
        const float* q0 = nullptr; int64_t ld0 = 0; int32_t nc0 = 0;
        if (warm && have_prev) { q0 = evecs_dev; ld0 = ldv; nc0 = k + 1; }
        else if (Q0_dev && !have_prev) { q0 = Q0_dev; ld0 = ldq0; nc0 = q0_cols; }
        fd_status est = fd_eigs(c, k, o->b, tol, o->max_applies, q0, ld0, nc0, lam.data(), evecs_dev, ldv, &info);
        // a probe whose residuals stalled above tol (noise-smeared spectrum at the operator's accuracy floor) still
        // gives eigenvalues far more accurate than the potential needs: keep it, flagged, if its residuals are small
        if (est == FD_ERR_NOT_CONVERGED && info.max_residual <= std::max(1e-4, 100.0 * tol) * std::fabs(lam[0])) { rec.flags |= 4; est = FD_OK; }
        if (est != FD_OK) return est;
        have_prev = true;
        rec.applies = info.applies;
        fill_potential(rec, lam.data(), k, N, eta);
        return FD_OK;
    };
    auto finish = [&](double bx, int oc, bool rerun) -> fd_status {
        if (rerun) {
            // bring the context and the outputs back to the selected probe
            fd_probe tmp;
            FD_TRY(run_probe(bx, tmp, true));
        }
        for (int i = 0; i <= k; ++i) evals_host[i] = lam[i];
        *beta_x_host = bx; *outcome = oc; *n_out = n;
        return FD_OK;
    };

    while (beta <= o->beta_max * (1 + 1e-12)) {
        if (n >= cap - 1) return fail(c, FD_ERR_INVALID, "fd_beta_flow: probe log full");
        fd_probe& rec = log[n];
        FD_TRY(run_probe(beta, rec, o->warm_start != 0));
        ++n;
        if (!(rec.g_P > kKappaP * eta)) {                                   // Eq. 12
            rec.flags |= 1;
            int last_safe = -1;
            for (int i = n - 2; i >= 0; --i)
                if (!(log[i].flags & 1)) { last_safe = i; break; }
            if (last_safe < 0) {
                *n_out = n; *outcome = FD_FLOW_PERRON_WALL; *beta_x_host = NAN;
                return fail(c, FD_ERR_PERRON_WALL, "first probe already at the Perron wall (g_P = %.3e)", rec.g_P);
            }
            return finish(log[last_safe].beta, FD_FLOW_PERRON_WALL, true);
        }
        if (n == 2 && log[1].V > log[0].V) return finish(log[0].beta, FD_FLOW_LEFT_EDGE, true);
        if (n >= 3 && brackets(log[n - 3], log[n - 2], log[n - 1])) {
            const double bv = parabola_vertex(log[n - 3], log[n - 2], log[n - 1]);
            fd_probe& fin = log[n];
            FD_TRY(run_probe(bv, fin, o->warm_start != 0));
            fin.flags |= 2;
            ++n;
            return finish(bv, FD_FLOW_VERTEX, false);
        }
        beta *= o->ratio;
    }
    if (n == 0) return fail(c, FD_ERR_INVALID, "fd_beta_flow: beta_start beyond beta_max");
    return finish(log[n - 1].beta, FD_FLOW_RIGHT_EDGE, false);
}

}  // namespace
}  // namespace fd

extern "C" fd_status fd_beta_flow(fd_ctx* c, const fd_flow_opts* o, const float* Q0_dev, int64_t ldq0, int32_t q0_cols,
                                  fd_probe* log, int32_t* n_probes, int32_t* outcome, double* beta_x_host,
                                  double* evals_host, float* evecs_dev, int64_t ldv) {
    if (!c) return FD_ERR_INVALID;
    if (!o || !log || !n_probes || *n_probes < 4 || !outcome || !beta_x_host || !evals_host || !evecs_dev)
        return fail(c, FD_ERR_INVALID, "fd_beta_flow: null argument or log capacity < 4");
    if (o->k < 1 || !(o->ratio > 1.0) || !(o->beta_max > 0)) return fail(c, FD_ERR_INVALID, "fd_beta_flow: bad options");
    const int cap = *n_probes;
    double beta = o->beta_start;
    if (!(beta > 0)) FD_TRY(fd_beta0(c, &beta));
    return flow_stage(c, o, FD_PREC_FP32, o->eta > 0 ? o->eta : 1e-7, o->tol, beta, Q0_dev, ldq0, q0_cols, log, cap, n_probes,
                      outcome, beta_x_host, evals_host, evecs_dev, ldv);
}

extern "C" fd_status fd_beta_flow_cascade(fd_ctx* c, const fd_flow_opts* o, const fd_cascade_stage* stages, int32_t n_stages,
                                          const float* Q0_dev, int64_t ldq0, int32_t q0_cols, fd_probe* log,
                                          int32_t* n_probes, int32_t* stage_first_probe, int32_t* outcome,
                                          double* beta_x_host, double* evals_host, float* evecs_dev, int64_t ldv) {
    if (!c) return FD_ERR_INVALID;
    if (!o || !stages || n_stages < 1 || n_stages > 8 || !log || !n_probes || *n_probes < 4 * n_stages || !stage_first_probe ||
        !outcome || !beta_x_host || !evals_host || !evecs_dev)
        return fail(c, FD_ERR_INVALID, "fd_beta_flow_cascade: null argument, bad stage count or log capacity < 4 per stage");
    if (o->k < 1 || !(o->ratio > 1.0) || !(o->beta_max > 0)) return fail(c, FD_ERR_INVALID, "fd_beta_flow_cascade: bad options");
    for (int s = 0; s < n_stages; ++s)
        if (stages[s].prec != FD_PREC_FP32 && stages[s].prec != FD_PREC_FAST) return fail(c, FD_ERR_INVALID, "fd_beta_flow_cascade: bad precision");
    const int cap = *n_probes;
    int used = 0;
    *n_probes = 0;
    double beta = o->beta_start;
    if (!(beta > 0)) FD_TRY(fd_beta0(c, &beta));
    for (int s = 0; s < n_stages; ++s) {
        const bool fast = stages[s].prec == FD_PREC_FAST;
        const double eta = stages[s].eta > 0 ? stages[s].eta : (fast ? 1e-3 : 1e-7);
        const double tol = stages[s].tol > 0 ? stages[s].tol : (fast ? 1e-3 : 1e-6);
        stage_first_probe[s] = used;
        int32_t n_stage = 0;
        // the first stage starts from the caller's basis, every later one from the previous stage's eigenvectors
        const float* q0 = s == 0 ? Q0_dev : evecs_dev;
        const int64_t ld0 = s == 0 ? ldq0 : ldv;
        const int32_t nc0 = s == 0 ? q0_cols : o->k + 1;
        fd_status st = flow_stage(c, o, stages[s].prec, eta, tol, beta, q0, ld0, nc0, log + used, cap - used, &n_stage, outcome,
                                  beta_x_host, evals_host, evecs_dev, ldv);
        used += n_stage;
        *n_probes = used;
        stage_first_probe[s + 1] = used;
        if (st != FD_OK) return st;
        beta = *beta_x_host / o->ratio;                  // the next stage restarts one grid step below this selection
    }
    return FD_OK;
}

extern "C" fd_status fd_nystrom(fd_ctx* c, const float* Xnew_dev, int64_t Nnew, int64_t ldxnew, const float* psi_dev,
                                int64_t ldpsi, int32_t m, const double* lambda_host, float* out_dev, int64_t ldout) {
    if (!c) return FD_ERR_INVALID;
    if (!c->have_s) return fail(c, FD_ERR_INVALID, "fd_nystrom before fd_degree");
    if (!Xnew_dev || !psi_dev || !lambda_host || !out_dev || Nnew < 1 || m < 1 || m > 1024)
        return fail(c, FD_ERR_INVALID, "fd_nystrom: bad argument");
    if (ldxnew < c->L.D || ldpsi < c->L.N || ldout < Nnew) return fail(c, FD_ERR_INVALID, "fd_nystrom: bad pitch");
    for (int j = 0; j < m; ++j)
        if (!(std::fabs(lambda_host[j]) > 1e-30)) return fail(c, FD_ERR_INVALID, "fd_nystrom: zero eigenvalue");
    const int64_t N = c->L.N;
    // right scaling q^-alpha (scratch vector w), eigenvalues to the device (scratch: sums buffer)
    FD_TRY(ew_pow(c, c->q(), -c->alpha, c->w(), N));
    double* lam_dev = c->at<double>(c->L.sums);
    FD_CUDA(c, cudaMemcpyAsync(lam_dev, lambda_host, sizeof(double) * (size_t)m, cudaMemcpyHostToDevice, c->stream));
    FD_CUDA(c, cudaStreamSynchronize(c->stream));
    float* den = c->at<float>(c->L.rowsq);                                  // N doubles of scratch = room for N floats
    for (int64_t r0 = 0; r0 < Nnew; r0 += N) {
        const int64_t n = std::min(N, Nnew - r0);
        const float* xr = Xnew_dev + r0 * ldxnew;
        // the denominator's right vector q^-alpha is positive: it may take the same kernel family as the numerators
        FD_TRY(apply_general(c, c->beta, nullptr, c->w(), true, xr, n, ldxnew, nullptr, N, 1, den, n, FD_PREC_FP32));
        for (int c0 = 0; c0 < m; c0 += c->L.b_max) {
            const int w = std::min<int>(c->L.b_max, m - c0);
            FD_TRY(fd_apply_general(c, c->beta, nullptr, c->w(), xr, n, ldxnew, psi_dev + (int64_t)c0 * ldpsi, ldpsi, w,
                                    out_dev + r0 + (int64_t)c0 * ldout, ldout, FD_PREC_FP32));
        }
        k_nystrom_finish<<<(unsigned)ceil_div(n, 256), 256, 0, c->stream>>>(out_dev + r0, ldout, m, den, lam_dev, n);
        FD_LAUNCH_CHECK(c, "k_nystrom_finish");
    }
    FD_CUDA(c, cudaStreamSynchronize(c->stream));
    return FD_OK;
}

extern "C" fd_status fd_ladder_start(fd_ctx* old_level, fd_ctx* new_level, const float* Xnew_dev, int64_t ldxnew,
                                     const float* evecs_old_dev, int64_t ldv_old, int32_t m, const double* evals_host,
                                     float* Q0_dev, int64_t ldq0) {
    if (!old_level || !new_level) return FD_ERR_INVALID;
    fd_ctx* c = new_level;
    if (!old_level->have_s || !new_level->have_s) return fail(c, FD_ERR_INVALID, "fd_ladder_start: both levels need fd_degree first");
    const int64_t n_old = old_level->L.N, n_new = new_level->L.N;
    if (n_new < n_old || old_level->L.D != new_level->L.D) return fail(c, FD_ERR_INVALID, "fd_ladder_start: levels are not nested");
    if (!Xnew_dev || !evecs_old_dev || !evals_host || !Q0_dev || m < 1 || ldv_old < n_old || ldq0 < n_new || ldxnew < c->L.D)
        return fail(c, FD_ERR_INVALID, "fd_ladder_start: bad argument");
    // Markov vectors on the old points, written into the first n_old rows of Q0
    FD_TRY(scale_cols_by_pow(old_level, evecs_old_dev, ldv_old, m, old_level->d(), -0.5, Q0_dev, ldq0, n_old));
    // their extension to the points that are new at this level
    if (n_new > n_old) {
        fd_status st = fd_nystrom(old_level, Xnew_dev + n_old * ldxnew, n_new - n_old, ldxnew, Q0_dev, ldq0, m, evals_host,
                                  Q0_dev + n_old, ldq0);
        if (st != FD_OK) return fail(c, st, "fd_ladder_start: extension failed: %s", fd_last_error(old_level));
    }
    // back to the symmetric operator's coordinates at the new level: v = d_new^1/2 * psi
    FD_TRY(scale_cols_by_pow(new_level, Q0_dev, ldq0, m, new_level->d(), 0.5, Q0_dev, ldq0, n_new));
    FD_CUDA(c, cudaStreamSynchronize(c->stream));
    return FD_OK;
}
