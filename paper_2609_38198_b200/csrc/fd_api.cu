// C-ABI entry points: context, degree passes, block product.  Argument checking and
// dispatch only; every O(N^2) and O(N) step runs in this library's own kernels.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "fd_internal.h"

namespace fd {

int64_t g_launches = 0;

fd_status fail(fd_ctx* c, fd_status st, const char* fmt, ...) {
    if (c) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        c->err = buf;
    }
    return st;
}

fd_status cuda_fail(fd_ctx* c, cudaError_t e, const char* what) {
    return fail(c, FD_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

static size_t carve(size_t& cur, size_t bytes) {
    size_t off = cur;
    cur += (size_t)round_up((int64_t)bytes, 256);
    return off;
}

Layout make_layout(int64_t N, int32_t D, int32_t b_max, int32_t m_max) {
    Layout L;
    L.N = N; L.D = D; L.b_max = b_max; L.m_max = m_max;
    L.DP = (int32_t)round_up(D, 4);
    // block-width-dependent buffers are sized by the widest column tile a kernel can launch for b <= b_max
    // (16, 32 or a multiple of 64), not by b_max itself: both kernel families pad a chunk of 33..64 columns to 64
    L.BP = b_max <= 16 ? 16 : b_max <= 32 ? 32 : (int32_t)round_up(b_max, 64);
    L.NP = round_up(N, kTileM * kRowTilesPerCta);
    L.K16 = (int32_t)ceil_div(D + 4, 16);
    size_t cur = 0;
    L.xs = carve(cur, (size_t)N * L.DP * 4);
    L.xrow = carve(cur, (size_t)N * L.DP * 4);
    L.mu = carve(cur, (size_t)(L.DP + 8) * 8);
    L.q = carve(cur, (size_t)N * 4);
    L.d = carve(cur, (size_t)N * 4);
    L.s = carve(cur, (size_t)N * 4);
    L.w = carve(cur, (size_t)N * 4);
    L.rowsq = carve(cur, (size_t)N * 8);
    L.sums = carve(cur, (size_t)(2 * 1024 + 8) * 8);
    L.wp = carve(cur, (size_t)N * L.BP * 4);
    // split-J partials of the SIMT kernel: only small problems split, so this is O(b_max), not O(N b_max)
    L.part_floats = (size_t)640 * 128 * (size_t)L.BP;
    L.part = carve(cur, L.part_floats * 4);
    // tensor-core operands: fp16 hi|lo rows of the augmented points, transposed fp16 hi / lo blocks
    L.xp_col = carve(cur, (size_t)L.NP * L.K16 * 64);
    L.xp_row = carve(cur, (size_t)L.NP * L.K16 * 64);
    L.wt_hi = carve(cur, (size_t)L.BP * L.NP * 2);
    L.wt_lo = carve(cur, (size_t)L.BP * L.NP * 2);
    L.colscale = carve(cur, (size_t)(L.BP + 8) * 4 * 2);
    L.status = carve(cur, 256);
    L.symsum = carve(cur, (size_t)N * 8);
    if (m_max > 0) {
        L.eig_q = carve(cur, (size_t)N * m_max * 4);
        L.eig_w = carve(cur, (size_t)N * m_max * 4);
        L.eig_x = carve(cur, (size_t)N * m_max * 4);
        L.eig_r = carve(cur, (size_t)N * L.BP * 4);
        L.eig_t = carve(cur, (size_t)N * L.BP * 4);
        // projection output + small right factors (2 * m_max * max(m_max, BP) doubles), then the per-chunk
        // partials of the A^T B kernel (up to 256 row chunks of m_max x BP)
        const size_t mm = (size_t)m_max * (size_t)(m_max > L.BP ? m_max : L.BP);
        size_t chunks = (size_t)ceil_div(N, 4096);
        if (chunks > 256) chunks = 256;
        if (chunks < 16) chunks = 16;     // small problems split finer so that a projection still fills the GPU
        L.eig_small_doubles = 2 * mm + chunks * mm;
        L.eig_small = carve(cur, L.eig_small_doubles * 8);
    }
    L.total = cur;
    return L;
}

fd_status apply_dispatch(fd_ctx* c, const ApplyArgs& a) {
    int path = c->opt_path;
    if (path == FD_PATH_TC) {
        if (!tc_supported(c, a)) return fail(c, FD_ERR_UNSUPPORTED, "tensor-core path does not cover this shape");
        c->last_path = FD_PATH_TC;
        return apply_tc(c, a);
    }
    if (path == FD_PATH_AUTO && tc_supported(c, a)) { c->last_path = FD_PATH_TC; return apply_tc(c, a); }
    c->last_path = FD_PATH_SIMT;
    return apply_simt(c, a);
}

}  // namespace fd

using namespace fd;

extern "C" {

size_t fd_workspace_bytes(int64_t N, int32_t D, int32_t b_max, int32_t m_max) {
    if (N < 1 || D < 1 || D > FD_MAX_D || b_max < 1 || b_max > 256 || m_max < 0) return 0;
    return make_layout(N, D, b_max, m_max).total;
}

fd_status fd_create(fd_ctx** out, const float* X_dev, int64_t N, int32_t D, int64_t ldx, int32_t center,
                    int32_t b_max, int32_t m_max, void* ws_dev, size_t ws_bytes, void* cuda_stream) {
    if (!out) return FD_ERR_INVALID;
    *out = nullptr;
    if (!X_dev || !ws_dev || N < 1 || D < 1 || ldx < D || b_max < 1 || b_max > 256 || m_max < 0)
        return FD_ERR_INVALID;
    if (D > FD_MAX_D) return FD_ERR_UNSUPPORTED;                 // no kernel covers more coordinates
    if (N > ((int64_t)1 << 31) - 1024) return FD_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(ws_dev) & 255) != 0) return FD_ERR_INVALID;
    Layout L = make_layout(N, D, b_max, m_max);
    if (ws_bytes < L.total) return FD_ERR_WORKSPACE;
    fd_ctx* c = new (std::nothrow) fd_ctx();
    if (!c) return FD_ERR_INVALID;
    c->L = L;
    c->ws = static_cast<char*>(ws_dev);
    c->stream = static_cast<cudaStream_t>(cuda_stream);
    c->centered = center ? 1 : 0;
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    if (e != cudaSuccess) { delete c; return FD_ERR_CUDA; }
    e = cudaMemsetAsync(c->at<unsigned int>(L.status), 0, 256, c->stream);
    if (e != cudaSuccess) { delete c; return FD_ERR_CUDA; }
    fd_status st = setup_points(c, X_dev, ldx);
    if (st != FD_OK) { delete c; return st; }
    *out = c;
    return FD_OK;
}

fd_status fd_destroy(fd_ctx* ctx) {
    if (ctx) {
        for (int i = 0; i < fd_ctx::kStageSlots; ++i) {
            if (ctx->stage_ev[i]) cudaEventDestroy(ctx->stage_ev[i]);
            if (ctx->stage[i]) cudaFreeHost(ctx->stage[i]);
        }
    }
    delete ctx;
    return FD_OK;
}

fd_status fd_set_option(fd_ctx* c, const char* name, double v) {
    if (!c || !name) return FD_ERR_INVALID;
    if (!strcmp(name, "path")) {
        if (v != FD_PATH_AUTO && v != FD_PATH_SIMT && v != FD_PATH_TC) return fail(c, FD_ERR_INVALID, "path must be 0, 1 or 2");
        c->opt_path = (int)v;
    } else if (!strcmp(name, "splits")) {
        if (v < 0 || v > 64) return fail(c, FD_ERR_INVALID, "splits out of range");
        c->opt_splits = (int)v;
    } else if (!strcmp(name, "flush")) {
        if (v < 0 || v > 1 << 20) return fail(c, FD_ERR_INVALID, "flush out of range");
        c->opt_flush = (int)v;
    } else if (!strcmp(name, "tail_split")) {
        if (v != 0 && v != 1) return fail(c, FD_ERR_INVALID, "tail_split must be 0 or 1");
        c->opt_tail_split = (int)v;
    } else if (!strcmp(name, "sym")) {
        if (v != 0 && v != 1) return fail(c, FD_ERR_INVALID, "sym must be 0 or 1");
        c->opt_sym = (int)v;
    } else if (!strcmp(name, "jt_chunk")) {
        if (v < 0 || v > 1 << 24) return fail(c, FD_ERR_INVALID, "jt_chunk out of range");
        c->opt_jt_chunk = (int)v;
    } else if (!strcmp(name, "tc_max_mag")) {
        if (!(v > 0)) return fail(c, FD_ERR_INVALID, "tc_max_mag must be positive");
        c->opt_tc_max_mag = v;
    } else if (!strcmp(name, "wait_selftest")) {
        if (!(v >= 1000) || v > 4e9) return fail(c, FD_ERR_INVALID, "wait_selftest: limit in cycles, 1e3..4e9");
        return tc_wait_selftest(c, (long long)v);
    } else {
        return fail(c, FD_ERR_INVALID, "unknown option %s", name);
    }
    return FD_OK;
}

fd_status fd_get_option(const fd_ctx* c, const char* name, double* v) {
    if (!c || !name || !v) return FD_ERR_INVALID;
    if (!strcmp(name, "path")) *v = c->opt_path;
    else if (!strcmp(name, "splits")) *v = c->opt_splits;
    else if (!strcmp(name, "flush")) *v = c->opt_flush;
    else if (!strcmp(name, "sym")) *v = c->opt_sym;
    else if (!strcmp(name, "tail_split")) *v = c->opt_tail_split;
    else if (!strcmp(name, "tc_max_mag")) *v = c->opt_tc_max_mag;
    else if (!strcmp(name, "last_path")) *v = c->last_path;
    else if (!strcmp(name, "tc_cycles")) {
        // SM cycles the first CTA of the most recent tensor-core block product spent (synchronises)
        long long cyc = 0;
        if (cudaStreamSynchronize(c->stream) != cudaSuccess ||
            cudaMemcpy(&cyc, c->at<unsigned int>(c->L.status) + 2, 8, cudaMemcpyDeviceToHost) != cudaSuccess) return FD_ERR_CUDA;
        *v = (double)cyc;
    }
    else if (!strcmp(name, "mean_sq")) *v = c->mean_sq;
    else if (!strcmp(name, "max_sq")) *v = c->max_sq;
    else if (!strcmp(name, "beta")) *v = c->beta;
    else return FD_ERR_INVALID;
    return FD_OK;
}

fd_status fd_beta0(fd_ctx* c, double* beta0_host) {
    if (!c || !beta0_host) return FD_ERR_INVALID;
    double est = c->mean_sq > 0 ? 1.0 / (2.0 * c->mean_sq) : 0.1;
    *beta0_host = est < 0.1 ? est : 0.1;
    return FD_OK;
}

fd_status fd_degree(fd_ctx* c, double beta, double alpha, fd_precision prec, float* q_dev, float* d_dev,
                    float* s_dev, double* S_off_host, double* S_off_2beta_host) {
    if (!c) return FD_ERR_INVALID;
    if (!(beta > 0) || !(beta < 1e30) || !(alpha >= 0) || alpha > 4) return fail(c, FD_ERR_INVALID, "beta or alpha out of range");
    if (prec != FD_PREC_FP32 && prec != FD_PREC_FAST) return fail(c, FD_ERR_INVALID, "bad precision");
    const int64_t N = c->L.N;
    c->have_s = false;
    double* rowsq = c->at<double>(c->L.rowsq);
    // pass 1: q = K 1 (and sum_j K_ij^2 per row)
    // (the rows this rank owns: all of them unless the context is row-sharded)
    const int64_t r0 = c->row0(), n = c->rows();
    ApplyArgs a{};
    a.xrow = c->xs() + r0 * c->L.DP; a.Nrow = n; a.rows_are_ctx = true; a.beta = beta;
    a.left = nullptr; a.right = nullptr; a.V = nullptr; a.ldv = N; a.b = 1;
    a.Y = c->q() + r0; a.ldy = N; a.rowsq = rowsq + r0; a.prec = prec;
    a.sym_ok = !c->sh.on;                                        // K = K^T, unit weights
    if (n > 0) FD_TRY(apply_dispatch(c, a));
    double sums[2] = {0.0, 0.0};
    if (n > 0) FD_TRY(reduce_sums(c, c->q() + r0, rowsq + r0, n, &sums[0], &sums[1]));
    FD_TRY(allreduce_host(c, sums, 2));
    FD_TRY(gather_rows(c, c->q(), N, 1));
    const double sum_q = sums[0], sum_sq = sums[1];
    if (!(sum_q == sum_q) || !(sum_q < 1e300)) return fail(c, FD_ERR_NONFINITE, "non-finite degree sum");
    if (alpha == 0.0) {
        // d = q, s = q^-1/2
        FD_CUDA(c, cudaMemcpyAsync(c->d(), c->q(), (size_t)N * 4, cudaMemcpyDeviceToDevice, c->stream));
        FD_TRY(ew_pow(c, c->q(), -0.5, c->s(), N));
    } else {
        // pass 2: d = q^-alpha * K q^-alpha
        FD_TRY(ew_pow(c, c->q(), -alpha, c->w(), N));
        ApplyArgs a2 = a;
        a2.left = c->w() + r0; a2.right = c->w(); a2.Y = c->d() + r0; a2.rowsq = nullptr; a2.right_pos = true;       // (sym_ok stays: left = right = q^-alpha in (0, 1])
        if (n > 0) FD_TRY(apply_dispatch(c, a2));
        FD_TRY(gather_rows(c, c->d(), N, 1));
        FD_TRY(ew_scale_vec(c, c->w(), c->d(), c->s(), N));
    }
    if (q_dev) FD_CUDA(c, cudaMemcpyAsync(q_dev, c->q(), (size_t)N * 4, cudaMemcpyDeviceToDevice, c->stream));
    if (d_dev) FD_CUDA(c, cudaMemcpyAsync(d_dev, c->d(), (size_t)N * 4, cudaMemcpyDeviceToDevice, c->stream));
    if (s_dev) FD_CUDA(c, cudaMemcpyAsync(s_dev, c->s(), (size_t)N * 4, cudaMemcpyDeviceToDevice, c->stream));
    FD_TRY(tc_check_status(c));
    // the diagonal of K is exactly 1 in both sums
    if (S_off_host) *S_off_host = sum_q - (double)N;
    if (S_off_2beta_host) *S_off_2beta_host = sum_sq - (double)N;
    c->beta = beta; c->alpha = alpha; c->have_s = true;
    return FD_OK;
}

static fd_status check_block(fd_ctx* c, const float* p, int64_t ld, int64_t rows, const char* what) {
    if (!p) return fail(c, FD_ERR_INVALID, "%s is null", what);
    if (ld < rows) return fail(c, FD_ERR_INVALID, "%s: leading dimension %lld < rows %lld", what, (long long)ld, (long long)rows);
    if ((reinterpret_cast<uintptr_t>(p) & 3) != 0) return fail(c, FD_ERR_INVALID, "%s is not 4-byte aligned", what);
    return FD_OK;
}

fd_status fd_apply_general(fd_ctx* c, double beta, const float* left_dev, const float* right_dev,
                           const float* Xrow_dev, int64_t Nrow, int64_t ldxrow, const float* V_dev, int64_t ldv,
                           int32_t b, float* Y_dev, int64_t ldy, fd_precision prec) {
    return fd::apply_general(c, beta, left_dev, right_dev, false, Xrow_dev, Nrow, ldxrow, V_dev, ldv, b, Y_dev, ldy, prec);
}

}  // extern "C"

namespace fd {

fd_status apply_general(fd_ctx* c, double beta, const float* left_dev, const float* right_dev, bool right_pos,
                        const float* Xrow_dev, int64_t Nrow, int64_t ldxrow, const float* V_dev, int64_t ldv, int32_t b,
                        float* Y_dev, int64_t ldy, fd_precision prec, bool gather_out) {
    if (!c) return FD_ERR_INVALID;
    if (!(beta > 0) || !(beta < 1e30)) return fail(c, FD_ERR_INVALID, "beta out of range");
    if (prec != FD_PREC_FP32 && prec != FD_PREC_FAST) return fail(c, FD_ERR_INVALID, "bad precision");
    if (b < 1 || b > c->L.b_max) return fail(c, FD_ERR_INVALID, "b = %d outside 1..b_max = %d", b, c->L.b_max);
    if (!V_dev && b != 1) return fail(c, FD_ERR_INVALID, "V null requires b = 1");
    const int64_t N = c->L.N;
    if (!Xrow_dev) Nrow = N;
    if (Nrow < 1) return fail(c, FD_ERR_INVALID, "Nrow < 1");
    if (Xrow_dev && ldxrow < c->L.D) return fail(c, FD_ERR_INVALID, "ldxrow < D");
    if (V_dev) FD_TRY(check_block(c, V_dev, ldv, N, "V"));
    FD_TRY(check_block(c, Y_dev, ldy, Nrow, "Y"));
    if (V_dev) {
        const char* v0 = (const char*)V_dev; const char* v1 = v0 + ((size_t)ldv * (b - 1) + N) * 4;
        const char* y0 = (const char*)Y_dev; const char* y1 = y0 + ((size_t)ldy * (b - 1) + Nrow) * 4;
        bool overlap = v0 < y1 && y0 < v1;
        if (overlap && ldv == ldy) {
            // two row ranges of one pitched panel (e.g. old rows in, new rows out, of the same basis) never touch
            const int64_t off = ((const float*)Y_dev - (const float*)V_dev);
            const int64_t r = ((off % ldv) + ldv) % ldv;          // first row of Y inside V's panel
            if (r >= N && r + Nrow <= ldv) overlap = false;
        }
        if (overlap) return fail(c, FD_ERR_INVALID, "V and Y overlap");
    }
    ApplyArgs a{};
    a.beta = beta; a.right = right_dev; a.V = V_dev; a.ldv = ldv; a.b = b; a.prec = prec; a.rowsq = nullptr;
    a.right_pos = right_pos;
    if (!Xrow_dev) {
        // square product: the rows this rank owns (all of them unless the context is row-sharded)
        const int64_t r0 = c->row0(), n = c->rows();
        a.xrow = c->xs() + r0 * c->L.DP; a.Nrow = n; a.rows_are_ctx = true;
        a.left = left_dev ? left_dev + r0 : nullptr; a.Y = Y_dev + r0; a.ldy = ldy;
        if (n > 0) FD_TRY(apply_dispatch(c, a));
        if (gather_out) FD_TRY(gather_rows(c, Y_dev, ldy, b));
        return FD_OK;
    }
    // rectangular product: stage the external rows chunk by chunk through the row scratch
    for (int64_t r0 = 0; r0 < Nrow; r0 += N) {
        int64_t n = Nrow - r0 < N ? Nrow - r0 : N;
        FD_TRY(stage_rows(c, Xrow_dev, ldxrow, r0, n));
        a.xrow = c->at<float>(c->L.xrow); a.Nrow = n; a.rows_are_ctx = false;
        a.left = left_dev ? left_dev + r0 : nullptr; a.Y = Y_dev + r0; a.ldy = ldy;
        FD_TRY(apply_dispatch(c, a));
    }
    return FD_OK;
}

}  // namespace fd

extern "C" {

fd_status fd_apply(fd_ctx* c, const float* V_dev, int64_t ldv, int32_t b, float* Y_dev, int64_t ldy, fd_precision prec) {
    if (!c) return FD_ERR_INVALID;
    if (!c->have_s) return fail(c, FD_ERR_INVALID, "fd_apply before fd_degree");
    if (!V_dev) return fail(c, FD_ERR_INVALID, "V is null");
    return fd_apply_general(c, c->beta, c->s(), c->s(), nullptr, c->L.N, 0, V_dev, ldv, b, Y_dev, ldy, prec);
}

fd_status fd_scale_by_degree(fd_ctx* c, const float* v_dev, int64_t ldv, int32_t cols, double power,
                             float* out_dev, int64_t ldout) {
    if (!c) return FD_ERR_INVALID;
    if (!c->have_s) return fail(c, FD_ERR_INVALID, "fd_scale_by_degree before fd_degree");
    if (cols < 1) return fail(c, FD_ERR_INVALID, "cols < 1");
    FD_TRY(check_block(c, v_dev, ldv, c->L.N, "v"));
    FD_TRY(check_block(c, out_dev, ldout, c->L.N, "out"));
    return scale_cols_by_pow(c, v_dev, ldv, cols, c->d(), power, out_dev, ldout, c->L.N);
}

fd_status fd_synchronize(fd_ctx* c) {
    if (!c) return FD_ERR_INVALID;
    return tc_check_status(c);
}

const char* fd_status_string(fd_status st) {
    switch (st) {
        case FD_OK: return "ok";
        case FD_ERR_INVALID: return "invalid argument";
        case FD_ERR_WORKSPACE: return "workspace too small or feature not provisioned";
        case FD_ERR_CUDA: return "CUDA runtime error";
        case FD_ERR_NOT_CONVERGED: return "eigensolver did not converge within max_applies";
        case FD_ERR_PERRON_WALL: return "Perron gap at or below the precision wall";
        case FD_ERR_UNSUPPORTED: return "unsupported shape";
        case FD_ERR_TIMEOUT: return "bounded device wait expired";
        case FD_ERR_NONFINITE: return "non-finite value";
        case FD_ERR_COMM: return "exchange callback of a row-sharded context failed";
    }
    return "unknown status";
}

const char* fd_last_error(const fd_ctx* c) { return c ? c->err.c_str() : ""; }
int32_t fd_version(void) { return 100; }
int64_t fd_launch_count(void) { return fd::g_launches; }

}  // extern "C"
