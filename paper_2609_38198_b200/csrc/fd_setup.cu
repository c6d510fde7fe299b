// O(N D) set-up: padded copy of the points, fp64 column means, mean and max of |x - mu|^2
// (the statistic Eq. 7 needs), and the O(N) elementwise / reduction helpers of the degree pass.
#include "fd_internal.h"

namespace fd {

namespace {

constexpr int kRedBlocks = 1024;

// dst[i * DP + k] = src[i * ld + k] for k < D, zero padding for D <= k < DP.
__global__ void k_pad_copy(const float* __restrict__ src, int64_t ld, int64_t n, int D, int DP, float* __restrict__ dst) {
    int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int64_t total = n * DP;
    for (; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        int64_t i = idx / DP;
        int k = (int)(idx - i * DP);
        dst[idx] = k < D ? src[i * ld + k] : 0.0f;
    }
}

// Stage 1 of the column sums: block b sums rows b, b + gridDim.x, ... into part[b * DP + k] (fp64).
__global__ void k_colsum_partial(const float* __restrict__ xs, int64_t n, int DP, double* __restrict__ part) {
    for (int k = threadIdx.x; k < DP; k += blockDim.x) {
        double acc = 0.0;
        for (int64_t i = blockIdx.x; i < n; i += gridDim.x) acc += (double)xs[i * DP + k];
        part[(size_t)blockIdx.x * DP + k] = acc;
    }
}

__global__ void k_colsum_final(const double* __restrict__ part, int blocks, int DP, int64_t n, int center, double* __restrict__ mu) {
    for (int k = threadIdx.x; k < DP; k += blockDim.x) {
        double acc = 0.0;
        for (int b = 0; b < blocks; ++b) acc += part[(size_t)b * DP + k];
        mu[k] = center ? acc / (double)n : 0.0;
    }
}

// Per block: sum and max over its rows of |x_i - mu|^2 in fp64.
__global__ void k_sqnorm_partial(const float* __restrict__ xs, int64_t n, int DP, const double* __restrict__ mu,
                                 double* __restrict__ part_sum, double* __restrict__ part_max) {
    __shared__ double s_sum[256];
    __shared__ double s_max[256];
    double acc = 0.0, mx = 0.0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        double r = 0.0;
        for (int k = 0; k < DP; ++k) {
            double v = (double)xs[i * DP + k] - mu[k];
            r += v * v;
        }
        acc += r;
        mx = r > mx ? r : mx;
    }
    s_sum[threadIdx.x] = acc; s_max[threadIdx.x] = mx;
    __syncthreads();
    for (int off = blockDim.x / 2; off > 0; off >>= 1) {
        if (threadIdx.x < off) {
            s_sum[threadIdx.x] += s_sum[threadIdx.x + off];
            double o = s_max[threadIdx.x + off];
            if (o > s_max[threadIdx.x]) s_max[threadIdx.x] = o;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) { part_sum[blockIdx.x] = s_sum[0]; part_max[blockIdx.x] = s_max[0]; }
}

__global__ void k_pow(const float* __restrict__ in, double p, float* __restrict__ out, int64_t n) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        // fp64 for the power: O(N) work, and s feeds every later product
        out[i] = (float)pow((double)in[i], p);
    }
}

__global__ void k_scale_vec(const float* __restrict__ qa, const float* __restrict__ d, float* __restrict__ s, int64_t n) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) s[i] = (float)((double)qa[i] / sqrt((double)d[i]));
}

__global__ void k_fill(float* __restrict__ out, float v, int64_t n) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = v;
}

// Stage 1: block partial sums (fixed assignment of elements to threads -> deterministic).
__global__ void k_sum_partial(const float* __restrict__ q, const double* __restrict__ rowsq, int64_t n,
                              double* __restrict__ part) {
    __shared__ double s_a[256];
    __shared__ double s_b[256];
    double a = 0.0, b = 0.0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        a += (double)q[i];
        if (rowsq) b += rowsq[i];
    }
    s_a[threadIdx.x] = a; s_b[threadIdx.x] = b;
    __syncthreads();
    for (int off = blockDim.x / 2; off > 0; off >>= 1) {
        if (threadIdx.x < off) { s_a[threadIdx.x] += s_a[threadIdx.x + off]; s_b[threadIdx.x] += s_b[threadIdx.x + off]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) { part[2 * blockIdx.x] = s_a[0]; part[2 * blockIdx.x + 1] = s_b[0]; }
}

__global__ void k_sum_final(const double* __restrict__ part, int blocks, double* __restrict__ out) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        double a = 0.0, b = 0.0;
        for (int i = 0; i < blocks; ++i) { a += part[2 * i]; b += part[2 * i + 1]; }
        out[0] = a; out[1] = b;
    }
}

__global__ void k_scale_cols_pow(const float* __restrict__ v, int64_t ldv, int cols, const float* __restrict__ d, double p,
                                 float* __restrict__ out, int64_t ldout, int64_t n) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float f = (float)pow((double)d[i], p);
    for (int c = 0; c < cols; ++c) out[i + (int64_t)c * ldout] = v[i + (int64_t)c * ldv] * f;
}

inline int grid_for(int64_t n, int block, int cap = 65535 * 8) {
    int64_t g = ceil_div(n, block);
    return (int)(g < 1 ? 1 : (g > cap ? cap : g));
}

}  // namespace

fd_status setup_points(fd_ctx* c, const float* X_dev, int64_t ldx) {
    const Layout& L = c->L;
    const int64_t N = L.N;
    k_pad_copy<<<grid_for(N * L.DP, 256, 148 * 16), 256, 0, c->stream>>>(X_dev, ldx, N, L.D, L.DP, c->xs());
    FD_LAUNCH_CHECK(c, "k_pad_copy");
    double* mu = c->at<double>(L.mu);
    double* scratch = c->at<double>(L.rowsq);     // reused: (kRedBlocks * DP) doubles needs N >= ... so cap blocks
    int blocks = (int)(N < kRedBlocks ? N : kRedBlocks);
    // scratch capacity is N doubles; blocks * DP must fit
    while ((int64_t)blocks * L.DP > N && blocks > 1) blocks /= 2;
    double* part = scratch;
    if ((int64_t)blocks * L.DP > N) {
        // tiny N with large D: fall back to the sums buffer (2 * 1024 + 8 doubles)
        part = c->at<double>(L.sums);
        blocks = 1;
        if (L.DP > 2 * 1024) return fail(c, FD_ERR_UNSUPPORTED, "D too large");
    }
    k_colsum_partial<<<blocks, 128, 0, c->stream>>>(c->xs(), N, L.DP, part);
    FD_LAUNCH_CHECK(c, "k_colsum_partial");
    k_colsum_final<<<1, 128, 0, c->stream>>>(part, blocks, L.DP, N, c->centered, mu);
    FD_LAUNCH_CHECK(c, "k_colsum_final");
    double* sums = c->at<double>(L.sums);
    int nb = grid_for(N, 256, 512);
    k_sqnorm_partial<<<nb, 256, 0, c->stream>>>(c->xs(), N, L.DP, mu, sums, sums + 1024);
    FD_LAUNCH_CHECK(c, "k_sqnorm_partial");
    double host[2048];
    FD_CUDA(c, cudaMemcpyAsync(host, sums, sizeof(double) * 2048, cudaMemcpyDeviceToHost, c->stream));
    FD_CUDA(c, cudaStreamSynchronize(c->stream));
    double tot = 0.0, mx = 0.0;
    for (int i = 0; i < nb; ++i) { tot += host[i]; if (host[1024 + i] > mx) mx = host[1024 + i]; }
    if (!(tot == tot) || !(tot < 1e300)) return fail(c, FD_ERR_NONFINITE, "non-finite input points");
    c->mean_sq = tot / (double)N;
    c->max_sq = mx;
    return FD_OK;
}

fd_status stage_rows(fd_ctx* c, const float* Xrow_dev, int64_t ldxrow, int64_t r0, int64_t n) {
    const Layout& L = c->L;
    k_pad_copy<<<grid_for(n * L.DP, 256, 148 * 16), 256, 0, c->stream>>>(Xrow_dev + r0 * ldxrow, ldxrow, n, L.D, L.DP,
                                                                         c->at<float>(L.xrow));
    FD_LAUNCH_CHECK(c, "k_pad_copy(rows)");
    // largest |x - mu|^2 among the staged rows: the Gram-form kernel's exponent budget must hold for them too, and
    // external rows may lie further from the centre than any of the context's own points (scratch: split partials)
    double* part = c->at<double>(L.part);
    const int nb = grid_for(n, 256, 512);
    k_sqnorm_partial<<<nb, 256, 0, c->stream>>>(c->at<float>(L.xrow), n, L.DP, c->at<double>(L.mu), part, part + 1024);
    FD_LAUNCH_CHECK(c, "k_sqnorm_partial(rows)");
    double host[2048];
    FD_CUDA(c, cudaMemcpyAsync(host, part, sizeof(double) * 2048, cudaMemcpyDeviceToHost, c->stream));
    FD_CUDA(c, cudaStreamSynchronize(c->stream));
    double tot = 0.0, mx = 0.0;
    for (int i = 0; i < nb; ++i) { tot += host[i]; if (host[1024 + i] > mx) mx = host[1024 + i]; }
    if (!(tot == tot) || !(tot < 1e300)) return fail(c, FD_ERR_NONFINITE, "non-finite row points");
    c->row_max_sq = mx;
    return FD_OK;
}

fd_status ew_pow(fd_ctx* c, const float* in, double p, float* out, int64_t n) {
    k_pow<<<grid_for(n, 256), 256, 0, c->stream>>>(in, p, out, n);
    FD_LAUNCH_CHECK(c, "k_pow");
    return FD_OK;
}

fd_status ew_scale_vec(fd_ctx* c, const float* qa, const float* d, float* s, int64_t n) {
    k_scale_vec<<<grid_for(n, 256), 256, 0, c->stream>>>(qa, d, s, n);
    FD_LAUNCH_CHECK(c, "k_scale_vec");
    return FD_OK;
}

fd_status ew_fill(fd_ctx* c, float* out, float v, int64_t n) {
    k_fill<<<grid_for(n, 256), 256, 0, c->stream>>>(out, v, n);
    FD_LAUNCH_CHECK(c, "k_fill");
    return FD_OK;
}

fd_status reduce_sums(fd_ctx* c, const float* q, const double* rowsq, int64_t n, double* sum_q, double* sum_sq) {
    double* sums = c->at<double>(c->L.sums);
    int nb = grid_for(n, 256, kRedBlocks);
    k_sum_partial<<<nb, 256, 0, c->stream>>>(q, rowsq, n, sums);
    FD_LAUNCH_CHECK(c, "k_sum_partial");
    k_sum_final<<<1, 32, 0, c->stream>>>(sums, nb, sums + 2 * kRedBlocks);
    FD_LAUNCH_CHECK(c, "k_sum_final");
    double host[2];
    FD_CUDA(c, cudaMemcpyAsync(host, sums + 2 * kRedBlocks, sizeof host, cudaMemcpyDeviceToHost, c->stream));
    FD_CUDA(c, cudaStreamSynchronize(c->stream));
    *sum_q = host[0]; *sum_sq = host[1];
    return FD_OK;
}

fd_status scale_cols_by_pow(fd_ctx* c, const float* v, int64_t ldv, int32_t cols, const float* d, double p,
                            float* out, int64_t ldout, int64_t n) {
    k_scale_cols_pow<<<grid_for(n, 256), 256, 0, c->stream>>>(v, ldv, cols, d, p, out, ldout, n);
    FD_LAUNCH_CHECK(c, "k_scale_cols_pow");
    return FD_OK;
}

}  // namespace fd
