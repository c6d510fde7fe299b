// Tall-skinny dense kernels for the eigensolver (HBM-bound O(N m b) work around the quadratic
// apply): A^T B with fp64 accumulation and a deterministic two-stage reduction, C = A S updates,
// column copies and conversions.  All blocks are column-major with N rows.
#include <algorithm>

#include "fd_dense.h"

namespace fd {

namespace {

constexpr int kTnI = 64;          // output tile of the A^T B kernel: 64 (columns of A) x 32 (columns of B)
constexpr int kTnJ = 32;
constexpr int kTnRows = 64;       // rows staged per step; one step is summed in fp32, steps are added in fp64

// part[chunk][i + j * m1] = sum over this chunk's rows of A[r, i] * B[r, j].
// 128 threads, each a 4 x 4 register tile.  Products of 64 consecutive rows are accumulated in fp32 (entries of
// orthonormal columns are ~N^-1/2, so a 64-term partial sum loses ~1e-10 absolute) and every such partial sum is
// added to an fp64 accumulator, which keeps the long sum over N rows at fp64 accuracy at fp32 FMA speed.
__global__ void __launch_bounds__(128)
k_tn_partial(const float* __restrict__ A, int64_t lda, int m1, const float* __restrict__ B, int64_t ldb, int m2,
             int64_t N, int64_t rows_per_chunk, double* __restrict__ part) {
    constexpr int PA = kTnI + 4, PB = kTnJ + 4;                 // padded pitches (keep float4 alignment)
    __shared__ __align__(16) float sa[kTnRows * PA];
    __shared__ __align__(16) float sb[kTnRows * PB];
    const int ti0 = blockIdx.x * kTnI, tj0 = blockIdx.y * kTnJ;
    const int64_t r_beg = (int64_t)blockIdx.z * rows_per_chunk;
    const int64_t r_end = r_beg + rows_per_chunk < N ? r_beg + rows_per_chunk : N;
    const int ti = threadIdx.x & 15, tj = threadIdx.x >> 4;     // i0 = 4 ti, j0 = 4 tj
    double acc[4][4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = 0.0;
    for (int64_t r0 = r_beg; r0 < r_end; r0 += kTnRows) {
        __syncthreads();
        for (int t = threadIdx.x; t < kTnRows * kTnI; t += 128) {
            const int rr = t % kTnRows, cc = t / kTnRows;       // rows fastest: coalesced along a column
            const int64_t r = r0 + rr;
            sa[rr * PA + cc] = (r < r_end && ti0 + cc < m1) ? A[r + (int64_t)(ti0 + cc) * lda] : 0.f;
        }
        for (int t = threadIdx.x; t < kTnRows * kTnJ; t += 128) {
            const int rr = t % kTnRows, cc = t / kTnRows;
            const int64_t r = r0 + rr;
            sb[rr * PB + cc] = (r < r_end && tj0 + cc < m2) ? B[r + (int64_t)(tj0 + cc) * ldb] : 0.f;
        }
        __syncthreads();
        float f[4][4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int v = 0; v < 4; ++v) f[u][v] = 0.f;
#pragma unroll 8
        for (int rr = 0; rr < kTnRows; ++rr) {
            const float4 a = *reinterpret_cast<const float4*>(&sa[rr * PA + 4 * ti]);
            const float4 b = *reinterpret_cast<const float4*>(&sb[rr * PB + 4 * tj]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) f[u][v] = fmaf(av[u], bv[v], f[u][v]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[u][v] += (double)f[u][v];
    }
    double* o = part + (size_t)blockIdx.z * m1 * m2;
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int i = ti0 + 4 * ti + u, j = tj0 + 4 * tj + v;
            if (i < m1 && j < m2) o[i + (size_t)j * m1] = acc[u][v];
        }
}

__global__ void k_tn_reduce(const double* __restrict__ part, int chunks, int64_t mm, double* __restrict__ out) {
    int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= mm) return;
    double acc = 0.0;
    for (int c = 0; c < chunks; ++c) acc += part[(size_t)c * mm + e];
    out[e] = acc;
}

// C[i, c] = alpha * sum_k A[i, k] S[k, c] + beta * C[i, c] for a strip of PT columns; one thread per row.
template <int PT>
__global__ void __launch_bounds__(128)
k_nn(const float* __restrict__ A, int64_t lda, int m, const float* __restrict__ S, int lds, int p,
     float* __restrict__ C, int64_t ldc, float alpha, float beta, int64_t N) {
    __shared__ __align__(16) float ss[64 * PT];
    const int64_t i = (int64_t)blockIdx.x * 128 + threadIdx.x;
    const int c0 = blockIdx.y * PT;
    float acc[PT];
#pragma unroll
    for (int c = 0; c < PT; ++c) acc[c] = 0.f;
    for (int k0 = 0; k0 < m; k0 += 64) {
        const int kn = m - k0 < 64 ? m - k0 : 64;
        __syncthreads();
        for (int t = threadIdx.x; t < kn * PT; t += 128) {
            int kk = t / PT, cc = t % PT;
            ss[kk * PT + cc] = (c0 + cc < p) ? S[(k0 + kk) + (size_t)(c0 + cc) * lds] : 0.f;
        }
        __syncthreads();
        if (i < N) {
#pragma unroll 4
            for (int kk = 0; kk < kn; ++kk) {
                const float a = A[i + (int64_t)(k0 + kk) * lda];
#pragma unroll
                for (int c4 = 0; c4 < PT / 4; ++c4) {
                    const float4 s4 = *reinterpret_cast<const float4*>(&ss[kk * PT + 4 * c4]);
                    acc[4 * c4 + 0] = fmaf(a, s4.x, acc[4 * c4 + 0]);
                    acc[4 * c4 + 1] = fmaf(a, s4.y, acc[4 * c4 + 1]);
                    acc[4 * c4 + 2] = fmaf(a, s4.z, acc[4 * c4 + 2]);
                    acc[4 * c4 + 3] = fmaf(a, s4.w, acc[4 * c4 + 3]);
                }
            }
        }
    }
    if (i >= N) return;
#pragma unroll
    for (int c = 0; c < PT; ++c) {
        if (c0 + c < p) {
            float* o = C + i + (int64_t)(c0 + c) * ldc;
            *o = beta == 0.f ? alpha * acc[c] : fmaf(alpha, acc[c], beta * *o);
        }
    }
}

// out[c] = sum_i A[i, c]^2 in fp64; one block per column, fixed summation order (bit-reproducible).
__global__ void __launch_bounds__(1024)
k_col_sqnorms(const float* __restrict__ A, int64_t lda, int64_t N, double* __restrict__ out) {
    __shared__ double sm[1024];
    const float* col = A + (int64_t)blockIdx.x * lda;
    double acc = 0.0;
    for (int64_t i0 = 0; i0 < N; i0 += 1024 * 8) {
        float f = 0.f;                               // 8 squares in fp32, then into the fp64 accumulator
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int64_t i = i0 + (int64_t)u * 1024 + threadIdx.x;
            if (i < N) { const float v = col[i]; f = fmaf(v, v, f); }
        }
        acc += (double)f;
    }
    sm[threadIdx.x] = acc;
    __syncthreads();
    for (int off = 512; off > 0; off >>= 1) {
        if ((int)threadIdx.x < off) sm[threadIdx.x] += sm[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) out[blockIdx.x] = sm[0];
}

__global__ void k_d2f(const double* __restrict__ in, float* __restrict__ out, int64_t n, double scale) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = (float)(in[i] * scale);
}

__global__ void k_scale_cols(float* __restrict__ A, int64_t lda, int p, const float* __restrict__ f, int64_t N) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    for (int c = 0; c < p; ++c) A[i + (int64_t)c * lda] *= f[c];
}

// Counter-based uniform(-1, 1) fill for cold-start blocks (hash of (seed, element index)).
__global__ void k_random_fill(float* __restrict__ A, int64_t lda, int p, int64_t N, int64_t row0, uint32_t seed) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    for (int c = 0; c < p; ++c) {
        uint64_t z = (uint64_t)(i + row0) * 0x9E3779B97F4A7C15ull + ((uint64_t)(c + 1) << 40) + seed;
        z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull; z ^= z >> 27; z *= 0x94D049BB133111EBull; z ^= z >> 31;
        A[i + (int64_t)c * lda] = (float)((double)(z >> 11) * (2.0 / 9007199254740992.0) - 1.0);
    }
}

__global__ void k_sqrt_vec(const float* __restrict__ d, float* __restrict__ out, int64_t N) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N) out[i] = (float)sqrt((double)d[i]);
}

}  // namespace

fd_status tn_product(fd_ctx* c, const float* A, int64_t lda, int m1, const float* B, int64_t ldb, int m2, int64_t N,
                     double* out_dev, double* scratch, size_t scratch_doubles) {
    if (m1 < 1 || m2 < 1) return FD_OK;
    const size_t mm = (size_t)m1 * m2;
    if (N < 1) {                                                  // a rank that owns no rows contributes zeros
        FD_CUDA(c, cudaMemsetAsync(out_dev, 0, mm * sizeof(double), c->stream));
        return FD_OK;
    }
    // Row chunks: at least 4096 rows each for large outputs, but enough chunks to put a few blocks on every SM when the
    // output is small (a 32 x 32 Gram matrix is a single output tile: with 4096-row chunks it would run on 32 blocks).
    const int64_t out_tiles = ceil_div(m1, kTnI) * ceil_div(m2, kTnJ);
    int64_t chunks = std::max<int64_t>(ceil_div(N, 4096), ceil_div((int64_t)c->sm_count * 4, out_tiles));
    if (chunks > 256) chunks = 256;
    if (chunks > ceil_div(N, kTnRows)) chunks = ceil_div(N, kTnRows);
    if ((size_t)chunks * mm > scratch_doubles) chunks = (int64_t)(scratch_doubles / mm);
    if (chunks < 1) return fail(c, FD_ERR_WORKSPACE, "projection scratch too small for %d x %d", m1, m2);
    int64_t rpc = round_up(ceil_div(N, chunks), kTnRows);
    chunks = ceil_div(N, rpc);
    dim3 grid((unsigned)ceil_div(m1, kTnI), (unsigned)ceil_div(m2, kTnJ), (unsigned)chunks);
    k_tn_partial<<<grid, 128, 0, c->stream>>>(A, lda, m1, B, ldb, m2, N, rpc, scratch);
    FD_LAUNCH_CHECK(c, "k_tn_partial");
    k_tn_reduce<<<(unsigned)ceil_div((int64_t)mm, 256), 256, 0, c->stream>>>(scratch, (int)chunks, (int64_t)mm, out_dev);
    FD_LAUNCH_CHECK(c, "k_tn_reduce");
    return FD_OK;
}

fd_status nn_product(fd_ctx* c, const float* A, int64_t lda, int m, const float* S_dev, int lds, int p, float* C,
                     int64_t ldc, float alpha, float beta, int64_t N) {
    if (p < 1 || N < 1) return FD_OK;
    if (m < 1) return fail(c, FD_ERR_INVALID, "nn_product: m < 1");
    if (p <= 8) {
        dim3 grid((unsigned)ceil_div(N, 128), (unsigned)ceil_div(p, 8));
        k_nn<8><<<grid, 128, 0, c->stream>>>(A, lda, m, S_dev, lds, p, C, ldc, alpha, beta, N);
    } else {
        dim3 grid((unsigned)ceil_div(N, 128), (unsigned)ceil_div(p, 32));
        k_nn<32><<<grid, 128, 0, c->stream>>>(A, lda, m, S_dev, lds, p, C, ldc, alpha, beta, N);
    }
    FD_LAUNCH_CHECK(c, "k_nn");
    return FD_OK;
}

fd_status col_sqnorms(fd_ctx* c, const float* A, int64_t lda, int p, int64_t N, double* out_dev) {
    if (p < 1) return FD_OK;
    if (N < 1) {
        FD_CUDA(c, cudaMemsetAsync(out_dev, 0, (size_t)p * sizeof(double), c->stream));
        return FD_OK;
    }
    k_col_sqnorms<<<(unsigned)p, 1024, 0, c->stream>>>(A, lda, N, out_dev);
    FD_LAUNCH_CHECK(c, "k_col_sqnorms");
    return FD_OK;
}

fd_status d2f(fd_ctx* c, const double* in, float* out, int64_t n, double scale) {
    k_d2f<<<(unsigned)ceil_div(n, 256), 256, 0, c->stream>>>(in, out, n, scale);
    FD_LAUNCH_CHECK(c, "k_d2f");
    return FD_OK;
}

fd_status scale_cols(fd_ctx* c, float* A, int64_t lda, int p, const float* f_dev, int64_t N) {
    k_scale_cols<<<(unsigned)ceil_div(N, 256), 256, 0, c->stream>>>(A, lda, p, f_dev, N);
    FD_LAUNCH_CHECK(c, "k_scale_cols");
    return FD_OK;
}

fd_status random_fill(fd_ctx* c, float* A, int64_t lda, int p, int64_t N, int64_t row0, uint32_t seed) {
    if (N < 1 || p < 1) return FD_OK;
    k_random_fill<<<(unsigned)ceil_div(N, 256), 256, 0, c->stream>>>(A, lda, p, N, row0, seed);
    FD_LAUNCH_CHECK(c, "k_random_fill");
    return FD_OK;
}

fd_status sqrt_vec(fd_ctx* c, const float* d, float* out, int64_t N) {
    if (N < 1) return FD_OK;
    k_sqrt_vec<<<(unsigned)ceil_div(N, 256), 256, 0, c->stream>>>(d, out, N);
    FD_LAUNCH_CHECK(c, "k_sqrt_vec");
    return FD_OK;
}

fd_status copy_cols(fd_ctx* c, const float* src, int64_t lds, float* dst, int64_t ldd, int p, int64_t N) {
    if (p < 1 || N < 1) return FD_OK;
    FD_CUDA(c, cudaMemcpy2DAsync(dst, (size_t)ldd * 4, src, (size_t)lds * 4, (size_t)N * 4, (size_t)p,
                                 cudaMemcpyDeviceToDevice, c->stream));
    return FD_OK;
}

}  // namespace fd
