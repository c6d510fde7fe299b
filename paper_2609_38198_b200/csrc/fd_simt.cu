// Direct-difference fp32 kernels on the FMA pipe (Eqs. 5-6 with the distance taken as
// sum_k (x_ik - x_jk)^2 instead of the Gram form of Eq. 4).
//
// This family serves the shapes where the Gram form is not accurate enough in fp32 (small D
// with large beta * |x|^2: the circle and 2-torus workloads) and every shape the tensor-core
// kernel does not cover.  One thread owns one row i; a CTA of 128 rows streams column tiles
// of 64 points through shared memory; all lanes of a warp read the same x_j / w_j (shared
// memory broadcast).  Small problems split the column range over gridDim.y and a second kernel
// adds the partials in a fixed order, so results are bit-reproducible run to run.
#include "fd_internal.h"

namespace fd {

namespace {

constexpr int kRows = 128;     // rows per CTA = threads per CTA
constexpr int kTJ = 64;        // points per column tile
constexpr int kFlushTiles = 32;  // column tiles between flushes of the fp32 tile accumulators

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// wp[j * BT + c] = right[j] * V[j + (c0 + c) * ldv] for c < bc, 0 for bc <= c < BT.
__global__ void k_pack_w(const float* __restrict__ V, int64_t ldv, const float* __restrict__ right, int64_t N,
                         int c0, int bc, int BT, float* __restrict__ wp) {
    __shared__ float tile[32][33];
    int64_t j0 = (int64_t)blockIdx.x * 32;
    int cb = blockIdx.y * 32;
    // read: threadIdx.x runs over j (coalesced along a column of V)
    for (int cc = threadIdx.y; cc < 32; cc += blockDim.y) {
        int c = cb + cc;
        int64_t j = j0 + threadIdx.x;
        float v = 0.0f;
        if (c < bc && j < N) {
            v = V ? V[j + (int64_t)(c0 + c) * ldv] : 1.0f;
            if (right) v *= right[j];
        }
        tile[cc][threadIdx.x] = v;
    }
    __syncthreads();
    // write: threadIdx.x runs over c (coalesced along a row of wp)
    for (int jj = threadIdx.y; jj < 32; jj += blockDim.y) {
        int c = cb + threadIdx.x;
        int64_t j = j0 + jj;
        if (c < BT && j < N) wp[j * BT + c] = tile[threadIdx.x][jj];
    }
}

// Block mode (BT > 0):  out[c * ld_out + i] = (left_i) * sum_j K_ij wp[j][c]   over this CTA's column range.
// Row-sum mode (BT == 0): sum_j K_ij w_j and sum_j K_ij^2 in fp64.
template <int DP4, int BT>
__global__ void __launch_bounds__(kRows)
k_simt(const float4* __restrict__ xrow, int64_t Nrow, const float4* __restrict__ xcol, int64_t N, float nbeta2,
       const float* __restrict__ wp, int64_t j_per_split, const float* __restrict__ left,
       float* __restrict__ out, int64_t ld_out, int64_t split_stride, int bstore,
       double* __restrict__ out_sum, double* __restrict__ out_sq, float* __restrict__ out_q) {
    constexpr int BTS = BT > 0 ? BT : 1;
    __shared__ float4 sx[kTJ * DP4];
    __shared__ __align__(16) float sw[kTJ * BTS];

    const int64_t i = (int64_t)blockIdx.x * kRows + threadIdx.x;
    const bool active = i < Nrow;
    float4 xi[DP4];
#pragma unroll
    for (int k = 0; k < DP4; ++k) xi[k] = active ? xrow[i * DP4 + k] : make_float4(0.f, 0.f, 0.f, 0.f);

    float acc[BTS], acc_hi[BTS];
#pragma unroll
    for (int c = 0; c < BTS; ++c) { acc[c] = 0.f; acc_hi[c] = 0.f; }
    float acc_sq = 0.f;
    double dsum = 0.0, dsq = 0.0;

    const int64_t jbeg = (int64_t)blockIdx.y * j_per_split;
    const int64_t jend = jbeg + j_per_split < N ? jbeg + j_per_split : N;
    int tiles_since_flush = 0;
    for (int64_t j0 = jbeg; j0 < jend; j0 += kTJ) {
        const int jn = (int)(jend - j0 < kTJ ? jend - j0 : kTJ);
        __syncthreads();
        for (int t = threadIdx.x; t < jn * DP4; t += kRows) sx[t] = xcol[j0 * DP4 + t];
        if (BT > 0) {
            const float4* src = reinterpret_cast<const float4*>(wp + j0 * BT);
            float4* dst = reinterpret_cast<float4*>(sw);
            for (int t = threadIdx.x; t < jn * (BTS / 4 > 0 ? BTS / 4 : 1); t += kRows) dst[t] = src[t];
        } else {
            for (int t = threadIdx.x; t < jn; t += kRows) sw[t] = wp ? wp[j0 + t] : 1.0f;
        }
        __syncthreads();
#pragma unroll 2
        for (int jj = 0; jj < jn; ++jj) {
            float h = 0.f;
#pragma unroll
            for (int k = 0; k < DP4; ++k) {
                const float4 xj = sx[jj * DP4 + k];
                float d0 = xi[k].x - xj.x, d1 = xi[k].y - xj.y, d2 = xi[k].z - xj.z, d3 = xi[k].w - xj.w;
                h = fmaf(d0, d0, h); h = fmaf(d1, d1, h); h = fmaf(d2, d2, h); h = fmaf(d3, d3, h);
            }
            const float kij = ex2_approx(h * nbeta2);
            if (BT > 0) {
#pragma unroll
                for (int c4 = 0; c4 < BTS / 4; ++c4) {
                    const float4 w = *reinterpret_cast<const float4*>(&sw[jj * BTS + 4 * c4]);
                    acc[4 * c4 + 0] = fmaf(kij, w.x, acc[4 * c4 + 0]);
                    acc[4 * c4 + 1] = fmaf(kij, w.y, acc[4 * c4 + 1]);
                    acc[4 * c4 + 2] = fmaf(kij, w.z, acc[4 * c4 + 2]);
                    acc[4 * c4 + 3] = fmaf(kij, w.w, acc[4 * c4 + 3]);
                }
            } else {
                acc[0] = fmaf(kij, sw[jj], acc[0]);
                acc_sq = fmaf(kij, kij, acc_sq);
            }
        }
        if (BT == 0) {
            // one column tile (<= 64 terms) in fp32, across tiles in fp64
            dsum += (double)acc[0]; dsq += (double)acc_sq;
            acc[0] = 0.f; acc_sq = 0.f;
        } else if (++tiles_since_flush == kFlushTiles) {
            // two-level summation keeps the rounding error of long column ranges at the 1e-7 level
#pragma unroll
            for (int c = 0; c < BTS; ++c) { acc_hi[c] += acc[c]; acc[c] = 0.f; }
            tiles_since_flush = 0;
        }
    }
    if (!active) return;
    if (BT > 0) {
        const float l = left ? left[i] : 1.0f;
        float* o = out + (int64_t)blockIdx.y * split_stride + i;
#pragma unroll
        for (int c = 0; c < BTS; ++c)
            if (c < bstore) o[(int64_t)c * ld_out] = (acc_hi[c] + acc[c]) * l;
    } else {
        if (out_q) {
            const double l = left ? (double)left[i] : 1.0;
            out_q[i] = (float)(dsum * l);
            if (out_sq) out_sq[i] = dsq;
        } else {
            out_sum[(int64_t)blockIdx.y * split_stride + i] = dsum;
            out_sq[(int64_t)blockIdx.y * split_stride + i] = dsq;
        }
    }
}

// Y[i + c * ldy] = left_i * sum_s part[s * split_stride + c * Nrow + i], s in a fixed order.
__global__ void k_reduce_block(const float* __restrict__ part, int splits, int64_t split_stride, int64_t Nrow, int bc,
                               const float* __restrict__ left, float* __restrict__ Y, int64_t ldy) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int c = blockIdx.y;
    if (i >= Nrow || c >= bc) return;
    float acc = 0.f;
    for (int s = 0; s < splits; ++s) acc += part[(int64_t)s * split_stride + (int64_t)c * Nrow + i];
    Y[i + (int64_t)c * ldy] = acc * (left ? left[i] : 1.0f);
}

__global__ void k_reduce_rowsum(const double* __restrict__ psum, const double* __restrict__ psq, int splits,
                                int64_t split_stride, int64_t Nrow, const float* __restrict__ left,
                                float* __restrict__ q, double* __restrict__ rowsq) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= Nrow) return;
    double a = 0.0, b = 0.0;
    for (int s = 0; s < splits; ++s) { a += psum[(int64_t)s * split_stride + i]; b += psq[(int64_t)s * split_stride + i]; }
    q[i] = (float)(a * (left ? (double)left[i] : 1.0));
    if (rowsq) rowsq[i] = b;
}

template <int DP4, int BT>
void launch_simt(dim3 grid, cudaStream_t st, const float* xrow, int64_t Nrow, const float* xcol, int64_t N, float nbeta2,
                 const float* wp, int64_t jps, const float* left, float* out, int64_t ld_out, int64_t split_stride, int bstore,
                 double* out_sum, double* out_sq, float* out_q) {
    k_simt<DP4, BT><<<grid, kRows, 0, st>>>(reinterpret_cast<const float4*>(xrow), Nrow,
                                            reinterpret_cast<const float4*>(xcol), N, nbeta2, wp, jps, left, out, ld_out,
                                            split_stride, bstore, out_sum, out_sq, out_q);
}

template <int DP4>
bool launch_simt_bt(int BT, dim3 grid, cudaStream_t st, const float* xrow, int64_t Nrow, const float* xcol, int64_t N,
                    float nbeta2, const float* wp, int64_t jps, const float* left, float* out, int64_t ld_out,
                    int64_t split_stride, int bstore, double* out_sum, double* out_sq, float* out_q) {
#define FD_CASE(B) case B: launch_simt<DP4, B>(grid, st, xrow, Nrow, xcol, N, nbeta2, wp, jps, left, out, ld_out, split_stride, bstore, out_sum, out_sq, out_q); return true;
    switch (BT) {
        FD_CASE(0) FD_CASE(4) FD_CASE(8) FD_CASE(16) FD_CASE(32) FD_CASE(64)
        default: return false;
    }
#undef FD_CASE
}

bool launch_simt_any(int DP4, int BT, dim3 grid, cudaStream_t st, const float* xrow, int64_t Nrow, const float* xcol,
                     int64_t N, float nbeta2, const float* wp, int64_t jps, const float* left, float* out, int64_t ld_out,
                     int64_t split_stride, int bstore, double* out_sum, double* out_sq, float* out_q) {
#define FD_CASE(Dq) case Dq: return launch_simt_bt<Dq>(BT, grid, st, xrow, Nrow, xcol, N, nbeta2, wp, jps, left, out, ld_out, split_stride, bstore, out_sum, out_sq, out_q);
    switch (DP4) {
        FD_CASE(1) FD_CASE(2) FD_CASE(3) FD_CASE(4) FD_CASE(5) FD_CASE(6) FD_CASE(7) FD_CASE(8)
        default: return false;
    }
#undef FD_CASE
}

int pick_bt(int bc) { return bc <= 4 ? 4 : bc <= 8 ? 8 : bc <= 16 ? 16 : bc <= 32 ? 32 : 64; }

}  // namespace

fd_status apply_simt(fd_ctx* c, const ApplyArgs& a) {
    const Layout& L = c->L;
    const int DP4 = L.DP / 4;
    if (DP4 > 8) return fail(c, FD_ERR_UNSUPPORTED, "SIMT path covers D <= 32 (got %d)", L.D);
    const int64_t N = L.N, Nrow = a.Nrow;
    const float nbeta2 = (float)(-a.beta * kLog2e);
    const int64_t row_tiles = ceil_div(Nrow, kRows);
    // split the column range when the row tiles alone cannot fill the GPU (4 CTAs of 128 threads per SM)
    const int64_t target = (int64_t)c->sm_count * 4;
    int64_t splits = c->opt_splits > 0 ? c->opt_splits : (row_tiles >= target ? 1 : ceil_div(target, row_tiles));
    const int64_t col_tiles = ceil_div(N, kTJ);
    if (splits > col_tiles) splits = col_tiles;
    if (splits > 64) splits = 64;
    if (splits < 1) splits = 1;

    const bool rowsum = (a.V == nullptr);
    if (rowsum) {
        // w_j = right_j (or 1); outputs q (float, left-scaled) and optionally sum_j K^2 (double)
        int64_t need = splits * 2 * Nrow * 2;                      // doubles counted in floats
        if (splits > 1 && (size_t)need > L.part_floats) splits = 1;
        const int64_t jps = round_up(ceil_div(N, splits), kTJ);
        splits = ceil_div(N, jps);
        dim3 grid((unsigned)row_tiles, (unsigned)splits);
        bool ok;
        if (splits == 1) {
            double* sq = a.rowsq;
            ok = launch_simt_any(DP4, 0, grid, c->stream, a.xrow, Nrow, c->xs(), N, nbeta2, a.right, jps, a.left, nullptr, 0, 0, 1,
                                 nullptr, sq, a.Y);
            if (!ok) return fail(c, FD_ERR_UNSUPPORTED, "no SIMT instantiation");
            FD_LAUNCH_CHECK(c, "k_simt(rowsum)");
        } else {
            double* psum = c->at<double>(L.part);
            double* psq = psum + splits * Nrow;
            ok = launch_simt_any(DP4, 0, grid, c->stream, a.xrow, Nrow, c->xs(), N, nbeta2, a.right, jps, nullptr, nullptr, 0,
                                 Nrow, 1, psum, psq, nullptr);
            if (!ok) return fail(c, FD_ERR_UNSUPPORTED, "no SIMT instantiation");
            FD_LAUNCH_CHECK(c, "k_simt(rowsum, split)");
            k_reduce_rowsum<<<(unsigned)ceil_div(Nrow, 256), 256, 0, c->stream>>>(psum, psq, (int)splits, Nrow, Nrow, a.left,
                                                                                a.Y, a.rowsq);
            FD_LAUNCH_CHECK(c, "k_reduce_rowsum");
        }
        return FD_OK;
    }

    float* wp = c->at<float>(L.wp);
    for (int c0 = 0; c0 < a.b; c0 += 64) {
        const int bc = a.b - c0 < 64 ? a.b - c0 : 64;
        const int BT = pick_bt(bc);
        if (BT > L.BP) return fail(c, FD_ERR_WORKSPACE, "column tile %d wider than the provisioned block buffers (%d)", BT, L.BP);
        dim3 pg((unsigned)ceil_div(N, 32), (unsigned)ceil_div(BT, 32));
        k_pack_w<<<pg, dim3(32, 8), 0, c->stream>>>(a.V, a.ldv, a.right, N, c0, bc, BT, wp);
        FD_LAUNCH_CHECK(c, "k_pack_w");
        int64_t sp = splits;
        if (sp > 1 && (size_t)(sp * BT * Nrow) > L.part_floats) sp = (int64_t)(L.part_floats / ((size_t)BT * Nrow));
        if (sp < 1) sp = 1;
        const int64_t jps = round_up(ceil_div(N, sp), kTJ);
        sp = ceil_div(N, jps);
        dim3 grid((unsigned)row_tiles, (unsigned)sp);
        float* Yc = a.Y + (int64_t)c0 * a.ldy;
        bool ok;
        if (sp == 1) {
            ok = launch_simt_any(DP4, BT, grid, c->stream, a.xrow, Nrow, c->xs(), N, nbeta2, wp, jps, a.left, Yc, a.ldy, 0, bc,
                                 nullptr, nullptr, nullptr);
            if (!ok) return fail(c, FD_ERR_UNSUPPORTED, "no SIMT instantiation");
            FD_LAUNCH_CHECK(c, "k_simt(block)");
            continue;
        }
        float* part = c->at<float>(L.part);
        ok = launch_simt_any(DP4, BT, grid, c->stream, a.xrow, Nrow, c->xs(), N, nbeta2, wp, jps, nullptr, part, Nrow,
                             (int64_t)BT * Nrow, BT, nullptr, nullptr, nullptr);
        if (!ok) return fail(c, FD_ERR_UNSUPPORTED, "no SIMT instantiation");
        FD_LAUNCH_CHECK(c, "k_simt(block, split)");
        dim3 rg((unsigned)ceil_div(Nrow, 256), (unsigned)bc);
        k_reduce_block<<<rg, 256, 0, c->stream>>>(part, (int)sp, (int64_t)BT * Nrow, Nrow, bc, a.left, Yc, a.ldy);
        FD_LAUNCH_CHECK(c, "k_reduce_block");
    }
    return FD_OK;
}

}  // namespace fd

// ================================================================================================
// fd_apply_general_static: the split direct-difference block product for callers that cannot
// allocate device memory.
//
// Some hosts of this library hold no allocator they may call at the point where they need a
// kernel product: code running inside another framework's stream callback or capture-adjacent
// region, a plug-in that is handed input and output buffers only, a process whose memory pool
// is owned and sized by someone else.  For them every byte of scratch the ordinary entry points
// take from the caller's workspace lives here instead, in one file-scope device array of fixed
// size that each GPU loading the library keeps until the process exits.
//
// Scratch layout inside the array (floats): padded copy of the points, packed right-hand block,
// split-column partial sums.  Nothing in it has to start at zero: every word a launch reads was
// written earlier in the same call.  All calls share the array, so two calls that overlap on the
// GPU (different streams, or different host threads) race; serialise them.
namespace fd {
namespace {

constexpr size_t kStaticXs = (size_t)FD_STATIC_MAX_N * FD_STATIC_MAX_D;          // padded points
constexpr size_t kStaticWp = (size_t)FD_STATIC_MAX_N * FD_STATIC_MAX_B;          // packed right block
constexpr size_t kStaticPart = (size_t)3 << 19;                                  // split partials (6 MiB)
constexpr size_t kStaticFloats = kStaticXs + kStaticWp + kStaticPart;            // 8 MiB in total

static __device__ __align__(256) float g_static_scratch[kStaticFloats];

// Device address of the array per device ordinal, resolved on the first call made with that device current.
// (In host code the symbol's name is only a handle; the address a kernel can use comes from the runtime.)
constexpr int kMaxDevices = 64;
float* g_static_ptr[kMaxDevices] = {};

__global__ void k_static_pad_copy(const float* __restrict__ src, int64_t ld, int64_t n, int D, int DP, float* __restrict__ dst) {
    int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t total = n * DP;
    for (; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = idx / DP;
        const int k = (int)(idx - i * DP);
        dst[idx] = k < D ? src[i * ld + k] : 0.0f;
    }
}

fd_status static_fail(char* errbuf, size_t errlen, fd_status st, const char* fmt, long long a = 0, long long b = 0) {
    if (errbuf && errlen) snprintf(errbuf, errlen, fmt, a, b);
    return st;
}

}  // namespace
}  // namespace fd

extern "C" fd_status fd_apply_general_static(const float* X_dev, int64_t N, int32_t D, int64_t ldx, double beta,
                                             const float* left_dev, const float* right_dev, const float* V_dev,
                                             int64_t ldv, int32_t b, float* Y_dev, int64_t ldy, void* cuda_stream,
                                             char* errbuf, size_t errbuf_len) {
    using namespace fd;
    if (errbuf && errbuf_len) errbuf[0] = 0;
    if (!X_dev || !V_dev || !Y_dev) return static_fail(errbuf, errbuf_len, FD_ERR_INVALID, "X, V and Y must be non-null");
    if (N < 1 || D < 1 || b < 1 || ldx < D || ldv < N || ldy < N || !(beta > 0) || !(beta < 1e30))
        return static_fail(errbuf, errbuf_len, FD_ERR_INVALID, "bad size, pitch or beta");
    if (N > FD_STATIC_MAX_N) return static_fail(errbuf, errbuf_len, FD_ERR_UNSUPPORTED, "N = %lld exceeds FD_STATIC_MAX_N = %lld", (long long)N, FD_STATIC_MAX_N);
    if (D > FD_STATIC_MAX_D) return static_fail(errbuf, errbuf_len, FD_ERR_UNSUPPORTED, "D = %lld exceeds FD_STATIC_MAX_D = %lld", D, FD_STATIC_MAX_D);
    if (b > FD_STATIC_MAX_B) return static_fail(errbuf, errbuf_len, FD_ERR_UNSUPPORTED, "b = %lld exceeds FD_STATIC_MAX_B = %lld", b, FD_STATIC_MAX_B);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    // set-up, once per device: resolve the device address of the scratch array
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return static_fail(errbuf, errbuf_len, FD_ERR_CUDA, "cudaGetDevice failed or device ordinal out of range");
    if (!g_static_ptr[dev]) {
        float* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) return static_fail(errbuf, errbuf_len, FD_ERR_CUDA, "cudaGetSymbolAddress failed (%lld)", (long long)e);
        g_static_ptr[dev] = ptr;
    }
    float* xs = g_static_ptr[dev];
    float* wp = xs + kStaticXs;
    float* part = wp + kStaticWp;

    const int DP = (int)round_up(D, 4), DP4 = DP / 4;
    const int BT = pick_bt(b);
    const float nbeta2 = (float)(-beta * kLog2e);
    int grid_copy = (int)ceil_div(N * DP, 256);
    k_static_pad_copy<<<grid_copy, 256, 0, stream>>>(X_dev, ldx, N, D, DP, xs);
    ++g_launches;
    dim3 pg((unsigned)ceil_div(N, 32), (unsigned)ceil_div(BT, 32));
    k_pack_w<<<pg, dim3(32, 8), 0, stream>>>(V_dev, ldv, right_dev, N, 0, b, BT, wp);
    ++g_launches;
    // split the column range so that ~600 CTAs run, within the partials' capacity
    const int64_t row_tiles = ceil_div(N, kRows);
    int64_t sp = row_tiles >= 592 ? 1 : ceil_div(592, row_tiles);
    const int64_t cap = (int64_t)(kStaticPart / ((size_t)BT * (size_t)N));
    if (sp > cap) sp = cap;
    if (sp > ceil_div(N, kTJ)) sp = ceil_div(N, kTJ);
    if (sp < 1) sp = 1;
    const int64_t jps = round_up(ceil_div(N, sp), kTJ);
    sp = ceil_div(N, jps);
    dim3 grid((unsigned)row_tiles, (unsigned)sp);
    bool ok;
    if (sp == 1) {
        ok = launch_simt_any(DP4, BT, grid, stream, xs, N, xs, N, nbeta2, wp, jps, left_dev, Y_dev, ldy, 0, b, nullptr, nullptr, nullptr);
        ++g_launches;
    } else {
        ok = launch_simt_any(DP4, BT, grid, stream, xs, N, xs, N, nbeta2, wp, jps, nullptr, part, N, (int64_t)BT * N, BT, nullptr,
                             nullptr, nullptr);
        ++g_launches;
        if (ok) {
            dim3 rg((unsigned)ceil_div(N, 256), (unsigned)b);
            k_reduce_block<<<rg, 256, 0, stream>>>(part, (int)sp, (int64_t)BT * N, N, b, left_dev, Y_dev, ldy);
            ++g_launches;
        }
    }
    if (!ok) return static_fail(errbuf, errbuf_len, FD_ERR_UNSUPPORTED, "no kernel instantiation for this D, b");
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return static_fail(errbuf, errbuf_len, FD_ERR_CUDA, "kernel launch failed (%lld)", (long long)e);
    return FD_OK;
}
