// Internal declarations shared by the translation units of libfd.so.
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>
#include <string>

#include "fd.h"

namespace fd {

constexpr double kLog2e = 1.4426950408889634074;

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }
inline int64_t ceil_div(int64_t x, int64_t m) { return (x + m - 1) / m; }

// ---- tensor-core path geometry ------------------------------------------------------------
constexpr int kTileM = 128;          // rows per row tile (TMEM lanes)
constexpr int kTileJ = 128;          // columns (points j) per column tile
constexpr int kRowTilesPerCta = 2;   // two row tiles share each staged column tile

// Byte offsets of everything the library keeps inside the caller's workspace.
struct Layout {
    int64_t N = 0; int32_t D = 0, DP = 0, b_max = 0, BP = 0, m_max = 0;
    int64_t NP = 0;                  // N rounded up to the tensor-core column tile
    int32_t K16 = 0;                 // 16-wide K slabs of the augmented Gram operand
    size_t xs = 0, xrow = 0, mu = 0, q = 0, d = 0, s = 0, w = 0, rowsq = 0, sums = 0;
    size_t wp = 0, part = 0, part_floats = 0;
    size_t xp_col = 0, xp_row = 0, wt_hi = 0, wt_lo = 0, colscale = 0, status = 0;
    size_t yacc = 0;
    size_t symsum = 0;               // N 64-bit fixed-point sums of the symmetric row-sum mode
    size_t eig_q = 0, eig_w = 0, eig_x = 0, eig_r = 0, eig_t = 0, eig_small = 0, eig_small_doubles = 0;
    size_t total = 0;
};
Layout make_layout(int64_t N, int32_t D, int32_t b_max, int32_t m_max);

}  // namespace fd

struct fd_ctx {
    fd::Layout L;
    char* ws = nullptr;
    cudaStream_t stream = nullptr;
    int device = 0;
    int sm_count = 148;
    int centered = 0;
    double mean_sq = 0.0;            // N^-1 sum |x_i - mu|^2 (Eq. 7)
    double max_sq = 0.0;             // max_i |x_i - mu|^2
    double row_max_sq = 0.0;         // the same maximum over the external rows staged most recently (rectangular products)
    // current operator state (set by fd_degree)
    bool have_s = false;
    double beta = 0.0, alpha = 0.0;
    double packed_beta = -1.0;       // bandwidth the tensor-core column operand is packed for
    // options
    int opt_path = FD_PATH_AUTO;
    int opt_splits = 0;
    int opt_flush = 0;
    int opt_tail_split = 1;          // block product, single column chunk: share the last round's row pairs between two CTAs each
    int opt_sym = 1;                 // symmetric half-work degree passes on the Gram-form kernels (0 = evaluate every tile)
    int opt_jt_chunk = 0;            // column tiles per L2-resident chunk of the tensor-core block product (0 = default)
    int last_path = 0;               // kernel family that served the most recent quadratic pass (FD_PATH_SIMT / FD_PATH_TC)
    fd_precision eigs_prec = FD_PREC_FP32;   // precision mode of fd_eigs's block products (set per stage by the cascade)
    double opt_tc_max_mag = 72.0;    // largest beta' * max|x - mu|^2 the Gram-form kernel is trusted with in fp32 mode
    std::string err;
    // pinned host staging ring for the eigensolver's small uploads (allocated on the first fd_eigs, freed by fd_destroy:
    // allocating and freeing page-locked memory on every call costs tens of milliseconds)
    static constexpr int kStageSlots = 4;
    float* stage[kStageSlots] = {nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t stage_ev[kStageSlots] = {nullptr, nullptr, nullptr, nullptr};
    size_t stage_floats = 0;
    // row-sharded operation (fd_set_shard): this rank owns rows [r0, r1) of every quadratic pass
    struct Shard {
        bool on = false;
        fd_shard h{};                // callbacks, rank, world, exchange buffer
        int64_t chunk = 0, r0 = 0, r1 = 0;
    } sh;
    int64_t row0() const { return sh.on ? sh.r0 : 0; }
    int64_t rows() const { return sh.on ? sh.r1 - sh.r0 : L.N; }

    template <class T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
    float* xs() const { return at<float>(L.xs); }
    float* q() const { return at<float>(L.q); }
    float* d() const { return at<float>(L.d); }
    float* s() const { return at<float>(L.s); }
    float* w() const { return at<float>(L.w); }
};

namespace fd {

extern int64_t g_launches;           // kernels launched by this library in this process

fd_status fail(fd_ctx* c, fd_status st, const char* fmt, ...);
fd_status cuda_fail(fd_ctx* c, cudaError_t e, const char* what);
#define FD_CUDA(ctx, call)                                                     \
    do {                                                                       \
        cudaError_t e__ = (call);                                              \
        if (e__ != cudaSuccess) return fd::cuda_fail((ctx), e__, #call);       \
    } while (0)
#define FD_TRY(expr)                                                           \
    do {                                                                       \
        fd_status st__ = (expr);                                               \
        if (st__ != FD_OK) return st__;                                        \
    } while (0)
#define FD_LAUNCH_CHECK(ctx, name)                                             \
    do {                                                                       \
        ++fd::g_launches;                                                      \
        cudaError_t e__ = cudaGetLastError();                                  \
        if (e__ != cudaSuccess) return fd::cuda_fail((ctx), e__, name);        \
    } while (0)

// ---- setup (fd_setup.cu) --------------------------------------------------------------------
// Copies X (row-major, pitch ldx) into the padded N x DP layout, computes column means in fp64,
// and mean / max of |x - mu|^2.  Synchronises.
fd_status setup_points(fd_ctx* c, const float* X_dev, int64_t ldx);
// Padded copy of an external row set into the row scratch (rows [r0, r0 + n)).
fd_status stage_rows(fd_ctx* c, const float* Xrow_dev, int64_t ldxrow, int64_t r0, int64_t n);

// ---- quadratic passes -----------------------------------------------------------------------
// General product on rows [0, Nrow) of `xrow` (padded N x DP layout, device) against the context's
// points:  Y = diag(left) K diag(right) V.  V == nullptr means the ones vector (b = 1).
struct ApplyArgs {
    const float* xrow; int64_t Nrow;        // padded row points (SIMT layout, uncentred)
    bool rows_are_ctx;                      // xrow is the context's own point set
    double beta;
    const float* left; const float* right;  // may be null
    const float* V; int64_t ldv; int32_t b;
    float* Y; int64_t ldy;
    double* rowsq;                          // optional: sum_j K_ij^2 per row (rowsum mode, b = 1, V null)
    bool right_pos;                         // caller guarantees right > 0 elementwise
    bool sym_ok;                            // square pass with left == right, weights in (0, 1]: the symmetric half-work row sums may serve it
    fd_precision prec;
};
fd_status apply_simt(fd_ctx* c, const ApplyArgs& a);
fd_status apply_tc(fd_ctx* c, const ApplyArgs& a);
bool tc_supported(const fd_ctx* c, const ApplyArgs& a);
fd_status apply_dispatch(fd_ctx* c, const ApplyArgs& a);
// Body of fd_apply_general with one more promise: right_pos = the caller guarantees right > 0 elementwise, which lets a
// row-sum (V == nullptr) with a right vector take the same kernel family as the block products of the same operator.
fd_status apply_general(fd_ctx* c, double beta, const float* left_dev, const float* right_dev, bool right_pos,
                        const float* Xrow_dev, int64_t Nrow, int64_t ldxrow, const float* V_dev, int64_t ldv, int32_t b,
                        float* Y_dev, int64_t ldy, fd_precision prec, bool gather_out = true);

// ---- row-sharded operation (fd_shard.cu) ----------------------------------------------------------
// Rows [begin, end) of rank `rank`: contiguous ranges of round_up(ceil(N / world), 256) rows.
void shard_range(int64_t N, int world, int rank, int64_t* begin, int64_t* end);
// A is column-major with pitch lda and `cols` columns; on entry every rank holds valid values in its own rows, on
// return in all N rows.  No-op for an unsharded context.  cols is split into groups of at most b_max internally.
fd_status gather_rows(fd_ctx* c, float* A, int64_t lda, int cols);
// In-place sum over the ranks of n host doubles.  No-op for an unsharded context.
fd_status allreduce_host(fd_ctx* c, double* buf, int64_t n);
// Reads and clears the tensor-core kernel's status word; FD_ERR_TIMEOUT if a bounded wait expired.  Synchronises.
fd_status tc_check_status(fd_ctx* c);
// Launches a one-thread kernel whose bounded wait must expire after limit_cycles (test of the time-out plumbing).
fd_status tc_wait_selftest(fd_ctx* c, long long limit_cycles);

// ---- small kernels (fd_elementwise.cu) ------------------------------------------------------
fd_status ew_pow(fd_ctx* c, const float* in, double p, float* out, int64_t n);            // out = in^p
fd_status ew_scale_vec(fd_ctx* c, const float* qa, const float* d, float* s, int64_t n);  // s = qa * d^-1/2
fd_status ew_fill(fd_ctx* c, float* out, float v, int64_t n);
// Deterministic fp64 sums of a float vector and a double vector (two-stage tree).  Synchronises.
fd_status reduce_sums(fd_ctx* c, const float* q, const double* rowsq, int64_t n, double* sum_q, double* sum_sq);
fd_status scale_cols_by_pow(fd_ctx* c, const float* v, int64_t ldv, int32_t cols, const float* d, double p,
                            float* out, int64_t ldout, int64_t n);

}  // namespace fd
