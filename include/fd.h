/* fd.h -- C ABI of the B200-native FlashDiffusion hot path.
 *
 * The library evaluates, without ever storing the N x N kernel, the Gaussian
 * application of Sec. 2.1-2.2 of the paper
 *
 *     K_ij = exp(-beta * |x_i - x_j|^2)                                  (Eq. 1)
 *     q = K 1,  K_alpha = diag(q)^-alpha K diag(q)^-alpha,  d = K_alpha 1,
 *     s = q^-alpha * d^-1/2,   M = diag(s) K diag(s)                     (Eq. 2)
 *     Y = M V = diag(s) K (diag(s) V)                                    (Eq. 3)
 *
 * tile by tile as in Eqs. 5-6, plus the drivers that sit on it: the block
 * Rayleigh-Ritz / Lanczos eigensolver (Sec. 2.3, first paragraph), the
 * bandwidth flow (Eqs. 7-14) and the out-of-sample extension used by the
 * (n, beta) ladder (Sec. 1).
 *
 * Conventions
 * -----------
 * Pointers: a name ending in _dev is DEVICE memory of the GPU that was current
 *   at fd_create; _host is host memory.  The library never allocates device
 *   memory: every device buffer, including the workspace, is allocated and
 *   freed by the caller and only borrowed for the duration of a call.  The
 *   library owns the fd_ctx host object alone.
 * Points:  X is row-major N x D float32 with row pitch ldx (elements).
 * Blocks:  V, Y, Q0 and eigenvector outputs are COLUMN-major float32,
 *   element (i, c) at [i + c * ld], ld >= number of rows.
 * Streams: all work is enqueued on the cudaStream_t given at fd_create (passed
 *   as void*; NULL = the legacy default stream).  fd_apply and fd_apply_general
 *   return without synchronising; calls that return host scalars synchronise
 *   that stream.
 * Errors:  every entry point returns an fd_status; argument errors are found
 *   before any launch; nothing aborts or throws.  There is no CPU fallback.
 * Threads: a context is not thread-safe.
 * k:       counts NONTRIVIAL eigenpairs; the Perron pair (eigenvalue 1) is
 *   returned in slot 0, so k + 1 pairs come back (Sec. 2.3, Sec. 3).
 */
#ifndef FD_H_
#define FD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fd_ctx fd_ctx;

typedef enum {
    FD_OK = 0,
    FD_ERR_INVALID = 1,        /* bad argument (null, range, alignment, ld)                    */
    FD_ERR_WORKSPACE = 2,      /* workspace too small / feature not provisioned at fd_create   */
    FD_ERR_CUDA = 3,           /* a CUDA runtime call failed; see fd_last_error                */
    FD_ERR_NOT_CONVERGED = 4,  /* fd_eigs hit max_applies; outputs hold the best Ritz pairs    */
    FD_ERR_PERRON_WALL = 5,    /* Eq. 12 failed: g_P <= kappa_P * eta                          */
    FD_ERR_UNSUPPORTED = 6,    /* shape outside what the kernels cover                         */
    FD_ERR_TIMEOUT = 7,        /* a bounded device-side wait expired (status word set)         */
    FD_ERR_NONFINITE = 8,      /* non-finite input or intermediate detected                    */
    FD_ERR_COMM = 9            /* an exchange callback of a row-sharded context reported failure */
} fd_status;

typedef enum {
    FD_PREC_FP32 = 0,          /* fp32-grade result (relative Frobenius error <= 1e-5)         */
    FD_PREC_FAST = 1           /* single 16-bit operands for K and V (<= 3e-3)                 */
} fd_precision;

/* Which kernel family serves the quadratic passes (fd_set_option "path"). */
enum { FD_PATH_AUTO = 0, FD_PATH_SIMT = 1, FD_PATH_TC = 2 };

/* Largest number of coordinates per point the kernels cover: D <= 32 on both kernel families, 33..FD_MAX_D on the
 * Gram-form tensor-core family only (a pass whose bandwidth exceeds that family's accuracy budget, beta * log2(e) *
 * max|x - mu|^2 >= "tc_max_mag", then returns FD_ERR_UNSUPPORTED).  fd_create refuses D > FD_MAX_D. */
#define FD_MAX_D 60

/* Bytes of device workspace fd_create needs.  O(N (D + b_max + m_max)); no N^2 term.
 * b_max: widest block passed to fd_apply / fd_apply_general (1..256).
 * m_max: basis capacity for fd_eigs (columns); 0 if fd_eigs will not be called. */
size_t fd_workspace_bytes(int64_t N, int32_t D, int32_t b_max, int32_t m_max);

/* Creates a context over N points.  Copies X into the library's padded layouts inside the
 * workspace (so X_dev may be released after the call), computes the column means and, if
 * center != 0, the centred copy used by the Gram-form kernels (Eq. 4) and by fd_beta0.
 * ws_dev must be 256-byte aligned and stay valid until fd_destroy.  Synchronises once. */
fd_status fd_create(fd_ctx** out, const float* X_dev, int64_t N, int32_t D, int64_t ldx,
                    int32_t center, int32_t b_max, int32_t m_max,
                    void* ws_dev, size_t ws_bytes, void* cuda_stream);
fd_status fd_destroy(fd_ctx* ctx);

/* Tuning / test knobs by name: "path" (FD_PATH_*), "splits" (0 = auto), "flush" (column tiles
 * between accumulator flushes of the tensor-core kernels; 0 = default: 1 in the fp32-grade mode, whose eigenvalue budget
 * the tensor core's round-toward-zero accumulation would otherwise eat, 8 in the reduced-precision mode), "tc_max_mag" (largest beta * log2(e) *
 * max|x - mu|^2 for which the Gram-form tensor-core kernel serves the fp32 mode), "jt_chunk" (column
 * tiles per L2-resident chunk of the tensor-core block product), "sym" (1, default: the degree passes on the Gram-form
 * kernels use K = K^T and evaluate only the tiles on or above the diagonal -- each off-diagonal tile gives the row sums
 * of its rows and, transposed, of its columns, N (N + 128) / 2 exponentials instead of N^2; 0: every tile; row-sharded
 * contexts always evaluate every tile of their rows), "tail_split" (1, default: in a block product with a single column
 * chunk the row pairs of the last, partly filled round of CTAs -- all pairs when there are fewer than CTAs -- are
 * shared by two CTAs each, half the columns per CTA, partial results added atomically; 0: off), "wait_selftest"
 * (value = limit in SM cycles: enqueues
 * a one-thread kernel whose bounded wait on a barrier that nothing completes must expire; the next
 * fd_synchronize then returns FD_ERR_TIMEOUT and the context stays usable).  fd_get_option also reports "last_path" (the
 * family that served the latest pass), "beta", "mean_sq", "max_sq" and "tc_cycles" (SM cycles the first CTA of the most
 * recent tensor-core quadratic kernel spent on its work items; synchronises; with the kernel's wall time it
 * gives the SM clock the kernel actually ran at).  Unknown name -> FD_ERR_INVALID. */
fd_status fd_set_option(fd_ctx* ctx, const char* name, double value);
fd_status fd_get_option(const fd_ctx* ctx, const char* name, double* value_host);

/* Eq. 7: beta0 = min(0.1, 1 / (2 * mean_i |x_i - mu|^2)). */
fd_status fd_beta0(fd_ctx* ctx, double* beta0_host);

/* Degree passes at bandwidth beta (Sec. 2.1 "entry fee"): q = K 1 and, for alpha != 0,
 * d = q^-alpha * K q^-alpha; then s = q^-alpha * d^-1/2 (alpha = 0: d = q).  Sets the
 * context's current (beta, alpha, q, d, s), which fd_apply and fd_eigs use afterwards.
 * q_dev, d_dev, s_dev: N floats each, any may be NULL.  S_off_host receives
 * sum_{i != j} K_ij and S_off_2beta_host the same sum for the kernel at 2 beta (obtained in
 * the same pass from sum K_ij^2, Sec. 2.3); either may be NULL.  Synchronises. */
fd_status fd_degree(fd_ctx* ctx, double beta, double alpha, fd_precision prec,
                    float* q_dev, float* d_dev, float* s_dev,
                    double* S_off_host, double* S_off_2beta_host);

/* Eq. 3: Y = diag(s) K diag(s) V with the context's current beta and s.  b in 1..b_max.
 * V_dev and Y_dev must not overlap.  Asynchronous. */
fd_status fd_apply(fd_ctx* ctx, const float* V_dev, int64_t ldv, int32_t b,
                   float* Y_dev, int64_t ldy, fd_precision prec);

/* Waits for everything the context has enqueued on its stream and reports a device-side
 * bounded-wait expiry of an earlier asynchronous call as FD_ERR_TIMEOUT (the status is cleared
 * once reported). */
fd_status fd_synchronize(fd_ctx* ctx);

/* The single primitive of Sec. 2.1 with both diagonal scalings explicit:
 *   Y = diag(left) K(Xrow, X) diag(right) V,  K_ij = exp(-beta |xrow_i - x_j|^2).
 * left_dev (Nrow floats) and right_dev (N floats) may be NULL (= ones); V_dev may be NULL
 * (= the ones vector, b must be 1).  Xrow_dev NULL means the context's own points
 * (Nrow = N); otherwise row-major Nrow x D with pitch ldxrow, in the same coordinates as the
 * X given to fd_create (this is the rectangular product the out-of-sample extension needs).
 * Does not change the context's current beta.  Asynchronous. */
fd_status fd_apply_general(fd_ctx* ctx, double beta, const float* left_dev, const float* right_dev,
                           const float* Xrow_dev, int64_t Nrow, int64_t ldxrow,
                           const float* V_dev, int64_t ldv, int32_t b,
                           float* Y_dev, int64_t ldy, fd_precision prec);

typedef struct {
    int32_t applies;           /* block applications of M performed                          */
    int32_t restarts;          /* thick restarts                                              */
    int32_t converged;         /* leading pairs (of k + 1) with residual <= tol * theta_0     */
    int32_t basis_cols;        /* columns in the basis at exit                                */
    double  max_residual;      /* largest residual norm among the k + 1 returned pairs       */
    double  seconds_apply;     /* host wall time spent inside the quadratic applies          */
    double  seconds_total;
} fd_eigs_info;

/* Leading k + 1 eigenpairs of M = diag(s) K diag(s) at the context's current (beta, s) by block
 * Krylov / Rayleigh-Ritz with residual expansion and thick restart (the paper names block
 * implicitly restarted Lanczos and gives no further detail; Sec. 2.3).  b = block size,
 * tol = residual tolerance relative to theta_0, Q0_dev = optional warm-start basis (N x q0_cols,
 * need not be orthonormal).  evals_host: k + 1 doubles, descending.  evecs_dev: N x (k + 1)
 * column-major, orthonormal.  Needs m_max >= 2 (k + 1) + b at fd_create; the thick restart keeps 3/5 of m_max, so a
 * capacity near 3 (k + 1) + 2 b keeps room for the rest of an eigenvalue cluster that the request cuts (on the
 * 6-torus, k = 128 cuts a 160-fold cluster: 129 of 129 pairs converge in 43 block products with m_max = 576, 73 of
 * 129 in 125 with 384).  info->converged counts the LEADING pairs below tol.  On FD_ERR_NOT_CONVERGED the outputs hold
 * the best current Ritz pairs.  Synchronous. */
fd_status fd_eigs(fd_ctx* ctx, int32_t k, int32_t b, double tol, int32_t max_applies,
                  const float* Q0_dev, int64_t ldq0, int32_t q0_cols,
                  double* evals_host, float* evecs_dev, int64_t ldv, fd_eigs_info* info);

/* One record per probe of the bandwidth flow (Eqs. 8-14). */
typedef struct {
    double beta, S_off, S_off_2beta, n_eff, d_hat, V_bias, V_stat, V_mach, V, g_P;
    double lambda1;            /* first nontrivial eigenvalue                                 */
    int32_t applies;           /* block applies the probe's eigensolve took                   */
    int32_t flags;             /* bit 0: inadmissible (Eq. 12); bit 1: final (vertex) probe;  */
                               /* bit 2: eigensolve stalled above tol (residuals <= max(1e-4, 100 tol)) */
} fd_probe;

typedef struct {
    double beta_start;         /* <= 0: use Eq. 7                                             */
    double beta_max;           /* grid end (inclusive)                                        */
    double ratio;              /* 2 (dyadic)                                                  */
    double alpha;
    double eta;                /* precision scale of Eq. 11; <= 0: 1e-7 (fp32)                */
    double tol;                /* eigensolver tolerance                                       */
    int32_t k, b, max_applies;
    int32_t warm_start;        /* 1: start each probe from the previous probe's eigenvectors  */
} fd_flow_opts;

enum { FD_FLOW_VERTEX = 0, FD_FLOW_PERRON_WALL = 1, FD_FLOW_LEFT_EDGE = 2, FD_FLOW_RIGHT_EDGE = 3 };

/* Dyadic bandwidth flow of Sec. 2.3: probes beta_start * ratio^j, potential of Eq. 13, bracket
 * rule and quadratic vertex, Perron wall of Eq. 12.  On return the context's current beta is
 * beta_x and evals/evecs hold that probe's pairs.  log: capacity *n_probes records in, number
 * written out.  Q0_dev: optional warm start for the first probe.  Synchronous. */
fd_status fd_beta_flow(fd_ctx* ctx, const fd_flow_opts* opts, const float* Q0_dev, int64_t ldq0,
                       int32_t q0_cols, fd_probe* log, int32_t* n_probes, int32_t* outcome,
                       double* beta_x_host, double* evals_host, float* evecs_dev, int64_t ldv);

/* Precision cascade of Sec. 2.3 (last paragraph): one sweep per requested data type, in order; the state a stage
 * selects initialises the next stage and the final bandwidth and eigenpairs are the last stage's.  Here a stage is a
 * precision mode of the kernels (FD_PREC_FAST explores, FD_PREC_FP32 resolves) with its own precision scale eta in
 * Eqs. 11-12 (footnote to Eq. 11: 8e-3 bf16, 1e-3 tf32, 1e-7 fp32; the reduced-precision mode here carries fp16
 * operands and behaves like the tf32 entry) and its own eigensolver tolerance (a reduced-precision operator has a
 * residual floor near its own error, about 2e-4).  Reading of "initialises": stage s + 1 restarts the dyadic sweep
 * at beta_x(s) / ratio, warm-started from stage s's eigenvectors.  opts->eta and opts->tol are ignored (each stage
 * has its own); everything else in opts applies to every stage.  log receives the probes of all stages back to
 * back and stage_first_probe[s] (n_stages + 1 entries) the index of stage s's first record; outcome, beta_x, evals
 * and evecs are the last stage's.  A stage that finds no admissible probe at all ends the cascade with
 * FD_ERR_PERRON_WALL.  Synchronous. */
typedef struct {
    fd_precision prec;
    double eta;                /* <= 0: 1e-7 for FD_PREC_FP32, 1e-3 for FD_PREC_FAST                        */
    double tol;                /* <= 0: 1e-6 for FD_PREC_FP32, 1e-3 for FD_PREC_FAST                        */
} fd_cascade_stage;
fd_status fd_beta_flow_cascade(fd_ctx* ctx, const fd_flow_opts* opts, const fd_cascade_stage* stages, int32_t n_stages,
                               const float* Q0_dev, int64_t ldq0, int32_t q0_cols, fd_probe* log, int32_t* n_probes,
                               int32_t* stage_first_probe, int32_t* outcome, double* beta_x_host, double* evals_host,
                               float* evecs_dev, int64_t ldv);

/* Out-of-sample extension of Markov eigenvectors from the context's points to new points
 * (Sec. 1, the (n, beta) ladder): psi_j(x) = sum_i K(x, x_i) q_i^-alpha psi_j(x_i) /
 * (lambda_j sum_i K(x, x_i) q_i^-alpha), at the context's current (beta, alpha, q).
 * psi_dev: N x m column-major (Markov vectors d^-1/2 * v); lambda_host: m values;
 * out_dev: Nnew x m column-major.  Two rectangular products (denominator, numerators), the
 * numerators b_max columns at a time.  Synchronous. */
fd_status fd_nystrom(fd_ctx* ctx, const float* Xnew_dev, int64_t Nnew, int64_t ldxnew,
                     const float* psi_dev, int64_t ldpsi, int32_t m, const double* lambda_host,
                     float* out_dev, int64_t ldout);

/* Start basis for the next level of the (n, beta) ladder (Sec. 1: find the eigenspace on n points, extend it to a
 * larger nested sample, re-solve there).  old_level: context over the first n_old points with its current
 * (beta, alpha, q, d); evecs_old_dev (n_old x m, column-major) and evals_host (m) are its eigenpairs of M.
 * new_level: context over N_new >= n_old points whose first n_old rows are the old points, after fd_degree (its d is
 * used); Xnew_dev: the new level's points (row-major, pitch ldxnew).  Writes Q0_dev (N_new x m, pitch ldq0):
 * Markov vectors psi = d_old^-1/2 * v on the old points, their out-of-sample extension (fd_nystrom) on the new
 * points, all rows times d_new^1/2.  Not orthonormalised: pass it to fd_eigs / fd_beta_flow as the warm start.
 * Synchronous. */
fd_status fd_ladder_start(fd_ctx* old_level, fd_ctx* new_level, const float* Xnew_dev, int64_t ldxnew,
                          const float* evecs_old_dev, int64_t ldv_old, int32_t m, const double* evals_host,
                          float* Q0_dev, int64_t ldq0);

/* Elementwise helper for the end of Sec. 2.3: out(i, c) = v(i, c) * d_i^power with the
 * context's current d (power = -0.5: Markov right eigenvectors from symmetric ones). */
fd_status fd_scale_by_degree(fd_ctx* ctx, const float* v_dev, int64_t ldv, int32_t cols,
                             double power, float* out_dev, int64_t ldout);

/* ---- Row-sharded operation: several processes, one GPU each (Sec. 3: multi-GPU runs are sharded over the row axis) ----
 *
 * Every rank creates its context on ALL N points (N D floats: tens of megabytes at most) and owns the rows
 * [row_begin, row_end) that fd_shard_rows assigns: `world` contiguous ranges of round_up(ceil(N / world), 256) rows,
 * the last ones shorter or empty.  Once fd_set_shard has been called,
 *   - every quadratic pass evaluates the owned rows only (N / world rows against all N columns);
 *   - fd_degree exchanges q and d (one column each) and sums its two scalars over the ranks;
 *   - fd_apply / fd_apply_general (square form) exchange the rows of Y, so Y is complete on every rank on return;
 *   - fd_eigs keeps the basis, its image and every tall-skinny product on the owned rows; per expansion it
 *     exchanges the rows of the new N x b block before the product and sums the small projected matrices over
 *     the ranks on the host; eigenvector outputs are complete on every rank; fd_beta_flow inherits all of this;
 *   - rectangular products (external rows), fd_nystrom and fd_ladder_start stay replicated: each rank computes all.
 * All ranks must make the same calls in the same order with the same arguments (the usual collective rule); the
 * host-side decisions of fd_eigs and fd_beta_flow depend only on summed quantities, which the callbacks must return
 * bit-identical on every rank (NCCL, gloo and MPI all-reduce do).
 *
 * The library links no communication library: the caller supplies two callbacks (torch.distributed / NCCL in the
 * Python binding) and the exchange buffer.
 *   allreduce_sum_host(user, buf, n): in-place sum over the ranks of n host doubles; blocking.
 *   allgather_dev(user, send_dev, recv_dev, count): every rank contributes count floats at send_dev; on return
 *     recv_dev holds world * count floats ordered by rank.  The callback is called with all earlier work of the
 *     context enqueued on the context's stream and must order itself after that work and before anything enqueued
 *     on that stream afterwards (a collective enqueued on that stream, or one that synchronises on both sides).
 *     send_dev and recv_dev lie inside xchg_dev.
 * Both return 0 on success; anything else makes the current call return FD_ERR_COMM.
 * xchg_dev: device buffer of at least fd_shard_exchange_bytes(N, b_max, world) bytes, 256-byte aligned, borrowed
 * until fd_destroy or fd_set_shard(ctx, NULL).  fd_set_shard(ctx, NULL) returns the context to unsharded operation. */
typedef struct {
    int32_t rank, world;
    int (*allreduce_sum_host)(void* user, double* buf, int64_t n);
    int (*allgather_dev)(void* user, const float* send_dev, float* recv_dev, int64_t count);
    void*   user;
    void*   xchg_dev;
    size_t  xchg_bytes;
} fd_shard;
/* Pure host arithmetic, no GPU needed. */
fd_status fd_shard_rows(int64_t N, int32_t world, int32_t rank, int64_t* row_begin, int64_t* row_end);
size_t    fd_shard_exchange_bytes(int64_t N, int32_t b_max, int32_t world);
fd_status fd_set_shard(fd_ctx* ctx, const fd_shard* shard);

/* No counterpart in the paper: an entry point for callers that cannot allocate device memory.
 *
 * Every other call borrows its scratch from a workspace the caller allocates.  Some callers have
 * no allocator to ask -- a plug-in that only receives input and output buffers, code that runs
 * where its host framework forbids allocation, a process whose device memory pool belongs to
 * someone else.  For them this variant of the direct-difference block product
 *     Y = diag(left) K(X, X) diag(right) V,   K_ij = exp(-beta |x_i - x_j|^2)
 * keeps its scratch (padded points, packed right block, split-column partial sums) in one
 * file-scope device array of 8 MiB that every GPU loading the library holds until the process
 * exits.  It calls no cudaMalloc / cudaFree and no allocating library routine; the caller passes
 * inputs and outputs only (X row-major N x D pitch ldx; V, Y column-major; left, right may be
 * NULL = ones; Y must not overlap V).  Limits: N <= FD_STATIC_MAX_N, D <= FD_STATIC_MAX_D,
 * b <= FD_STATIC_MAX_B; anything larger is refused with FD_ERR_UNSUPPORTED and a message in
 * errbuf (optional, may be NULL).  The first call made with a given device current resolves the
 * array's device address (cudaGetSymbolAddress); make that first call outside any stream capture.
 * All calls share the array and it keeps the last call's contents: nothing in it needs clearing
 * (every word read was written earlier in the same call), but two calls that overlap on the GPU
 * race -- keep them on one stream or otherwise serialised.  Asynchronous on cuda_stream. */
#define FD_STATIC_MAX_N 8192
#define FD_STATIC_MAX_D 32
#define FD_STATIC_MAX_B 32
fd_status fd_apply_general_static(const float* X_dev, int64_t N, int32_t D, int64_t ldx, double beta,
                                  const float* left_dev, const float* right_dev,
                                  const float* V_dev, int64_t ldv, int32_t b,
                                  float* Y_dev, int64_t ldy, void* cuda_stream,
                                  char* errbuf, size_t errbuf_len);

/* Measured unit throughput of the GPU that is current, for the roofline of the quadratic kernels (their bound is
 * on-chip arithmetic -- one exponential per pair, Sec. 2.2 -- not memory bandwidth, so the denominators are per-clock
 * unit rates): exponentials (MUFU ex2), fused multiply-adds, fp32 -> packed fp16 conversions, logic and add
 * instructions per clock per SM, and SM cycles per tcgen05.mma (kind::f16, M = 128, K = 16, fp32 accumulation) with
 * N = 64 / 128 and the A operand in tensor memory (ts) or shared memory (ss).  Rates are counted in SM cycles, so they
 * do not depend on the clock the GPU runs at.  scratch_dev: 256-byte aligned device buffer of at least
 * sm_count * 4104 + 256 bytes (1 MiB is plenty), borrowed for the call.  Synchronises. */
typedef struct {
    int32_t sm_count;
    double  ex2_per_clk_sm, ffma_per_clk_sm, cvt_f16x2_per_clk_sm, lop_per_clk_sm, fadd_per_clk_sm;
    double  clk_mma_ts_n64, clk_mma_ts_n128, clk_mma_ss_n64, clk_mma_ss_n128;
} fd_unit_rates;
fd_status fd_unit_peaks(void* scratch_dev, size_t scratch_bytes, void* cuda_stream, fd_unit_rates* out_host);

const char* fd_status_string(fd_status st);
const char* fd_last_error(const fd_ctx* ctx);
int32_t     fd_version(void);
/* Number of kernels this library has launched in the calling process (all contexts). */
int64_t     fd_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* FD_H_ */
