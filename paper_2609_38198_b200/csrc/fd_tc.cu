// Gram-form kernel on the 5th-generation tensor cores (tcgen05 + TMEM), Eqs. 4-6.
//
// Per (row tile I, column tile J) of 128 x 128 pairs:
//   1. Gram MMA (fp16 hi/lo split, three products per 16-wide K slab, fp32 accumulation in TMEM)
//      of AUGMENTED points, so the tile leaves the tensor core already as the base-2 exponent
//        S_ij = 2 b' x_i.x_j - b' r_i - b' r_j + bias            (b' = beta log2 e, Eq. 4)
//      the norms ride along as extra K columns ([.., e_i, 1] . [.., 1, e_j]), each norm carried by
//      two hi/lo pairs so it is exact to fp32.
//   2. Two warpgroups (one per row tile; thread = row) read S from TMEM, take 2^S on the MUFU,
//      split P = 2^S into fp16 hi + lo (mask / subtract), and write both halves back IN PLACE over
//      the S columns as the TMEM A operand.
//   3. Product MMA  Y_I += P_hi W_hi + P_lo W_hi + P_hi W_lo  with W = diag(right) V pre-split into
//      fp16 hi / lo (per-column power-of-two scaling), fp32 accumulation in TMEM (Eq. 6).
//   4. Every `flush` column tiles the TMEM accumulator is added into fp32 registers and restarted,
//      so tensor-core accumulation error does not grow with N.
// S tiles flow through a ring of TMEM buffers shared by both row tiles, so the tensor core runs ahead of
// the warpgroups and the product MMA of a tile overlaps the exponentials of the next ones.
// Row-sum mode (rectangular and row-sharded passes): no product MMA; the warpgroups add P (and P^2) on the FMA pipe,
// fp32 within a column tile and fp64 across tiles; a positive right vector enters through e_j.
// Symmetric row-sum mode (the degree passes of a whole data set, K = K^T): only the tiles on or above the diagonal are
// evaluated; the S tile is built with the streamed points on the TMEM lanes, so one thread adds up both what a tile gives
// its streamed point (one fixed-point atomic per tile) and, in 128 per-thread accumulators reduced across lanes every
// 64 tiles, what it gives the resident points.
//
// One persistent CTA per SM: warps 0-3 / 4-7 = the two exponential warpgroups (raised to 232 registers);
// warp 8 = TMA producer, warps 9 / 10 = product-MMA issuers for row tile 0 / 1, warp 11 = Gram-MMA issuer
// (lowered to 40 registers).  Three issuing threads because the per-tile bookkeeping of a lone issuer
// (waits, commits, descriptors) cost about as much as its MMAs and left the tensor pipe idle.  Column tiles are staged by TMA (every CTA loads its own copy) through a 4-deep ring.
// Every mbarrier wait is bounded; on expiry the CTA raises a status word, drains and exits.
#include <cuda.h>

#include <algorithm>
#include <cmath>

#include "fd_tc_common.h"

namespace fd {

namespace {

using namespace tc;

// ------------------------------------------------------------------------------------------------ shared memory map
template <int BT, int MODE>
struct Smem {
    static constexpr int kXChunk = 128 * 64;                       // one K slab (hi|lo) of 128 points: 8 KB
    static constexpr int kWHalf = is_rowsum(MODE) ? 0 : BT * 128;   // 64 j x BT columns fp16
    static constexpr int kWBytes = is_rowsum(MODE) ? 0 : 4 * kWHalf;   // [W_hi j-half 0][W_hi j-half 1][W_lo 0][W_lo 1]
    // symmetric row-sum mode: per-warp column partial sums, [row tile][parity][warp quarter][128 columns] floats
    static constexpr int kColPartBytes = (MODE == kModeRowsumSym) ? 2 * 2 * 4 * 128 * 4 + 64 : 0;   // + four mbarriers (col_ready[row tile][parity])
    static __host__ __device__ constexpr int stage_bytes(int K16) { return K16 * kXChunk + kWBytes; }
    static __host__ __device__ constexpr int total(int K16) {
        return 1024 /*align slack*/ + kStages * stage_bytes(K16) + 2 * K16 * kXChunk + 1024 /*barriers*/ + kColPartBytes;
    }
};

constexpr int kMaxBuf = 4;

struct Barriers {
    uint64_t full[kStages], empty[kStages];
    uint64_t xfull, xempty;
    // Ring-buffer barriers are indexed [buffer][row tile]: each one then has a single producer role and a single
    // consumer role that waits on EVERY one of its phases.  (A parity wait is only unambiguous if the waiter has seen
    // the previous phase complete; a barrier per buffer alone, shared by both row tiles, lets a waiter that skips
    // alternate phases pass one phase early.)
    uint64_t s_full[kMaxBuf][2];            // S tile ready in ring buffer (Gram issuer -> warpgroup)
    uint64_t s_done[kMaxBuf][2];            // block mode: P written in place; row-sum mode: S consumed (warpgroup -> issuer)
    uint64_t p_half[kMaxBuf][2];            // block mode: first 64 columns of P written (lets the product MMA start early)
    uint64_t kw_done[kMaxBuf][2];           // block mode: product MMAs that read P from this buffer have completed
    uint64_t y_full[2], y_empty[2];         // accumulator flush hand-off (per row tile)
    uint32_t tmem_base;
    int abort_flag;
};

// ------------------------------------------------------------------------------------------------ work items
// Work item w of a CTA -> (row pair, first column tile, number of column tiles, column chunk).
//   block / row-sum modes: (column chunk c, row pair r) with c outermost, r = blockIdx.x + k * gridDim.x;
//   block mode with tail split: full rounds first, then one half-range item of a tail pair (see TcParams);
//   symmetric row-sum mode: only tiles on or above the diagonal.  Row pair r needs column tiles 2 r .. num_jt - 1; pairing r
//     with num_work - 1 - r gives work units of equal length (num_jt + 2 tiles): unit u = blockIdx.x + k * gridDim.x is the
//     two items {u, num_work - 1 - u} (the middle pair of an odd count stands alone: its second item is empty).
struct ItemGeometry { int item, j0, num_jt, cch; bool tail_item; };

template <int MODE>
__device__ __forceinline__ ItemGeometry item_geometry(const TcParams& p, int w, int my_rows) {
    ItemGeometry g;
    if constexpr (MODE == kModeRowsumSym) {
        const int unit = (int)blockIdx.x + (w >> 1) * (int)gridDim.x;
        g.cch = 0;
        g.item = (w & 1) ? p.num_work - 1 - unit : unit;
        g.j0 = 2 * g.item;
        g.num_jt = ((w & 1) && g.item == unit) ? 0 : p.num_jt - g.j0;
        g.tail_item = false;
    } else if constexpr (MODE == kModeBlockTail) {
        const int full_rounds = p.tail_first / (int)gridDim.x;
        const int half = (p.num_jt + 1) / 2;
        g.cch = 0;
        g.tail_item = w >= full_rounds;
        const int part = g.tail_item ? (int)blockIdx.x / p.tail_pairs : 0;
        g.item = g.tail_item ? p.tail_first + (int)blockIdx.x % p.tail_pairs : (int)blockIdx.x + w * (int)gridDim.x;
        g.j0 = g.tail_item ? part * half : 0;
        g.num_jt = g.tail_item ? (part == 0 ? half : p.num_jt - half) : p.num_jt;
    } else {
        g.cch = w / my_rows;
        g.item = (int)blockIdx.x + (w % my_rows) * (int)gridDim.x;
        g.j0 = g.cch * p.jt_chunk;
        g.num_jt = (p.num_jt - g.j0 < p.jt_chunk) ? p.num_jt - g.j0 : p.jt_chunk;
        g.tail_item = false;
    }
    return g;
}

// ------------------------------------------------------------------------------------------------ the kernel
// Tiles of one work item are numbered n = 2 j + t (column tile j, row tile t) and flow through a ring of NBUF
// S buffers in TMEM (3 in block mode, 4 in row-sum mode), so the tensor core runs up to NBUF tiles ahead of the
// warpgroups and neither warpgroup waits for the product MMA of its previous tile.
template <int BT, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
k_tc(const __grid_constant__ CUtensorMap map_xrow, const __grid_constant__ CUtensorMap map_xcol,
     const __grid_constant__ CUtensorMap map_whi, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    using SM = Smem<BT, MODE>;
    constexpr int NBUF = is_rowsum(MODE) ? 4 : 3;
    constexpr uint32_t kRingPeriod = (NBUF & 1) ? 2 * NBUF : NBUF;   // tiles between two uses of a buffer by the same row tile
    constexpr uint32_t kYCol = 384;                    // block mode: Y_t at columns 384 + 64 t
    const int K16 = p.K16;
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_base = base;
    uint8_t* xi_base = base + kStages * SM::stage_bytes(K16);                 // 2 row tiles x K16 slabs
    Barriers* bars = (Barriers*)(xi_base + 2 * K16 * SM::kXChunk);
    volatile int* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        // a column stage is released by the Gram issuer alone (row-sum mode) or by both product issuers (block mode)
        for (int s = 0; s < kStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], is_rowsum(MODE) ? 1 : 2); }
        mbar_init(&bars->xfull, 1); mbar_init(&bars->xempty, 1);
        for (int u = 0; u < kMaxBuf; ++u)
            for (int t = 0; t < 2; ++t) {
                mbar_init(&bars->s_full[u][t], 1); mbar_init(&bars->s_done[u][t], 4);
                mbar_init(&bars->kw_done[u][t], 1); mbar_init(&bars->p_half[u][t], 4);
            }
        for (int t = 0; t < 2; ++t) { mbar_init(&bars->y_full[t], 1); mbar_init(&bars->y_empty[t], 4); }
        if constexpr (MODE == kModeRowsumSym) {
            uint64_t* col_ready = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(bars) + 1024 + 2 * 2 * 4 * 128 * 4);
            for (int u = 0; u < 4; ++u) mbar_init(&col_ready[u], 4);          // the four warps' column partials of a tile are written
        }
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;
    const long long t_begin = clock64();

    // Work items of this CTA: (column chunk c, row-pair tile r) with c outermost, r = blockIdx.x + k * gridDim.x.  Every CTA
    // sweeps chunk c for all of its rows before chunk c + 1, so the whole grid reads the same L2-sized slice of the
    // column operands at about the same time; a row's partial results always come from the same threads, in order.
    // (item_geometry above has the other modes' orders.)
    constexpr bool kSym = MODE == kModeRowsumSym;
    constexpr bool kTail = MODE == kModeBlockTail;
    const int my_rows = kSym ? ((p.num_work + 1) / 2 - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x
                             : (p.num_work - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int my_items = kSym ? 2 * my_rows
                       : kTail ? p.tail_first / (int)gridDim.x + ((int)blockIdx.x < 2 * p.tail_pairs ? 1 : 0) : my_rows * p.num_chunks;
#define FD_ITEM_GEOMETRY(w)                                                                         \
    const ItemGeometry geo_ = item_geometry<MODE>(p, (w), my_rows);                                 \
    const int cch = geo_.cch;                                                                       \
    const int item = geo_.item;                                                                     \
    const int j0 = geo_.j0;                                                                         \
    const int num_jt = geo_.num_jt;                                                                 \
    const bool tail_item = geo_.tail_item;                                                          \
    const int tiles_per_item = 2 * num_jt;                                                          \
    (void)tail_item;                                                                                \
    (void)item; (void)tiles_per_item; (void)cch
    const int flush = p.flush;

    if (warp >= 8) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(40));
      if (warp == 8) {
        // =============================================================== TMA producer (one thread)
        if (lane == 0) {
            prefetch_tmap(&map_xrow); prefetch_tmap(&map_xcol);
            if (!is_rowsum(MODE)) prefetch_tmap(&map_whi);
            uint32_t it = 0;
            bool ok = true;
            for (int w = 0; w < my_items && ok; ++w) {
                FD_ITEM_GEOMETRY(w);
                ok = mbar_wait(&bars->xempty, (w & 1) ^ 1, abort_flag, p.status, 1);
                if (!ok) break;
                mbar_expect_tx(&bars->xfull, 2 * K16 * SM::kXChunk);
                for (int t = 0; t < 2; ++t)
                    for (int c = 0; c < K16; ++c)
                        tma_load_2d(xi_base + (t * K16 + c) * SM::kXChunk, &map_xrow, 0,
                                    (int)(c * p.np_rows + (int64_t)item * 256 + t * 128), &bars->xfull);
                for (int j = 0; j < num_jt; ++j, ++it) {
                    const int s = it % kStages;
                    ok = mbar_wait(&bars->empty[s], ((it / kStages) & 1) ^ 1, abort_flag, p.status, 2);
                    if (!ok) break;
                    uint8_t* st = stage_base + s * SM::stage_bytes(K16);
                    mbar_expect_tx(&bars->full[s], SM::stage_bytes(K16));
                    for (int c = 0; c < K16; ++c)
                        tma_load_2d(st + c * SM::kXChunk, &map_xcol, 0, (int)(c * p.np_cols + (int64_t)(j0 + j) * 128), &bars->full[s]);
                    if (!is_rowsum(MODE)) {
                        uint8_t* wst = st + K16 * SM::kXChunk;
                        tma_load_2d(wst, &map_whi, (j0 + j) * 128, 0, &bars->full[s]);
                        tma_load_2d(wst + SM::kWHalf, &map_whi, (j0 + j) * 128 + 64, 0, &bars->full[s]);
                        // (W_hi and W_lo are rows 0.. and lo_row.. of one array: one tensor map, and a parameter block that
                        // stays below 640 bytes -- above it the kernel measured 2.5 % more SM cycles)
                        tma_load_2d(wst + 2 * SM::kWHalf, &map_whi, (j0 + j) * 128, p.lo_row, &bars->full[s]);
                        tma_load_2d(wst + 3 * SM::kWHalf, &map_whi, (j0 + j) * 128 + 64, p.lo_row, &bars->full[s]);
                    }
                }
            }
            if (!ok) {
                // aborted: let the copies already in flight land before the CTA exits (bounded)
                const uint32_t issued = it;
                for (uint32_t k = (issued > (uint32_t)kStages ? issued - kStages : 0); k < issued; ++k) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&bars->full[k % kStages], (k / kStages) & 1) && clock64() - t0 < 20000000ll) {}
                }
            }
        }
      } else if (warp == 11) {
        // =============================================================== Gram MMA issuer (one thread)
        // Issues S(n) = A_t B_j^T for every tile as soon as its ring buffer is free again; runs up to NBUF tiles ahead.
        if (lane == 0) {
          if constexpr (is_rowsum(MODE)) {
            // Row-sum mode: the MUFU binds and the tensor pipe is mostly idle; descriptors are rebuilt per MMA, which paces
            // the Gram MMAs between the warpgroups' TMEM loads (issuing them in tight bursts measured 5 % slower).
            constexpr uint32_t idesc_g = idesc_f16(128);
            uint32_t it0 = 0, gn0 = 0;
            bool ok = true;
            for (int w = 0; w < my_items && ok; ++w) {
                FD_ITEM_GEOMETRY(w);
                ok = mbar_wait(&bars->xfull, w & 1, abort_flag, p.status, 3);
                if (!ok) break;
                tc_fence_after();
                for (int n = 0; n < tiles_per_item && ok; ++n) {
                    const uint32_t g = gn0 + (uint32_t)n;
                    const int buf = g % NBUF;
                    const uint32_t itj = it0 + (uint32_t)(n >> 1);
                    const int s = itj % kStages;
                    if (g >= (uint32_t)NBUF) {
                        // the tile that used this buffer last (NBUF tiles ago, possibly of the other row tile) must be finished
                        const uint32_t gp = g - NBUF;
                        uint64_t* fb = is_rowsum(MODE) ? &bars->s_done[buf][gp & 1] : &bars->kw_done[buf][gp & 1];
                        ok = mbar_wait(fb, (gp / kRingPeriod) & 1, abort_flag, p.status, 5);
                        if (!ok) break;
                    }
                    if ((n & 1) == 0) {
                        ok = mbar_wait(&bars->full[s], (itj / kStages) & 1, abort_flag, p.status, 4);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    // The two small cross terms (hi x lo) go first and the large hi x hi term last: each MMA rounds its
                    // result at the magnitude of its largest addend, so only the final one rounds at full magnitude.
                    const uint32_t s_addr = tmem + 128u * buf;
                    const int t = n & 1;
                    uint8_t* st = stage_base + s * SM::stage_bytes(K16);
                    // (symmetric mode: the streamed tile is the M operand, so TMEM lanes = streamed points)
                    for (int c = 0; c < K16; ++c) {
                        uint64_t a = smem_desc(smem_u32(xi_base + (t * K16 + c) * SM::kXChunk), 512, 4);
                        uint64_t b = smem_desc(smem_u32(st + c * SM::kXChunk), 512, 4);
                        if (MODE == kModeRowsumSym) { const uint64_t x = a; a = b; b = x; }
                        mma_ss(s_addr, a, b + 2, idesc_g, c > 0);          // + 2: the lo half starts 32 B into the row
                        mma_ss(s_addr, a + 2, b, idesc_g, 1);
                    }
                    for (int c = 0; c < K16; ++c) {
                        uint64_t a = smem_desc(smem_u32(xi_base + (t * K16 + c) * SM::kXChunk), 512, 4);
                        uint64_t b = smem_desc(smem_u32(st + c * SM::kXChunk), 512, 4);
                        if (MODE == kModeRowsumSym) { const uint64_t x = a; a = b; b = x; }
                        mma_ss(s_addr, a, b, idesc_g, 1);
                    }
                    tc_commit(&bars->s_full[buf][n & 1]);
                    if (is_rowsum(MODE) && (n & 1)) tc_commit(&bars->empty[s]);   // both Gram MMAs of this column tile issued
                }
                if (ok) tc_commit(&bars->xempty);                  // the row operand tiles may be replaced
                it0 += (uint32_t)num_jt;
                gn0 += (uint32_t)tiles_per_item;
            }
          } else {
            constexpr uint32_t idesc_g = idesc_f16(128);
            // Operand descriptors as (low, high) words and ring positions as counters: this thread shares its scheduler
            // with busy warps, so every instruction it does not issue shortens the gap between two MMAs.
            const uint64_t xd = smem_desc(smem_u32(xi_base), 512, 4);      // 64 B rows (SWIZZLE_64B), 512 B between 8-row groups
            const uint32_t xi_lo = (uint32_t)xd, xdesc_hi = (uint32_t)(xd >> 32);
            const uint32_t stage_lo = (uint32_t)smem_desc(smem_u32(stage_base), 512, 4);
            const uint32_t stage_step = (uint32_t)(SM::stage_bytes(K16) >> 4);
            constexpr uint32_t kSlab = SM::kXChunk >> 4;
            uint32_t itj = 0, buf = 0, gr = 0, ph = 0;              // column-tile counter; tile index mod NBUF, mod kRingPeriod, ring phase
            bool first_round = true;                                // no buffer has been used yet
            bool ok = true;
            for (int w = 0; w < my_items && ok; ++w) {
                FD_ITEM_GEOMETRY(w);
                ok = mbar_wait(&bars->xfull, w & 1, abort_flag, p.status, 3);
                if (!ok) break;
                tc_fence_after();
                for (int n = 0; n < tiles_per_item && ok; ++n) {
                    const int t = n & 1;
                    const int s = itj % kStages;
                    if (!first_round) {
                        // the tile that used this buffer last (NBUF tiles ago, possibly of the other row tile) must be finished
                        const int tp = (NBUF & 1) ? (t ^ 1) : t;
                        const uint32_t php = gr >= (uint32_t)NBUF ? ph : ph ^ 1u;
                        uint64_t* fb = is_rowsum(MODE) ? &bars->s_done[buf][tp] : &bars->kw_done[buf][tp];
                        ok = mbar_wait(fb, php, abort_flag, p.status, 5);
                        if (!ok) break;
                    }
                    if (t == 0) {
                        ok = mbar_wait(&bars->full[s], (itj / kStages) & 1, abort_flag, p.status, 4);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    // The two small cross terms (hi x lo) go first and the large hi x hi term last: each MMA rounds its
                    // result at the magnitude of its largest addend, so only the final one rounds at full magnitude.
                    const uint32_t s_addr = tmem + 128u * buf;
                    const uint32_t a0 = xi_lo + (uint32_t)(t * K16) * kSlab, b0 = stage_lo + (uint32_t)s * stage_step;
                    if (K16 == 1) {
                        mma_ss2<0>(s_addr, a0, xdesc_hi, b0 + 2, xdesc_hi, idesc_g);          // + 2: the lo half starts 32 B into the row
                        mma_ss2<1>(s_addr, a0 + 2, xdesc_hi, b0, xdesc_hi, idesc_g);
                        mma_ss2<1>(s_addr, a0, xdesc_hi, b0, xdesc_hi, idesc_g);
                    } else {
                        for (int c = 0; c < K16; ++c) {
                            const uint32_t a = a0 + (uint32_t)c * kSlab, b = b0 + (uint32_t)c * kSlab;
                            if (c == 0) mma_ss2<0>(s_addr, a, xdesc_hi, b + 2, xdesc_hi, idesc_g);
                            else mma_ss2<1>(s_addr, a, xdesc_hi, b + 2, xdesc_hi, idesc_g);
                            mma_ss2<1>(s_addr, a + 2, xdesc_hi, b, xdesc_hi, idesc_g);
                        }
                        for (int c = 0; c < K16; ++c)
                            mma_ss2<1>(s_addr, a0 + (uint32_t)c * kSlab, xdesc_hi, b0 + (uint32_t)c * kSlab, xdesc_hi, idesc_g);
                    }
                    tc_commit(&bars->s_full[buf][t]);
                    if (t == 1) {
                        if (is_rowsum(MODE)) tc_commit(&bars->empty[s]);   // both Gram MMAs of this column tile issued
                        ++itj;
                    }
                    if (++buf == (uint32_t)NBUF) { buf = 0; first_round = false; }
                    if (++gr == kRingPeriod) { gr = 0; ph ^= 1u; }
                }
                if (ok) tc_commit(&bars->xempty);                  // the row operand tiles may be replaced
            }
          }
        }
      } else if (!is_rowsum(MODE)) {
        // =============================================================== product MMA issuers: warp 9 -> row tile 0, warp 10 -> row tile 1
        // Two issuing threads so that the per-tile bookkeeping of one overlaps the MMAs of the other.
        if (lane == 0) {
            constexpr uint32_t idesc_y = idesc_f16(BT);
            const int t = warp - 9;
            // W stage descriptor as (low, high) words: 128 B rows (SWIZZLE_128B), 1024 B between 8-row groups
            const uint64_t wd = smem_desc(smem_u32(stage_base + K16 * SM::kXChunk), 1024, 2);
            const uint32_t wbase_lo = (uint32_t)wd, wdesc_hi = (uint32_t)(wd >> 32);
            const uint32_t stage_step = (uint32_t)(SM::stage_bytes(K16) >> 4);
            constexpr uint32_t kLoOff = (uint32_t)((2 * SM::kWHalf) >> 4);          // W_lo tiles follow the two W_hi tiles of a stage
            uint32_t itj = 0, n_grp = 0;
            uint32_t buf = (uint32_t)t % NBUF, gr = (uint32_t)t, ph = 0;            // this row tile's tile index mod NBUF, mod kRingPeriod, ring phase
            bool ok = true;
            const uint32_t y_addr = tmem + kYCol + 64 * t;
            for (int w = 0; w < my_items && ok; ++w) {
                FD_ITEM_GEOMETRY(w);
                int in_group = 0;                                  // tiles accumulated in the current group (no division in the hot loop)
                for (int j = 0; j < num_jt && ok; ++j, ++itj) {
                    const int s = itj % kStages;
                    ok = mbar_wait(&bars->p_half[buf][t], ph, abort_flag, p.status, 7);
                    if (!ok) break;
                    const bool group_start = in_group == 0;
                    const bool group_end = in_group + 1 == flush || j + 1 == num_jt;
                    in_group = group_end ? 0 : in_group + 1;
                    if (group_start && n_grp > 0) {
                        ok = mbar_wait(&bars->y_empty[t], (n_grp - 1) & 1, abort_flag, p.status, 6);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    // Y_t += P W : 8 K steps of 16 columns j; K step ks reads P_hi at S-buffer columns [16 ks, 16 ks + 8)
                    // and P_lo at [16 ks + 8, 16 ks + 16) (the warpgroup wrote them in place over S).  The first four K steps
                    // start as soon as the first half of P is written, the rest once the tile is complete.
                    const uint32_t w_lo = wbase_lo + (uint32_t)s * stage_step;
                    const uint32_t p_addr = tmem + 128u * buf;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        if (ks == 4) {
                            ok = mbar_wait(&bars->s_done[buf][t], ph, abort_flag, p.status, 7);
                            if (!ok) break;
                            tc_fence_after();
                        }
                        const uint32_t off = (uint32_t)(((ks >> 2) * SM::kWHalf + (ks & 3) * 32) >> 4);
                        const uint32_t a_hi = p_addr + 16 * ks;
                        if (ks == 0 && group_start) mma_ts2<0>(y_addr, a_hi, w_lo + off, wdesc_hi, idesc_y);
                        else mma_ts2<1>(y_addr, a_hi, w_lo + off, wdesc_hi, idesc_y);
                        mma_ts2<1>(y_addr, a_hi + 8, w_lo + off, wdesc_hi, idesc_y);
                        mma_ts2<1>(y_addr, a_hi, w_lo + kLoOff + off, wdesc_hi, idesc_y);
                    }
                    if (!ok) break;
                    tc_commit(&bars->kw_done[buf][t]);
                    if (group_end) { tc_commit(&bars->y_full[t]); ++n_grp; }
                    tc_commit(&bars->empty[s]);
                    buf += 2; if (buf >= (uint32_t)NBUF) buf -= NBUF;
                    gr += 2; if (gr >= kRingPeriod) { gr -= kRingPeriod; ph ^= 1u; }
                }
            }
        }
      }
    } else {
        // =============================================================== exponential warpgroups
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(232));
        const int t = warp >> 2;                       // row tile of this warpgroup
        const int wq = warp & 3;                       // TMEM lane quarter this warp may access
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        const int row_in_tile = wq * 32 + lane;
        uint32_t gn0 = 0, n_grp = 0;
        uint32_t ncol = 0;                             // symmetric row-sum mode: off-diagonal tiles this row tile has finished
        bool ok = true;

        for (int w = 0; w < my_items && ok; ++w) {
            FD_ITEM_GEOMETRY(w);
            const int64_t row = (int64_t)item * 256 + t * 128 + row_in_tile;
            if constexpr (MODE == kModeRowsumSym) {
                // Symmetric half-work row sums.  The S tile is built the other way round here (lanes = points of the
                // STREAMED tile J, columns = points of the CTA's resident tile It), so a thread owns one streamed point:
                //   * its sum over the 128 columns is that point's share of tile (J, It): one fixed-point atomic per tile;
                //   * acc[c] += P[., c] collects, over the whole sweep, the resident point c's sum over the streamed
                //     points that fall on this lane; the 128 lanes are reduced (butterfly of shuffles, the four warps
                //     through shared memory) only every kSymFlush tiles, which also bounds the fp32 accumulation length.
                // J < It is the mirror of a tile another resident tile evaluates (skipped: only J = 2 item for the second
                // resident tile); J == It counts once (resident side only); J > It counts for both sides.  Sums go to one
                // 64-bit fixed-point integer per point: integer additions commute, so the result does not depend on the
                // order in which CTAs arrive.
                constexpr int kSymFlush = 64;
                constexpr bool kWantSq = BT == 16;             // the sum of squares rides along in the first degree pass only (BT = 32: without)
                float* colpart = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(bars) + 1024);
                uint64_t* col_ready = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(bars) + 1024 + 2 * 2 * 4 * 128 * 4);
                const double fix = (double)(1ull << p.sym_shift);
                const int It = 2 * item + t;
                float acc[128];
#pragma unroll
                for (int c = 0; c < 128; ++c) acc[c] = 0.f;
                double dsq = 0.0;
                int pending = 0;                               // tiles accumulated in acc since the last reduction
                // reduces acc over the 128 lanes of the resident tile and adds the sums to the resident points
                auto reduce_acc = [&]() -> bool {
                    const uint32_t slot = ncol & 1u;
                    float* mine = colpart + (((t * 2 + (int)slot) * 4 + wq) * 128);
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
#pragma unroll
                        for (int m = 16; m >= 1; m >>= 1) {
                            const bool up = (lane & m) != 0;
#pragma unroll
                            for (int k = 0; k < m; ++k) {
                                const float send = up ? acc[32 * ch + k] : acc[32 * ch + k + m];
                                const float keep = up ? acc[32 * ch + k + m] : acc[32 * ch + k];
                                acc[32 * ch + k] = keep + __shfl_xor_sync(0xffffffffu, send, m);
                            }
                        }
                        mine[ch * 32 + lane] = acc[32 * ch];
                    }
#pragma unroll
                    for (int c = 0; c < 128; ++c) acc[c] = 0.f;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&col_ready[t * 2 + slot]);
                    if (!mbar_wait(&col_ready[t * 2 + slot], (ncol >> 1) & 1u, abort_flag, p.status, 11)) return false;
                    const float* all = colpart + ((t * 2 + (int)slot) * 4) * 128;
                    const int cidx = wq * 32 + lane;
                    const float csum = (all[cidx] + all[128 + cidx]) + (all[256 + cidx] + all[384 + cidx]);
                    const int64_t pt = (int64_t)It * 128 + cidx;
                    if (pt < p.N) atomicAdd(p.symsum + pt, (unsigned long long)__double2ll_rn((double)csum * fix));
                    ++ncol;
                    return true;
                };
                for (int j = 0; j < num_jt && ok; ++j) {
                    const uint32_t g = gn0 + 2u * j + t;
                    const int buf = g % NBUF;
                    ok = mbar_wait(&bars->s_full[buf][t], (g / kRingPeriod) & 1, abort_flag, p.status, 8);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t addr = tmem + lane_addr + 128u * buf;
                    const int J = j0 + j;
                    const bool use = J >= It;
                    float r0 = 0.f, r1 = 0.f, q0 = 0.f, q1 = 0.f;
                    uint32_t sv[2][32];
                    tmem_ld32(addr, sv[0]);
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        tmem_wait_ld();
                        if (ch < 3) tmem_ld32(addr + 32 * (ch + 1), sv[(ch + 1) & 1]);
                        if (use) {
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                const float p0 = ex2f(__uint_as_float(sv[ch & 1][i])), p1 = ex2f(__uint_as_float(sv[ch & 1][i + 1]));
                                acc[32 * ch + i] += p0; acc[32 * ch + i + 1] += p1;
                                r0 += p0; r1 += p1;
                                if (kWantSq) { q0 = fmaf(p0, p0, q0); q1 = fmaf(p1, p1, q1); }
                            }
                        }
                    }
                    // the buffer can be refilled: its values are in registers or consumed
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->s_done[buf][t]);
                    if (!use) continue;                            // mirrored tile: evaluated by the other resident tile
                    const bool offdiag = J > It;
                    dsq += (double)(q0 + q1) * (offdiag ? 2.0 : 1.0);
                    if (offdiag) {
                        const int64_t pt = (int64_t)J * 128 + row_in_tile;
                        if (pt < p.N) atomicAdd(p.symsum + pt, (unsigned long long)__double2ll_rn((double)(r0 + r1) * fix));
                    }
                    if (++pending == kSymFlush) { ok = reduce_acc(); pending = 0; if (!ok) break; }
                }
                if (ok && pending > 0) ok = reduce_acc();
                if (ok && num_jt > 0 && row < p.Nrow && p.rowsq)
                    // this thread's share of sum_ij K_ij^2: only the total over all threads is meaningful.  (A thread whose
                    // slot It * 128 + r lies beyond N has only seen streamed points J * 128 + r >= N, i.e. zeros.)
                    p.rowsq[row] = dsq * (1.0 / ((double)(1 << kBias) * (double)(1 << kBias)));
            } else if (MODE == kModeRowsum) {
                double dsum = 0.0, dsq = 0.0;
                for (int j = 0; j < num_jt && ok; ++j) {
                    const uint32_t g = gn0 + 2u * j + t;
                    const int buf = g % NBUF;
                    ok = mbar_wait(&bars->s_full[buf][t], (g / kRingPeriod) & 1, abort_flag, p.status, 8);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t addr = tmem + lane_addr + 128u * buf;
                    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f, q0 = 0.f, q1 = 0.f;
                    uint32_t sv[4][32];
#pragma unroll
                    for (int qd = 0; qd < 4; ++qd) tmem_ld32(addr + 32 * qd, sv[qd]);
                    tmem_wait_ld();
                    // the buffer can be refilled as soon as its values are in registers
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->s_done[buf][t]);
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4) {
                            const float p0 = ex2f(__uint_as_float(sv[ch][i])), p1 = ex2f(__uint_as_float(sv[ch][i + 1]));
                            const float p2 = ex2f(__uint_as_float(sv[ch][i + 2])), p3 = ex2f(__uint_as_float(sv[ch][i + 3]));
                            a0 += p0; a1 += p1; a2 += p2; a3 += p3;
                            if (BT == 16) {                // (BT = 32: the instantiation without the sum of squares)
                                q0 = fmaf(p0, p0, q0); q1 = fmaf(p1, p1, q1); q0 = fmaf(p2, p2, q0); q1 = fmaf(p3, p3, q1);
                            }
                        }
                    }
                    dsum += (double)((a0 + a1) + (a2 + a3));
                    dsq += (double)(q0 + q1);
                }
                if (ok && row < p.Nrow) {
                    // undo the 2^bias scaling of P (exact powers of two)
                    const double l = (p.left ? (double)p.left[row] : 1.0) * (1.0 / (double)(1 << kBias));
                    p.q[row] = (float)(dsum * l);
                    if (p.rowsq) p.rowsq[row] = dsq * (1.0 / ((double)(1 << kBias) * (double)(1 << kBias)));
                }
            } else {
                float acc[BT];
#pragma unroll
                for (int c = 0; c < BT; ++c) acc[c] = 0.f;
                bool pending = false;
                // Adds the finished TMEM accumulator of this row tile into the registers and hands it back.
                // The tensor core adds each K step into the TMEM accumulator with round-toward-zero.  For a sum whose partial
                // sums keep one sign, n additions lose n / 4 ulp of the result on average (half an ulp each, at a running
                // magnitude that averages half the final one): measured 2.85e-8 per addition against 2^-25 = 2.98e-8.  The
                // flush adds that expected loss back (one FMA instead of one add), which removes the common scale error of
                // M V that would otherwise shift every eigenvalue by ~7e-7 per column tile in the group.
                auto do_flush = [&](int tiles_in_group) -> bool {
                    const float corr = 1.0f + (float)(tiles_in_group * 8 * 3) * 2.98023224e-8f;
                    if (!mbar_wait(&bars->y_full[t], n_grp & 1, abort_flag, p.status, 10)) return false;
                    ++n_grp;
                    tc_fence_after();
                    const uint32_t yaddr = tmem + lane_addr + kYCol + 64 * t;
                    // all loads first, one wait (the S registers are free between tiles), and the accumulator is handed
                    // back before the additions
                    uint32_t v[BT / 16][16];
#pragma unroll
                    for (int c0 = 0; c0 < BT / 16; ++c0) tmem_ld16(yaddr + 16 * c0, v[c0]);
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->y_empty[t]);
#pragma unroll
                    for (int c0 = 0; c0 < BT / 16; ++c0)
#pragma unroll
                        for (int i = 0; i < 16; ++i) acc[16 * c0 + i] = fmaf(__uint_as_float(v[c0][i]), corr, acc[16 * c0 + i]);
                    return true;
                };
                int in_group = 0;
                for (int j = 0; j < num_jt && ok; ++j) {
                    const uint32_t g = gn0 + 2u * j + t;
                    const int buf = g % NBUF;
                    ok = mbar_wait(&bars->s_full[buf][t], (g / kRingPeriod) & 1, abort_flag, p.status, 9);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t addr = tmem + lane_addr + 128u * buf;
                    // whole S row into registers first (the four loads overlap), then exponentials and in-place stores
                    uint32_t sv[4][32];
#pragma unroll
                    for (int qd = 0; qd < 4; ++qd) tmem_ld32(addr + 32 * qd, sv[qd]);
                    tmem_wait_ld();
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch) {
                        uint32_t hi[8], lo[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float p0 = ex2f(__uint_as_float(sv[ch >> 1][16 * (ch & 1) + 2 * i]));
                            const float p1 = ex2f(__uint_as_float(sv[ch >> 1][16 * (ch & 1) + 2 * i + 1]));
                            const float h0 = __uint_as_float(__float_as_uint(p0) & 0xFFFFE000u);
                            const float h1 = __uint_as_float(__float_as_uint(p1) & 0xFFFFE000u);
                            hi[i] = pack_f16x2(h0, h1);
                            lo[i] = pack_f16x2(p0 - h0, p1 - h1);
                        }
                        tmem_st8(addr + 16 * ch, hi);
                        tmem_st8(addr + 16 * ch + 8, lo);
                        if (ch == 3) {
                            tmem_wait_st();
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&bars->p_half[buf][t]);
                        }
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->s_done[buf][t]);
                    // flush of the accumulator group that ended with the PREVIOUS tile of this row tile (its product
                    // MMA has had a whole tile of time to finish); the last group of the work item is flushed at once
                    if (pending) { ok = do_flush(flush); pending = false; if (!ok) break; }
                    ++in_group;
                    if (in_group == flush || j + 1 == num_jt) {
                        if (j + 1 == num_jt) { ok = do_flush(in_group); if (!ok) break; }
                        else pending = true;
                        in_group = 0;
                    }
                }
                if (ok && row < p.Nrow) {
                    const float l = p.left ? p.left[row] : 1.0f;
#pragma unroll
                    for (int c = 0; c < BT; ++c)
                        if (c < p.b) {
                            float* o = p.Y + row + (int64_t)c * p.ldy;
                            const float v = acc[c] * l * p.colscale_inv[c];
                            if (kTail && tail_item) atomicAdd(o, v);   // the other half of the column range arrives from another CTA
                            // later column chunks add to the partial result of the same thread; streaming loads and stores:
                            // the partial results are touched once per chunk round and should not push the fp16 operands,
                            // which every CTA re-reads, out of L2
                            else __stcs(o, cch == 0 ? v : __ldcs(o) + v);
                        }
                }
            }
            gn0 += (uint32_t)tiles_per_item;
        }
    }
    tc_fence_before();
    __syncthreads();
    // SM cycles CTA 0 spent on its work items (status words 2-3): lets the host relate the kernel time to the SM clock
    if (blockIdx.x == 0 && threadIdx.x == 0) *reinterpret_cast<long long*>(p.status + 2) = clock64() - t_begin;
    if (warp == 8) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// Exercises the bounded-wait path without any fault: one thread waits on a barrier that nothing will ever complete,
// with a short limit; the wait gives up, records its code in the status word and the kernel returns normally.
__global__ void k_wait_selftest(unsigned int* status, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(&bar, 0, &abort_flag, status, 0x7f, limit_cycles);
    }
}

// ------------------------------------------------------------------------------------------------ operand packing
// Augmented fp16 hi|lo operand rows.  role 0 (rows of the product): [c x, e, 1]; role 1 (columns): [c x, 1, e] with
// c = sqrt(2 b'), e = -b' |x - mu|^2 (+ the bias for role 1, + log2 of a positive weight vector when one is given).
// Layout: slab s (16 augmented columns) of point p at out[(s * np + p) * 32 ..]: 16 hi then 16 lo halves.
__global__ void k_pack_points(const float* __restrict__ xs, int DP, int D, int64_t n, int64_t np, const double* __restrict__ mu,
                              double bprime, int role, double bias, const float* __restrict__ logw_src, int K16,
                              __half* __restrict__ out) {
    int64_t pidx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (pidx >= np) return;
    const bool valid = pidx < n;
    const double cs = sqrt(2.0 * bprime);
    double r = 0.0;
    if (valid)
        for (int k = 0; k < D; ++k) { double v = (double)xs[pidx * DP + k] - mu[k]; r += v * v; }
    double e = -bprime * r;
    if (logw_src && valid) e += log2((double)logw_src[pidx]);     // a positive weight rides in the exponent
    if (role == 1) e += bias;
    if (!valid) e = -30000.0;                           // padded point: 2^e = 0 (its row / column contributes nothing)
    // norm pieces: two hi/lo pairs carry e to beyond fp32 precision
    const __half e_h1 = __double2half(e);
    const double r1 = e - (double)__half2float(e_h1);
    const __half e_l1 = __double2half(r1);
    const double r2 = r1 - (double)__half2float(e_l1);
    const __half e_h2 = __double2half(r2);
    const __half e_l2 = __double2half(r2 - (double)__half2float(e_h2));
    const __half one = __float2half(1.0f), zero = __float2half(0.0f);
    for (int s = 0; s < K16; ++s) {
        __half* o = out + ((int64_t)s * np + pidx) * 32;
        for (int kk = 0; kk < 16; ++kk) {
            const int col = s * 16 + kk;
            __half h = zero, l = zero;
            if (col < D) {
                if (valid) {
                    const double v = cs * ((double)xs[pidx * DP + col] - mu[col]);
                    h = __double2half(v);
                    l = __double2half(v - (double)__half2float(h));
                }
            } else if (col == D || col == D + 1) {          // row-norm slots: role 0 carries e, role 1 carries 1
                if (role == 0) { h = col == D ? e_h1 : e_h2; l = col == D ? e_l1 : e_l2; }
                else h = one;
            } else if (col == D + 2 || col == D + 3) {      // column-norm slots
                if (role == 1) { h = col == D + 2 ? e_h1 : e_h2; l = col == D + 2 ? e_l1 : e_l2; }
                else h = one;
            }
            o[kk] = h;
            o[16 + kk] = l;
        }
    }
}

// Stage 1: per-block maxima of |right_j V_jc| for each column c.
__global__ void k_colmax_partial(const float* __restrict__ V, int64_t ldv, const float* __restrict__ right, int64_t N, int c0,
                                 int bc, float* __restrict__ part) {
    __shared__ float sm[256];
    const int c = blockIdx.y;
    float m = 0.f;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < N; j += (int64_t)gridDim.x * blockDim.x) {
        float v = V[j + (int64_t)(c0 + c) * ldv];
        if (right) v *= right[j];
        m = fmaxf(m, fabsf(v));
    }
    sm[threadIdx.x] = m;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if (threadIdx.x < off) sm[threadIdx.x] = fmaxf(sm[threadIdx.x], sm[threadIdx.x + off]);
        __syncthreads();
    }
    if (threadIdx.x == 0) part[(size_t)c * gridDim.x + blockIdx.x] = sm[0];
    (void)bc;
}
// Stage 2: column scale = power of two that puts the column maximum in [2^12, 2^13); stores the scale and the
// epilogue factor 2^-bias / scale.
__global__ void k_colscale(const float* __restrict__ part, int blocks, int bc, int BT, float* __restrict__ scale,
                           float* __restrict__ inv) {
    const int c = threadIdx.x;
    if (c >= BT) return;
    float m = 0.f;
    if (c < bc)
        for (int b = 0; b < blocks; ++b) m = fmaxf(m, part[(size_t)c * blocks + b]);
    float sc = 1.0f;
    if (m > 0.f && isfinite(m)) {
        int e;
        frexpf(m, &e);                               // m = f * 2^e, f in [0.5, 1)
        sc = ldexpf(1.0f, 13 - e);
    }
    scale[c] = sc;
    inv[c] = ldexpf(1.0f, -kBias) / sc;
}
// wt_hi / wt_lo [c * np + j] = fp16 split of scale_c * right_j * V[j, c0 + c]; zero padding for j >= N and c >= bc.
__global__ void k_pack_wt(const float* __restrict__ V, int64_t ldv, const float* __restrict__ right, int64_t N, int64_t np,
                          int c0, int bc, const float* __restrict__ scale, __half* __restrict__ hi, __half* __restrict__ lo) {
    const int c = blockIdx.y;
    const float sc = scale[c];
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < np; j += (int64_t)gridDim.x * blockDim.x) {
        float v = 0.f;
        if (c < bc && j < N) {
            v = V[j + (int64_t)(c0 + c) * ldv];
            if (right) v *= right[j];
            v *= sc;
        }
        const __half h = __float2half_rn(v);
        hi[(int64_t)c * np + j] = h;
        if (lo) lo[(int64_t)c * np + j] = __float2half_rn(v - __half2float(h));
    }
}

// Symmetric row-sum mode: fixed-point sums -> q.
__global__ void k_sym_finish(const unsigned long long* __restrict__ sums, int64_t n, double scale, float* __restrict__ q) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) q[i] = (float)((double)(long long)sums[i] * scale);
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

bool make_map_2d(CUtensorMap* m, void* base, uint64_t inner, uint64_t outer, uint64_t row_bytes, uint32_t box_inner,
                 uint32_t box_outer, CUtensorMapSwizzle sw) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {row_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BT, int MODE>
fd_status launch_tc(fd_ctx* c, const CUtensorMap& mr, const CUtensorMap& mc, const CUtensorMap& mh, const TcParams& p, int grid) {
    const int smem = Smem<BT, MODE>::total(p.K16);
    if (smem > 227 * 1024) return fail(c, FD_ERR_UNSUPPORTED, "tensor-core kernel needs %d B of shared memory", smem);
    // the attribute is per device: set it on every launch (cheap) rather than remembering one device
    FD_CUDA(c, cudaFuncSetAttribute(k_tc<BT, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    k_tc<BT, MODE><<<grid, kThreads, smem, c->stream>>>(mr, mc, mh, p);
    FD_LAUNCH_CHECK(c, "k_tc");
    return FD_OK;
}

}  // namespace

bool tc_supported(const fd_ctx* c, const ApplyArgs& a) {
    const Layout& L = c->L;
    if (!c->centered) return false;
    if (L.K16 > 4) return false;                                   // D <= 60
    if ((int64_t)L.K16 * L.NP >= ((int64_t)1 << 31)) return false;    // TMA row coordinates are 32-bit
    if (a.Nrow > L.N) return false;
    // The decision depends only on the data set, the bandwidth and the precision mode -- never on the kind of pass --
    // so the degree passes and the block products of one operator always run on the same kernel family (their
    // common rounding bias then cancels in diag(s) K diag(s)).
    // small problems: the split direct-difference kernel fills the GPU better (it covers D <= 32 only)
    if (c->opt_path != FD_PATH_TC && L.N < 16384 && L.DP <= 32) return false;
    const double bprime = a.beta * kLog2e;
    // exponent magnitude the fp16 hi/lo norm pieces and the fp32 Gram accumulation can carry accurately
    const double mag = bprime * (a.rows_are_ctx ? c->max_sq : std::max(c->max_sq, c->row_max_sq));
    if (!(mag < (a.prec == FD_PREC_FAST ? 2000.0 : c->opt_tc_max_mag))) return false;
    if (a.V == nullptr && a.right != nullptr && !a.right_pos) return false;   // row-sum mode folds a POSITIVE right vector into e_j
    return true;
}

fd_status apply_tc(fd_ctx* c, const ApplyArgs& a) {
    const Layout& L = c->L;
    const int64_t N = L.N, NP = L.NP;
    if (!encode_fn()) return fail(c, FD_ERR_CUDA, "cuTensorMapEncodeTiled entry point unavailable");
    const double bprime = a.beta * kLog2e;
    const bool rowsum = a.V == nullptr;
    const double* mu = c->at<double>(L.mu);
    __half* xp_col = c->at<__half>(L.xp_col);
    __half* xp_row = c->at<__half>(L.xp_row);
    unsigned int* status = c->at<unsigned int>(L.status);
    const int K16 = L.K16;
    const int pk_blocks = (int)ceil_div(NP, 256);
    // operands: columns (role 1) always from the context's points, rows (role 0) from a.xrow
    // the same bias in both modes: the S tiles of the degree pass and of the block product are then bit-identical, so
    // any rounding bias of the Gram accumulation is common to q and to K and cancels in diag(s) K diag(s)
    k_pack_points<<<pk_blocks, 256, 0, c->stream>>>(c->xs(), L.DP, L.D, N, NP, mu, bprime, 1, (double)kBias,
                                                   rowsum ? a.right : nullptr, K16, xp_col);
    FD_LAUNCH_CHECK(c, "k_pack_points(col)");
    // Symmetric row sums (K = K^T): a square pass over the context's own points whose left and right weights are the same
    // vector (the degree passes) evaluates only the tiles on or above the diagonal; the weight is folded into both exponents.
    const bool sym = rowsum && a.sym_ok && c->opt_sym != 0 && a.rows_are_ctx && a.xrow == c->xs() && a.Nrow == N &&
                     a.left == a.right && L.symsum != 0;
    k_pack_points<<<pk_blocks, 256, 0, c->stream>>>(a.xrow, L.DP, L.D, a.Nrow, NP, mu, bprime, 0, 0.0, sym ? a.right : nullptr, K16,
                                                   xp_row);
    FD_LAUNCH_CHECK(c, "k_pack_points(row)");

    CUtensorMap mr, mc, mh;
    if (!make_map_2d(&mr, xp_row, 32, (uint64_t)K16 * NP, 64, 32, 128, CU_TENSOR_MAP_SWIZZLE_64B) ||
        !make_map_2d(&mc, xp_col, 32, (uint64_t)K16 * NP, 64, 32, 128, CU_TENSOR_MAP_SWIZZLE_64B))
        return fail(c, FD_ERR_CUDA, "cuTensorMapEncodeTiled failed for the point operands");

    TcParams p{};
    p.Nrow = a.Nrow; p.N = N;
    p.num_work = (int)ceil_div(a.Nrow, 256);
    p.num_jt = (int)ceil_div(N, 128);
    // column chunk: ~1024 tiles (40 MB of fp16 operands at b = 64) stay resident in the 126 MB L2 while every CTA sweeps them
    p.jt_chunk = rowsum ? p.num_jt : (c->opt_jt_chunk > 0 ? c->opt_jt_chunk : 1024);
    if (p.jt_chunk > p.num_jt) p.jt_chunk = p.num_jt;
    p.num_chunks = (int)ceil_div(p.num_jt, p.jt_chunk);
    p.np_rows = NP; p.np_cols = NP; p.K16 = K16;
    p.left = a.left; p.status = status;
    p.flush = c->opt_flush > 0 ? c->opt_flush : 1;
    const int grid = std::min(p.num_work, c->sm_count);

    if (rowsum && sym) {
        p.num_jt = (int)(NP / 128);                      // even: every row pair's two diagonal tiles exist (padding gives 2^e = 0)
        p.jt_chunk = p.num_jt; p.num_chunks = 1;
        p.left = nullptr;
        p.q = a.Y; p.rowsq = a.rowsq; p.b = 1;
        p.symsum = c->at<unsigned long long>(L.symsum);
        // sums are at most NP * 2^bias in the kernel's scaled units: the fixed-point unit keeps them below 2^61
        int lg = 0;
        while (((int64_t)1 << lg) < NP) ++lg;
        p.sym_shift = 61 - kBias - lg;
        FD_CUDA(c, cudaMemsetAsync(p.symsum, 0, (size_t)N * 8, c->stream));
        const int sym_grid = std::min((p.num_work + 1) / 2, c->sm_count);
        if (p.rowsq) FD_TRY((launch_tc<16, kModeRowsumSym>(c, mr, mc, mc, p, sym_grid)));
        else FD_TRY((launch_tc<32, kModeRowsumSym>(c, mr, mc, mc, p, sym_grid)));
        k_sym_finish<<<(unsigned)ceil_div(N, 256), 256, 0, c->stream>>>(p.symsum, N, std::ldexp(1.0, -(kBias + (int)p.sym_shift)), a.Y);
        FD_LAUNCH_CHECK(c, "k_sym_finish");
    } else if (rowsum) {
        p.q = a.Y; p.rowsq = a.rowsq; p.b = 1;
        if (p.rowsq) FD_TRY((launch_tc<16, kModeRowsum>(c, mr, mc, mc, p, grid)));
        else FD_TRY((launch_tc<32, kModeRowsum>(c, mr, mc, mc, p, grid)));
    } else {
        __half* wt_hi = c->at<__half>(L.wt_hi);
        __half* wt_lo = c->at<__half>(L.wt_lo);
        float* scale = c->at<float>(L.colscale);
        float* inv = scale + L.BP + 8;
        float* part = c->at<float>(L.part);
        const bool fast = a.prec == FD_PREC_FAST;
        // widest column chunk whose stages fit in shared memory: 64 columns up to D = 28, 32 up to D = 44, 16 beyond (the
        // fp32-grade kernel stages W_hi and W_lo; the reduced-precision kernel stages one of them and always fits 64)
        const int limit = 227 * 1024;
        const int cw = fast || Smem<64, kModeBlock>::total(K16) <= limit ? 64 : Smem<32, kModeBlock>::total(K16) <= limit ? 32 : 16;
        for (int c0 = 0; c0 < a.b; c0 += cw) {
            const int bc = std::min(cw, a.b - c0);
            const int BT = bc <= 16 ? 16 : bc <= 32 ? 32 : 64;
            if (BT > L.BP) return fail(c, FD_ERR_WORKSPACE, "column tile %d wider than the provisioned block buffers (%d)", BT, L.BP);
            const int cm_blocks = (int)std::min<int64_t>(256, ceil_div(N, 1024));
            k_colmax_partial<<<dim3(cm_blocks, bc), 256, 0, c->stream>>>(a.V, a.ldv, a.right, N, c0, bc, part);
            FD_LAUNCH_CHECK(c, "k_colmax_partial");
            k_colscale<<<1, 64, 0, c->stream>>>(part, cm_blocks, bc, BT, scale, inv);
            FD_LAUNCH_CHECK(c, "k_colscale");
            k_pack_wt<<<dim3((unsigned)std::min<int64_t>(1024, ceil_div(NP, 256)), BT), 256, 0, c->stream>>>(
                a.V, a.ldv, a.right, N, NP, c0, bc, scale, wt_hi, fast ? nullptr : wt_lo);
            FD_LAUNCH_CHECK(c, "k_pack_wt");
            // one map over W_hi (rows 0 .. BT) and, in the fp32-grade mode, W_lo behind it (rows BP .. BP + BT of the same array)
            if (wt_lo != wt_hi + (size_t)L.BP * NP) return fail(c, FD_ERR_INVALID, "W_hi and W_lo are not adjacent in the workspace");
            p.lo_row = L.BP;
            if (!make_map_2d(&mh, wt_hi, (uint64_t)NP, (uint64_t)(fast ? BT : L.BP + BT), (uint64_t)NP * 2, 64, BT, CU_TENSOR_MAP_SWIZZLE_128B))
                return fail(c, FD_ERR_CUDA, "cuTensorMapEncodeTiled failed for the block operands");
            p.b = bc; p.colscale_inv = inv; p.Y = a.Y + (int64_t)c0 * a.ldy; p.ldy = a.ldy;
            if (fast) {
                // reduced-precision mode (single fp16 operands): the one-row-tile kernel with sixteen exponential warps
                TcParams pb = p;                   // 128-row work items
                pb.num_work = (int)ceil_div(a.Nrow, 128);
                // the accumulator is flushed every 8 column tiles here: the round-toward-zero loss of the longer groups
                // (a few 1e-6) is far below this mode's own error (3e-4), and the flushes cost 4 %
                if (c->opt_flush <= 0) pb.flush = 8;
                FD_TRY(launch_fast_product(c, BT, mr, mc, mh, pb, std::min(pb.num_work, c->sm_count)));
                continue;
            }
            // Tail split: with a single column chunk (N up to about 2^17) the row pairs of the last, partly filled round --
            // or all pairs when there are fewer than CTAs -- are each shared by two CTAs (half the column range each).
            int bgrid = grid;
            p.tail_split = 0;
            if (p.num_chunks == 1 && p.num_jt >= 2 && c->opt_tail_split != 0) {
                const int tail = p.num_work % grid;                  // pairs in the last round (grid = min(pairs, SMs))
                const int tail_pairs = p.num_work < c->sm_count ? p.num_work : tail;
                if (tail_pairs > 0 && 2 * tail_pairs <= c->sm_count) {
                    p.tail_split = 2;
                    p.tail_pairs = tail_pairs;
                    p.tail_first = p.num_work - tail_pairs;
                    bgrid = std::max(grid, 2 * tail_pairs);
                    const int64_t r0t = (int64_t)p.tail_first * 256;
                    FD_CUDA(c, cudaMemset2DAsync(p.Y + r0t, (size_t)p.ldy * 4, 0, (size_t)(a.Nrow - r0t) * 4, (size_t)bc, c->stream));
                }
            }
            if (p.tail_split == 2) {
                switch (BT) {
                    case 16: FD_TRY((launch_tc<16, kModeBlockTail>(c, mr, mc, mh, p, bgrid))); break;
                    case 32: FD_TRY((launch_tc<32, kModeBlockTail>(c, mr, mc, mh, p, bgrid))); break;
                    default: FD_TRY((launch_tc<64, kModeBlockTail>(c, mr, mc, mh, p, bgrid))); break;
                }
                continue;
            }
            switch (BT) {
                case 16: FD_TRY((launch_tc<16, kModeBlock>(c, mr, mc, mh, p, grid))); break;
                case 32: FD_TRY((launch_tc<32, kModeBlock>(c, mr, mc, mh, p, grid))); break;
                default: FD_TRY((launch_tc<64, kModeBlock>(c, mr, mc, mh, p, grid))); break;
            }
        }
    }
    return FD_OK;
}

fd_status tc_wait_selftest(fd_ctx* c, long long limit_cycles) {
    k_wait_selftest<<<1, 32, 0, c->stream>>>(c->at<unsigned int>(c->L.status), limit_cycles);
    FD_LAUNCH_CHECK(c, "k_wait_selftest");
    return FD_OK;
}

// Reads the kernel's status word (after the stream has been synchronised by the caller).
fd_status tc_check_status(fd_ctx* c) {
    unsigned int h = 0;
    FD_CUDA(c, cudaMemcpyAsync(&h, c->at<unsigned int>(c->L.status), 4, cudaMemcpyDeviceToHost, c->stream));
    FD_CUDA(c, cudaStreamSynchronize(c->stream));
    if (h != 0) {
        FD_CUDA(c, cudaMemsetAsync(c->at<unsigned int>(c->L.status), 0, 4, c->stream));
        return fail(c, FD_ERR_TIMEOUT, "tensor-core kernel: bounded wait expired (code 0x%x)", h);
    }
    return FD_OK;
}

}  // namespace fd
