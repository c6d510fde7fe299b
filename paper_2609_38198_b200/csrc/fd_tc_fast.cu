// Reduced-precision block product Y_I += K_IJ W_J on tcgen05 / TMEM (Eqs. 5-6): the kernel behind fd_apply with
// FD_PREC_FAST on the Gram-form path (single fp16 operands for K and W; relative Frobenius error ~2e-4, bound 3e-3).
//
// Per (row tile I, column tile J) of 128 x 128 pairs:
//   1. Gram MMA of augmented fp16 hi|lo points: the tile leaves the tensor core as the base-2 exponent
//        S_ij = 2 b' x_i.x_j - b' r_i - b' r_j + bias      (Eq. 4; the norms ride as extra K columns)
//      into one of three 128-column TMEM buffers.
//   2. Exponential warps (thread = row, 64 columns each) read S, take 2^S on the MUFU, round P to fp16 and write it
//      back IN PLACE as the TMEM A operand of the product.
//   3. Product MMA per 16-column K step:  Y += P W  with W = diag(right) V in fp16, fp32 accumulation in TMEM.
//   4. Every `flush` column tiles a separate warpgroup adds Y into fp32 registers and the accumulator restarts, so
//      tensor-core accumulation error does not grow with N.
//
// One persistent CTA per SM works on one 128-row tile at a time.  24 warps:
//   warps 0-15   exponential warps, four warpgroups: warpgroup k takes column half (k & 1) of every tile whose running
//                index has parity (k >> 1).  Two tiles are always being exponentiated while a third S buffer is with the
//                tensor core, so neither the MUFU (four warps per scheduler, in different phases) nor the tensor pipe
//                waits for the other in steady state;
//   warps 16-19  flush warpgroup: owns the fp32 accumulator registers and the epilogue;
//   warp 20      TMA producer (4-stage ring of column tiles; every CTA loads its own copy);
//   warp 21 / 22 product-MMA issuer / Gram-MMA issuer (one thread each: two independent dependency chains).
// TMEM (512 columns): three S/P buffers at [0, 384), accumulator at [384, 384 + BT).
// Registers: compiled for 80 per thread (65536 / 768 rounded down to the allocation unit); setmaxnreg then moves
// registers from the utility and exponential warps to the flush warpgroup; the total is conserved exactly (an increase
// that the decreases do not cover would block for ever), and the host checks the compiled count before launching.
// Every mbarrier wait is bounded; on expiry the CTA raises a status word, drains and exits.
//
// The fp32-grade product (fp16 hi + lo pieces of P and W, three MMA terms) stays on the two-row-tile kernel of
// fd_tc.cu: with three times the tensor work per tile the GPU runs at its power limit, and sharing each staged column
// tile between two row tiles costs less energy per pair than this layout (measured at N = 2^20: 537 ms against 582 ms).
#include <algorithm>

#include "fd_tc_common.h"

namespace fd {

namespace {

using namespace tc;

constexpr int kThreadsBp = 768;
constexpr int kRegsLaunch = 80, kRegsExp = 72, kRegsFlush = 152, kRegsUtil = 40;
static_assert(kThreadsBp * kRegsLaunch == 512 * kRegsExp + 128 * kRegsFlush + 128 * kRegsUtil,
              "setmaxnreg must conserve the register total");

template <int BT>
struct SmemP {
    static constexpr int kXChunk = 128 * 64;                          // one K slab (hi|lo) of 128 points: 8 KB
    static constexpr int kWHalf = BT * 128;                           // 64 j x BT columns fp16
    static constexpr int kWBytes = 2 * kWHalf;                        // [W j-half 0][W j-half 1]
    static __host__ __device__ constexpr int stage_bytes(int K16) { return K16 * kXChunk + kWBytes; }
    static __host__ __device__ constexpr int total(int K16) {
        return 1024 /*align slack*/ + kStages * stage_bytes(K16) + K16 * kXChunk + 1024 /*barriers*/;
    }
};

struct BarriersP {
    uint64_t full[kStages], empty[kStages];   // column stage: TMA -> issuers; product issuer -> TMA
    uint64_t xfull, xempty;                   // row operand tile of a work item
    uint64_t s_full[6];                       // [tile index mod 6]: exponent tile ready (Gram issuer -> one pair of warpgroups)
    uint64_t p_done[3][2];                    // [S buffer][half]: P half written in place (warpgroup -> product issuer)
    uint64_t kw_done[3];                      // [S buffer]: product MMAs that read it have completed (-> Gram issuer)
    uint64_t y_full, y_empty;                 // accumulator flush hand-off (product issuer <-> flush warpgroup)
    uint32_t tmem_base;
    int abort_flag;
};

template <int BT>
__global__ void __launch_bounds__(kThreadsBp, 1)
k_bp(const __grid_constant__ CUtensorMap map_xrow, const __grid_constant__ CUtensorMap map_xcol,
     const __grid_constant__ CUtensorMap map_whi, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    using SM = SmemP<BT>;
    constexpr uint32_t kYCol = 384;                    // accumulator: columns [384, 384 + BT)
    const int K16 = p.K16;
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_base = base;
    uint8_t* xi_base = base + kStages * SM::stage_bytes(K16);                 // K16 slabs of the row tile
    BarriersP* bars = (BarriersP*)(xi_base + K16 * SM::kXChunk);
    volatile int* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
        mbar_init(&bars->xfull, 1); mbar_init(&bars->xempty, 1);
        for (int u = 0; u < 6; ++u) mbar_init(&bars->s_full[u], 1);
        for (int u = 0; u < 3; ++u) {
            mbar_init(&bars->kw_done[u], 1);
            mbar_init(&bars->p_done[u][0], 4); mbar_init(&bars->p_done[u][1], 4);
        }
        mbar_init(&bars->y_full, 1); mbar_init(&bars->y_empty, 4);
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 20) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;
    const long long t_begin = clock64();

    // Work items of this CTA: (column chunk c, row tile r), c outermost, r = blockIdx.x + k * gridDim.x.  Every CTA sweeps
    // chunk c for all of its rows before chunk c + 1, so the whole grid reads the same L2-sized slice of the column
    // operands at about the same time; a row's partial results always come from the same thread, in order.
    // Tiles are numbered by a running index gt across work items; S buffer = gt mod 3, exponential pair = gt mod 2.
    const int my_rows = (p.num_work - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int my_items = my_rows * p.num_chunks;
#define FD_ITEM_P(w)                                                                                \
    const int cch = (w) / my_rows;                                                                  \
    const int item = (int)blockIdx.x + ((w) % my_rows) * (int)gridDim.x;                            \
    const int j0 = cch * p.jt_chunk;                                                                \
    const int num_jt = (p.num_jt - j0 < p.jt_chunk) ? p.num_jt - j0 : p.jt_chunk;                   \
    (void)item; (void)cch; (void)j0
    const int flush = p.flush;

    if (warp >= 20) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsUtil));
      if (warp == 20) {
        // =============================================================== TMA producer (one thread)
        if (lane == 0) {
            prefetch_tmap(&map_xrow); prefetch_tmap(&map_xcol); prefetch_tmap(&map_whi);
            uint32_t it = 0;
            bool ok = true;
            for (int w = 0; w < my_items && ok; ++w) {
                FD_ITEM_P(w);
                ok = mbar_wait(&bars->xempty, (w & 1) ^ 1, abort_flag, p.status, 1);
                if (!ok) break;
                mbar_expect_tx(&bars->xfull, K16 * SM::kXChunk);
                for (int c = 0; c < K16; ++c)
                    tma_load_2d(xi_base + c * SM::kXChunk, &map_xrow, 0, (int)(c * p.np_rows + (int64_t)item * 128), &bars->xfull);
                for (int j = 0; j < num_jt; ++j, ++it) {
                    const int s = it % kStages;
                    ok = mbar_wait(&bars->empty[s], ((it / kStages) & 1) ^ 1, abort_flag, p.status, 2);
                    if (!ok) break;
                    uint8_t* st = stage_base + s * SM::stage_bytes(K16);
                    mbar_expect_tx(&bars->full[s], SM::stage_bytes(K16));
                    for (int c = 0; c < K16; ++c)
                        tma_load_2d(st + c * SM::kXChunk, &map_xcol, 0, (int)(c * p.np_cols + (int64_t)(j0 + j) * 128), &bars->full[s]);
                    uint8_t* wst = st + K16 * SM::kXChunk;
                    const int x0 = (j0 + j) * 128;
                    tma_load_2d(wst, &map_whi, x0, 0, &bars->full[s]);
                    tma_load_2d(wst + SM::kWHalf, &map_whi, x0 + 64, 0, &bars->full[s]);
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
      } else if (warp == 22) {
        // =============================================================== Gram MMA issuer (one thread)
        // S(gt) = A_I B_J^T as soon as its buffer is free again (the product MMAs of tile gt - 3 have completed); runs up to
        // three tiles ahead of the product.
        if (lane == 0) {
            constexpr uint32_t idesc_g = idesc_f16(128);
            // descriptors as (low, high) words: 64 B rows (SWIZZLE_64B), 512 B between 8-row groups
            const uint64_t xd = smem_desc(smem_u32(xi_base), 512, 4);
            const uint32_t xi_lo = (uint32_t)xd, xdesc_hi = (uint32_t)(xd >> 32);
            const uint32_t stage_lo = (uint32_t)smem_desc(smem_u32(stage_base), 512, 4);
            const uint32_t stage_step = (uint32_t)(SM::stage_bytes(K16) >> 4);
            uint32_t gt = 0, slot = 0, use = 0, six = 0;            // tile index; gt mod 3; gt / 3; gt mod 6
            bool ok = true;
            for (int w = 0; w < my_items && ok; ++w) {
                FD_ITEM_P(w);
                ok = mbar_wait(&bars->xfull, w & 1, abort_flag, p.status, 3);
                if (!ok) break;
                for (int j = 0; j < num_jt && ok; ++j, ++gt) {
                    const int s = gt % kStages;
                    if (use > 0) {
                        ok = mbar_wait(&bars->kw_done[slot], (use - 1) & 1, abort_flag, p.status, 5);
                        if (!ok) break;
                    }
                    ok = mbar_wait(&bars->full[s], (gt / kStages) & 1, abort_flag, p.status, 4);
                    if (!ok) break;
                    tc_fence_after();
                    // The two small cross terms (hi x lo) go first and the large hi x hi term last: each MMA rounds its
                    // result at the magnitude of its largest addend, so only the final one rounds at full magnitude.
                    const uint32_t s_addr = tmem + 128u * slot;
                    const uint32_t b_lo = stage_lo + (uint32_t)s * stage_step;
                    if (K16 == 1) {
                        mma_ss2<0>(s_addr, xi_lo, xdesc_hi, b_lo + 2, xdesc_hi, idesc_g);      // + 2: the lo half starts 32 B into the row
                        mma_ss2<1>(s_addr, xi_lo + 2, xdesc_hi, b_lo, xdesc_hi, idesc_g);
                        mma_ss2<1>(s_addr, xi_lo, xdesc_hi, b_lo, xdesc_hi, idesc_g);
                    } else {
                        for (int c = 0; c < K16; ++c) {
                            const uint32_t a = xi_lo + (uint32_t)c * (SM::kXChunk >> 4), b = b_lo + (uint32_t)c * (SM::kXChunk >> 4);
                            if (c == 0) mma_ss2<0>(s_addr, a, xdesc_hi, b + 2, xdesc_hi, idesc_g);
                            else mma_ss2<1>(s_addr, a, xdesc_hi, b + 2, xdesc_hi, idesc_g);
                            mma_ss2<1>(s_addr, a + 2, xdesc_hi, b, xdesc_hi, idesc_g);
                        }
                        for (int c = 0; c < K16; ++c) {
                            const uint32_t a = xi_lo + (uint32_t)c * (SM::kXChunk >> 4), b = b_lo + (uint32_t)c * (SM::kXChunk >> 4);
                            mma_ss2<1>(s_addr, a, xdesc_hi, b, xdesc_hi, idesc_g);
                        }
                    }
                    tc_commit(&bars->s_full[six]);
                    if (++slot == 3) { slot = 0; ++use; }
                    if (++six == 6) six = 0;
                }
                if (ok) tc_commit(&bars->xempty);                  // the row operand tile may be replaced
            }
        }
      } else if (warp == 21) {
        // =============================================================== product MMA issuer (one thread)
        if (lane == 0) {
            constexpr uint32_t idesc_y = idesc_f16(BT);
            const uint32_t y_addr = tmem + kYCol;
            // W stage descriptor as (low, high) words: 128 B rows (SWIZZLE_128B), 1024 B between 8-row groups
            const uint64_t wd = smem_desc(smem_u32(stage_base + K16 * SM::kXChunk), 1024, 2);
            const uint32_t wbase_lo = (uint32_t)wd, wdesc_hi = (uint32_t)(wd >> 32);
            const uint32_t stage_step = (uint32_t)(SM::stage_bytes(K16) >> 4);
            uint32_t gt = 0, slot = 0, use = 0, n_grp = 0;
            bool ok = true;
            for (int w = 0; w < my_items && ok; ++w) {
                FD_ITEM_P(w);
                int in_group = 0;                                  // tiles accumulated in the current group
                for (int j = 0; j < num_jt && ok; ++j, ++gt) {
                    const int s = gt % kStages;
                    const bool group_start = in_group == 0;
                    const bool group_end = in_group + 1 == flush || j + 1 == num_jt;
                    in_group = group_end ? 0 : in_group + 1;
                    const uint32_t w_lo = wbase_lo + (uint32_t)s * stage_step;
                    const uint32_t p_addr = tmem + 128u * slot;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        ok = mbar_wait(&bars->p_done[slot][h], use & 1, abort_flag, p.status, 7);
                        if (!ok) break;
                        if (h == 0 && group_start && n_grp > 0) {
                            ok = mbar_wait(&bars->y_empty, (n_grp - 1) & 1, abort_flag, p.status, 6);
                            if (!ok) break;
                        }
                        tc_fence_after();
                        // W tile of column half h; K step k of the half starts 32 B (two 16-byte units) further into the
                        // 128 B rows.  K step ks reads P at S-buffer columns [16 ks, 16 ks + 8).
                        const uint32_t bh = w_lo + (uint32_t)((h * SM::kWHalf) >> 4);
                        const uint32_t ph = p_addr + 64u * h;
                        if (h == 0 && group_start) mma_ts2<0>(y_addr, ph, bh, wdesc_hi, idesc_y);
                        else mma_ts2<1>(y_addr, ph, bh, wdesc_hi, idesc_y);
#pragma unroll
                        for (int k = 1; k < 4; ++k) mma_ts2<1>(y_addr, ph + 16 * k, bh + 2 * k, wdesc_hi, idesc_y);
                    }
                    if (!ok) break;
                    tc_commit(&bars->kw_done[slot]);
                    if (group_end) { tc_commit(&bars->y_full); ++n_grp; }
                    tc_commit(&bars->empty[s]);
                    if (++slot == 3) { slot = 0; ++use; }
                }
            }
        }
      }
    } else if (warp >= 16) {
        // =============================================================== flush warpgroup (thread = row)
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsFlush));
        const int wq = warp & 3;                       // TMEM lane quarter this warp may access
        const uint32_t y_addr = tmem + ((uint32_t)(wq * 32) << 16) + kYCol;
        const int row_in_tile = wq * 32 + lane;
        uint32_t n_grp = 0;
        bool ok = true;
        for (int w = 0; w < my_items && ok; ++w) {
            FD_ITEM_P(w);
            const int64_t row = (int64_t)item * 128 + row_in_tile;
            float acc[BT];
#pragma unroll
            for (int c = 0; c < BT; ++c) acc[c] = 0.f;
            // The tensor core adds each K step into the TMEM accumulator with round-toward-zero.  For a sum whose partial sums
            // keep one sign, n additions lose n / 4 ulp of the result on average (half an ulp each, at a running magnitude
            // that averages half the final one): measured 2.85e-8 per addition against 2^-25 = 2.98e-8.  The flush adds that
            // expected loss back (one FMA instead of one add); it is far below this mode's own rounding error.
            int left_tiles = num_jt;
            while (left_tiles > 0 && ok) {
                const int tiles_in_group = left_tiles < flush ? left_tiles : flush;
                left_tiles -= tiles_in_group;
                const float corr = 1.0f + (float)(tiles_in_group * 8) * 2.98023224e-8f;
                ok = mbar_wait(&bars->y_full, n_grp & 1, abort_flag, p.status, 10);
                if (!ok) break;
                ++n_grp;
                tc_fence_after();
                uint32_t v[BT / 16][16];
#pragma unroll
                for (int c0 = 0; c0 < BT / 16; ++c0) tmem_ld16(y_addr + 16 * c0, v[c0]);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->y_empty);        // handed back before the additions
#pragma unroll
                for (int c = 0; c < BT; ++c) acc[c] = fmaf(__uint_as_float(v[c / 16][c % 16]), corr, acc[c]);
            }
            if (ok && row < p.Nrow) {
                const float l = p.left ? p.left[row] : 1.0f;
#pragma unroll
                for (int c = 0; c < BT; ++c)
                    if (c < p.b) {
                        float* o = p.Y + row + (int64_t)c * p.ldy;
                        const float v = acc[c] * l * p.colscale_inv[c];
                        __stcs(o, cch == 0 ? v : __ldcs(o) + v);   // later column chunks add to the partial result of the same thread (streaming: touched once per chunk round)
                    }
            }
        }
    } else {
        // =============================================================== exponential warps
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsExp));
        const int wg = warp >> 2;                      // warpgroup 0..3
        const int pr = wg >> 1;                        // takes the tiles whose running index has this parity
        const int h = wg & 1;                          // column half of every tile it takes
        const int wq = warp & 3;                       // TMEM lane quarter this warp may access
        const uint32_t lane_addr = ((uint32_t)(wq * 32) << 16) + 64u * h;
        uint32_t gt = 0, slot = 0, six = 0, use6 = 0;  // running tile index; gt mod 3; gt mod 6; gt / 6
        bool ok = true;
        for (int w = 0; w < my_items && ok; ++w) {
            FD_ITEM_P(w);
            for (int j = 0; j < num_jt && ok; ++j, ++gt) {
                if ((int)(gt & 1) == pr) {
                    ok = mbar_wait(&bars->s_full[six], use6 & 1, abort_flag, p.status, 9);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t addr = tmem + lane_addr + 128u * slot;
#pragma unroll
                    for (int q32 = 0; q32 < 2; ++q32) {
                        uint32_t sv[32];
                        tmem_ld32(addr + 32 * q32, sv);
                        tmem_wait_ld();
#pragma unroll
                        for (int ch = 0; ch < 2; ++ch) {
                            uint32_t hi[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const float p0 = ex2f(__uint_as_float(sv[16 * ch + 2 * i]));
                                const float p1 = ex2f(__uint_as_float(sv[16 * ch + 2 * i + 1]));
                                hi[i] = pack_f16x2(p0, p1);
                            }
                            tmem_st8(addr + 32 * q32 + 16 * ch, hi);
                        }
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->p_done[slot][h]);
                }
                if (++slot == 3) slot = 0;
                if (++six == 6) { six = 0; ++use6; }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    // SM cycles CTA 0 spent on its work items (status words 2-3): lets the host relate the kernel time to the SM clock
    if (blockIdx.x == 0 && threadIdx.x == 0) *reinterpret_cast<long long*>(p.status + 2) = clock64() - t_begin;
    if (warp == 20) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

template <int BT>
fd_status launch_one(fd_ctx* c, const CUtensorMap& mr, const CUtensorMap& mc, const CUtensorMap& mh, const TcParams& p, int grid) {
    const int smem = SmemP<BT>::total(p.K16);
    if (smem > 227 * 1024) return fail(c, FD_ERR_UNSUPPORTED, "tensor-core kernel needs %d B of shared memory", smem);
    // the attribute is per device: set it on every launch (cheap) rather than remembering one device
    FD_CUDA(c, cudaFuncSetAttribute(k_bp<BT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    cudaFuncAttributes fa;
    FD_CUDA(c, cudaFuncGetAttributes(&fa, k_bp<BT>));
    if (fa.numRegs != kRegsLaunch)
        return fail(c, FD_ERR_UNSUPPORTED, "fast block-product kernel compiled with %d registers per thread, %d expected", fa.numRegs, kRegsLaunch);
    k_bp<BT><<<grid, kThreadsBp, smem, c->stream>>>(mr, mc, mh, p);
    FD_LAUNCH_CHECK(c, "k_bp");
    return FD_OK;
}

}  // namespace

namespace tc {

fd_status launch_fast_product(fd_ctx* c, int BT, const CUtensorMap& mr, const CUtensorMap& mc, const CUtensorMap& mh,
                              const TcParams& p, int grid) {
    switch (BT) {
        case 16: return launch_one<16>(c, mr, mc, mh, p, grid);
        case 32: return launch_one<32>(c, mr, mc, mh, p, grid);
        case 64: return launch_one<64>(c, mr, mc, mh, p, grid);
    }
    return fail(c, FD_ERR_UNSUPPORTED, "no fast block-product instantiation for column tile %d", BT);
}

}  // namespace tc

}  // namespace fd
