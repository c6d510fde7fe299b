// Row-sharded operation over several processes with one GPU each (Sec. 3 of the paper shards its multi-GPU runs over
// the row axis).  Every rank holds all N points and owns a contiguous range of rows; the quadratic passes evaluate the
// owned rows against all columns, and the only data exchanged are N x b blocks (rows gathered from their owners) and
// small host matrices (summed).  The library links no communication library: the two collectives are callbacks.
#include <algorithm>

#include "fd_internal.h"

namespace fd {

void shard_range(int64_t N, int world, int rank, int64_t* begin, int64_t* end) {
    const int64_t chunk = round_up(ceil_div(N, world), 256);
    const int64_t b = std::min<int64_t>(N, (int64_t)rank * chunk);
    *begin = b;
    *end = std::min<int64_t>(N, b + chunk);
}

fd_status allreduce_host(fd_ctx* c, double* buf, int64_t n) {
    if (!c->sh.on || n < 1) return FD_OK;
    if (c->sh.h.allreduce_sum_host(c->sh.h.user, buf, n) != 0) return fail(c, FD_ERR_COMM, "allreduce_sum_host callback failed");
    return FD_OK;
}

fd_status gather_rows(fd_ctx* c, float* A, int64_t lda, int cols) {
    if (!c->sh.on || cols < 1) return FD_OK;
    const fd_ctx::Shard& sh = c->sh;
    const int64_t N = c->L.N, chunk = sh.chunk, n_own = sh.r1 - sh.r0;
    const int group = c->L.BP;                                   // the exchange buffer holds BP columns per rank
    float* send = static_cast<float*>(sh.h.xchg_dev);
    float* recv = send + (size_t)group * chunk;
    for (int c0 = 0; c0 < cols; c0 += group) {
        const int w = std::min(group, cols - c0);
        float* Ac = A + (int64_t)c0 * lda;
        // own rows -> contiguous [w][chunk] (rows beyond the owned range of a short last shard are never read back)
        if (n_own > 0)
            FD_CUDA(c, cudaMemcpy2DAsync(send, (size_t)chunk * 4, Ac + sh.r0, (size_t)lda * 4, (size_t)n_own * 4, (size_t)w,
                                         cudaMemcpyDeviceToDevice, c->stream));
        if (sh.h.allgather_dev(sh.h.user, send, recv, (int64_t)w * chunk) != 0)
            return fail(c, FD_ERR_COMM, "allgather_dev callback failed");
        for (int r = 0; r < sh.h.world; ++r) {
            if (r == sh.h.rank) continue;
            int64_t b, e;
            shard_range(N, sh.h.world, r, &b, &e);
            if (e <= b) continue;
            FD_CUDA(c, cudaMemcpy2DAsync(Ac + b, (size_t)lda * 4, recv + (size_t)r * w * chunk, (size_t)chunk * 4,
                                         (size_t)(e - b) * 4, (size_t)w, cudaMemcpyDeviceToDevice, c->stream));
        }
    }
    return FD_OK;
}

}  // namespace fd

using namespace fd;

extern "C" {

fd_status fd_shard_rows(int64_t N, int32_t world, int32_t rank, int64_t* row_begin, int64_t* row_end) {
    if (N < 1 || world < 1 || rank < 0 || rank >= world || !row_begin || !row_end) return FD_ERR_INVALID;
    shard_range(N, world, rank, row_begin, row_end);
    return FD_OK;
}

size_t fd_shard_exchange_bytes(int64_t N, int32_t b_max, int32_t world) {
    if (N < 1 || b_max < 1 || b_max > 256 || world < 1) return 0;
    const int64_t chunk = round_up(ceil_div(N, world), 256);
    const int64_t BP = make_layout(N, 1, b_max, 0).BP;
    return (size_t)(world + 1) * (size_t)BP * (size_t)chunk * 4;
}

fd_status fd_set_shard(fd_ctx* c, const fd_shard* shard) {
    if (!c) return FD_ERR_INVALID;
    if (!shard) { c->sh = fd_ctx::Shard{}; return FD_OK; }
    if (shard->world < 1 || shard->rank < 0 || shard->rank >= shard->world) return fail(c, FD_ERR_INVALID, "bad rank / world");
    if (!shard->allreduce_sum_host || !shard->allgather_dev) return fail(c, FD_ERR_INVALID, "missing exchange callback");
    if (!shard->xchg_dev || (reinterpret_cast<uintptr_t>(shard->xchg_dev) & 255) != 0)
        return fail(c, FD_ERR_INVALID, "exchange buffer null or not 256-byte aligned");
    if (shard->xchg_bytes < fd_shard_exchange_bytes(c->L.N, c->L.b_max, shard->world))
        return fail(c, FD_ERR_WORKSPACE, "exchange buffer smaller than fd_shard_exchange_bytes");
    c->sh.on = true;
    c->sh.h = *shard;
    c->sh.chunk = round_up(ceil_div(c->L.N, shard->world), 256);
    shard_range(c->L.N, shard->world, shard->rank, &c->sh.r0, &c->sh.r1);
    c->have_s = false;                                           // the operator state must be rebuilt by fd_degree
    return FD_OK;
}

}  // extern "C"
