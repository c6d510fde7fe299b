// fd_unit_peaks: measured per-SM throughput of the units the hot path leans on, for the roofline denominators.
//
// The Gaussian block product is bound by on-chip arithmetic, not by HBM: one exponential per pair on the MUFU, the
// hi/lo split on the ALU and FMA pipes, and the Gram / product contractions on the tensor cores.  The roofline in the
// benchmark therefore needs per-clock unit rates rather than a copy bandwidth; this file measures them with tiny
// kernels that count SM cycles (clock64), so the results are rates per clock per SM and do not depend on the clock the
// GPU happens to run at.  Each probe keeps 1024 threads per SM busy with eight independent dependency chains per
// thread; the tensor-core probe issues back-to-back tcgen05.mma instructions of the shapes the kernels use from one
// thread and waits for their completion through a bounded mbarrier wait.
#include <vector>

#include "fd_tc_common.h"

namespace fd {

namespace {

using namespace tc;

enum Probe { kEx2 = 0, kFfma = 1, kCvtF16x2 = 2, kLop = 3, kFadd = 4 };

template <int OP>
__global__ void __launch_bounds__(1024, 1) k_probe_alu(long long* __restrict__ cycles, float* __restrict__ sink, int iters, float seed) {
    float x[8];
    uint32_t u[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { x[i] = seed - 0.001f * (float)(threadIdx.x + i); u[i] = __float_as_uint(x[i]); }
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (OP == kEx2) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(x[i]));
            if (OP == kFfma) asm volatile("fma.rn.f32 %0, %0, %0, %0;" : "+f"(x[i]));
            if (OP == kCvtF16x2) { asm volatile("cvt.rn.f16x2.f32 %0, %1, %1;" : "=r"(u[i]) : "f"(x[i])); x[i] = __uint_as_float(u[i]); }
            if (OP == kLop) asm volatile("xor.b32 %0, %0, %1;" : "+r"(u[i]) : "r"(u[(i + 1) & 7]));    // not foldable: the operand changes
            if (OP == kFadd) asm volatile("add.f32 %0, %0, %0;" : "+f"(x[i]));
        }
    }
    const long long t1 = clock64();
    float s = 0.f;
    uint32_t v = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { s += x[i]; v ^= u[i]; }
    sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = s + __uint_as_float(v);
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// Back-to-back tcgen05.mma kind::f16, M = 128, K = 16, fp32 accumulation in TMEM; A from TMEM (TS) or shared memory (SS).
// Operands are whatever the zero-filled buffers hold: only the time matters.
template <int N, int TS>
__global__ void __launch_bounds__(128, 1) k_probe_mma(long long* __restrict__ cycles, int iters) {
    extern __shared__ uint8_t raw[];
    uint8_t* base = (uint8_t*)(((uintptr_t)raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar;
    __shared__ uint32_t tbase;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
    for (int i = threadIdx.x; i < 48 * 1024 / 4; i += blockDim.x) ((uint32_t*)base)[i] = 0u;
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tbase)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tbase;
    if (warp == 0 && lane == 0) {
        const uint64_t a = smem_desc(smem_u32(base), 1024, 2), b = smem_desc(smem_u32(base + 16384), 1024, 2);
        const long long t0 = clock64();
        for (int i = 0; i < iters; ++i) {
            if (TS) mma_ts(tmem + 256, tmem + (uint32_t)(i & 7) * 8u, b + 2 * (i & 3), idesc_f16(N), 1);
            else mma_ss(tmem + 256, a + 2 * (i & 3), b + 2 * (i & 3), idesc_f16(N), 1);
        }
        tc_commit(&bar);
        long long guard = 0;
        while (!mbar_try_wait(&bar, 0) && ++guard < 50000000ll) {}
        cycles[blockIdx.x] = guard < 50000000ll ? clock64() - t0 : -1;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

template <int OP>
cudaError_t run_alu(cudaStream_t st, int sms, long long* cyc_dev, float* sink_dev, double* per_clk_sm) {
    const int iters = 2000;
    k_probe_alu<OP><<<sms, 1024, 0, st>>>(cyc_dev, sink_dev, 20, -1.5f);            // warm-up
    k_probe_alu<OP><<<sms, 1024, 0, st>>>(cyc_dev, sink_dev, iters, -1.5f);
    fd::g_launches += 2;
    std::vector<long long> h(sms);
    cudaError_t e = cudaMemcpyAsync(h.data(), cyc_dev, sizeof(long long) * sms, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return e;
    double c = 0;
    for (int i = 0; i < sms; ++i) c += (double)h[i];
    c /= sms;
    *per_clk_sm = 1024.0 * iters * 8.0 / c;
    return cudaSuccess;
}

template <int N, int TS>
cudaError_t run_mma(cudaStream_t st, int sms, long long* cyc_dev, double* clk_per_mma) {
    const int iters = 2048, smem = 50 * 1024;
    cudaError_t e = cudaFuncSetAttribute(k_probe_mma<N, TS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    k_probe_mma<N, TS><<<sms, 128, smem, st>>>(cyc_dev, 64);
    k_probe_mma<N, TS><<<sms, 128, smem, st>>>(cyc_dev, iters);
    fd::g_launches += 2;
    std::vector<long long> h(sms);
    e = cudaMemcpyAsync(h.data(), cyc_dev, sizeof(long long) * sms, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return e;
    double c = 0;
    for (int i = 0; i < sms; ++i) { if (h[i] < 0) return cudaErrorUnknown; c += (double)h[i]; }
    *clk_per_mma = c / sms / iters;
    return cudaSuccess;
}

}  // namespace
}  // namespace fd

using namespace fd;

extern "C" fd_status fd_unit_peaks(void* scratch_dev, size_t scratch_bytes, void* cuda_stream, fd_unit_rates* out_host) {
    if (!scratch_dev || !out_host) return FD_ERR_INVALID;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return FD_ERR_CUDA;
    const size_t need = (size_t)sms * 1024 * 4 + (size_t)sms * 8 + 256;
    if (scratch_bytes < need) return FD_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(scratch_dev) & 255) != 0) return FD_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    long long* cyc = static_cast<long long*>(scratch_dev);
    float* sink = reinterpret_cast<float*>(static_cast<char*>(scratch_dev) + (((size_t)sms * 8 + 255) & ~(size_t)255));
    fd_unit_rates r{};
    r.sm_count = sms;
    cudaError_t e = cudaSuccess;
    if (e == cudaSuccess) e = run_alu<kEx2>(st, sms, cyc, sink, &r.ex2_per_clk_sm);
    if (e == cudaSuccess) e = run_alu<kFfma>(st, sms, cyc, sink, &r.ffma_per_clk_sm);
    if (e == cudaSuccess) e = run_alu<kCvtF16x2>(st, sms, cyc, sink, &r.cvt_f16x2_per_clk_sm);
    if (e == cudaSuccess) e = run_alu<kLop>(st, sms, cyc, sink, &r.lop_per_clk_sm);
    if (e == cudaSuccess) e = run_alu<kFadd>(st, sms, cyc, sink, &r.fadd_per_clk_sm);
    if (e == cudaSuccess) e = run_mma<64, 1>(st, sms, cyc, &r.clk_mma_ts_n64);
    if (e == cudaSuccess) e = run_mma<128, 1>(st, sms, cyc, &r.clk_mma_ts_n128);
    if (e == cudaSuccess) e = run_mma<64, 0>(st, sms, cyc, &r.clk_mma_ss_n64);
    if (e == cudaSuccess) e = run_mma<128, 0>(st, sms, cyc, &r.clk_mma_ss_n128);
    if (e != cudaSuccess) return FD_ERR_CUDA;
    *out_host = r;
    return FD_OK;
}
