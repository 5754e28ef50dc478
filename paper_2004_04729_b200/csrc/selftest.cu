// Self-test of the bounded waits: every wait inside the tensor-core kernels polls an mbarrier
// against a clock budget and, when the budget runs out, records the fact and lets the kernel
// return. This kernel runs that same wait on a barrier that nobody ever arrives on, with a small
// budget, so that the expiry path (flag set, every thread returns, context still usable) can be
// exercised without disturbing any product kernel.
#include "tc_common.cuh"

namespace dbp {

namespace {

__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(long long budget, int *err_flag) {
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    // phase 0 never completes: there is no arrival anywhere in this kernel
    if (threadIdx.x == 0) tc::mbar_wait(&bar, 0u, err_flag, budget);
}

// fp32 FMA rate: every thread runs eight independent chains of dependent FMAs (enough to cover the
// pipeline's latency with 4 warps per scheduler... the grid puts 2048 threads on every SM)
__global__ void __launch_bounds__(256) fma_chain_kernel(float *out, int iters, float a, float b) {
    float x0 = threadIdx.x, x1 = x0 + 1.f, x2 = x0 + 2.f, x3 = x0 + 3.f, x4 = x0 + 4.f, x5 = x0 + 5.f, x6 = x0 + 6.f, x7 = x0 + 7.f;
#pragma unroll 1
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            x0 = fmaf(x0, a, b); x1 = fmaf(x1, a, b); x2 = fmaf(x2, a, b); x3 = fmaf(x3, a, b);
            x4 = fmaf(x4, a, b); x5 = fmaf(x5, a, b); x6 = fmaf(x6, a, b); x7 = fmaf(x7, a, b);
        }
    }
    const float s = ((x0 + x1) + (x2 + x3)) + ((x4 + x5) + (x6 + x7));
    if (s == 123.456f) out[0] = s;             // keeps the chains alive; practically never true
}

}  // namespace

int measure_fma_peak(dbp_ctx *ctx, double *tflops) {
    float *out = nullptr;
    if (cudaMalloc(&out, sizeof(float)) != cudaSuccess) return DBP_ENOMEM;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) { cudaFree(out); return DBP_ECUDA; }
    const int blocks = ctx->sm_count * 8, iters = 4096;
    double best = 0.0;
    for (int rep = 0; rep < 4; ++rep) {
        cudaEventRecord(e0, ctx->stream);
        note_launch();
        fma_chain_kernel<<<blocks, 256, 0, ctx->stream>>>(out, iters, 0.999f, 0.001f);
        cudaEventRecord(e1, ctx->stream);
        if (cudaEventSynchronize(e1) != cudaSuccess) { cudaFree(out); return fail_cuda("FMA rate kernel"); }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double flops = 2.0 * 64.0 * iters * 256.0 * blocks;
        if (rep > 0 && ms > 0.f && flops / (ms * 1e-3) / 1e12 > best) best = flops / (ms * 1e-3) / 1e12;
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1); cudaFree(out);
    *tflops = best;
    return DBP_OK;
}

int launch_bounded_wait_selftest(dbp_ctx *ctx, long long budget) {
    note_launch();
    bounded_wait_selftest_kernel<<<1, 32, 0, ctx->stream>>>(budget, &ctx->state->tc_timeout);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dbp
