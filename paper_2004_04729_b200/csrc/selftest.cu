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

}  // namespace

int launch_bounded_wait_selftest(dbp_ctx *ctx, long long budget) {
    bounded_wait_selftest_kernel<<<1, 32, 0, ctx->stream>>>(budget, &ctx->state->tc_timeout);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dbp
