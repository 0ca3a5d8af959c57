// Self-test of the give-up-and-return path of the bounded device-side waits.  Every pipeline wait in this library
// (TMA arrival, stage release, accumulator hand-over) polls an mbarrier a limited number of times; when the limit runs
// out the kernel records SMALL_ERR_TIMEOUT in the context's status word and returns normally - it never traps and never
// spins without bound.  This kernel makes exactly that happen without any copy in flight: it waits, with the context's
// limit and the same wait routine the layer kernels use, on a barrier that nothing ever arms.
#include "common.cuh"
#include "sm100.cuh"

namespace small {
namespace {

__global__ void wait_on_unarmed_barrier_kernel(int *status, uint32_t limit, unsigned long long *polls_out) {
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = sm100::smem_u32(&bar);
    if (threadIdx.x == 0) {
        sm100::mbar_init(b, 1);
        sm100::mbar_fence_init();
    }
    __syncthreads();
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = sm100::mbar_wait(b, 0, limit) ? 1 : 0;     // one lane per warp polls, as in the layer kernels
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok && threadIdx.x == 0) {
        atomicExch(status, (int)SMALL_ERR_TIMEOUT);
        if (polls_out) *polls_out = limit;
    }
}

}  // namespace
}  // namespace small

using namespace small;

SMALL_API int small_selftest_wait_timeout(small_ctx *ctx, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    wait_on_unarmed_barrier_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(ctx->dev_status, ctx->wait_iters, nullptr);
    return check_launch(ctx);
}
