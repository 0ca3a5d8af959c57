// Issue-rate probe for the TF32 tensor-core pipe: every SM runs a long chain of tcgen05.mma kind::tf32 (M = 128, N as
// requested, K = 8) on operands that already sit in shared memory, so nothing but the pipe limits it.  The result is
// the dense TF32 rate this part sustains, the denominator for the tensor-bound rooflines of the convolution.
#include "common.cuh"

namespace small {
namespace {

__device__ __forceinline__ uint32_t probe_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__global__ void __launch_bounds__(128, 1) tf32_peak_kernel(int n, int iters, long long *cycles, int *status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (probe_smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - probe_smem_u32(smem_raw));
    __shared__ __align__(8) unsigned long long bar;
    __shared__ uint32_t tmem_slot;
    const uint32_t a_addr = base, b_addr = base + 128 * 128;
    // operands: small finite values (the pipe's timing does not depend on them)
    float *ops = reinterpret_cast<float *>(base_ptr);
    for (int i = threadIdx.x; i < (128 + n) * 32; i += blockDim.x) ops[i] = (float)((i * 2654435761u >> 20) & 255) * (1.0f / 256.0f);
    const uint32_t bar_addr = probe_smem_u32(&bar);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_addr) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(probe_smem_u32(&tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_slot;
    if (threadIdx.x == 0) {
        const uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
        const uint32_t a_lo = ((a_addr & 0x3FFFFu) >> 4) | (1u << 16), b_lo = ((b_addr & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
        // Eight MMA chains per loop trip, round robin over the independent accumulators that fit in tensor memory,
        // issued as straight-line code: with index arithmetic or branches between the MMAs the issuing thread, not
        // the pipe, sets the pace for small n.
        const int slots = 512 / n > 8 ? 8 : 512 / n;
        uint32_t dd[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) dd[j] = tmem + (uint32_t)((j % slots) * n);
        const long long t0 = clock64();
        for (int i = 0; i < iters; i += 8) {
            const uint32_t acc = i > 0 ? 1u : 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    asm volatile(
                        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
                        "setp.ne.b32 p, %5, 0;\n\t"
                        "mov.b64 da, {%1, %3};\n\t"
                        "mov.b64 db, {%2, %3};\n\t"
                        "tcgen05.mma.cta_group::1.kind::tf32 [%0], da, db, %4, p;\n\t}"
                        ::"r"(dd[j]), "r"(a_lo + 2u * k), "r"(b_lo + 2u * k), "r"(desc_hi), "r"(idesc), "r"(k > 0 ? 1u : acc) : "memory");
                }
            }
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_addr) : "memory");
        bool done = false;
        for (uint32_t it = 0; it < (1u << 26) && !done; ++it) {
            uint32_t ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(bar_addr) : "memory");
            done = ok != 0;
        }
        if (!done) atomicExch(status, (int)SMALL_ERR_TIMEOUT);
        cycles[blockIdx.x] = clock64() - t0;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

}  // namespace
}  // namespace small

using namespace small;

SMALL_API int small_measure_tf32_peak(small_ctx *ctx, int n, int iters, long long *cycles_dev, double *tflops,
                                      double *cycles_per_mma, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!cycles_dev || !tflops || !cycles_per_mma) return SMALL_ERR_INVALID_ARG;
    if ((n != 32 && n != 64 && n != 128 && n != 256) || iters < 8 || iters > (1 << 20) || iters % 8) return SMALL_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t smem = 1024 + (size_t)(128 + n) * 128;
    cudaError_t e = cudaFuncSetAttribute(tf32_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    float ms = 0.f;
    if (e == cudaSuccess) {
        tf32_peak_kernel<<<ctx->sm_count, 128, smem, st>>>(n, iters, cycles_dev, ctx->dev_status);   // warm-up
        cudaEventRecord(e0, st);
        tf32_peak_kernel<<<ctx->sm_count, 128, smem, st>>>(n, iters, cycles_dev, ctx->dev_status);
        cudaEventRecord(e1, st);
        e = cudaEventSynchronize(e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    }
    long long first = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&first, cycles_dev, sizeof(first), cudaMemcpyDeviceToHost);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    const double flops = 2.0 * 128.0 * n * 8.0 * 4.0 * iters * ctx->sm_count;
    *tflops = flops / (ms * 1e-3) / 1e12;
    *cycles_per_mma = (double)first / (4.0 * iters);
    return SMALL_OK;
}
