// Full reduction (paper Section 3.2 item 5): the fully connected layer on blocked [N][J][1][1] -> [N][K][1][1].
// The lane is the output channel, as in the convolution kernels.  Two mappings of the (image, block of 32 outputs)
// units: one thread block per unit, its eight warps sharing out the input's channel blocks, so that a long reduction
// (a classifier head behind a wide last layer) is eight short chains combined through shared memory instead of one
// long one; and, when there are units enough to fill the GPU many times over, one warp per unit with no block-wide
// synchronisation.
#include "common.cuh"

namespace small {

__global__ void __launch_bounds__(256) fc_kernel(const float *__restrict__ in, const float *__restrict__ w,
                                                 const float *__restrict__ bias, float *__restrict__ out,
                                                 int N, int JB, int K, int KB, bool relu) {
    grid_dep_sync();
    grid_dep_trigger();
    __shared__ float part[8][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long units = (long long)N * KB;
    for (long long u = blockIdx.x; u < units; u += gridDim.x) {
        const int kb = (int)(u % KB);
        const long long n = u / KB;
        const float *x = in + n * JB * 32;
        const float *wt = w + (size_t)kb * JB * 32 * 32 + lane;
        float acc = 0.0f;
        for (int jb = warp; jb < JB; jb += 8) {
            const float xv = x[jb * 32 + lane];
#pragma unroll
            for (int j = 0; j < 32; ++j) acc = fmaf(__shfl_sync(0xffffffffu, xv, j), wt[(jb * 32 + j) * 32], acc);
        }
        part[warp][lane] = acc;
        __syncthreads();
        if (warp == 0) {
            const int k = kb * 32 + lane;
            float v = (bias && k < K) ? bias[k] : 0.0f;
#pragma unroll
            for (int i = 0; i < 8; ++i) v += part[i][lane];
            if (relu) v = v > 0.f ? v : 0.f;
            out[u * 32 + lane] = k < K ? v : 0.0f;
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256) fc_warp_kernel(const float *__restrict__ in, const float *__restrict__ w,
                                                      const float *__restrict__ bias, float *__restrict__ out,
                                                      int N, int JB, int K, int KB, bool relu) {
    grid_dep_sync();
    grid_dep_trigger();
    const int lane = threadIdx.x & 31;
    const long long warps = (long long)N * KB;
    for (long long wid = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5; wid < warps;
         wid += ((long long)gridDim.x * blockDim.x) >> 5) {
        const int kb = (int)(wid % KB);
        const long long n = wid / KB;
        const int k = kb * 32 + lane;
        float acc = (bias && k < K) ? bias[k] : 0.0f;
        const float *x = in + n * JB * 32;
        const float *wt = w + (size_t)kb * JB * 32 * 32 + lane;
        for (int jb = 0; jb < JB; ++jb) {
            const float xv = x[jb * 32 + lane];
#pragma unroll
            for (int j = 0; j < 32; ++j) acc = fmaf(__shfl_sync(0xffffffffu, xv, j), wt[(jb * 32 + j) * 32], acc);
        }
        if (relu) acc = acc > 0.f ? acc : 0.f;
        out[wid * 32 + lane] = k < K ? acc : 0.0f;
    }
}

// Abstract fused layer (Section 6): a global average pool (single channel reduction over the whole plane) and the full
// reduction behind it - the classifier head of the networks - as one kernel.  One thread block per image: its eight
// warps share out the pixels of each channel block (lane = channel, whole 128-byte lines), combine through shared
// memory into the averaged vector (rounded to float as the pooling layer would store it), then run the full
// reduction on it exactly as fc_kernel does.  The pooled tensor never goes to global memory.
__global__ void __launch_bounds__(256) gap_fc_kernel(const float *__restrict__ in, const float *__restrict__ w,
                                                     const float *__restrict__ bias, float *__restrict__ out,
                                                     int N, int JB, int HW, int K, int KB, bool relu) {
    grid_dep_sync();
    grid_dep_trigger();
    extern __shared__ float avg[];            // JB x 32 averaged channels
    __shared__ float part[8][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float hw = (float)HW;
    for (int n = blockIdx.x; n < N; n += gridDim.x) {
        for (int jb = 0; jb < JB; ++jb) {
            const float *plane = in + ((size_t)n * JB + jb) * HW * 32 + lane;
            float s0 = 0.0f, s1 = 0.0f;
            int p = warp;
            for (; p + 8 < HW; p += 16) { s0 += plane[(size_t)p * 32]; s1 += plane[(size_t)(p + 8) * 32]; }
            if (p < HW) s0 += plane[(size_t)p * 32];
            part[warp][lane] = s0 + s1;
            __syncthreads();
            if (warp == 0) {
                float v = 0.0f;
#pragma unroll
                for (int i = 0; i < 8; ++i) v += part[i][lane];
                avg[jb * 32 + lane] = v / hw;
            }
            __syncthreads();
        }
        for (int kb = 0; kb < KB; ++kb) {
            const float *wt = w + (size_t)kb * JB * 32 * 32 + lane;
            float acc = 0.0f;
            for (int jb = warp; jb < JB; jb += 8) {
#pragma unroll
                for (int j = 0; j < 32; ++j) acc = fmaf(avg[jb * 32 + j], wt[(jb * 32 + j) * 32], acc);
            }
            part[warp][lane] = acc;
            __syncthreads();
            if (warp == 0) {
                const int k = kb * 32 + lane;
                float v = (bias && k < K) ? bias[k] : 0.0f;
#pragma unroll
                for (int i = 0; i < 8; ++i) v += part[i][lane];
                if (relu) v = v > 0.f ? v : 0.f;
                out[((size_t)n * KB + kb) * 32 + lane] = k < K ? v : 0.0f;
            }
            __syncthreads();
        }
    }
}

int launch_gap_fc(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, int N, int C, int H, int W, int K,
                  bool relu, cudaStream_t st) {
    const int JB = blocks_of(C), KB = blocks_of(K);
    const size_t smem = (size_t)JB * 32 * sizeof(float);
    if (smem > 40 * 1024) return SMALL_ERR_UNSUPPORTED;
    const long long cap = (long long)ctx->sm_count * 8;
    launch_kernel(ctx, gap_fc_kernel, dim3((unsigned)(N < cap ? N : cap)), dim3(256), smem, st, in, w, bias, out, N, JB, H * W, K, KB, relu);
    return check_launch(ctx);
}

int launch_fc(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, int N, int J, int K, bool relu, cudaStream_t st) {
    int JB = blocks_of(J), KB = blocks_of(K);
    long long units = (long long)N * KB, cap = (long long)ctx->sm_count * 8;
    if (units >= 64LL * ctx->sm_count) {      // every SM gets 64 units or more: a warp each
        long long want = (units + 7) / 8, capw = (long long)ctx->sm_count * 16;
        launch_kernel(ctx, fc_warp_kernel, dim3((unsigned)(want < capw ? want : capw)), dim3(256), 0, st, in, w, bias, out, N, JB, K, KB, relu);
        return check_launch(ctx);
    }
    launch_kernel(ctx, fc_kernel, dim3((unsigned)(units < cap ? units : cap)), dim3(256), 0, st, in, w, bias, out, N, JB, K, KB, relu);
    return check_launch(ctx);
}

}  // namespace small
