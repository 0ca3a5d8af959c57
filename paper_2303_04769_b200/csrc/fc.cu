// Full reduction (paper Section 3.2 item 5): the fully connected layer on blocked [N][J][1][1] -> [N][K][1][1].
// One warp per (image, block of 32 outputs); the lane is the output channel, as in the convolution kernels.
#include "common.cuh"

namespace small {

__global__ void __launch_bounds__(256) fc_kernel(const float *__restrict__ in, const float *__restrict__ w,
                                                 const float *__restrict__ bias, float *__restrict__ out,
                                                 int N, int JB, int K, int KB, bool relu) {
    grid_dep_sync();
    grid_dep_trigger();
    const int lane = threadIdx.x & 31;
    const long long warps = (long long)N * KB;
    for (long long wid = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5; wid < warps;
         wid += ((long long)gridDim.x * blockDim.x) >> 5) {
        int kb = (int)(wid % KB);
        long long n = wid / KB;
        int k = kb * 32 + lane;
        float acc = (bias && k < K) ? bias[k] : 0.0f;
        const float *x = in + n * JB * 32;
        const float *wt = w + (size_t)kb * JB * 32 * 32 + lane;
        for (int jb = 0; jb < JB; ++jb) {
            float xv = x[jb * 32 + lane];
#pragma unroll
            for (int j = 0; j < 32; ++j) acc = fmaf(__shfl_sync(0xffffffffu, xv, j), wt[(jb * 32 + j) * 32], acc);
        }
        if (relu) acc = acc > 0.f ? acc : 0.f;
        out[wid * 32 + lane] = k < K ? acc : 0.0f;
    }
}

int launch_fc(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, int N, int J, int K, bool relu, cudaStream_t st) {
    int JB = blocks_of(J), KB = blocks_of(K);
    long long warps = (long long)N * KB;
    long long want = (warps + 7) / 8, cap = (long long)ctx->sm_count * 16;
    launch_kernel(ctx, fc_kernel, dim3((unsigned)(want < cap ? want : cap)), dim3(256), 0, st, in, w, bias, out, N, JB, K, KB, relu);
    return check_launch(ctx);
}

}  // namespace small
