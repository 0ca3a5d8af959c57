// Single element reductions (paper Section 3.2 item 1): ReLU (the Max kernel against zero) and addition.
// Bandwidth-bound: 128-bit loads and stores over the channel block, several independent loads in flight per thread.
#include "common.cuh"

namespace small {

__device__ __forceinline__ float relu1(float v) { return v > 0.0f ? v : 0.0f; }   // -0 and negatives -> +0
__device__ __forceinline__ float4 relu4(float4 v) { return make_float4(relu1(v.x), relu1(v.y), relu1(v.z), relu1(v.w)); }

template <int UNROLL>
__global__ void __launch_bounds__(256) relu_kernel(const float4 *__restrict__ in, float4 *__restrict__ out, size_t n4) {
    grid_dep_sync();
    grid_dep_trigger();
    size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    for (; i + (UNROLL - 1) * stride < n4; i += UNROLL * stride) {
        float4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) v[u] = __ldcs(in + i + u * stride);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) __stcs(out + i + u * stride, relu4(v[u]));
    }
    for (; i < n4; i += stride) __stcs(out + i, relu4(__ldcs(in + i)));
}

template <int UNROLL>
__global__ void __launch_bounds__(256) add_kernel(const float4 *__restrict__ a, const float4 *__restrict__ b,
                                                  float4 *__restrict__ out, size_t n4, bool relu) {
    grid_dep_sync();
    grid_dep_trigger();
    size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    for (; i + (UNROLL - 1) * stride < n4; i += UNROLL * stride) {
        float4 x[UNROLL], y[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) { x[u] = __ldcs(a + i + u * stride); y[u] = __ldcs(b + i + u * stride); }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            float4 r = make_float4(x[u].x + y[u].x, x[u].y + y[u].y, x[u].z + y[u].z, x[u].w + y[u].w);
            __stcs(out + i + u * stride, relu ? relu4(r) : r);
        }
    }
    for (; i < n4; i += stride) {
        float4 x = __ldcs(a + i), y = __ldcs(b + i);
        float4 r = make_float4(x.x + y.x, x.y + y.y, x.z + y.z, x.w + y.w);
        __stcs(out + i, relu ? relu4(r) : r);
    }
}

// Launch shape from a sweep on B200: tensors well beyond L2 stream best with few loads per thread and 4 CTAs per SM;
// smaller ones (where ramp-up and tail are a large part of the run) want 8 CTAs per SM and 8 loads in flight each.
static int stream_grid(small_ctx *ctx, size_t n4, int unroll, int ctas_per_sm) {
    size_t want = (n4 + 256ull * unroll - 1) / (256ull * unroll);
    size_t cap = (size_t)ctx->sm_count * ctas_per_sm;
    if (want < 1) want = 1;
    return (int)(want < cap ? want : cap);
}
static bool is_large(size_t n4) { return n4 * 16 >= (size_t)64 << 20; }

// Batch normalisation at inference (paper Table 2: single element, FMA): out = scale[c] * in + shift[c].  One thread =
// four channels of one pixel; the channel's scale and shift come from the 128-byte line position (chunk of the block),
// pad lanes (c >= C) are written as +0.
__global__ void __launch_bounds__(256) scale_shift_kernel(const float4 *__restrict__ in, const float *__restrict__ scale,
                                                          const float *__restrict__ shift, float4 *__restrict__ out,
                                                          size_t n4, int C, int CB, size_t plane4, bool relu) {
    size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4; i += stride) {
        const int cb = (int)((i / plane4) % CB);            // plane4 = H * W * 8 vectors per (image, channel block)
        const int c = cb * 32 + (int)(i & 7) * 4;
        const float4 v = __ldcs(in + i);
        float4 r;
        r.x = c + 0 < C ? fmaf(scale[c + 0], v.x, shift[c + 0]) : 0.0f;
        r.y = c + 1 < C ? fmaf(scale[c + 1], v.y, shift[c + 1]) : 0.0f;
        r.z = c + 2 < C ? fmaf(scale[c + 2], v.z, shift[c + 2]) : 0.0f;
        r.w = c + 3 < C ? fmaf(scale[c + 3], v.w, shift[c + 3]) : 0.0f;
        __stcs(out + i, relu ? relu4(r) : r);
    }
}

// Upsample (paper Table 2: nearest neighbour): out[n][cb][oh][ow] = in[n][cb][oh / f][ow / f]; one thread writes four
// channels of one output pixel, so a warp writes four whole output lines.
__global__ void __launch_bounds__(256) upsample_nearest_kernel(const float4 *__restrict__ in, float4 *__restrict__ out,
                                                               size_t n4_out, int H, int W, int f) {
    const int OW = W * f, OH = H * f;
    size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n4_out; i += stride) {
        const int j = (int)(i & 7);
        size_t p = i >> 3;
        const int ow = (int)(p % OW); p /= OW;
        const int oh = (int)(p % OH); p /= OH;             // p = image * channel blocks + block
        __stcs(out + i, __ldg(in + ((p * H + oh / f) * W + ow / f) * 8 + j));
    }
}

int launch_scale_shift(small_ctx *ctx, const float *in, const float *scale, const float *shift, float *out,
                       int N, int C, int H, int W, bool relu, cudaStream_t st) {
    const int CB = blocks_of(C);
    const size_t plane4 = (size_t)H * W * 8, n4 = (size_t)N * CB * plane4;
    scale_shift_kernel<<<stream_grid(ctx, n4, 1, 8), 256, 0, st>>>(reinterpret_cast<const float4 *>(in), scale, shift,
                                                                  reinterpret_cast<float4 *>(out), n4, C, CB, plane4, relu);
    return check_launch(ctx);
}

int launch_upsample_nearest(small_ctx *ctx, const float *in, float *out, int N, int C, int H, int W, int f, cudaStream_t st) {
    const size_t n4 = (size_t)N * blocks_of(C) * H * f * W * f * 8;
    upsample_nearest_kernel<<<stream_grid(ctx, n4, 1, 8), 256, 0, st>>>(reinterpret_cast<const float4 *>(in),
                                                                        reinterpret_cast<float4 *>(out), n4, H, W, f);
    return check_launch(ctx);
}

int launch_relu(small_ctx *ctx, const float *in, float *out, size_t n, cudaStream_t st) {
    size_t n4 = n / 4;   // a blocked tensor is a whole number of 32-float lines
    const float4 *i4 = reinterpret_cast<const float4 *>(in);
    float4 *o4 = reinterpret_cast<float4 *>(out);
    if (is_large(n4)) launch_kernel(ctx, relu_kernel<2>, dim3((unsigned)(stream_grid(ctx, n4, 2, 4))), dim3(256), 0, st, i4, o4, n4);
    else launch_kernel(ctx, relu_kernel<8>, dim3((unsigned)(stream_grid(ctx, n4, 8, 8))), dim3(256), 0, st, i4, o4, n4);
    return check_launch(ctx);
}

int launch_add(small_ctx *ctx, const float *a, const float *b, float *out, size_t n, bool relu, cudaStream_t st) {
    size_t n4 = n / 4;
    const float4 *a4 = reinterpret_cast<const float4 *>(a), *b4 = reinterpret_cast<const float4 *>(b);
    float4 *o4 = reinterpret_cast<float4 *>(out);
    if (is_large(n4)) launch_kernel(ctx, add_kernel<2>, dim3((unsigned)(stream_grid(ctx, n4, 2, 4))), dim3(256), 0, st, a4, b4, o4, n4, relu);
    else launch_kernel(ctx, add_kernel<4>, dim3((unsigned)(stream_grid(ctx, n4, 4, 8))), dim3(256), 0, st, a4, b4, o4, n4, relu);
    return check_launch(ctx);
}

}  // namespace small
