// Layout kernels: NCHW <-> blocked activations (paper Section 4.4, Figure 2) and the one-time filter packing.
#include "common.cuh"

namespace small {

// One 32-channel x 32-pixel tile per iteration: read along the plane (NCHW's fast axis), write along the
// channel block (the blocked layout's fast axis), transposing through shared memory.
__global__ void __launch_bounds__(256) pack_kernel(const float *__restrict__ nchw, float *__restrict__ blk,
                                                   int C, int HW, int CB, long long tiles, int ptiles) {
    __shared__ float tile[32][33];
    const int tx = threadIdx.x, ty = threadIdx.y;
    for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        int pt = (int)(t % ptiles);
        long long ncb = t / ptiles;
        int cb = (int)(ncb % CB);
        long long n = ncb / CB;
        int p = pt * 32 + tx;
#pragma unroll
        for (int cl = ty; cl < 32; cl += 8) {
            int c = cb * 32 + cl;
            tile[cl][tx] = (c < C && p < HW) ? nchw[(n * C + c) * HW + p] : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int pl = ty; pl < 32; pl += 8) {
            int po = pt * 32 + pl;
            if (po < HW) blk[(ncb * HW + po) * 32 + tx] = tile[tx][pl];
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256) unpack_kernel(const float *__restrict__ blk, float *__restrict__ nchw,
                                                     int C, int HW, int CB, long long tiles, int ptiles) {
    __shared__ float tile[32][33];
    const int tx = threadIdx.x, ty = threadIdx.y;
    for (long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        int pt = (int)(t % ptiles);
        long long ncb = t / ptiles;
        int cb = (int)(ncb % CB);
        long long n = ncb / CB;
#pragma unroll
        for (int pl = ty; pl < 32; pl += 8) {
            int po = pt * 32 + pl;
            tile[pl][tx] = po < HW ? blk[(ncb * HW + po) * 32 + tx] : 0.0f;
        }
        __syncthreads();
        int p = pt * 32 + tx;
#pragma unroll
        for (int cl = ty; cl < 32; cl += 8) {
            int c = cb * 32 + cl;
            if (c < C && p < HW) nchw[(n * C + c) * HW + p] = tile[tx][cl];
        }
        __syncthreads();
    }
}

static int tile_grid(small_ctx *ctx, long long tiles) {
    long long cap = (long long)ctx->sm_count * 16;
    return (int)(tiles < cap ? tiles : cap);
}

int launch_pack(small_ctx *ctx, const float *nchw, float *blk, int N, int C, int H, int W, cudaStream_t st) {
    int HW = H * W, CB = blocks_of(C), ptiles = ceil_div(HW, 32);
    long long tiles = (long long)N * CB * ptiles;
    pack_kernel<<<tile_grid(ctx, tiles), dim3(32, 8), 0, st>>>(nchw, blk, C, HW, CB, tiles, ptiles);
    return check_launch(ctx);
}

int launch_unpack(small_ctx *ctx, const float *blk, float *nchw, int N, int C, int H, int W, cudaStream_t st) {
    int HW = H * W, CB = blocks_of(C), ptiles = ceil_div(HW, 32);
    long long tiles = (long long)N * CB * ptiles;
    unpack_kernel<<<tile_grid(ctx, tiles), dim3(32, 8), 0, st>>>(blk, nchw, C, HW, CB, tiles, ptiles);
    return check_launch(ctx);
}

// ---- filters -------------------------------------------------------------------------------------

__device__ __forceinline__ float round_tf32(float x) {
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
    return __uint_as_float(u);
}

// FP32 section: [KB][CB][FH][FW][32 ci][32 ko], ko fastest; channels beyond C / K hold zeros.
__global__ void pack_conv_w_fp32_kernel(const float *__restrict__ w, float *__restrict__ wb, int C, int K, int FH, int FW, size_t total) {
    int CB = (C + 31) / 32;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i;
        int ko = (int)(r % 32); r /= 32;
        int ci = (int)(r % 32); r /= 32;
        int y = (int)(r % FW); r /= FW;
        int x = (int)(r % FH); r /= FH;
        int cb = (int)(r % CB); r /= CB;
        int kb = (int)r;
        int k = kb * 32 + ko, c = cb * 32 + ci;
        wb[i] = (k < K && c < C) ? w[(((size_t)k * C + c) * FH + x) * FW + y] : 0.0f;
    }
}

// Group convolution (Section 3.1.2-3.1.3: G groups of K filters, group g reduces channels g*S_C .. g*S_C + F_C - 1;
// filters given as [G][K][F_C][FH][FW]).  Packed for the FP32 kernel as [KB][span][FH][FW][32 ci][32 ko]: block j of
// filter block kb is channel block cb0(kb) + j, cb0 = channel block of kb's first group; a (channel, filter) pair of
// different groups is stored as zero, so the kernel needs no group logic in its inner loops.
__global__ void pack_group_conv_w_kernel(const float *__restrict__ w, float *__restrict__ wb, int C, int F_C, int S_C, int Kg, int G,
                                         int span, int FH, int FW, size_t total) {
    const int OC = Kg * G;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i;
        int ko = (int)(r % 32); r /= 32;
        int ci = (int)(r % 32); r /= 32;
        int y = (int)(r % FW); r /= FW;
        int x = (int)(r % FH); r /= FH;
        int j = (int)(r % span); r /= span;
        int kb = (int)r;
        const int oc = kb * 32 + ko;
        float v = 0.0f;
        if (oc < OC) {
            const int g = oc / Kg;
            const int cb0 = ((kb * 32) / Kg * S_C) / 32;
            const int c = (cb0 + j) * 32 + ci;
            const int rel = c - g * S_C;
            if (c < C && rel >= 0 && rel < F_C) v = w[(((size_t)oc * F_C + rel) * FH + x) * FW + y];
        }
        wb[i] = v;
    }
}

// Tensor-core sections: [CB][FH*FW][KB*32 k][32 ci], ci fastest (the K-major B operand: one 128-byte row per
// output channel and input block).  hi = round-to-nearest TF32 of w; lo = TF32 of the exact residual w - hi.
__global__ void pack_conv_w_tc_kernel(const float *__restrict__ w, float *__restrict__ hi, float *__restrict__ lo,
                                      int C, int K, int FH, int FW, size_t total) {
    int Kp = ((K + 31) / 32) * 32, T = FH * FW;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i;
        int ci = (int)(r % 32); r /= 32;
        int k = (int)(r % Kp); r /= Kp;
        int tap = (int)(r % T); r /= T;
        int cb = (int)r;
        int c = cb * 32 + ci;
        float v = (k < K && c < C) ? w[((size_t)k * C + c) * T + tap] : 0.0f;
        float h = round_tf32(v);
        hi[i] = h;
        if (lo) lo[i] = round_tf32(v - h);
    }
}

// Depthwise: [CB][FH*FW][32 c].
__global__ void pack_dw_w_kernel(const float *__restrict__ w, float *__restrict__ wb, int C, int T, size_t total) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int ci = (int)(i % 32);
        int tap = (int)((i / 32) % T);
        int cb = (int)(i / 32 / T);
        int c = cb * 32 + ci;
        wb[i] = c < C ? w[(size_t)c * T + tap] : 0.0f;
    }
}

// Fully connected: [KB][JB*32 j][32 ko], ko fastest.

static int flat_grid(small_ctx *ctx, size_t total) {
    size_t b = (total + 255) / 256, cap = (size_t)ctx->sm_count * 8;
    return (int)(b < cap ? (b ? b : 1) : cap);
}

int launch_pack_conv_weights(small_ctx *ctx, const float *w, float *wb, int C, int K, int FH, int FW, unsigned math, cudaStream_t st) {
    size_t nA = conv_w_fp32_elems(C, K, FH, FW), nB = conv_w_tc_elems(C, K, FH, FW);
    pack_conv_w_fp32_kernel<<<flat_grid(ctx, nA), 256, 0, st>>>(w, wb, C, K, FH, FW, nA);
    if (int s = check_launch(ctx)) return s;
    if (math != SMALL_MATH_FP32) {
        float *hi = wb + nA, *lo = math == SMALL_MATH_3XTF32 ? hi + nB : nullptr;
        pack_conv_w_tc_kernel<<<flat_grid(ctx, nB), 256, 0, st>>>(w, hi, lo, C, K, FH, FW, nB);
        if (int s = check_launch(ctx)) return s;
    }
    return SMALL_OK;
}

// Tensor-core sections of a group convolution whose groups are whole channel blocks (F_C = S_C, multiples of 32, K a
// multiple of 32): [F_C/32][FH*FW][G*K rows][32 ci] - row g*K + k holds filter k of group g, so one box of K rows is one
// group's filter tile.  hi = TF32 rounding, lo = TF32 of the residual.
__global__ void pack_group_conv_w_tc_kernel(const float *__restrict__ w, float *__restrict__ hi, float *__restrict__ lo,
                                            int F_C, int K, int G, int FH, int FW, size_t total) {
    const int T = FH * FW, rows = G * K;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i;
        int ci = (int)(r % 32); r /= 32;
        int row = (int)(r % rows); r /= rows;
        int tap = (int)(r % T); r /= T;
        int cb = (int)r;
        const float v = w[((size_t)row * F_C + cb * 32 + ci) * T + tap];
        const float h = round_tf32(v);
        hi[i] = h;
        lo[i] = round_tf32(v - h);
    }
}

size_t group_conv_w_tc_elems(int F_C, int K, int G, int FH, int FW) { return (size_t)(F_C / 32) * FH * FW * G * K * 32; }

int launch_pack_group_conv_weights_tc(small_ctx *ctx, const float *w, float *hi, float *lo, int F_C, int K, int G, int FH, int FW, cudaStream_t st) {
    const size_t total = group_conv_w_tc_elems(F_C, K, G, FH, FW);
    pack_group_conv_w_tc_kernel<<<flat_grid(ctx, total), 256, 0, st>>>(w, hi, lo, F_C, K, G, FH, FW, total);
    return check_launch(ctx);
}

int group_conv_span(int C, int F_C, int S_C, int Kg) {
    const int G = (C - F_C) / S_C + 1, OC = Kg * G, KB = blocks_of(OC);
    int span = 1;
    for (int kb = 0; kb < KB; ++kb) {
        const int g0 = (kb * 32) / Kg;
        int g1 = (kb * 32 + 31) / Kg;
        if (g1 > G - 1) g1 = G - 1;
        const int need = (g1 * S_C + F_C - 1) / 32 - (g0 * S_C) / 32 + 1;
        if (need > span) span = need;
    }
    return span;
}

int launch_pack_group_conv_weights(small_ctx *ctx, const float *w, float *wb, int C, int F_C, int S_C, int Kg, int FH, int FW, cudaStream_t st) {
    const int G = (C - F_C) / S_C + 1, span = group_conv_span(C, F_C, S_C, Kg);
    const size_t total = (size_t)blocks_of(Kg * G) * span * FH * FW * 32 * 32;
    pack_group_conv_w_kernel<<<flat_grid(ctx, total), 256, 0, st>>>(w, wb, C, F_C, S_C, Kg, G, span, FH, FW, total);
    return check_launch(ctx);
}

int launch_pack_dw_weights(small_ctx *ctx, const float *w, float *wb, int C, int FH, int FW, cudaStream_t st) {
    size_t total = (size_t)blocks_of(C) * FH * FW * 32;
    pack_dw_w_kernel<<<flat_grid(ctx, total), 256, 0, st>>>(w, wb, C, FH * FW, total);
    return check_launch(ctx);
}

}  // namespace small
