// Quantised inference (paper Sections 5.1 and 5.5: uint8 tensors; Section 5.3: int32 accumulation) over the same
// blocked layout with one byte per channel: uint8[N][ceil(C/32)][H][W][32], a pixel of a channel block = 32 bytes = 8
// words of 4 channels; pad lanes hold 0.  This file: the layout moves, the filter packing, the bandwidth-bound layers
// (depthwise, max pool, ReLU) and the C ABI of the quantised layers; the full channel reduction runs the quantised
// form of the register-tiled kernel (conv_direct.cu).  Arithmetic: acc = bias + sum (q_in - z_in)(q_w - z_w) in int32,
// q_out = clamp(z_out + floor((acc * mult + 2^(shift-1)) / 2^shift), lo, 255) with a 64-bit product, lo = z_out under
// ReLU.  Max pooling and ReLU act on the bytes themselves (the affine map keeps order).
#include "common.cuh"

namespace small {

namespace {

__device__ __forceinline__ int requantize(int acc, int mult, int shift, int zo, int lo) {
    const long long r = ((long long)acc * (long long)mult + (1ll << (shift - 1))) >> shift;
    const long long z = (long long)zo + r;
    return (int)(z < lo ? lo : z > 255 ? 255 : z);
}

// one thread = one word (4 channels) of one pixel of the blocked tensor
__global__ void q_pack_kernel(const uint8_t *__restrict__ nchw, uint32_t *__restrict__ blk, int C, int HW, int CB, size_t words) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < words; i += (size_t)gridDim.x * blockDim.x) {
        const int c4 = (int)(i & 7);
        size_t r = i >> 3;
        const int p = (int)(r % HW); r /= HW;
        const int cb = (int)(r % CB);
        const size_t n = r / CB;
        uint32_t word = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int c = cb * 32 + c4 * 4 + b;
            if (c < C) word |= (uint32_t)nchw[(n * C + c) * HW + p] << (8 * b);
        }
        blk[i] = word;
    }
}

__global__ void q_unpack_kernel(const uint32_t *__restrict__ blk, uint8_t *__restrict__ nchw, int C, int HW, int CB, size_t words) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < words; i += (size_t)gridDim.x * blockDim.x) {
        const int c4 = (int)(i & 7);
        size_t r = i >> 3;
        const int p = (int)(r % HW); r /= HW;
        const int cb = (int)(r % CB);
        const size_t n = r / CB;
        const uint32_t word = blk[i];
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int c = cb * 32 + c4 * 4 + b;
            if (c < C) nchw[(n * C + c) * HW + p] = (uint8_t)(word >> (8 * b));
        }
    }
}

// filters [K][C][FH][FW] bytes -> words [KB][CB][T][8 c4][32 ko], a word = 4 consecutive channels of one filter and tap
__global__ void pack_q_conv_w_kernel(const uint8_t *__restrict__ w, uint32_t *__restrict__ wb, int C, int K, int T, size_t words) {
    const int CB = (C + 31) / 32;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < words; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i;
        const int ko = (int)(r & 31); r >>= 5;
        const int c4 = (int)(r & 7); r >>= 3;
        const int t = (int)(r % T); r /= T;
        const int cb = (int)(r % CB);
        const int kb = (int)(r / CB);
        const int k = kb * 32 + ko;
        uint32_t word = 0;
        if (k < K)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int c = cb * 32 + c4 * 4 + b;
                if (c < C) word |= (uint32_t)w[((size_t)k * C + c) * T + t] << (8 * b);
            }
        wb[i] = word;
    }
}

// per filter and tap the sum of the weight bytes over the channels [K][T], then per filter over everything [K]
__global__ void q_conv_tables_kernel(const uint8_t *__restrict__ w, int *__restrict__ tab, int C, int K, int T) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < K * T) {
        const int k = i / T, t = i - k * T;
        int s = 0;
        for (int c = 0; c < C; ++c) s += w[((size_t)k * C + c) * T + t];
        tab[i] = s;
    } else if (i < K * T + K) {
        const int k = i - K * T;
        int s = 0;
        for (int j = 0; j < C * T; ++j) s += w[(size_t)k * C * T + j];
        tab[i] = s;
    }
}

// depthwise filters [C][FH][FW] bytes -> [CB][T][32] bytes, pad lanes 0
__global__ void pack_q_dw_w_kernel(const uint8_t *__restrict__ w, uint8_t *__restrict__ wb, int C, int T, int total) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int lane = i & 31, t = (i >> 5) % T, cb = (i >> 5) / T;
    const int c = cb * 32 + lane;
    wb[i] = c < C ? w[(size_t)c * T + t] : (uint8_t)0;
}

struct QPlaneArgs {
    const uint32_t *in; uint32_t *out; const uint32_t *w; const int *bias;
    int N, C, CB, H, W, FH, FW, S, pt, pl, OH, OW;
    int zx, zw, zo, mult, shift, lo;
};

// one thread = 4 channels of one output pixel; any window, stride and padding
__global__ void q_dwconv_kernel(const QPlaneArgs a) {
    const size_t words = (size_t)a.N * a.CB * a.OH * a.OW * 8;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < words; i += (size_t)gridDim.x * blockDim.x) {
        const int c4 = (int)(i & 7);
        size_t r = i >> 3;
        const int ow = (int)(r % a.OW); r /= a.OW;
        const int oh = (int)(r % a.OH); r /= a.OH;
        const int cb = (int)(r % a.CB);
        const size_t n = r / a.CB;
        const uint32_t *plane = a.in + ((n * a.CB + cb) * a.H * a.W) * 8 + c4;
        int acc[4] = {0, 0, 0, 0};
        for (int x = 0; x < a.FH; ++x) {
            const int ih = oh * a.S + x - a.pt;
            if (ih < 0 || ih >= a.H) continue;
            for (int y = 0; y < a.FW; ++y) {
                const int iw = ow * a.S + y - a.pl;
                if (iw < 0 || iw >= a.W) continue;
                const uint32_t xv = plane[((size_t)ih * a.W + iw) * 8];
                const uint32_t wv = a.w[((size_t)cb * a.FH * a.FW + x * a.FW + y) * 8 + c4];
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    acc[b] += ((int)((xv >> (8 * b)) & 255u) - a.zx) * ((int)((wv >> (8 * b)) & 255u) - a.zw);
            }
        }
        uint32_t word = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int c = cb * 32 + c4 * 4 + b;
            if (c < a.C) word |= (uint32_t)requantize(acc[b] + (a.bias ? a.bias[c] : 0), a.mult, a.shift, a.zo, a.lo) << (8 * b);
        }
        a.out[i] = word;
    }
}

__device__ __forceinline__ uint32_t lane_mask(int C, int cb, int c4) {      // 0xff in the bytes of real channels
    uint32_t m = 0;
#pragma unroll
    for (int b = 0; b < 4; ++b)
        if (cb * 32 + c4 * 4 + b < C) m |= 0xffu << (8 * b);
    return m;
}

__global__ void q_maxpool_kernel(const QPlaneArgs a) {
    const size_t words = (size_t)a.N * a.CB * a.OH * a.OW * 8;
    const uint32_t z4 = (uint32_t)a.zx * 0x01010101u;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < words; i += (size_t)gridDim.x * blockDim.x) {
        const int c4 = (int)(i & 7);
        size_t r = i >> 3;
        const int ow = (int)(r % a.OW); r /= a.OW;
        const int oh = (int)(r % a.OH); r /= a.OH;
        const int cb = (int)(r % a.CB);
        const size_t n = r / a.CB;
        const uint32_t *plane = a.in + ((n * a.CB + cb) * a.H * a.W) * 8 + c4;
        uint32_t best = 0;
        bool any = false;
        for (int x = 0; x < a.FH; ++x) {
            const int ih = oh * a.S + x - a.pt;
            if (ih < 0 || ih >= a.H) continue;
            for (int y = 0; y < a.FW; ++y) {
                const int iw = ow * a.S + y - a.pl;
                if (iw < 0 || iw >= a.W) continue;
                best = __vmaxu4(best, plane[((size_t)ih * a.W + iw) * 8]);
                any = true;
            }
        }
        a.out[i] = (any ? best : z4) & lane_mask(a.C, cb, c4);
    }
}

__global__ void q_relu_kernel(const uint32_t *__restrict__ in, uint32_t *__restrict__ out, int C, int CB, int HW, int z, size_t words) {
    const uint32_t z4 = (uint32_t)z * 0x01010101u;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < words; i += (size_t)gridDim.x * blockDim.x) {
        const int c4 = (int)(i & 7);
        const int cb = (int)((i >> 3) / HW % CB);
        out[i] = __vmaxu4(in[i], z4) & lane_mask(C, cb, c4);
    }
}

int grid_for(small_ctx *ctx, size_t items) {
    const size_t want = (items + 255) / 256, cap = (size_t)ctx->sm_count * 16;
    return (int)(want < cap ? (want ? want : 1) : cap);
}

bool qparams_ok(int zx, int zw, int zo, int mult, int shift) {
    return zx >= 0 && zx <= 255 && zw >= 0 && zw <= 255 && zo >= 0 && zo <= 255 && mult >= 0 && shift >= 1 && shift <= 62;
}

size_t q_conv_words(int C, int K, int FH, int FW) { return (size_t)blocks_of(K) * blocks_of(C) * FH * FW * 8 * 32; }

}  // namespace

bool q_conv_supported(const Geom &g);
int launch_q_conv(small_ctx *ctx, const uint8_t *in, const uint32_t *w_words, const int *tables, const int *bias, uint8_t *out,
                  const Geom &g, bool relu, int zx, int zw, int zo, int mult, int shift, cudaStream_t st);

}  // namespace small

using namespace small;

SMALL_API size_t small_q_packed_bytes(int N, int C, int H, int W) { return packed_elems(N, C, H, W); }

SMALL_API int small_q_pack(small_ctx *ctx, const uint8_t *nchw, uint8_t *blk, int N, int C, int H, int W, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!nchw || !blk) return SMALL_ERR_INVALID_ARG;
    if (!aligned16(blk)) return SMALL_ERR_ALIGN;
    if (N < 1 || C < 1 || H < 1 || W < 1 || (long long)H * W > (1ll << 24)) return SMALL_ERR_SHAPE;
    const size_t words = packed_elems(N, C, H, W) / 4;
    if (ranges_overlap(nchw, (size_t)N * C * H * W, blk, words * 4)) return SMALL_ERR_OVERLAP;
    q_pack_kernel<<<grid_for(ctx, words), 256, 0, static_cast<cudaStream_t>(stream)>>>(nchw, reinterpret_cast<uint32_t *>(blk), C, H * W, blocks_of(C), words);
    return check_launch(ctx);
}

SMALL_API int small_q_unpack(small_ctx *ctx, const uint8_t *blk, uint8_t *nchw, int N, int C, int H, int W, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!nchw || !blk) return SMALL_ERR_INVALID_ARG;
    if (!aligned16(blk)) return SMALL_ERR_ALIGN;
    if (N < 1 || C < 1 || H < 1 || W < 1 || (long long)H * W > (1ll << 24)) return SMALL_ERR_SHAPE;
    const size_t words = packed_elems(N, C, H, W) / 4;
    if (ranges_overlap(nchw, (size_t)N * C * H * W, blk, words * 4)) return SMALL_ERR_OVERLAP;
    q_unpack_kernel<<<grid_for(ctx, words), 256, 0, static_cast<cudaStream_t>(stream)>>>(reinterpret_cast<const uint32_t *>(blk), nchw, C, H * W, blocks_of(C), words);
    return check_launch(ctx);
}

SMALL_API size_t small_q_conv_weight_bytes(int C, int K, int FH, int FW) {
    if (C < 1 || K < 1 || FH < 1 || FW < 1) return 0;
    return q_conv_words(C, K, FH, FW) * 4 + ((size_t)K * FH * FW + K) * sizeof(int);
}

SMALL_API int small_q_pack_conv_weights(small_ctx *ctx, const uint8_t *w, void *wb, int C, int K, int FH, int FW, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!w || !wb) return SMALL_ERR_INVALID_ARG;
    if (!aligned16(wb)) return SMALL_ERR_ALIGN;
    if (C < 1 || K < 1 || FH < 1 || FW < 1 || (long long)K * FH * FW > (1ll << 28)) return SMALL_ERR_SHAPE;
    if (ranges_overlap(w, (size_t)K * C * FH * FW, wb, small_q_conv_weight_bytes(C, K, FH, FW))) return SMALL_ERR_OVERLAP;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t words = q_conv_words(C, K, FH, FW);
    const int T = FH * FW;
    pack_q_conv_w_kernel<<<grid_for(ctx, words), 256, 0, st>>>(w, static_cast<uint32_t *>(wb), C, K, T, words);
    q_conv_tables_kernel<<<(K * T + K + 127) / 128, 128, 0, st>>>(w, reinterpret_cast<int *>(static_cast<uint32_t *>(wb) + words), C, K, T);
    return check_launch(ctx);
}

SMALL_API int small_q_conv2d(small_ctx *ctx, const uint8_t *in, const void *w_blk, const int32_t *bias, uint8_t *out,
                             int N, int C, int K, int H, int W, int FH, int FW, int stride, int pt, int pb, int pl, int pr,
                             int z_in, int z_w, int z_out, int mult, int shift, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~SMALL_RELU) return SMALL_ERR_INVALID_ARG;
    if (!in || !w_blk || !out || !qparams_ok(z_in, z_w, z_out, mult, shift)) return SMALL_ERR_INVALID_ARG;
    if (!aligned16(in) || !aligned16(w_blk) || !aligned16(out) || (bias && (reinterpret_cast<uintptr_t>(bias) & 3u))) return SMALL_ERR_ALIGN;
    Geom g;
    if (int s = make_geom(g, N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr)) return s;
    if ((long long)C * FH * FW > 33000) return SMALL_ERR_SHAPE;      // the raw sums of byte products must stay inside 32 bits
    if (ranges_overlap(in, packed_elems(N, C, H, W), out, packed_elems(N, K, g.OH, g.OW))) return SMALL_ERR_OVERLAP;
    if (!q_conv_supported(g)) return SMALL_ERR_UNSUPPORTED;
    const uint32_t *words = static_cast<const uint32_t *>(w_blk);
    const int *tables = reinterpret_cast<const int *>(words + q_conv_words(C, K, FH, FW));
    return launch_q_conv(ctx, in, words, tables, bias, out, g, flags & SMALL_RELU, z_in, z_w, z_out, mult, shift, static_cast<cudaStream_t>(stream));
}

SMALL_API size_t small_q_dw_weight_bytes(int C, int FH, int FW) {
    if (C < 1 || FH < 1 || FW < 1) return 0;
    return (size_t)blocks_of(C) * FH * FW * 32;
}

SMALL_API int small_q_pack_dw_weights(small_ctx *ctx, const uint8_t *w, uint8_t *wb, int C, int FH, int FW, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!w || !wb) return SMALL_ERR_INVALID_ARG;
    if (!aligned16(wb)) return SMALL_ERR_ALIGN;
    if (C < 1 || FH < 1 || FW < 1 || (long long)blocks_of(C) * FH * FW * 32 > (1ll << 30)) return SMALL_ERR_SHAPE;
    const int total = (int)small_q_dw_weight_bytes(C, FH, FW);
    if (ranges_overlap(w, (size_t)C * FH * FW, wb, total)) return SMALL_ERR_OVERLAP;
    pack_q_dw_w_kernel<<<(total + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(w, wb, C, FH * FW, total);
    return check_launch(ctx);
}

SMALL_API int small_q_dwconv2d(small_ctx *ctx, const uint8_t *in, const uint8_t *w_blk, const int32_t *bias, uint8_t *out,
                               int N, int C, int H, int W, int FH, int FW, int stride, int pt, int pb, int pl, int pr,
                               int z_in, int z_w, int z_out, int mult, int shift, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~SMALL_RELU) return SMALL_ERR_INVALID_ARG;
    if (!in || !w_blk || !out || !qparams_ok(z_in, z_w, z_out, mult, shift)) return SMALL_ERR_INVALID_ARG;
    if (!aligned16(in) || !aligned16(w_blk) || !aligned16(out) || (bias && (reinterpret_cast<uintptr_t>(bias) & 3u))) return SMALL_ERR_ALIGN;
    Geom g;
    if (int s = make_geom(g, N, C, C, H, W, FH, FW, stride, pt, pb, pl, pr)) return s;
    if ((long long)FH * FW > 33000) return SMALL_ERR_SHAPE;
    if (ranges_overlap(in, packed_elems(N, C, H, W), out, packed_elems(N, C, g.OH, g.OW))) return SMALL_ERR_OVERLAP;
    QPlaneArgs a{reinterpret_cast<const uint32_t *>(in), reinterpret_cast<uint32_t *>(out), reinterpret_cast<const uint32_t *>(w_blk), bias,
                 N, C, g.CB, H, W, FH, FW, stride, pt, pl, g.OH, g.OW, z_in, z_w, z_out, mult, shift, (flags & SMALL_RELU) ? z_out : 0};
    q_dwconv_kernel<<<grid_for(ctx, packed_elems(N, C, g.OH, g.OW) / 4), 256, 0, static_cast<cudaStream_t>(stream)>>>(a);
    return check_launch(ctx);
}

SMALL_API int small_q_maxpool2d(small_ctx *ctx, const uint8_t *in, uint8_t *out, int N, int C, int H, int W, int FH, int FW,
                                int stride, int pt, int pb, int pl, int pr, int z, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!in || !out || z < 0 || z > 255) return SMALL_ERR_INVALID_ARG;
    if (!aligned16(in) || !aligned16(out)) return SMALL_ERR_ALIGN;
    Geom g;
    if (int s = make_geom(g, N, C, C, H, W, FH, FW, stride, pt, pb, pl, pr)) return s;
    if (ranges_overlap(in, packed_elems(N, C, H, W), out, packed_elems(N, C, g.OH, g.OW))) return SMALL_ERR_OVERLAP;
    QPlaneArgs a{reinterpret_cast<const uint32_t *>(in), reinterpret_cast<uint32_t *>(out), nullptr, nullptr,
                 N, C, g.CB, H, W, FH, FW, stride, pt, pl, g.OH, g.OW, z, 0, 0, 0, 1, 0};
    q_maxpool_kernel<<<grid_for(ctx, packed_elems(N, C, g.OH, g.OW) / 4), 256, 0, static_cast<cudaStream_t>(stream)>>>(a);
    return check_launch(ctx);
}

SMALL_API int small_q_relu(small_ctx *ctx, const uint8_t *in, uint8_t *out, int N, int C, int H, int W, int z, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!in || !out || z < 0 || z > 255) return SMALL_ERR_INVALID_ARG;
    if (!aligned16(in) || !aligned16(out)) return SMALL_ERR_ALIGN;
    const size_t bytes = packed_elems(N, C, H, W);
    if (bytes == 0) return SMALL_ERR_SHAPE;
    if (in != out && ranges_overlap(in, bytes, out, bytes)) return SMALL_ERR_OVERLAP;
    q_relu_kernel<<<grid_for(ctx, bytes / 4), 256, 0, static_cast<cudaStream_t>(stream)>>>(reinterpret_cast<const uint32_t *>(in), reinterpret_cast<uint32_t *>(out),
                                                                                         C, blocks_of(C), H * W, z, bytes / 4);
    return check_launch(ctx);
}
