// Single channel reduction with weights (paper Section 3.2 item 2; Table 1: F_C = 1, K = 1, G = I_C): depthwise
// convolution on the blocked layout.  The channel block is the vector dimension (G_b = C_b, Section 4.2.1): one
// thread owns four adjacent channels (a 128-bit lane) of an output pixel, so a warp reads whole 128-byte lines.
#include "common.cuh"

namespace small {

struct DwArgs {
    const float *in; const float *w; const float *bias; float *out;
    int H, W, FH, FW, S, pt, pl, OH, OW, C, CB;
    long long planes;
    bool relu;
};

__device__ __forceinline__ void fma4(float4 &a, const float4 &v, const float4 &w) {
    a.x = fmaf(v.x, w.x, a.x); a.y = fmaf(v.y, w.y, a.y); a.z = fmaf(v.z, w.z, a.z); a.w = fmaf(v.w, w.w, a.w);
}

// Generic window / stride: one output pixel x four channels per thread.
__global__ void __launch_bounds__(256) dwconv_generic_kernel(DwArgs a) {
    const long long total = a.planes * a.OH * a.OW * 8;
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
        int q = (int)(t & 7);
        long long pix = t >> 3;
        int ow = (int)(pix % a.OW);
        long long r = pix / a.OW;
        int oh = (int)(r % a.OH);
        long long plane = r / a.OH;
        int cb = (int)(plane % a.CB);
        const float4 *src = reinterpret_cast<const float4 *>(a.in + plane * a.H * a.W * 32) + q;
        const float4 *wt = reinterpret_cast<const float4 *>(a.w + (size_t)cb * a.FH * a.FW * 32) + q;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        int cbase = cb * 32 + q * 4;
        if (a.bias) {   // bias has exactly C entries
            if (cbase + 0 < a.C) acc.x = a.bias[cbase + 0];
            if (cbase + 1 < a.C) acc.y = a.bias[cbase + 1];
            if (cbase + 2 < a.C) acc.z = a.bias[cbase + 2];
            if (cbase + 3 < a.C) acc.w = a.bias[cbase + 3];
        }
        int h0 = oh * a.S - a.pt, w0 = ow * a.S - a.pl;
        for (int x = 0; x < a.FH; ++x) {
            int h = h0 + x;
            if (h < 0 || h >= a.H) continue;
            for (int y = 0; y < a.FW; ++y) {
                int w = w0 + y;
                if (w < 0 || w >= a.W) continue;
                fma4(acc, src[(h * a.W + w) * 8], __ldg(wt + (x * a.FW + y) * 8));
            }
        }
        if (a.relu) {
            acc.x = acc.x > 0.f ? acc.x : 0.f; acc.y = acc.y > 0.f ? acc.y : 0.f;
            acc.z = acc.z > 0.f ? acc.z : 0.f; acc.w = acc.w > 0.f ? acc.w : 0.f;
        }
        reinterpret_cast<float4 *>(a.out)[t] = acc;
    }
}

int launch_dwconv(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, const Geom &g, bool relu, cudaStream_t st) {
    DwArgs a{in, w, bias, out, g.H, g.W, g.FH, g.FW, g.S, g.pt, g.pl, g.OH, g.OW, g.C, g.CB, (long long)g.N * g.CB, relu};
    long long total = a.planes * g.OH * g.OW * 8;
    long long want = (total + 255) / 256, cap = (long long)ctx->sm_count * 32;
    int grid = (int)(want < cap ? want : cap);
    dwconv_generic_kernel<<<grid, 256, 0, st>>>(a);
    return check_launch(ctx);
}

}  // namespace small
