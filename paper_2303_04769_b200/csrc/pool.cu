// Single channel reductions without weights (paper Section 3.2 item 2): max and average pooling on the blocked
// layout.  One thread owns four adjacent channels of one output pixel (a 128-bit lane of the 32-channel line),
// so a warp reads and writes four whole 128-byte lines per window position.
#include "common.cuh"

namespace small {

struct PoolArgs {
    const float *in; float *out; int32_t *idx;
    int H, W, FH, FW, S, pt, pl, OH, OW;
    long long planes;   // N * channel blocks
    int C, CB;
};

template <bool MAX, bool IDX>
__global__ void __launch_bounds__(256) pool_kernel(PoolArgs a) {
    const long long total = a.planes * a.OH * a.OW * 8;
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
        int q = (int)(t & 7);
        long long pix = t >> 3;
        int ow = (int)(pix % a.OW);
        long long r = pix / a.OW;
        int oh = (int)(r % a.OH);
        long long plane = r / a.OH;
        const float4 *src = reinterpret_cast<const float4 *>(a.in + plane * a.H * a.W * 32) + q;
        int h0 = oh * a.S - a.pt, w0 = ow * a.S - a.pl;
        int hs = h0 < 0 ? 0 : h0, he = h0 + a.FH > a.H ? a.H : h0 + a.FH;
        int ws = w0 < 0 ? 0 : w0, we = w0 + a.FW > a.W ? a.W : w0 + a.FW;
        float4 acc;
        int4 bi = make_int4(0, 0, 0, 0);
        if (MAX) {
            // the first in-range element starts the scan; later ones replace it only when strictly greater
            int first = hs * a.W + ws;
            acc = src[first * 8];
            bi = make_int4(first, first, first, first);
            for (int h = hs; h < he; ++h)
                for (int w = ws; w < we; ++w) {
                    int p = h * a.W + w;
                    float4 v = src[p * 8];
                    if (v.x > acc.x) { acc.x = v.x; bi.x = p; }
                    if (v.y > acc.y) { acc.y = v.y; bi.y = p; }
                    if (v.z > acc.z) { acc.z = v.z; bi.z = p; }
                    if (v.w > acc.w) { acc.w = v.w; bi.w = p; }
                }
        } else {
            acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int h = hs; h < he; ++h)
                for (int w = ws; w < we; ++w) {
                    float4 v = src[(h * a.W + w) * 8];
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
            float cnt = (float)((he - hs) * (we - ws));
            acc.x /= cnt; acc.y /= cnt; acc.z /= cnt; acc.w /= cnt;
        }
        // pad lanes of the last channel block stay +0 (index 0)
        int cbase = (int)(plane % a.CB) * 32 + q * 4;
        if (cbase + 3 >= a.C) {
            if (cbase + 0 >= a.C) { acc.x = 0.f; bi.x = 0; }
            if (cbase + 1 >= a.C) { acc.y = 0.f; bi.y = 0; }
            if (cbase + 2 >= a.C) { acc.z = 0.f; bi.z = 0; }
            if (cbase + 3 >= a.C) { acc.w = 0.f; bi.w = 0; }
        }
        reinterpret_cast<float4 *>(a.out)[t] = acc;
        if (IDX) reinterpret_cast<int4 *>(a.idx)[t] = bi;
    }
}

int launch_pool(small_ctx *ctx, const float *in, float *out, int32_t *idx, const Geom &g, int mode, cudaStream_t st) {
    PoolArgs a{in, out, idx, g.H, g.W, g.FH, g.FW, g.S, g.pt, g.pl, g.OH, g.OW, (long long)g.N * g.CB, g.C, g.CB};
    long long total = a.planes * g.OH * g.OW * 8;
    long long want = (total + 255) / 256, cap = (long long)ctx->sm_count * 32;
    int grid = (int)(want < cap ? want : cap);
    if (mode == SMALL_POOL_MAX) {
        if (idx) pool_kernel<true, true><<<grid, 256, 0, st>>>(a);
        else pool_kernel<true, false><<<grid, 256, 0, st>>>(a);
    } else {
        pool_kernel<false, false><<<grid, 256, 0, st>>>(a);
    }
    return check_launch(ctx);
}

}  // namespace small
