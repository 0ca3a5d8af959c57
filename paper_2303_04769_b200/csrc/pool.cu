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
    grid_dep_sync();
    grid_dep_trigger();
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

// 2x2 window, stride 2, no padding, no indices (the pooling of the workloads): every input line is read exactly once,
// so this is a pure stream.  Two output pixels per thread = eight independent 128-bit loads in flight.
__global__ void __launch_bounds__(256) maxpool2x2_kernel(const float4 *__restrict__ in, float4 *__restrict__ out, long long planes,
                                                         int H, int W, int OH, int OW, int C, int CB) {
    grid_dep_sync();
    grid_dep_trigger();
    const long long total = planes * OH * OW * 8, stride = (long long)gridDim.x * blockDim.x;
    for (long long t0 = blockIdx.x * (long long)blockDim.x + threadIdx.x; t0 < total; t0 += 2 * stride) {
        float4 v[2][4];
        bool ok[2];
        int cbase[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const long long t = t0 + u * stride;
            ok[u] = t < total;
            if (ok[u]) {
                const int q = (int)(t & 7);
                const long long p = t >> 3;
                const int ow = (int)(p % OW);
                const long long r = p / OW;
                const int oh = (int)(r % OH);
                const long long plane = r / OH;
                cbase[u] = (int)(plane % CB) * 32 + q * 4;
                const float4 *s = in + ((plane * H + oh * 2) * W + ow * 2) * 8 + q;
                v[u][0] = __ldcs(s); v[u][1] = __ldcs(s + 8); v[u][2] = __ldcs(s + W * 8); v[u][3] = __ldcs(s + W * 8 + 8);
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (ok[u]) {
                float4 m = v[u][0];          // row-major scan, strictly greater replaces: the first maximum wins
#pragma unroll
                for (int k = 1; k < 4; ++k) {
                    m.x = v[u][k].x > m.x ? v[u][k].x : m.x; m.y = v[u][k].y > m.y ? v[u][k].y : m.y;
                    m.z = v[u][k].z > m.z ? v[u][k].z : m.z; m.w = v[u][k].w > m.w ? v[u][k].w : m.w;
                }
                if (cbase[u] + 3 >= C) {     // pad lanes stay +0
                    if (cbase[u] + 0 >= C) m.x = 0.f;
                    if (cbase[u] + 1 >= C) m.y = 0.f;
                    if (cbase[u] + 2 >= C) m.z = 0.f;
                    if (cbase[u] + 3 >= C) m.w = 0.f;
                }
                __stcs(out + t0 + u * stride, m);
            }
        }
    }
}

// Large windows (global pooling): one warp per (plane, output pixel).  Lane = (4-channel group q, one of four subsets
// of the window positions), so 32 independent loads are in flight per step instead of one thread walking the whole
// window; the four subsets are combined by shuffles.  Sums and maxima do not depend on the order of combination
// beyond rounding (average) or not at all (maximum), and indices are not produced here.
template <bool MAX>
__global__ void __launch_bounds__(256) pool_window_kernel(PoolArgs a) {
    grid_dep_sync();
    grid_dep_trigger();
    const int lane = threadIdx.x & 31, q = lane & 7, sub = lane >> 3;
    const long long warps = a.planes * a.OH * a.OW;
    for (long long wid = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5; wid < warps; wid += ((long long)gridDim.x * blockDim.x) >> 5) {
        const int ow = (int)(wid % a.OW);
        const long long r = wid / a.OW;
        const int oh = (int)(r % a.OH);
        const long long plane = r / a.OH;
        const float4 *src = reinterpret_cast<const float4 *>(a.in + plane * a.H * a.W * 32) + q;
        const int h0 = oh * a.S - a.pt, w0 = ow * a.S - a.pl;
        const int hs = h0 < 0 ? 0 : h0, he = h0 + a.FH > a.H ? a.H : h0 + a.FH;
        const int ws = w0 < 0 ? 0 : w0, we = w0 + a.FW > a.W ? a.W : w0 + a.FW;
        const int ww = we - ws, cnt = (he - hs) * ww;
        float4 acc = MAX ? src[(hs * a.W + ws) * 8] : make_float4(0.f, 0.f, 0.f, 0.f);
        for (int i = sub; i < cnt; i += 4) {
            const int h = hs + i / ww, w = ws + i % ww;
            const float4 v = src[(h * a.W + w) * 8];
            if (MAX) { acc.x = fmaxf(acc.x, v.x); acc.y = fmaxf(acc.y, v.y); acc.z = fmaxf(acc.z, v.z); acc.w = fmaxf(acc.w, v.w); }
            else { acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w; }
        }
#pragma unroll
        for (int d = 8; d < 32; d <<= 1) {
            float4 o;
            o.x = __shfl_xor_sync(0xffffffffu, acc.x, d); o.y = __shfl_xor_sync(0xffffffffu, acc.y, d);
            o.z = __shfl_xor_sync(0xffffffffu, acc.z, d); o.w = __shfl_xor_sync(0xffffffffu, acc.w, d);
            if (MAX) { acc.x = fmaxf(acc.x, o.x); acc.y = fmaxf(acc.y, o.y); acc.z = fmaxf(acc.z, o.z); acc.w = fmaxf(acc.w, o.w); }
            else { acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w; }
        }
        if (sub == 0) {
            if (!MAX) { const float c = (float)cnt; acc.x /= c; acc.y /= c; acc.z /= c; acc.w /= c; }
            const int cbase = (int)(plane % a.CB) * 32 + q * 4;   // pad lanes stay +0
            if (cbase + 0 >= a.C) acc.x = 0.f;
            if (cbase + 1 >= a.C) acc.y = 0.f;
            if (cbase + 2 >= a.C) acc.z = 0.f;
            if (cbase + 3 >= a.C) acc.w = 0.f;
            reinterpret_cast<float4 *>(a.out)[wid * 8 + q] = acc;
        }
    }
}

int launch_pool(small_ctx *ctx, const float *in, float *out, int32_t *idx, const Geom &g, int mode, cudaStream_t st) {
    PoolArgs a{in, out, idx, g.H, g.W, g.FH, g.FW, g.S, g.pt, g.pl, g.OH, g.OW, (long long)g.N * g.CB, g.C, g.CB};
    long long total = a.planes * g.OH * g.OW * 8;
    long long want = (total + 255) / 256, cap = (long long)ctx->sm_count * 32;
    int grid = (int)(want < cap ? want : cap);
    if (mode == SMALL_POOL_MAX && !idx && g.FH == 2 && g.FW == 2 && g.S == 2 && !(g.pt | g.pb | g.pl | g.pr)) {
        long long w2 = (total + 511) / 512, cap2 = (long long)ctx->sm_count * 8;
        launch_kernel(ctx, maxpool2x2_kernel, dim3((unsigned)((int)(w2 < cap2 ? w2 : cap2))), dim3(256), 0, st, reinterpret_cast<const float4 *>(in), reinterpret_cast<float4 *>(out),
                                                                     a.planes, g.H, g.W, g.OH, g.OW, g.C, g.CB);
        return check_launch(ctx);
    }
    if (!idx && g.FH * g.FW >= 16) {
        const long long warps = a.planes * g.OH * g.OW;
        long long wb = (warps + 7) / 8, capb = (long long)ctx->sm_count * 16;
        const int gridb = (int)(wb < capb ? wb : capb);
        if (mode == SMALL_POOL_MAX) launch_kernel(ctx, pool_window_kernel<true>, dim3((unsigned)(gridb)), dim3(256), 0, st, a);
        else launch_kernel(ctx, pool_window_kernel<false>, dim3((unsigned)(gridb)), dim3(256), 0, st, a);
        return check_launch(ctx);
    }
    if (mode == SMALL_POOL_MAX) {
        if (idx) launch_kernel(ctx, pool_kernel<true, true>, dim3((unsigned)(grid)), dim3(256), 0, st, a);
        else launch_kernel(ctx, pool_kernel<true, false>, dim3((unsigned)(grid)), dim3(256), 0, st, a);
    } else {
        launch_kernel(ctx, pool_kernel<false, false>, dim3((unsigned)(grid)), dim3(256), 0, st, a);
    }
    return check_launch(ctx);
}

}  // namespace small
