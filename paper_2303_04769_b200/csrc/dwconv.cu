// Single channel reduction with weights (paper Section 3.2 item 2; Table 1: F_C = 1, K = 1, G = I_C): depthwise
// convolution on the blocked layout.  The channel block is the vector dimension (G_b = C_b, Section 4.2.1): one
// thread owns four adjacent channels (a 128-bit lane), so a warp reads whole 128-byte lines.  The 3x3 kernel stages
// halo tiles in shared memory with TMA (whole tiles in flight per SM, padding supplied by the out-of-range zero fill,
// double buffered) and each thread walks down a column of output pixels with the 3x3 window held in registers (the
// paper's O_wb register tile turned by 90 degrees): one new row of three pixels per output instead of nine, and
// every input line leaves HBM once.  Other window shapes use the generic kernel (one output pixel per thread).
#include "common.cuh"
#include "sm100.cuh"

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

// 3x3 window, stride ST (1 or 2).  Tile = nn images x one channel block x a strip of TR output rows; its input box
// (nn x Hb x Wb pixels of 128 bytes) arrives by TMA.  Thread = (image, output column, 4-channel lane group).
struct Dw3Args {
    const float *w; const float *bias; float *out; int *status;
    int N, C, CB, OH, OW, pt, pl;
    int nn, TR, Hb, Wb, strips, groups;    // groups = ceil(N / nn)
    int segs, rps;                         // a column's TR rows are walked by `segs` threads, `rps` rows each
    long long tiles;
    uint32_t stage_bytes;
    uint32_t wait_iters;                   // limit of the bounded waits (polls)
    bool relu;
};

template <int ST>
__global__ void __launch_bounds__(256) dwconv3x3_tma_kernel(const __grid_constant__ CUtensorMap map_in, const Dw3Args a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (sm100::smem_u32(smem_raw) + 127u) & ~127u;
    const float4 *stage_ptr[2];
    stage_ptr[0] = reinterpret_cast<const float4 *>(smem_raw + (base - sm100::smem_u32(smem_raw)));
    stage_ptr[1] = reinterpret_cast<const float4 *>(smem_raw + (base - sm100::smem_u32(smem_raw)) + a.stage_bytes);
    __shared__ __align__(8) unsigned long long bars[2];
    __shared__ int failed;
    const uint32_t bar0 = sm100::smem_u32(&bars[0]);

    auto issue = [&](long long t, int s) {       // one elected thread: arm the barrier and start the tile's copy
        const int strip = (int)(t % a.strips);
        const long long r = t / a.strips;
        const int cb = (int)(r % a.CB);
        const int grp = (int)(r / a.CB);
        sm100::mbar_expect_tx(bar0 + 8 * s, a.stage_bytes);
        sm100::tma_load_5d(base + s * a.stage_bytes, &map_in, bar0 + 8 * s, 0, -a.pl, strip * a.TR * ST - a.pt, cb, grp * a.nn);
    };
    if (threadIdx.x == 0) {
        sm100::mbar_init(bar0, 1);
        sm100::mbar_init(bar0 + 8, 1);
        sm100::mbar_fence_init();
        failed = 0;
    }
    __syncthreads();
    grid_dep_sync();
    grid_dep_trigger();
    const long long first = blockIdx.x, stride = gridDim.x;
    if (threadIdx.x == 0) {
        if (first < a.tiles) issue(first, 0);
        if (first + stride < a.tiles) issue(first + stride, 1);
    }
    const int q = threadIdx.x & 7;
    const int cols = a.nn * a.OW;                 // output columns of a tile (all images)
    uint32_t it = 0;
    for (long long t = first; t < a.tiles; t += stride, ++it) {
        const int s = it & 1;
        // one lane per warp polls, the rest wait at the shuffle
        int ok = 1;
        if ((threadIdx.x & 31) == 0) ok = sm100::mbar_wait(bar0 + 8 * s, (it >> 1) & 1, a.wait_iters) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) { failed = 1; atomicExch(a.status, (int)SMALL_ERR_TIMEOUT); }
        const int strip = (int)(t % a.strips);
        const long long r = t / a.strips;
        const int cb = (int)(r % a.CB);
        const int grp = (int)(r / a.CB);
        if (ok) {
            const float4 *tile = stage_ptr[s];
            const float4 *wt = reinterpret_cast<const float4 *>(a.w + (size_t)cb * 9 * 32) + q;
            float4 w[9];
#pragma unroll
            for (int i = 0; i < 9; ++i) w[i] = __ldg(wt + i * 8);
            float4 bias4 = make_float4(0.f, 0.f, 0.f, 0.f);
            const int cbase = cb * 32 + q * 4;
            if (a.bias) {   // bias has exactly C entries
                if (cbase + 0 < a.C) bias4.x = a.bias[cbase + 0];
                if (cbase + 1 < a.C) bias4.y = a.bias[cbase + 1];
                if (cbase + 2 < a.C) bias4.z = a.bias[cbase + 2];
                if (cbase + 3 < a.C) bias4.w = a.bias[cbase + 3];
            }
            const int oh0 = strip * a.TR, rows = min(a.TR, a.OH - oh0);
            // unit = (row segment, column): narrow tiles (few columns) split each column's rows over several threads so
            // that all 32 column slots of the block have work
            for (int u = threadIdx.x >> 3; u < cols * a.segs; u += 32) {
                const int seg = u / cols, c = u - seg * cols;
                const int img = c / a.OW, ow = c - img * a.OW;
                const int n = grp * a.nn + img;
                const int i0 = seg * a.rps, i1 = min(rows, i0 + a.rps);
                if (n >= a.N || i0 >= i1) continue;
                const float4 *col = tile + ((size_t)img * a.Hb * a.Wb + (size_t)i0 * ST * a.Wb + ow * ST) * 8 + q;     // window's top-left pixel
                float4 *dst = reinterpret_cast<float4 *>(a.out) + ((((size_t)n * a.CB + cb) * a.OH + oh0 + i0) * a.OW + ow) * 8 + q;
                float4 r0[3], r1[3], r2[3];
#pragma unroll
                for (int y = 0; y < 3; ++y) { r0[y] = col[y * 8]; r1[y] = col[(a.Wb + y) * 8]; }
                const float4 *next = col + 2 * a.Wb * 8;
                for (int i = i0; i < i1; ++i) {
#pragma unroll
                    for (int y = 0; y < 3; ++y) r2[y] = next[y * 8];
                    float4 acc = bias4;
#pragma unroll
                    for (int y = 0; y < 3; ++y) { fma4(acc, r0[y], w[y]); fma4(acc, r1[y], w[3 + y]); fma4(acc, r2[y], w[6 + y]); }
                    if (a.relu) {
                        acc.x = acc.x > 0.f ? acc.x : 0.f; acc.y = acc.y > 0.f ? acc.y : 0.f;
                        acc.z = acc.z > 0.f ? acc.z : 0.f; acc.w = acc.w > 0.f ? acc.w : 0.f;
                    }
                    __stcs(dst, acc);
                    dst += a.OW * 8;
                    if (ST == 1) {
#pragma unroll
                        for (int y = 0; y < 3; ++y) { r0[y] = r1[y]; r1[y] = r2[y]; }
                        next += a.Wb * 8;
                    } else {
#pragma unroll
                        for (int y = 0; y < 3; ++y) r0[y] = r2[y];
                        if (i + 1 < i1) {
#pragma unroll
                            for (int y = 0; y < 3; ++y) r1[y] = next[(a.Wb + y) * 8];
                        }
                        next += 2 * a.Wb * 8;
                    }
                }
            }
        }
        __syncthreads();                           // everyone is done with stage s
        if (threadIdx.x == 0 && !failed && t + 2 * stride < a.tiles) issue(t + 2 * stride, s);
        if (failed) break;
    }
    // after a timeout: give copies that may still be in flight a bounded grace period before the CTA exits
    if (failed && threadIdx.x == 0)
        for (uint32_t k = 0; k < (1u << 14); ++k) __nanosleep(200);
}

// Picks the tile of the TMA kernel; false if the shape does not fit (then the generic kernel runs).
static bool plan_dw3(const Geom &g, int sms, Dw3Args &a) {
    const int S = g.S;
    a.Wb = (g.OW - 1) * S + 3;
    if (a.Wb > 256) return false;
    const size_t row_bytes = (size_t)a.Wb * 128;
    const size_t budget = 48 * 1024;                              // per stage: two stages, two CTAs per SM
    const int hb_plane = (g.OH - 1) * S + 3;
    if ((size_t)hb_plane * row_bytes <= budget) {
        a.TR = g.OH; a.Hb = hb_plane; a.strips = 1;
        a.nn = (int)(budget / ((size_t)hb_plane * row_bytes));
        if (a.nn > g.N) a.nn = g.N;
        if (a.nn > 256) a.nn = 256;
        // keep at least a few tiles per SM so that the double buffer has something to overlap
        while (a.nn > 1 && (long long)ceil_div(g.N, a.nn) * g.CB < 4LL * sms) --a.nn;
    } else {
        a.nn = 1;
        int hb = (int)(budget / row_bytes);
        if (hb > 256) hb = 256;
        a.TR = (hb - 3) / S + 1;
        if (hb < 3 || a.TR < 1) return false;
        a.strips = ceil_div(g.OH, a.TR);
        a.TR = ceil_div(g.OH, a.strips);                          // balanced strips
        a.Hb = (a.TR - 1) * S + 3;
    }
    a.groups = ceil_div(g.N, a.nn);
    // 256 threads = 32 column slots x 8 lane groups; a tile with fewer columns splits its rows (at least 3 per thread)
    const int cols = a.nn * g.OW;
    a.segs = cols >= 32 ? 1 : 32 / cols;
    if (a.segs > a.TR / 3) a.segs = a.TR / 3 > 0 ? a.TR / 3 : 1;
    a.rps = ceil_div(a.TR, a.segs);
    a.segs = ceil_div(a.TR, a.rps);
    a.tiles = (long long)a.groups * g.CB * a.strips;
    a.stage_bytes = (uint32_t)((size_t)a.nn * a.Hb * row_bytes);
    return true;
}

int launch_dwconv(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, const Geom &g, bool relu, cudaStream_t st) {
    DwArgs a{in, w, bias, out, g.H, g.W, g.FH, g.FW, g.S, g.pt, g.pl, g.OH, g.OW, g.C, g.CB, (long long)g.N * g.CB, relu};
    Dw3Args t{};
    if (g.FH == 3 && g.FW == 3 && (g.S == 1 || g.S == 2) && plan_dw3(g, ctx->sm_count, t)) {
        t.w = w; t.bias = bias; t.out = out; t.status = ctx->dev_status; t.wait_iters = ctx->wait_iters;
        t.N = g.N; t.C = g.C; t.CB = g.CB; t.OH = g.OH; t.OW = g.OW; t.pt = g.pt; t.pl = g.pl; t.relu = relu;
        CUtensorMap map;
        CUresult r = sm100::encode_blocked_map(ctx->encode_tiled, &map, in, g.N, g.CB, g.H, g.W, t.Wb, t.Hb, t.nn);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
        const size_t smem = 2 * (size_t)t.stage_bytes + 128;
        const long long cap = 2LL * ctx->sm_count;                 // persistent: two CTAs per SM
        const unsigned grid = (unsigned)(t.tiles < cap ? t.tiles : cap);
        auto kern = g.S == 1 ? dwconv3x3_tma_kernel<1> : dwconv3x3_tma_kernel<2>;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
        launch_kernel(ctx, kern, dim3(grid), dim3(256), smem, st, map, t);
        return check_launch(ctx);
    }
    long long total = a.planes * g.OH * g.OW * 8;
    long long want = (total + 255) / 256, cap = (long long)ctx->sm_count * 32;
    int grid = (int)(want < cap ? want : cap);
    launch_kernel(ctx, dwconv_generic_kernel, dim3(grid), dim3(256), 0, st, a);
    return check_launch(ctx);
}

}  // namespace small
