// Full channel reduction on CUDA cores (paper Section 3.2 item 4; Algorithms 1 and 2), FP32 FMA, any window,
// stride and padding.  It is the path for SMALL_MATH_FP32 and for shapes the tensor-core kernel does not take.
//
// Mapping of the paper's loop nest (Algorithm 1) onto a thread block:
//   g / k block loops ("in parallel")  -> the grid: one CTA per (image, block of 32 filters, 8 x PIX output tile)
//   i loop over F_C in steps of F_Cb    -> the cb loop over 32-channel input blocks (F_Cb = C_b = 32)
//   kernel tile O_wb x K_b              -> PIX output pixels per thread (registers) x 32 filters per warp (lanes)
//   LOAD / COMPUTE / STORE phases       -> accumulators start at zero; the epilogue adds bias and, when the
//                                          accumulate flag is set, the tile already in `out`; then ReLU; then store
// The lane is the output channel, so a warp's store of one pixel is one 128-byte line of the blocked layout and
// the filter reads from shared memory are conflict-free; the input pixel is a shared-memory broadcast.
#include "common.cuh"

namespace small {

struct ConvArgs {
    const float *in; const float *w; const float *bias; float *out;
    int C, K, H, W, FH, FW, S, pt, pl, OH, OW, CB, KB;
    int tiles_h, tiles_w, rows, cols;   // output tiles per plane; input tile extent in shared memory
    // Partial channel reduction (group convolution, Section 3.1.2): the 32 filters of block kb only read the
    // input channel blocks [cb0(kb), cb0(kb) + span); the packed filters hold zeros where a (channel, filter)
    // pair lies in different groups.  A full reduction has span = CB and cb0 = 0.
    int span, Kg, S_C;                  // blocks per filter block; filters per group; channel step between groups
    bool relu, accumulate;
};

template <int PIX, int ST>
__global__ void __launch_bounds__(256) conv_fp32_kernel(ConvArgs a) {
    grid_dep_sync();     // no early trigger: see launch_conv_fp32
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int S = ST ? ST : a.S;

    int b = blockIdx.x;
    const int tw = b % a.tiles_w; b /= a.tiles_w;
    const int th = b % a.tiles_h; b /= a.tiles_h;
    const int kb = b % a.KB;
    const int n = b / a.KB;
    const int oh0 = th * 8, ow0 = tw * PIX;
    const int ih0 = oh0 * S - a.pt, iw0 = ow0 * S - a.pl;

    float acc[PIX];
#pragma unroll
    for (int p = 0; p < PIX; ++p) acc[p] = 0.0f;

    const int max_ci4 = a.C >= 32 ? 8 : (a.C + 3) / 4;     // float4 groups per pixel in the shared tile
    float4 *in_tile = reinterpret_cast<float4 *>(smem);
    float *w_tile = smem + (size_t)a.rows * a.cols * max_ci4 * 4;

    const int cb0 = a.Kg > 0 ? ((kb * 32) / a.Kg * a.S_C) / 32 : 0;       // first channel block of this filter block's groups
    for (int cbj = 0; cbj < a.span; ++cbj) {
        const int cb = cb0 + cbj;
        if (cb >= a.CB) break;
        const int ci_n = min(32, a.C - cb * 32);
        const int ci4 = (ci_n + 3) >> 2;
        __syncthreads();   // the previous block's tile is no longer read
        // input halo tile: rows x cols pixels x ci4 float4; outside the plane reads as zero (the padding)
        const float4 *src = reinterpret_cast<const float4 *>(a.in + ((size_t)n * a.CB + cb) * a.H * a.W * 32);
        const int tile_elems = a.rows * a.cols * ci4;
        for (int e = threadIdx.x; e < tile_elems; e += 256) {
            int q = e % ci4;
            int pc = e / ci4;
            int c = pc % a.cols, r = pc / a.cols;
            int gh = ih0 + r, gw = iw0 + c;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (gh >= 0 && gh < a.H && gw >= 0 && gw < a.W) v = src[(gh * a.W + gw) * 8 + q];
            in_tile[e] = v;
        }
        for (int x = 0; x < a.FH; ++x) {
            __syncthreads();   // input tile visible (first x); previous filter row no longer read
            // filter row x of (kb, cb): [FW][ci][32 ko], only the channels that exist
            const float *wsrc = a.w + ((((size_t)kb * a.span + cbj) * a.FH + x) * a.FW) * 32 * 32;
            const int w_elems = a.FW * ci4 * 4 * 32;
            for (int e = threadIdx.x; e < w_elems; e += 256) {
                int ko = e & 31;
                int r = e >> 5;
                int ci = r % (ci4 * 4), y = r / (ci4 * 4);
                w_tile[e] = wsrc[(y * 32 + ci) * 32 + ko];
            }
            __syncthreads();
            const float4 *row = in_tile + ((warp * S + x) * a.cols) * ci4;
            for (int y = 0; y < a.FW; ++y) {
                for (int q = 0; q < ci4; ++q) {
                    const float *wp = w_tile + ((y * ci4 + q) * 4) * 32 + lane;
                    const float w0 = wp[0], w1 = wp[32], w2 = wp[64], w3 = wp[96];
#pragma unroll
                    for (int p = 0; p < PIX; ++p) {
                        const float4 v = row[(p * S + y) * ci4 + q];
                        acc[p] = fmaf(v.x, w0, acc[p]);
                        acc[p] = fmaf(v.y, w1, acc[p]);
                        acc[p] = fmaf(v.z, w2, acc[p]);
                        acc[p] = fmaf(v.w, w3, acc[p]);
                    }
                }
            }
        }
    }

    // epilogue: bias, optional accumulate, optional ReLU; pad lanes (k >= K) are written as +0
    const int oh = oh0 + warp;
    if (oh < a.OH) {
        const int k = kb * 32 + lane;
        const float bv = (a.bias && k < a.K) ? a.bias[k] : 0.0f;
        float *dst = a.out + ((((size_t)n * a.KB + kb) * a.OH + oh) * a.OW + ow0) * 32 + lane;
#pragma unroll
        for (int p = 0; p < PIX; ++p) {
            if (ow0 + p < a.OW) {
                float v = acc[p] + bv;
                if (a.accumulate) v += dst[p * 32];
                if (a.relu) v = v > 0.f ? v : 0.f;
                dst[p * 32] = k < a.K ? v : 0.0f;
            }
        }
    }
}

template <int PIX, int ST>
static int launch_variant(small_ctx *ctx, ConvArgs &a, long long blocks, size_t smem, cudaStream_t st) {
    auto kern = conv_fp32_kernel<PIX, ST>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    }
    // Always an ordinary launch, and the kernel lets its successor start only as its blocks leave.  Its blocks are small
    // and many per SM; started beside the big-shared-memory blocks of a persistent kernel in front of it, they would
    // inherit that kernel's shared-memory / L1 split for the whole launch (measured: the depthwise-separable network
    // in FP32 mode ran 12 % slower with this kernel as a dependent launch).
    const int dependent = ctx->dependent;
    ctx->dependent = 0;
    launch_kernel(ctx, kern, dim3((unsigned)blocks), dim3(256), smem, st, a);
    ctx->dependent = dependent;
    return check_launch(ctx);
}

int launch_conv_fp32(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, const Geom &g,
                     bool relu, bool accumulate, cudaStream_t st, int span, int Kg, int S_C) {
    const int PIX = g.OW <= 8 ? 8 : 16;
    ConvArgs a{in, w, bias, out, g.C, g.K, g.H, g.W, g.FH, g.FW, g.S, g.pt, g.pl, g.OH, g.OW, g.CB, g.KB,
               ceil_div(g.OH, 8), ceil_div(g.OW, PIX), 0, 0, span > 0 ? span : g.CB, span > 0 ? Kg : 0, S_C, relu, accumulate};
    // the shared input tile covers the whole 8 x PIX thread tile, so threads whose outputs fall outside the plane
    // still read inside the allocation (their results are not stored)
    a.rows = 7 * g.S + g.FH;
    a.cols = (PIX - 1) * g.S + g.FW;
    int max_ci4 = g.C >= 32 ? 8 : (g.C + 3) / 4;
    size_t smem = ((size_t)a.rows * a.cols * max_ci4 * 4 + (size_t)g.FW * max_ci4 * 4 * 32) * sizeof(float);
    if (smem > ctx->max_smem_optin) return SMALL_ERR_UNSUPPORTED;
    long long blocks = (long long)g.N * g.KB * a.tiles_h * a.tiles_w;
    if (blocks > 0x7fffffffLL) return SMALL_ERR_SHAPE;
    if (PIX == 8) {
        if (g.S == 1) return launch_variant<8, 1>(ctx, a, blocks, smem, st);
        if (g.S == 2) return launch_variant<8, 2>(ctx, a, blocks, smem, st);
        return launch_variant<8, 0>(ctx, a, blocks, smem, st);
    }
    if (g.S == 1) return launch_variant<16, 1>(ctx, a, blocks, smem, st);
    if (g.S == 2) return launch_variant<16, 2>(ctx, a, blocks, smem, st);
    return launch_variant<16, 0>(ctx, a, blocks, smem, st);
}

}  // namespace small
