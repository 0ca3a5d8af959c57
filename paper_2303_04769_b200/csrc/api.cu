// C ABI of the library: context, argument validation and dispatch.  Every step of a layer runs in the
// kernels of the neighbouring .cu files; this file only checks arguments and launches.
#include <cstdio>
#include <cstring>
#include <initializer_list>
#include <new>

#include "common.cuh"

namespace small {

int make_geom(Geom &g, int N, int C, int K, int H, int W, int FH, int FW, int S, int pt, int pb, int pl, int pr) {
    if (N < 1 || C < 1 || K < 1 || H < 1 || W < 1 || FH < 1 || FW < 1 || S < 1) return SMALL_ERR_SHAPE;
    if (pt < 0 || pb < 0 || pl < 0 || pr < 0) return SMALL_ERR_SHAPE;
    if (pt >= FH || pb >= FH || pl >= FW || pr >= FW) return SMALL_ERR_SHAPE;  // a window never lies wholly in the pad
    int OH = out_size(H, FH, S, pt, pb), OW = out_size(W, FW, S, pl, pr);
    if (OH < 1 || OW < 1) return SMALL_ERR_SHAPE;
    // 32-bit index arithmetic inside a plane, 64-bit across planes: keep planes and rows well inside int range
    if ((long long)H * W > (1ll << 24) || (long long)N * blocks_of(C) > (1ll << 30) || (long long)N * blocks_of(K) > (1ll << 30))
        return SMALL_ERR_SHAPE;
    g = Geom{N, C, K, H, W, FH, FW, S, pt, pb, pl, pr, OH, OW, blocks_of(C), blocks_of(K)};
    return SMALL_OK;
}

size_t conv_w_fp32_elems(int C, int K, int FH, int FW) {
    return (size_t)blocks_of(K) * blocks_of(C) * FH * FW * SMALL_CB * SMALL_CB;
}
size_t conv_w_tc_elems(int C, int K, int FH, int FW) {
    return (size_t)blocks_of(C) * FH * FW * blocks_of(K) * SMALL_CB * SMALL_CB;
}

static int check_ptrs(std::initializer_list<const void *> required, std::initializer_list<const void *> optional = {}) {
    for (const void *p : required) {
        if (!p) return SMALL_ERR_INVALID_ARG;
        if (!aligned16(p)) return SMALL_ERR_ALIGN;
    }
    for (const void *p : optional)
        if (p && !aligned16(p)) return SMALL_ERR_ALIGN;
    return SMALL_OK;
}

static unsigned math_of(unsigned flags) { return flags & SMALL_MATH_MASK; }
static bool math_valid(unsigned m) { return m == SMALL_MATH_FP32 || m == SMALL_MATH_TF32 || m == SMALL_MATH_3XTF32; }

}  // namespace small

using namespace small;

SMALL_API int small_channel_block(void) { return SMALL_CB; }
SMALL_API size_t small_packed_elems(int N, int C, int H, int W) { return packed_elems(N, C, H, W); }
SMALL_API int small_out_size(int I, int F, int stride, int pa, int pb) {
    if (pa < 0 || pb < 0) return 0;
    return out_size(I, F, stride, pa, pb);
}

SMALL_API const char *small_strerror(int s) {
    switch (s) {
        case SMALL_OK: return "ok";
        case SMALL_ERR_INVALID_ARG: return "invalid argument (null pointer, unknown flag or mode)";
        case SMALL_ERR_SHAPE: return "invalid shape (dimension < 1, empty output, pad >= window, or too large)";
        case SMALL_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case SMALL_ERR_OVERLAP: return "input and output ranges overlap";
        case SMALL_ERR_WORKSPACE: return "workspace too small or slot id out of range";
        case SMALL_ERR_UNSUPPORTED: return "request outside what the kernels cover";
        case SMALL_ERR_CUDA: return "CUDA call failed (see small_last_cuda_error)";
        case SMALL_ERR_TIMEOUT: return "bounded device-side wait ran out";
        case SMALL_ERR_NOT_INIT: return "context is null or shut down";
        default: return "unknown status";
    }
}

SMALL_API int small_init(int device, small_ctx **out) {
    if (!out) return SMALL_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess) return SMALL_ERR_CUDA;
    if (device < 0 || device >= count) return SMALL_ERR_INVALID_ARG;
    if ((e = cudaSetDevice(device)) != cudaSuccess) return SMALL_ERR_CUDA;
    small_ctx *c = new (std::nothrow) small_ctx();
    if (!c) return SMALL_ERR_INVALID_ARG;
    c->device = device;
    c->last_cuda = 0;
    c->encode_tiled = nullptr;
    cudaDeviceProp prop;
    if ((e = cudaGetDeviceProperties(&prop, device)) != cudaSuccess) { delete c; return SMALL_ERR_CUDA; }
    c->sm_count = prop.multiProcessorCount;
    c->max_smem_optin = prop.sharedMemPerBlockOptin;
    if (prop.major != 10) { delete c; return SMALL_ERR_UNSUPPORTED; }  // kernels are built for sm_100a only
    void *block = nullptr;
    if ((e = cudaMalloc(&block, 256)) != cudaSuccess) { delete c; return SMALL_ERR_CUDA; }
    cudaMemset(block, 0, 256);
    c->dev_status = static_cast<int *>(block);
    cudaDriverEntryPointQueryResult q;
    void *fn = nullptr;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) {
        cudaFree(block);
        delete c;
        return SMALL_ERR_CUDA;
    }
    c->encode_tiled = fn;
    c->static_workspace = nullptr;
    c->tc_cache = nullptr;
    c->mma_cache = nullptr;
    c->wait_iters = 1u << 22;     // with the polls' nanosleep back-off: seconds
    if (resolve_static_workspace(c) != SMALL_OK) {      // loads the library's device code here, not inside a later call
        cudaFree(block);
        delete c;
        return SMALL_ERR_CUDA;
    }
    c->overlap = 1;
    c->dependent = 0;
    c->conv_path = SMALL_CONV_PATH_AUTO;
    c->net_fusion = SMALL_FUSE_DWPW | SMALL_FUSE_CONVPOOL | SMALL_FUSE_FC_CHAIN | SMALL_FUSE_POOLFC;
    c->branch_overlap = 1;
    c->side_stream = c->ev_fork = c->ev_join = nullptr;
    {
        cudaStream_t side;
        cudaEvent_t f, j;
        if (cudaStreamCreateWithFlags(&side, cudaStreamNonBlocking) == cudaSuccess) c->side_stream = side;
        if (cudaEventCreateWithFlags(&f, cudaEventDisableTiming) == cudaSuccess) c->ev_fork = f;
        if (cudaEventCreateWithFlags(&j, cudaEventDisableTiming) == cudaSuccess) c->ev_join = j;
        if (!c->side_stream || !c->ev_fork || !c->ev_join) c->branch_overlap = 0;
        c->copy_stream = nullptr; c->host_ws = nullptr; c->host_parity = 0; c->host_used[0] = c->host_used[1] = 0;
        cudaStream_t cs;
        bool ok = cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking) == cudaSuccess;
        for (int i = 0; i < 2; ++i) {
            cudaEvent_t a = nullptr, b = nullptr;
            ok = ok && cudaEventCreateWithFlags(&a, cudaEventDisableTiming) == cudaSuccess && cudaEventCreateWithFlags(&b, cudaEventDisableTiming) == cudaSuccess;
            c->ev_h2d[i] = a; c->ev_pack[i] = b;
        }
        if (ok) c->copy_stream = cs;
    }
    *out = c;
    return SMALL_OK;
}

SMALL_API int small_shutdown(small_ctx *ctx) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    cudaSetDevice(ctx->device);
    if (ctx->dev_status) cudaFree(ctx->dev_status);
    free_tc_cache(ctx);
    free_mma_cache(ctx);
    if (ctx->ev_fork) cudaEventDestroy(static_cast<cudaEvent_t>(ctx->ev_fork));
    if (ctx->ev_join) cudaEventDestroy(static_cast<cudaEvent_t>(ctx->ev_join));
    if (ctx->side_stream) cudaStreamDestroy(static_cast<cudaStream_t>(ctx->side_stream));
    for (int i = 0; i < 2; ++i) {
        if (ctx->ev_h2d[i]) cudaEventDestroy(static_cast<cudaEvent_t>(ctx->ev_h2d[i]));
        if (ctx->ev_pack[i]) cudaEventDestroy(static_cast<cudaEvent_t>(ctx->ev_pack[i]));
    }
    if (ctx->copy_stream) cudaStreamDestroy(static_cast<cudaStream_t>(ctx->copy_stream));
    delete ctx;
    return SMALL_OK;
}

SMALL_API int small_last_cuda_error(small_ctx *ctx) { return ctx ? ctx->last_cuda : 0; }

SMALL_API int small_set_layer_overlap(small_ctx *ctx, int on) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    ctx->overlap = on ? 1 : 0;
    return SMALL_OK;
}

SMALL_API int small_set_wait_limit(small_ctx *ctx, unsigned polls) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (polls < 16u) return SMALL_ERR_INVALID_ARG;
    ctx->wait_iters = polls;
    return SMALL_OK;
}

SMALL_API int small_set_fc_chain_tile(small_ctx *ctx, int images) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (images != 0 && images != 32 && images != 64 && images != 128) return SMALL_ERR_INVALID_ARG;
    ctx->fc_chain_tile = images;
    return SMALL_OK;
}

SMALL_API int small_set_branch_overlap(small_ctx *ctx, int on) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    ctx->branch_overlap = (on && ctx->side_stream && ctx->ev_fork && ctx->ev_join) ? 1 : 0;
    return SMALL_OK;
}

SMALL_API int small_set_conv_path(small_ctx *ctx, int path) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (path < SMALL_CONV_PATH_AUTO || path > SMALL_CONV_PATH_WARP_MMA) return SMALL_ERR_INVALID_ARG;
    ctx->conv_path = path;
    return SMALL_OK;
}

SMALL_API int small_device_status(small_ctx *ctx, int *status, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!status) return SMALL_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int host = 0;
    cudaError_t e = cudaMemcpyAsync(&host, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->dev_status, 0, sizeof(int), st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    *status = host;
    return SMALL_OK;
}

// ---- layout ----
SMALL_API int small_pack(small_ctx *ctx, const float *nchw, float *blk, int N, int C, int H, int W, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (int s = check_ptrs({nchw, blk})) return s;
    if (N < 1 || C < 1 || H < 1 || W < 1 || (long long)H * W > (1ll << 24)) return SMALL_ERR_SHAPE;
    if (ranges_overlap(nchw, sizeof(float) * (size_t)N * C * H * W, blk, sizeof(float) * packed_elems(N, C, H, W))) return SMALL_ERR_OVERLAP;
    return launch_pack(ctx, nchw, blk, N, C, H, W, static_cast<cudaStream_t>(stream));
}

SMALL_API int small_unpack(small_ctx *ctx, const float *blk, float *nchw, int N, int C, int H, int W, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (int s = check_ptrs({nchw, blk})) return s;
    if (N < 1 || C < 1 || H < 1 || W < 1 || (long long)H * W > (1ll << 24)) return SMALL_ERR_SHAPE;
    if (ranges_overlap(nchw, sizeof(float) * (size_t)N * C * H * W, blk, sizeof(float) * packed_elems(N, C, H, W))) return SMALL_ERR_OVERLAP;
    return launch_unpack(ctx, blk, nchw, N, C, H, W, static_cast<cudaStream_t>(stream));
}

// ---- filters ----
SMALL_API size_t small_conv_weight_elems(int C, int K, int FH, int FW, unsigned math) {
    if (C < 1 || K < 1 || FH < 1 || FW < 1 || !math_valid(math)) return 0;
    size_t n = conv_w_fp32_elems(C, K, FH, FW);
    if (math != SMALL_MATH_FP32) n += conv_w_tc_elems(C, K, FH, FW);
    if (math == SMALL_MATH_3XTF32) n += conv_w_tc_elems(C, K, FH, FW);
    return n;
}

SMALL_API int small_pack_conv_weights(small_ctx *ctx, const float *w, float *wb, int C, int K, int FH, int FW,
                                      unsigned math, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!math_valid(math)) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({w, wb})) return s;
    if (C < 1 || K < 1 || FH < 1 || FW < 1) return SMALL_ERR_SHAPE;
    if (ranges_overlap(w, sizeof(float) * (size_t)K * C * FH * FW, wb, sizeof(float) * small_conv_weight_elems(C, K, FH, FW, math)))
        return SMALL_ERR_OVERLAP;
    return launch_pack_conv_weights(ctx, w, wb, C, K, FH, FW, math, static_cast<cudaStream_t>(stream));
}

// ---- group convolution (partial channel reduction)
static bool group_shape_ok(int C, int F_C, int S_C, int K) {
    return C >= 1 && F_C >= 1 && F_C <= C && S_C >= 1 && K >= 1 && (C - F_C) % S_C == 0;
}

SMALL_API int small_group_count(int C, int F_C, int S_C) {
    if (C < 1 || F_C < 1 || F_C > C || S_C < 1 || (C - F_C) % S_C != 0) return 0;
    return (C - F_C) / S_C + 1;
}

// groups that are whole channel blocks with a multiple of 32 filters each can run on the tensor-core kernel
static bool group_tc_layout(int F_C, int S_C, int K) { return F_C == S_C && F_C % 32 == 0 && K % 32 == 0 && K <= 256; }
static size_t group_fp32_elems(int C, int F_C, int S_C, int K, int FH, int FW) {
    const int G = (C - F_C) / S_C + 1;
    return (size_t)blocks_of(K * G) * group_conv_span(C, F_C, S_C, K) * FH * FW * SMALL_CB * SMALL_CB;
}

SMALL_API size_t small_group_conv_weight_elems(int C, int F_C, int S_C, int K, int FH, int FW) {
    if (!group_shape_ok(C, F_C, S_C, K) || FH < 1 || FW < 1) return 0;
    const int G = (C - F_C) / S_C + 1;
    size_t n = group_fp32_elems(C, F_C, S_C, K, FH, FW);
    if (group_tc_layout(F_C, S_C, K)) n += 2 * group_conv_w_tc_elems(F_C, K, G, FH, FW);    // TF32 part and residual
    return n;
}

SMALL_API int small_pack_group_conv_weights(small_ctx *ctx, const float *w, float *wb, int C, int F_C, int S_C, int K,
                                            int FH, int FW, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (int s = check_ptrs({w, wb})) return s;
    if (!group_shape_ok(C, F_C, S_C, K) || FH < 1 || FW < 1) return SMALL_ERR_SHAPE;
    const int G = (C - F_C) / S_C + 1;
    if (ranges_overlap(w, sizeof(float) * (size_t)G * K * F_C * FH * FW, wb,
                       sizeof(float) * small_group_conv_weight_elems(C, F_C, S_C, K, FH, FW)))
        return SMALL_ERR_OVERLAP;
    if (int s = launch_pack_group_conv_weights(ctx, w, wb, C, F_C, S_C, K, FH, FW, static_cast<cudaStream_t>(stream))) return s;
    if (group_tc_layout(F_C, S_C, K)) {
        float *hi = wb + group_fp32_elems(C, F_C, S_C, K, FH, FW);
        return launch_pack_group_conv_weights_tc(ctx, w, hi, hi + group_conv_w_tc_elems(F_C, K, G, FH, FW), F_C, K, G, FH, FW,
                                                 static_cast<cudaStream_t>(stream));
    }
    return SMALL_OK;
}

SMALL_API int small_group_conv2d(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out,
                                 int N, int C, int F_C, int S_C, int K, int H, int W, int FH, int FW, int stride,
                                 int pt, int pb, int pl, int pr, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~(SMALL_RELU | SMALL_ACCUMULATE | SMALL_MATH_MASK)) return SMALL_ERR_INVALID_ARG;
    if (!math_valid(math_of(flags))) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({in, w, out}, {bias})) return s;
    if (!group_shape_ok(C, F_C, S_C, K)) return SMALL_ERR_SHAPE;
    const int G = (C - F_C) / S_C + 1;
    if ((long long)K * G > 0x7fffffLL) return SMALL_ERR_SHAPE;
    Geom g;
    if (int s = make_geom(g, N, C, K * G, H, W, FH, FW, stride, pt, pb, pl, pr)) return s;
    if (ranges_overlap(in, sizeof(float) * packed_elems(N, C, H, W), out, sizeof(float) * packed_elems(N, K * G, g.OH, g.OW)))
        return SMALL_ERR_OVERLAP;
    // tensor-core modes: groups of whole channel blocks run on the tensor-core kernel, one filter tile per group
    const unsigned math = math_of(flags);
    if (math != SMALL_MATH_FP32 && G > 1 && group_tc_layout(F_C, S_C, K) && (reinterpret_cast<uintptr_t>(out) & 31u) == 0) {
        Geom gg;
        if (make_geom(gg, N, F_C, K * G, H, W, FH, FW, stride, pt, pb, pl, pr) == SMALL_OK &&
            conv_tc_supported(gg, math == SMALL_MATH_3XTF32, G)) {
            const float *w_hi = w + group_fp32_elems(C, F_C, S_C, K, FH, FW);
            const float *w_lo = w_hi + group_conv_w_tc_elems(F_C, K, G, FH, FW);
            return launch_conv_tc(ctx, in, w_hi, w_lo, bias, out, gg, flags & SMALL_RELU, flags & SMALL_ACCUMULATE, math,
                                  static_cast<cudaStream_t>(stream), G);
        }
    }
    // everything else runs the FP32 kernel (tighter than the tensor-core modes promise)
    return launch_conv_fp32(ctx, in, w, bias, out, g, flags & SMALL_RELU, flags & SMALL_ACCUMULATE, static_cast<cudaStream_t>(stream),
                            group_conv_span(C, F_C, S_C, K), K, S_C);
}

SMALL_API size_t small_dw_weight_elems(int C, int FH, int FW) {
    if (C < 1 || FH < 1 || FW < 1) return 0;
    return (size_t)blocks_of(C) * FH * FW * SMALL_CB;
}

SMALL_API int small_pack_dw_weights(small_ctx *ctx, const float *w, float *wb, int C, int FH, int FW, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (int s = check_ptrs({w, wb})) return s;
    if (C < 1 || FH < 1 || FW < 1) return SMALL_ERR_SHAPE;
    if (ranges_overlap(w, sizeof(float) * (size_t)C * FH * FW, wb, sizeof(float) * small_dw_weight_elems(C, FH, FW))) return SMALL_ERR_OVERLAP;
    return launch_pack_dw_weights(ctx, w, wb, C, FH, FW, static_cast<cudaStream_t>(stream));
}

// A fully-connected layer's filters [K][J] are a 1x1 convolution's [K][C = J][1][1], and the packed FP32 section of the
// two is the same array; the tensor-core sections come with the math mode the buffer is packed for.
SMALL_API size_t small_fc_weight_elems(int J, int K, unsigned math) {
    return small_conv_weight_elems(J, K, 1, 1, math);
}

SMALL_API int small_pack_fc_weights(small_ctx *ctx, const float *w, float *wb, int J, int K, unsigned math, void *stream) {
    return small_pack_conv_weights(ctx, w, wb, J, K, 1, 1, math, stream);
}

// ---- layers ----
// Which kernel family a full channel reduction takes under a tensor-core math mode.  The tensor-core kernel's MMAs are
// 128 x N x 8 with N = the layer's filters: with few channels each still occupies the pipe for its floor of 40 to 50
// cycles, and a launch carries some microseconds of pipeline set-up and drain.  The register-tiled FP32 kernel (whose
// result meets every mode's tolerance) has neither cost but sustains about half the FP32 FMA rate.  Measured on the
// residual network's layers at batch 256 (tensor cores TF32 / 3xTF32 against CUDA cores, microseconds): 1x1 stride 2
// 16->32: 9.9 / 13.6 against 8.8; 3x3 stride 2 16->32: 20.1 / 29.5 against 25.3; 3x3 16->16: 25.7 / 39.3 against 44.4;
// 1x1 stride 2 32->64: 8.1 / 9.0 against 11.0.  Hence: CUDA cores for C * K <= 512 when the window is 1 x 1, or when the
// mode is 3xTF32 and the stride 2 (the stride-2 view spends two or three MMAs per product on four phase planes).
static bool prefer_cuda_cores(const small_ctx *ctx, const Geom &g, unsigned math) {
    if (ctx && ctx->conv_path == SMALL_CONV_PATH_TENSOR) return false;
    if (ctx && ctx->conv_path == SMALL_CONV_PATH_CUDA_CORES) return true;
    if ((long long)g.C * g.K > 512) return false;
    return g.FH * g.FW == 1 || (math == SMALL_MATH_3XTF32 && g.S == 2);
}

static int conv2d_path(const small_ctx *ctx, const Geom &g, unsigned math, bool out_aligned32) {
    if (ctx && ctx->conv_path == SMALL_CONV_PATH_WARP_MMA && math != SMALL_MATH_FP32 && conv_mma_supported(g, math == SMALL_MATH_3XTF32)) return 4;
    if (conv_thin_supported(g)) return 0;          // a reduction of a few dozen terms: CUDA cores in every math mode
    if (ctx && ctx->conv_path == SMALL_CONV_PATH_GENERAL) return 2;
    bool direct = conv_direct_supported(g);
    // the register-tiled kernel computes runs of 8 output columns per thread and 256 to 2048 outputs x 8 to 64 filters per
    // thread block: planes narrower than 4 columns leave it mostly idle, and a layer that gives it fewer blocks than half
    // the SMs runs faster on the general kernel's many small blocks (measured on the depthwise-separable network)
    if (direct && !(ctx && ctx->conv_path == SMALL_CONV_PATH_CUDA_CORES) &&
        (g.OW < 4 || conv_direct_blocks(g) < (ctx ? ctx->sm_count : 148) / 2))
        direct = false;
    if (math == SMALL_MATH_FP32) return direct ? 1 : 2;
    // One channel block and at most 32 filters (64 with a 1x1 window): the warp-level MMA (see conv_mma.cu), which measured faster than both
    // other families on such layers (residual CNN at batch 256, microseconds, TF32 / 3xTF32, block-level tensor-core
    // kernel against warp-level: 3x3 16->16 25.3 / 37.4 against 17.3 / 28.7; 3x3 stride 2 16->32 19.9 / 28.3 against
    // 12.2 / 15.8; 1x1 stride 2 16->32 10.2 / 14.3 against 7.1 / 7.6; 3x3 32->32 on 16x16 planes 15.5 / 27.2 against
    // 14.8 / 23.9, on 8x8 planes 10.2 / 13.4 against 8.1 / 9.1; 1x1 stride 2 32->64 8.3 / 9.8 against 7.1 / 7.7; but 3x3
    // stride 2 32->64 15.4 / 18.4 against 15.4 / 23.6, so 3x3 layers with more than 32 filters stay where they were).
    if (!(ctx && (ctx->conv_path == SMALL_CONV_PATH_TENSOR || ctx->conv_path == SMALL_CONV_PATH_CUDA_CORES)) &&
        ((ctx && ctx->conv_path == SMALL_CONV_PATH_WARP_MMA) || g.K <= 32 || (g.K <= 64 && g.FH * g.FW == 1)) && conv_mma_supported(g, math == SMALL_MATH_3XTF32))
        return 4;
    if (ctx && ctx->conv_path == SMALL_CONV_PATH_WARP_MMA) return direct ? 1 : 2;
    const bool tc = out_aligned32 && conv_tc_supported(g, math == SMALL_MATH_3XTF32);
    if (tc && !(direct && prefer_cuda_cores(ctx, g, math))) return 3;
    return direct ? 1 : 2;
}

SMALL_API int small_conv2d_uses_tensor_cores(int N, int C, int K, int H, int W, int FH, int FW, int stride,
                                             int pt, int pb, int pl, int pr) {
    Geom g;
    if (make_geom(g, N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr) != SMALL_OK) return 0;
    return conv2d_path(nullptr, g, SMALL_MATH_TF32, true) >= 3 ? 1 : 0;     // block-level or warp-level MMAs
}

SMALL_API int small_conv2d_path(small_ctx *ctx, int N, int C, int K, int H, int W, int FH, int FW, int stride,
                                int pt, int pb, int pl, int pr, unsigned math) {
    Geom g;
    if (!ctx || !math_valid(math) || make_geom(g, N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr) != SMALL_OK) return -1;
    return conv2d_path(ctx, g, math, true);
}

SMALL_API int small_conv2d(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out,
                           int N, int C, int K, int H, int W, int FH, int FW, int stride,
                           int pt, int pb, int pl, int pr, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~(SMALL_RELU | SMALL_ACCUMULATE | SMALL_MATH_MASK)) return SMALL_ERR_INVALID_ARG;
    unsigned math = math_of(flags);
    if (!math_valid(math)) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({in, w, out}, {bias})) return s;
    Geom g;
    if (int s = make_geom(g, N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr)) return s;
    if (ranges_overlap(in, sizeof(float) * packed_elems(N, C, H, W), out, sizeof(float) * packed_elems(N, K, g.OH, g.OW)))
        return SMALL_ERR_OVERLAP;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    bool relu = flags & SMALL_RELU, acc = flags & SMALL_ACCUMULATE;
    // the tensor-core epilogue may store 32 bytes per thread: an output that is only 16-byte aligned takes a CUDA-core kernel
    switch (conv2d_path(ctx, g, math, (reinterpret_cast<uintptr_t>(out) & 31u) == 0)) {
        case 0: return launch_conv_thin(ctx, in, w, bias, out, g, relu, acc, st);
        case 1: return launch_conv_direct(ctx, in, w, bias, out, g, relu, acc, st);
        case 3: {
            const float *w_hi = w + conv_w_fp32_elems(C, K, FH, FW);
            const float *w_lo = w_hi + conv_w_tc_elems(C, K, FH, FW);
            return launch_conv_tc(ctx, in, w_hi, math == SMALL_MATH_3XTF32 ? w_lo : nullptr, bias, out, g, relu, acc, math, st);
        }
        case 4: {
            const float *w_hi = w + conv_w_fp32_elems(C, K, FH, FW);
            const float *w_lo = w_hi + conv_w_tc_elems(C, K, FH, FW);
            return launch_conv_mma(ctx, in, w_hi, math == SMALL_MATH_3XTF32 ? w_lo : nullptr, bias, out, g, relu, acc, math, st);
        }
        default: return launch_conv_fp32(ctx, in, w, bias, out, g, relu, acc, st);
    }
}

// ---- fused convolution -> 2 x 2 stride-2 max pool
SMALL_API int small_conv_maxpool_fused(int N, int C, int K, int H, int W, int FH, int FW, int stride, int pt, int pb, int pl, int pr) {
    Geom g;
    if (make_geom(g, N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr) != SMALL_OK) return 0;
    return conv_direct_pool_supported(g) ? 1 : 0;
}

SMALL_API int small_conv_maxpool2d(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, float *scratch,
                                   int N, int C, int K, int H, int W, int FH, int FW, int stride,
                                   int pt, int pb, int pl, int pr, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~(SMALL_RELU | SMALL_MATH_MASK)) return SMALL_ERR_INVALID_ARG;
    if (!math_valid(math_of(flags))) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({in, w, out}, {bias, scratch})) return s;
    Geom g;
    if (int s = make_geom(g, N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr)) return s;
    if (g.OH < 2 || g.OW < 2) return SMALL_ERR_SHAPE;                  // the pool's output would be empty
    const size_t in_b = sizeof(float) * packed_elems(N, C, H, W), out_b = sizeof(float) * packed_elems(N, K, g.OH / 2, g.OW / 2);
    if (ranges_overlap(in, in_b, out, out_b)) return SMALL_ERR_OVERLAP;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // one kernel: the register-tiled FP32 kernel pools in its STORE phase (FP32 FMAs meet every math mode's tolerance)
    if (conv_direct_pool_supported(g)) return launch_conv_direct_pool(ctx, in, w, bias, out, g, flags & SMALL_RELU, st);
    // the two layers one after the other, through the caller's scratch tensor
    if (!scratch) return SMALL_ERR_WORKSPACE;
    const size_t mid_b = sizeof(float) * packed_elems(N, K, g.OH, g.OW);
    if (ranges_overlap(scratch, mid_b, in, in_b) || ranges_overlap(scratch, mid_b, out, out_b)) return SMALL_ERR_OVERLAP;
    if (int s = small_conv2d(ctx, in, w, bias, scratch, N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr, flags, stream)) return s;
    return small_pool2d(ctx, scratch, out, nullptr, N, K, g.OH, g.OW, 2, 2, 2, 0, 0, 0, 0, SMALL_POOL_MAX, stream);
}

SMALL_API int small_dwconv2d(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out,
                             int N, int C, int H, int W, int FH, int FW, int stride,
                             int pt, int pb, int pl, int pr, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~(SMALL_RELU | SMALL_MATH_MASK)) return SMALL_ERR_INVALID_ARG;
    if (!math_valid(math_of(flags))) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({in, w, out}, {bias})) return s;
    Geom g;
    if (int s = make_geom(g, N, C, C, H, W, FH, FW, stride, pt, pb, pl, pr)) return s;
    if (ranges_overlap(in, sizeof(float) * packed_elems(N, C, H, W), out, sizeof(float) * packed_elems(N, C, g.OH, g.OW)))
        return SMALL_ERR_OVERLAP;
    return launch_dwconv(ctx, in, w, bias, out, g, flags & SMALL_RELU, static_cast<cudaStream_t>(stream));
}

// ---- fused depthwise 3x3 -> 1x1 convolution
static bool dwpw_geoms(Geom &gd, Geom &gp, int N, int C, int K, int H, int W, int stride, int pt, int pb, int pl, int pr) {
    if (make_geom(gd, N, C, C, H, W, 3, 3, stride, pt, pb, pl, pr) != SMALL_OK) return false;
    return make_geom(gp, N, C, K, gd.OH, gd.OW, 1, 1, 1, 0, 0, 0, 0) == SMALL_OK;
}

SMALL_API int small_dwpw_fused(int N, int C, int K, int H, int W, int stride, int pt, int pb, int pl, int pr, unsigned math) {
    if (math != SMALL_MATH_TF32 && math != SMALL_MATH_3XTF32) return 0;
    if (stride != 1 && stride != 2) return 0;
    Geom gd, gp;
    if (!dwpw_geoms(gd, gp, N, C, K, H, W, stride, pt, pb, pl, pr)) return 0;
    DwFuse f{nullptr, nullptr, C, H, W, stride, pt, pl, 0};
    return conv_tc_supported(gp, math == SMALL_MATH_3XTF32, 1, &f) ? 1 : 0;
}

SMALL_API int small_dwpw_conv2d(small_ctx *ctx, const float *in, const float *dw_w, const float *dw_bias,
                                const float *pw_w, const float *pw_bias, float *out, float *scratch,
                                int N, int C, int K, int H, int W, int stride,
                                int pt, int pb, int pl, int pr, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~(SMALL_RELU | SMALL_RELU_MID | SMALL_MATH_MASK)) return SMALL_ERR_INVALID_ARG;
    const unsigned math = math_of(flags);
    if (!math_valid(math)) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({in, dw_w, pw_w, out}, {dw_bias, pw_bias, scratch})) return s;
    Geom gd, gp;
    if (int s = make_geom(gd, N, C, C, H, W, 3, 3, stride, pt, pb, pl, pr)) return s;
    if (int s = make_geom(gp, N, C, K, gd.OH, gd.OW, 1, 1, 1, 0, 0, 0, 0)) return s;
    if (ranges_overlap(in, sizeof(float) * packed_elems(N, C, H, W), out, sizeof(float) * packed_elems(N, K, gd.OH, gd.OW)))
        return SMALL_ERR_OVERLAP;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool relu = flags & SMALL_RELU, relu_mid = flags & SMALL_RELU_MID;
    if (math != SMALL_MATH_FP32 && (stride == 1 || stride == 2) && (reinterpret_cast<uintptr_t>(out) & 31u) == 0) {
        DwFuse f{dw_w, dw_bias, C, H, W, stride, pt, pl, relu_mid ? 1 : 0};
        if (conv_tc_supported(gp, math == SMALL_MATH_3XTF32, 1, &f)) {
            const float *w_hi = pw_w + conv_w_fp32_elems(C, K, 1, 1);
            const float *w_lo = w_hi + conv_w_tc_elems(C, K, 1, 1);
            return launch_conv_tc(ctx, in, w_hi, math == SMALL_MATH_3XTF32 ? w_lo : nullptr, pw_bias, out, gp, relu, false, math, st, 1, &f);
        }
    }
    // the two layers one after the other, through the caller's scratch tensor
    if (!scratch) return SMALL_ERR_WORKSPACE;
    const size_t mid = sizeof(float) * packed_elems(N, C, gd.OH, gd.OW);
    if (ranges_overlap(scratch, mid, in, sizeof(float) * packed_elems(N, C, H, W)) ||
        ranges_overlap(scratch, mid, out, sizeof(float) * packed_elems(N, K, gd.OH, gd.OW)))
        return SMALL_ERR_OVERLAP;
    if (int s = launch_dwconv(ctx, in, dw_w, dw_bias, scratch, gd, relu_mid, st)) return s;
    return small_conv2d(ctx, scratch, pw_w, pw_bias, out, N, C, K, gd.OH, gd.OW, 1, 1, 1, 0, 0, 0, 0,
                        (relu ? SMALL_RELU : 0u) | math, stream);
}

SMALL_API int small_pool2d(small_ctx *ctx, const float *in, float *out, int32_t *idx,
                           int N, int C, int H, int W, int FH, int FW, int stride,
                           int pt, int pb, int pl, int pr, int mode, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (mode != SMALL_POOL_MAX && mode != SMALL_POOL_AVG) return SMALL_ERR_INVALID_ARG;
    if (idx && mode != SMALL_POOL_MAX) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({in, out}, {idx})) return s;
    Geom g;
    if (int s = make_geom(g, N, C, C, H, W, FH, FW, stride, pt, pb, pl, pr)) return s;
    size_t in_b = sizeof(float) * packed_elems(N, C, H, W), out_b = sizeof(float) * packed_elems(N, C, g.OH, g.OW);
    if (ranges_overlap(in, in_b, out, out_b)) return SMALL_ERR_OVERLAP;
    if (idx && (ranges_overlap(in, in_b, idx, out_b) || ranges_overlap(out, out_b, idx, out_b))) return SMALL_ERR_OVERLAP;
    return launch_pool(ctx, in, out, idx, g, mode, static_cast<cudaStream_t>(stream));
}

SMALL_API int small_relu(small_ctx *ctx, const float *in, float *out, int N, int C, int H, int W, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (int s = check_ptrs({in, out})) return s;
    size_t n = packed_elems(N, C, H, W);
    if (n == 0) return SMALL_ERR_SHAPE;
    if (in != out && ranges_overlap(in, n * sizeof(float), out, n * sizeof(float))) return SMALL_ERR_OVERLAP;
    return launch_relu(ctx, in, out, n, static_cast<cudaStream_t>(stream));
}

SMALL_API int small_scale_shift(small_ctx *ctx, const float *in, const float *scale, const float *shift, float *out,
                                int N, int C, int H, int W, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~SMALL_RELU) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({in, out}, {})) return s;
    if (!scale || !shift) return SMALL_ERR_INVALID_ARG;
    size_t n = packed_elems(N, C, H, W);
    if (n == 0) return SMALL_ERR_SHAPE;
    if (in != out && ranges_overlap(in, n * sizeof(float), out, n * sizeof(float))) return SMALL_ERR_OVERLAP;
    return launch_scale_shift(ctx, in, scale, shift, out, N, C, H, W, flags & SMALL_RELU, static_cast<cudaStream_t>(stream));
}

SMALL_API int small_upsample_nearest(small_ctx *ctx, const float *in, float *out, int N, int C, int H, int W, int factor, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (int s = check_ptrs({in, out})) return s;
    if (factor < 1 || factor > 64) return SMALL_ERR_INVALID_ARG;
    size_t n = packed_elems(N, C, H, W);
    if (n == 0 || (long long)H * factor > 0x7fffffLL || (long long)W * factor > 0x7fffffLL) return SMALL_ERR_SHAPE;
    if (ranges_overlap(in, n * sizeof(float), out, n * sizeof(float) * factor * factor)) return SMALL_ERR_OVERLAP;
    return launch_upsample_nearest(ctx, in, out, N, C, H, W, factor, static_cast<cudaStream_t>(stream));
}

SMALL_API int small_add(small_ctx *ctx, const float *a, const float *b, float *out, int N, int C, int H, int W,
                        unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~SMALL_RELU) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({a, b, out})) return s;
    size_t n = packed_elems(N, C, H, W);
    if (n == 0) return SMALL_ERR_SHAPE;
    if (a != out && ranges_overlap(a, n * sizeof(float), out, n * sizeof(float))) return SMALL_ERR_OVERLAP;
    if (b != out && ranges_overlap(b, n * sizeof(float), out, n * sizeof(float))) return SMALL_ERR_OVERLAP;
    return launch_add(ctx, a, b, out, n, flags & SMALL_RELU, static_cast<cudaStream_t>(stream));
}

// Above this much work a full reduction under a tensor-core math mode runs on the tensor-core kernel as a 1x1
// convolution over a 1x1 plane (the images are the pixels); below it the CUDA-core kernel's 3 microseconds win over the
// tensor-core kernel's set-up (measured on the classifier heads and the autoencoder's layers).
static const double kFcTensorCoreFlops = 4e6;

SMALL_API int small_fc_uses_tensor_cores(int N, int J, int K, unsigned math) {
    if (math != SMALL_MATH_TF32 && math != SMALL_MATH_3XTF32) return 0;
    if (2.0 * N * J * K < kFcTensorCoreFlops) return 0;
    Geom g;
    if (make_geom(g, N, J, K, 1, 1, 1, 1, 1, 0, 0, 0, 0) != SMALL_OK) return 0;
    return conv_tc_supported(g, math == SMALL_MATH_3XTF32) ? 1 : 0;
}

SMALL_API int small_fc(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out,
                       int N, int J, int K, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~(SMALL_RELU | SMALL_MATH_MASK)) return SMALL_ERR_INVALID_ARG;
    const unsigned math = math_of(flags);
    if (!math_valid(math)) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({in, w, out}, {bias})) return s;
    if (N < 1 || J < 1 || K < 1 || (long long)N * blocks_of(J) > (1ll << 30) || (long long)N * blocks_of(K) > (1ll << 30)) return SMALL_ERR_SHAPE;
    if (ranges_overlap(in, sizeof(float) * packed_elems(N, J, 1, 1), out, sizeof(float) * packed_elems(N, K, 1, 1))) return SMALL_ERR_OVERLAP;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (small_fc_uses_tensor_cores(N, J, K, math) && (reinterpret_cast<uintptr_t>(out) & 31u) == 0 &&
        ctx->conv_path != SMALL_CONV_PATH_CUDA_CORES) {
        Geom g;
        make_geom(g, N, J, K, 1, 1, 1, 1, 1, 0, 0, 0, 0);
        const float *w_hi = w + conv_w_fp32_elems(J, K, 1, 1);
        const float *w_lo = w_hi + conv_w_tc_elems(J, K, 1, 1);
        return launch_conv_tc(ctx, in, w_hi, math == SMALL_MATH_3XTF32 ? w_lo : nullptr, bias, out, g, flags & SMALL_RELU, false, math, st);
    }
    return launch_fc(ctx, in, w, bias, out, N, J, K, flags & SMALL_RELU, st);
}

// ---- global average pool -> full reduction as one fused layer
SMALL_API int small_gap_fc_fused(int N, int C, int K, unsigned math) {
    if (N < 1 || C < 1 || K < 1 || !math_valid(math)) return 0;
    if ((size_t)blocks_of(C) * 32 * sizeof(float) > 40 * 1024) return 0;
    return small_fc_uses_tensor_cores(N, C, K, math) ? 0 : 1;       // large full reductions keep their tensor-core route
}

SMALL_API int small_gap_fc(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, float *scratch,
                           int N, int C, int H, int W, int K, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~(SMALL_RELU | SMALL_MATH_MASK)) return SMALL_ERR_INVALID_ARG;
    const unsigned math = math_of(flags);
    if (!math_valid(math)) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({in, w, out}, {bias, scratch})) return s;
    if (N < 1 || C < 1 || K < 1 || H < 1 || W < 1 || (long long)H * W > (1ll << 24) || (long long)N * blocks_of(C) > (1ll << 30) ||
        (long long)N * blocks_of(K) > (1ll << 30))
        return SMALL_ERR_SHAPE;
    const size_t in_b = sizeof(float) * packed_elems(N, C, H, W), out_b = sizeof(float) * packed_elems(N, K, 1, 1);
    if (ranges_overlap(in, in_b, out, out_b)) return SMALL_ERR_OVERLAP;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (small_gap_fc_fused(N, C, K, math))
        return launch_gap_fc(ctx, in, w, bias, out, N, C, H, W, K, flags & SMALL_RELU, st);
    // the two layers one after the other, through the caller's scratch tensor [N][C][1][1]
    if (!scratch) return SMALL_ERR_UNSUPPORTED;
    if (!aligned16(scratch)) return SMALL_ERR_ALIGN;
    const size_t mid_b = sizeof(float) * packed_elems(N, C, 1, 1);
    if (ranges_overlap(scratch, mid_b, in, in_b) || ranges_overlap(scratch, mid_b, out, out_b)) return SMALL_ERR_OVERLAP;
    if (int s = small_pool2d(ctx, in, scratch, nullptr, N, C, H, W, H, W, 1, 0, 0, 0, 0, SMALL_POOL_AVG, stream)) return s;
    return small_fc(ctx, scratch, w, bias, out, N, C, K, flags, stream);
}

// ---- a chain of full reductions as one fused kernel
SMALL_API int small_fc_chain_fused(const int *widths, int L, unsigned math) {
    if (!widths) return 0;
    return fc_chain_supported(widths, L, math) ? 1 : 0;
}

SMALL_API int small_fc_chain(small_ctx *ctx, const float *in, const float *const *w_blk, const float *const *bias, const int *widths,
                             const int *relu, float *out, float *scratch, int L, int N, unsigned flags, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (flags & ~SMALL_MATH_MASK) return SMALL_ERR_INVALID_ARG;
    const unsigned math = math_of(flags);
    if (!math_valid(math) || !w_blk || !widths || !relu || L < 1 || L > 64) return SMALL_ERR_INVALID_ARG;
    if (int s = check_ptrs({in, out}, {scratch})) return s;
    if (N < 1) return SMALL_ERR_SHAPE;
    int widest = 0;
    for (int i = 0; i <= L; ++i) {
        if (widths[i] < 1) return SMALL_ERR_SHAPE;
        if (i > 0 && i < L && widths[i] > widest) widest = widths[i];
    }
    for (int l = 0; l < L; ++l) {
        if (!w_blk[l]) return SMALL_ERR_INVALID_ARG;
        if (!aligned16(w_blk[l]) || (bias && bias[l] && !aligned16(bias[l]))) return SMALL_ERR_ALIGN;
    }
    const size_t in_b = sizeof(float) * packed_elems(N, widths[0], 1, 1), out_b = sizeof(float) * packed_elems(N, widths[L], 1, 1);
    if (ranges_overlap(in, in_b, out, out_b)) return SMALL_ERR_OVERLAP;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (fc_chain_supported(widths, L, math) && (reinterpret_cast<uintptr_t>(out) & 31u) == 0 && ctx->conv_path != SMALL_CONV_PATH_CUDA_CORES)
        return launch_fc_chain(ctx, in, w_blk, bias, widths, relu, out, L, N, math, st);
    // layer by layer, through the two halves of the caller's scratch tensor
    if (L == 1) return small_fc(ctx, in, w_blk[0], bias ? bias[0] : nullptr, out, N, widths[0], widths[1], (relu[0] ? SMALL_RELU : 0u) | math, stream);
    if (!scratch) return SMALL_ERR_WORKSPACE;
    const size_t half = packed_elems(N, widest, 1, 1);
    if (ranges_overlap(scratch, 2 * half * sizeof(float), in, in_b) || ranges_overlap(scratch, 2 * half * sizeof(float), out, out_b)) return SMALL_ERR_OVERLAP;
    const float *src = in;
    for (int l = 0; l < L; ++l) {
        float *dst = l == L - 1 ? out : scratch + (size_t)(l & 1) * half;
        if (int s = small_fc(ctx, src, w_blk[l], bias ? bias[l] : nullptr, dst, N, widths[l], widths[l + 1], (relu[l] ? SMALL_RELU : 0u) | math, stream)) return s;
        src = dst;
    }
    return SMALL_OK;
}
