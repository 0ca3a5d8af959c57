// Shared host-side declarations of the library: context, launch checks, argument validation.
#pragma once

#include <cuda_runtime.h>
#include <cstddef>
#include <cstdint>

#include "small.h"

#define SMALL_CB 32          // channel block of the blocked layout (floats): one 128-byte line
#define SMALL_API extern "C" __attribute__((visibility("default")))

struct small_ctx {
    int device;
    int last_cuda;           // last cudaError_t / CUresult seen
    int *dev_status;         // device status word (timeouts of bounded waits)
    void *encode_tiled;      // cuTensorMapEncodeTiled, resolved through the runtime
    int sm_count;
    size_t max_smem_optin;
    int overlap;             // small_run_net launches every layer after the first as a dependent launch (see launch_kernel)
    int dependent;           // set by small_run_net while it issues those layers
    unsigned wait_iters;     // limit (polls) of every bounded device-side wait; small_set_wait_limit
    void *tc_cache;          // finished launches of the tensor-core kernel by (shape, mode, tensors); conv_tc.cu
    void *mma_cache;         // the same for the warp-level tensor-core kernel; conv_mma.cu
    void *static_workspace;  // device address of the library's built-in workspace array on this device (net_static.cu)
    int branch_overlap;      // small_run_net runs independent neighbouring layers side by side (side stream)
    void *side_stream, *ev_fork, *ev_join;   // cudaStream_t / cudaEvent_t of that
    void *copy_stream, *ev_h2d[2], *ev_pack[2];   // small_run_net_host: input copies on their own stream, two staging areas
    void *host_ws; int host_parity, host_used[2];
    unsigned net_fusion;     // SMALL_FUSE_*: which neighbouring layers small_run_net runs as one fused layer
    int conv_path;           // SMALL_CONV_PATH_*: automatic, or one kernel family forced where it takes the shape
    int fc_chain_tile;       // images per thread block of the fused chain of full reductions: 0 = by batch size, else 32, 64 or 128
};

namespace small {

static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
static inline int blocks_of(int C) { return (C + SMALL_CB - 1) / SMALL_CB; }
static inline size_t packed_elems(int N, int C, int H, int W) {
    if (N < 1 || C < 1 || H < 1 || W < 1) return 0;
    return (size_t)N * blocks_of(C) * SMALL_CB * (size_t)H * W;
}
static inline int out_size(int I, int F, int S, int pa, int pb) {
    if (I < 1 || F < 1 || S < 1) return 0;
    int span = I + pa + pb - F;
    if (span < 0) return 0;
    return span / S + 1;
}
static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline bool ranges_overlap(const void *a, size_t na, const void *b, size_t nb) {
    uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + nb && b0 < a0 + na;
}
static inline int check_launch(small_ctx *ctx) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    return SMALL_OK;
}

// Dependent launches.  Every layer kernel of this library executes grid_dep_sync() before its first access to global
// memory that an earlier kernel of the stream may have written (or may still read), and nothing it does before that
// touches such memory; it also executes grid_dep_trigger().  A kernel launched with programmatic stream serialisation
// may therefore start while the kernel in front of it in the stream is still draining: its blocks become resident as
// that kernel's blocks leave, set up their shared memory, barriers and tensor memory, and then wait at
// grid_dep_sync() until the earlier kernel has completed and its writes are visible.  Launched the ordinary way,
// both instructions do nothing.  Chains stay ordered: a kernel cannot complete before its own grid_dep_sync()
// returns, so completion of kernel i implies completion of every kernel before it.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dep_sync() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline void launch_kernel(small_ctx *ctx, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->dependent ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
    (void)e;   // picked up by check_launch through cudaGetLastError
}
#endif

// Geometry of one windowed layer, validated once on the host and passed to kernels by value.
struct Geom {
    int N, C, K, H, W, FH, FW, S, pt, pb, pl, pr, OH, OW;
    int CB, KB;   // channel blocks of input and output
};

// Fills g and returns SMALL_OK, or the status that describes what is wrong.
int make_geom(Geom &g, int N, int C, int K, int H, int W, int FH, int FW, int S, int pt, int pb, int pl, int pr);

void free_tc_cache(small_ctx *);             // conv_tc.cu
void free_mma_cache(small_ctx *);            // conv_mma.cu
int resolve_static_workspace(small_ctx *);   // net_static.cu; called by small_init with the context's device current

// ---- kernel launchers (each in its own .cu); all return a small_status ----
int launch_pack(small_ctx *, const float *nchw, float *blk, int N, int C, int H, int W, cudaStream_t);
int launch_unpack(small_ctx *, const float *blk, float *nchw, int N, int C, int H, int W, cudaStream_t);
int launch_pack_conv_weights(small_ctx *, const float *w, float *wb, int C, int K, int FH, int FW, unsigned math, cudaStream_t);
int launch_pack_dw_weights(small_ctx *, const float *w, float *wb, int C, int FH, int FW, cudaStream_t);
int launch_relu(small_ctx *, const float *in, float *out, size_t n, cudaStream_t);
int launch_add(small_ctx *, const float *a, const float *b, float *out, size_t n, bool relu, cudaStream_t);
int launch_scale_shift(small_ctx *, const float *in, const float *scale, const float *shift, float *out, int N, int C, int H, int W,
                       bool relu, cudaStream_t);
int launch_upsample_nearest(small_ctx *, const float *in, float *out, int N, int C, int H, int W, int f, cudaStream_t);
int launch_pool(small_ctx *, const float *in, float *out, int32_t *idx, const Geom &, int mode, cudaStream_t);
int launch_dwconv(small_ctx *, const float *in, const float *w, const float *bias, float *out, const Geom &, bool relu, cudaStream_t);
int launch_fc(small_ctx *, const float *in, const float *w, const float *bias, float *out, int N, int J, int K, bool relu, cudaStream_t);
// global average pool over the H x W plane and the full reduction behind it as one kernel; w as launch_fc takes it
int launch_gap_fc(small_ctx *, const float *in, const float *w, const float *bias, float *out, int N, int C, int H, int W, int K,
                  bool relu, cudaStream_t);
// span > 0: group convolution - filter block kb reads `span` channel blocks from that of its first group on
// (Kg filters per group, groups S_C channels apart); span = 0: full reduction over all channel blocks
int launch_conv_fp32(small_ctx *, const float *in, const float *w, const float *bias, float *out, const Geom &,
                     bool relu, bool accumulate, cudaStream_t, int span = 0, int Kg = 0, int S_C = 0);
// register-tiled FP32 kernel: windows 1 or 3 wide, strides 1 and 2 (group convolutions as launch_conv_fp32 takes them)
bool conv_direct_supported(const Geom &, int span = 0, int Kg = 0, int S_C = 0);
long long conv_direct_blocks(const Geom &);     // thread blocks its plan launches (0: shape not taken)
int launch_conv_direct(small_ctx *, const float *in, const float *w, const float *bias, float *out, const Geom &,
                       bool relu, bool accumulate, cudaStream_t, int span = 0, int Kg = 0, int S_C = 0);
// the same kernel with a 2 x 2 stride-2 max pool taken in its STORE phase: out is [N][K][OH/2][OW/2]
bool conv_direct_pool_supported(const Geom &);
int launch_conv_direct_pool(small_ctx *, const float *in, const float *w, const float *bias, float *out, const Geom &, bool relu, cudaStream_t);
// a run of 2 to 8 full reductions of width <= 128 as one tensor-core kernel (fc_chain.cu); widths has L + 1 entries
bool fc_chain_supported(const int *widths, int L, unsigned math);
int launch_fc_chain(small_ctx *, const float *in, const float *const *w_blk, const float *const *bias, const int *widths,
                    const int *relu, float *out, int L, int N, unsigned math, cudaStream_t);
// at most four input channels, 3 x 3 (strides 1, 2) or the 10 x 4 stride-2 window: FP32 FMAs with the filters in registers
bool conv_thin_supported(const Geom &);
// nchw_in: `in` is the NCHW tensor float[N][C][H][W] instead of the blocked one (used at a network's edge)
int launch_conv_thin(small_ctx *, const float *in, const float *w, const float *bias, float *out, const Geom &,
                     bool relu, bool accumulate, cudaStream_t, bool nchw_in = false);
int group_conv_span(int C, int F_C, int S_C, int Kg);      // channel blocks a filter block of a group convolution needs
int launch_pack_group_conv_weights(small_ctx *, const float *w, float *wb, int C, int F_C, int S_C, int Kg, int FH, int FW, cudaStream_t);
// tensor-core implicit GEMM; mode is SMALL_MATH_TF32 or SMALL_MATH_3XTF32
// x3: with the doubled stages of 3xTF32.  groups > 1: a group convolution whose groups are whole channel blocks; the
// Geom then holds one group's channels (C = F_C) and all filters (K = groups x filters per group).
// A depthwise 3x3 fused in front of a 1x1 convolution: the Geom given to the two functions below is the 1x1 layer over
// the depthwise output (H = W = that output's size); this describes the depthwise layer and its input.
struct DwFuse { const float *w; const float *bias; int C, H, W, s, pt, pl, relu; };
bool conv_tc_supported(const Geom &, bool x3 = false, int groups = 1, const DwFuse *dw = nullptr);
int launch_conv_tc(small_ctx *, const float *in, const float *w_hi, const float *w_lo, const float *bias, float *out,
                   const Geom &, bool relu, bool accumulate, unsigned mode, cudaStream_t, int groups = 1, const DwFuse *dw = nullptr);
// warp-level tensor-core kernel (conv_mma.cu): one channel block, filters in tiles of 32, strides 1 and 2; reads the same
// filter sections as launch_conv_tc
bool conv_mma_supported(const Geom &, bool x3);
int launch_conv_mma(small_ctx *, const float *in, const float *w_hi, const float *w_lo, const float *bias, float *out,
                    const Geom &, bool relu, bool accumulate, unsigned mode, cudaStream_t);
// tensor-core filter sections of a group convolution: [F_C/32][FH*FW][G*K][32 ci], TF32 part and residual
size_t group_conv_w_tc_elems(int F_C, int K, int G, int FH, int FW);
int launch_pack_group_conv_weights_tc(small_ctx *, const float *w, float *hi, float *lo, int F_C, int K, int G, int FH, int FW, cudaStream_t);

// Sizes (in floats) of the sections of a packed convolution filter buffer.
size_t conv_w_fp32_elems(int C, int K, int FH, int FW);   // [KB][CB][FH][FW][32 ci][32 ko]
size_t conv_w_tc_elems(int C, int K, int FH, int FW);     // [CB][FH*FW][KB*32][32 ci]

}  // namespace small
