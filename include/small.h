/*
 * small.h - C ABI of a B200 (sm_100a) implementation of the SMaLL layer set
 * (arXiv 2303.04769): one loop-nest family specialised per layer by its
 * dimensions, every layer reading and writing the same blocked-channel layout
 * so that no layer reformats data.
 *
 * GENERAL CONVENTIONS
 *
 * Blocked layout (paper Section 4.4, Figure 2).  An activation tensor with N
 * images, C channels and an H x W plane is stored as
 *     float[N][ceil(C / Cb)][H][W][Cb]          Cb = small_channel_block() = 32
 * channels fastest, then width, height, channel block, image.  Channels C ..
 * ceil(C/Cb)*Cb - 1 of the last block ("pad lanes") are +0.0f: small_pack writes
 * them so and every layer keeps them so.  Input and output of every layer use
 * this one layout (the paper's premise); only small_pack / small_unpack touch
 * NCHW.
 *
 * Pointers.  Unless a parameter says "host", every pointer is a DEVICE pointer
 * on the context's device, 16-byte aligned, to memory the CALLER owns and keeps
 * alive until the work queued on `stream` has finished.  The library allocates
 * no device memory in any layer call.  Input and output ranges must not overlap
 * unless the function says so.
 *
 * Streams and errors.  `stream` is a cudaStream_t passed as void* (NULL = the
 * default stream).  Calls only enqueue work.  Every function returns a
 * small_status; argument errors are found on the host before anything is
 * launched (nothing is enqueued when the result is not SMALL_OK).  A CUDA
 * launch failure gives SMALL_ERR_CUDA and keeps the CUDA code for
 * small_last_cuda_error().  Device-side pipeline waits are bounded; one that
 * runs out records SMALL_ERR_TIMEOUT in a status word read by
 * small_device_status().
 *
 * Layer parameters are the paper's (Section 3.1): input channels C (I_C),
 * filters / output channels K, plane H x W (I_H, I_W), window FH x FW (F_H,
 * F_W), one stride for both plane dimensions (S_H = S_W), plus explicit zero
 * padding on the four sides, which the paper leaves to the code around its
 * kernels (Section 4.2.1).  Output extent: O = floor((I + pad_a + pad_b - F) /
 * stride) + 1, which is Section 3.1.2's formula when the pads are zero.
 */
#ifndef SMALL_H
#define SMALL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct small_ctx small_ctx; /* opaque; one per device; not thread-safe */

typedef enum {
    SMALL_OK = 0,
    SMALL_ERR_INVALID_ARG = 1, /* NULL where a pointer is required, unknown flag or mode */
    SMALL_ERR_SHAPE = 2,       /* a dimension < 1, an empty output, pad >= window, size overflow */
    SMALL_ERR_ALIGN = 3,       /* a device pointer is not 16-byte aligned */
    SMALL_ERR_OVERLAP = 4,     /* input and output ranges overlap where that is not allowed */
    SMALL_ERR_WORKSPACE = 5,   /* workspace too small or a slot id out of range */
    SMALL_ERR_UNSUPPORTED = 6, /* valid request outside what the kernels cover */
    SMALL_ERR_CUDA = 7,        /* a CUDA runtime / driver call failed */
    SMALL_ERR_TIMEOUT = 8,     /* a bounded device-side wait ran out */
    SMALL_ERR_NOT_INIT = 9     /* ctx is NULL or was shut down */
} small_status;

/* flags for the weighted layers and small_add */
enum {
    SMALL_RELU = 1u,       /* out = max(out, 0) after bias (Table 2: ReLU = Max), fused in the epilogue */
    SMALL_ACCUMULATE = 2u, /* out = out_previous + result (+ bias): the LOAD phase of the paper's kernel
                              (Algorithm 2) picking up an existing partial result; used for residual joins */
    SMALL_MATH_FP32 = 0u << 4,   /* FP32 FMA on CUDA cores, FP32 accumulate */
    SMALL_MATH_TF32 = 1u << 4,   /* TF32 tensor-core products, FP32 accumulate */
    SMALL_MATH_3XTF32 = 2u << 4, /* three TF32 products per term (hi*hi + hi*lo + lo*hi), FP32 accumulate */
    SMALL_RELU_MID = 4u,   /* small_dwpw_conv2d only: max(x, 0) on the depthwise result, before the 1x1 convolution */
    SMALL_MATH_MASK = 3u << 4
};

enum { SMALL_POOL_MAX = 0, SMALL_POOL_AVG = 1 };

/* ---- context ------------------------------------------------------------------------------- */

/* Creates the context for CUDA device `device` (makes it current, loads the driver entry point
 * used to encode tensor maps, allocates a 256-byte device status block - the only device
 * allocation the library ever makes).  *ctx receives the handle.  Errors: INVALID_ARG, CUDA,
 * UNSUPPORTED (the device is not compute capability 10.x). */
int small_init(int device, small_ctx **ctx);
/* Frees the context.  Work still queued on any stream must have finished. */
int small_shutdown(small_ctx *ctx);
/* Cb, the channel block of the blocked layout (Section 4.4: a machine-specific parameter). 32 here:
 * one 128-byte line per pixel and block, the width of a warp and of the tensor-core swizzle row. */
int small_channel_block(void);
/* Number of floats of a blocked tensor: N * ceil(C/Cb)*Cb * H * W; 0 if a dimension is < 1. */
size_t small_packed_elems(int N, int C, int H, int W);
/* floor((I + pad_before + pad_after - F) / stride) + 1, or 0 when that window does not fit (Section 3.1.2). */
int small_out_size(int I, int F, int stride, int pad_before, int pad_after);
const char *small_strerror(int status);
/* Last cudaError_t / CUresult seen by this context (0 if none). */
int small_last_cuda_error(small_ctx *ctx);
/* Layer overlap inside small_run_net (on by default; `on` = 0 switches it off).  When on, every layer behind the
 * first is launched with programmatic stream serialisation: its thread blocks may become resident and set up shared
 * memory, barriers and tensor memory while the layer in front of it is still draining, and they wait on the device
 * until that layer has completed before they read or write a tensor.  Results are the same either way.  The paper
 * has no counterpart. */
int small_set_layer_overlap(small_ctx *ctx, int on);
/* Branch overlap inside small_run_net (on by default; `on` = 0 switches it off).  When on, two neighbouring layers of the
 * list that share no tensor except as readers - a residual stage's convolution and its shortcut convolution - run at the
 * same time: the second one on a stream of the context's own (created in small_init), forked from and joined to the
 * caller's stream by events, which a stream capture records as a fork and a join.  Results are the same either way.  The
 * paper has no counterpart (its layers are consecutive calls). */
int small_set_branch_overlap(small_ctx *ctx, int on);
/* Limit, in polls, of every bounded device-side wait (default 2^22: seconds, with the polls' back-off); at least 16.
 * A wait that runs out makes its kernel record SMALL_ERR_TIMEOUT, let its copies in flight land, free its tensor memory
 * and return; the affected outputs are undefined and later calls work normally.  The paper has no counterpart. */
int small_set_wait_limit(small_ctx *ctx, unsigned polls);
/* Runs the give-up-and-return path on purpose, harmlessly: one small kernel waits - with the context's limit and the wait
 * routine of the layer kernels - on a barrier that nothing arms (no copy is in flight), records SMALL_ERR_TIMEOUT and
 * returns.  Lower the limit first (a few hundred polls) or the call takes seconds.  small_device_status then reads
 * SMALL_ERR_TIMEOUT once and the context works as before. */
int small_selftest_wait_timeout(small_ctx *ctx, void *stream);
/* Kernel family of the full channel reductions under the tensor-core math modes.  AUTO (the default): per layer,
 * whichever of the tensor-core kernel and the register-tiled FP32 kernel is the faster one for its channel counts
 * (FP32 FMAs meet every mode's tolerance); layers of one channel block and at most 32 filters take the warp-level
 * tensor-core kernel.  TENSOR (the block-level tensor-core kernel) / CUDA_CORES / WARP_MMA force one family wherever it
 * takes the shape, GENERAL the general FP32 kernel (any window and stride) everywhere except the network stems.  For
 * measurements and comparisons; results stay within the mode's tolerance either way.  The paper has no counterpart. */
enum { SMALL_CONV_PATH_AUTO = 0, SMALL_CONV_PATH_TENSOR = 1, SMALL_CONV_PATH_CUDA_CORES = 2, SMALL_CONV_PATH_GENERAL = 3,
       SMALL_CONV_PATH_WARP_MMA = 4 };
int small_set_conv_path(small_ctx *ctx, int path);
/* Which kernel small_conv2d runs for this shape and math mode (with a 32-byte aligned output) under the context's
 * path setting: 0 = few-input-channel kernel (network stems), 1 = register-tiled FP32 kernel, 2 = general FP32 kernel,
 * 3 = block-level tensor-core kernel (tcgen05), 4 = warp-level tensor-core kernel (few channels and filters);
 * -1 for invalid arguments. */
int small_conv2d_path(small_ctx *ctx, int N, int C, int K, int H, int W, int FH, int FW, int stride,
                      int pad_t, int pad_b, int pad_l, int pad_r, unsigned math);
/* Synchronises `stream`, then reads and clears the device status word: *status is SMALL_OK or
 * SMALL_ERR_TIMEOUT (a tensor-core pipeline wait gave up; the affected outputs are undefined). */
int small_device_status(small_ctx *ctx, int *status, void *stream);

/* Measures the dense TF32 tensor-core rate of this device: every SM issues `iters` x 4 back-to-back
 * tcgen05.mma kind::tf32 of shape 128 x n x 8 (n = 32, 64, 128 or 256; iters a multiple of 8) on operands resident in
 * shared memory.
 * cycles_dev: device buffer of one 64-bit word per SM (receives each SM's cycle count).  *tflops: whole-device rate
 * from CUDA events; *cycles_per_mma: SM 0's cycles per MMA instruction.  Synchronises `stream`.  This is the
 * measured denominator of the tensor-bound rooflines (the paper has no counterpart: its kernels are CPU SIMD). */
int small_measure_tf32_peak(small_ctx *ctx, int n, int iters, long long *cycles_dev, double *tflops,
                            double *cycles_per_mma, void *stream);

/* ---- layout (Section 4.4) ------------------------------------------------------------------ */

/* NCHW float[N][C][H][W] -> blocked; pad lanes are written as +0.  Bit-exact move. */
int small_pack(small_ctx *ctx, const float *nchw, float *blk, int N, int C, int H, int W, void *stream);
/* blocked -> NCHW, dropping pad lanes.  Bit-exact move. */
int small_unpack(small_ctx *ctx, const float *blk, float *nchw, int N, int C, int H, int W, void *stream);

/* ---- filters: packed once, off the timed path (Section 4.4: the filter tensor has its own blocked
 * layout).  The packed layouts are private to the library; `math` is SMALL_MATH_FP32/TF32/3XTF32 and
 * decides which copies the packed buffer holds (FP32 always; TF32-rounded K-major tiles for the two
 * tensor-core modes; the low-order residual tiles for 3XTF32).  A layer call may use any math mode
 * whose copies the buffer holds, i.e. any mode <= the one it was packed for. */
size_t small_conv_weight_elems(int C, int K, int FH, int FW, unsigned math);
/* w_kcrs: device float[K][C][FH][FW].  w_blk: device, small_conv_weight_elems floats. */
int small_pack_conv_weights(small_ctx *ctx, const float *w_kcrs, float *w_blk, int C, int K, int FH, int FW,
                            unsigned math, void *stream);
/* Group convolution filters (Section 3.1.3: the filter tensor is F_H x F_W x F_C x K x G).
 * w_gkcrs: device float[G][K][F_C][FH][FW], G = small_group_count(C, F_C, S_C) (0 if the channel window does
 * not tile the channels: (C - F_C) must be a multiple of S_C). */
int small_group_count(int C, int F_C, int S_C);
size_t small_group_conv_weight_elems(int C, int F_C, int S_C, int K, int FH, int FW);
int small_pack_group_conv_weights(small_ctx *ctx, const float *w_gkcrs, float *w_blk, int C, int F_C, int S_C, int K,
                                  int FH, int FW, void *stream);
size_t small_dw_weight_elems(int C, int FH, int FW);
/* w_crs: device float[C][FH][FW] (one filter per channel: Table 1, single channel reduction). */
int small_pack_dw_weights(small_ctx *ctx, const float *w_crs, float *w_blk, int C, int FH, int FW, void *stream);
size_t small_fc_weight_elems(int J, int K, unsigned math);
/* w_kj: device float[K][J]. */
int small_pack_fc_weights(small_ctx *ctx, const float *w_kj, float *w_blk, int J, int K, unsigned math, void *stream);

/* ---- layers -------------------------------------------------------------------------------- */

/* Full channel reduction (Section 3.2 item 4; Table 1: F_C = I_C, K = O_C, G = 1): standard and 1x1
 * convolution, cross-correlation form, zero padding, with the bias / accumulate / ReLU epilogue:
 *   out[n,k,oh,ow] = [out[n,k,oh,ow] +] bias[k] + sum_{c,x,y} in[n,c,oh*s+x-pad_t,ow*s+y-pad_l] * w[k,c,x,y]
 * in: blocked [N][C][H][W]; out: blocked [N][K][OH][OW]; bias: K floats or NULL.
 * flags: SMALL_RELU | SMALL_ACCUMULATE | one SMALL_MATH_*.  The tensor-core modes apply to the shapes
 * small_conv2d_uses_tensor_cores accepts (stride 1 or 2, padded row within the kernel's tile, at most 64
 * taps in the stride-1 view of the window); any other shape runs the FP32 kernel (tighter accuracy, no
 * error).  3XTF32 needs roughly twice the shared memory per tile and falls back the same way where even
 * its smallest tile does not fit.  `out` must be 32-byte aligned for the tensor-core kernel (16 otherwise).
 * Layers of one channel block (C <= 32) with at most 32 filters (64 with a 1 x 1 window) run warp-level tensor-core
 * MMAs instead of the 128-row block-level ones, which such layers leave mostly empty; same modes, same tolerances.
 * Layers with at most four input channels and a 3 x 3 window (stride 1 or 2), or one channel and a 10 x 4
 * stride-2 window - the first layer of a network - run FP32 FMAs on the CUDA cores in every math mode (a reduction
 * of a few dozen terms is no dense contraction; the result meets each mode's tolerance).
 * Errors: NOT_INIT, INVALID_ARG, SHAPE (dims < 1, empty output, pad >= window), ALIGN, OVERLAP,
 * UNSUPPORTED (window so large that one input tile exceeds shared memory). */
int small_conv2d(small_ctx *ctx, const float *in, const float *w_blk, const float *bias, float *out,
                 int N, int C, int K, int H, int W, int FH, int FW, int stride,
                 int pad_t, int pad_b, int pad_l, int pad_r, unsigned flags, void *stream);
/* Partial channel reduction (Section 3.1.2, Figure 1; Table 1 "group convolution"): the window also slides over
 * the channels.  Group g = 0..G-1 reduces input channels g*S_C .. g*S_C + F_C - 1 with its own K filters and
 * writes output channels g*K .. g*K + K - 1 (O_C = K*G); S_C = F_C is the usual grouped convolution, S_C < F_C
 * gives overlapping groups, F_C = S_C = 1 with K = 1 is a depthwise convolution.  Same epilogue, flags, padding
 * and errors as small_conv2d; bias has K*G entries.  Under SMALL_MATH_TF32 / 3XTF32, groups that are whole channel
 * blocks (F_C = S_C a multiple of 32) with K a multiple of 32 (at most 256) run on the tensor-core kernel, one filter
 * tile per group; every other shape, and SMALL_MATH_FP32, runs the FP32 kernel. */
int small_group_conv2d(small_ctx *ctx, const float *in, const float *w_blk, const float *bias, float *out,
                       int N, int C, int F_C, int S_C, int K, int H, int W, int FH, int FW, int stride,
                       int pad_t, int pad_b, int pad_l, int pad_r, unsigned flags, void *stream);
/* Abstract fused layer (Section 6, future directions): depthwise 3x3 (+ dw_bias, + ReLU with SMALL_RELU_MID) followed
 * by a 1x1 convolution to K channels (+ pw_bias, + ReLU with SMALL_RELU), as one layer:
 *   out = act( pw( act_mid( dw(in) + dw_bias ) ) + pw_bias )
 * in: blocked [N][C][H][W]; out: blocked [N][K][OH][OW], OH/OW from the depthwise window (3x3, `stride`, the pads).
 * dw_w_blk from small_pack_dw_weights(C, 3, 3); pw_w_blk from small_pack_conv_weights(C, K, 1, 1, math).
 * Under SMALL_MATH_TF32 / 3XTF32, shapes small_dwpw_fused accepts run as ONE kernel: the depthwise result is computed
 * in shared memory and feeds the tensor cores without going to global memory.  Otherwise the two layers run one after
 * the other through `scratch` (device, small_packed_elems(N, C, OH, OW) floats; may be NULL when the fused kernel
 * runs - SMALL_ERR_WORKSPACE if it is needed and NULL).  Errors as small_conv2d. */
int small_dwpw_conv2d(small_ctx *ctx, const float *in, const float *dw_w_blk, const float *dw_bias,
                      const float *pw_w_blk, const float *pw_bias, float *out, float *scratch,
                      int N, int C, int K, int H, int W, int stride,
                      int pad_t, int pad_b, int pad_l, int pad_r, unsigned flags, void *stream);
/* 1 if small_dwpw_conv2d runs this shape as one fused kernel under the given tensor-core math mode, else 0. */
int small_dwpw_fused(int N, int C, int K, int H, int W, int stride, int pad_t, int pad_b, int pad_l, int pad_r, unsigned math);
/* Abstract fused layer (Section 6): convolution (+ bias, + ReLU with SMALL_RELU) followed by a 2 x 2 stride-2 max pool
 * (no padding; an odd last row or column is dropped, as Section 3.1.2's size rule says), as one layer:
 *   out[n,k,i,j] = max over the 2 x 2 block (2i.., 2j..) of act(conv(in)[n,k,.,.] + bias[k])
 * in: blocked [N][C][H][W]; out: blocked [N][K][OH/2][OW/2] with OH, OW the convolution's output size.  Shapes
 * small_conv_maxpool_fused accepts (windows 1 or 3 wide, stride 1 or 2, an even number of convolution rows per tile) run
 * as ONE kernel whose STORE phase pools in registers and by one warp shuffle, so the convolution's output never reaches
 * memory; it computes FP32 FMAs on the CUDA cores in every math mode (within each mode's tolerance).  Other shapes run the
 * two layers through `scratch` (device, small_packed_elems(N, K, OH, OW) floats; may be NULL when the fused kernel runs -
 * SMALL_ERR_WORKSPACE if it is needed and NULL).  flags: SMALL_RELU | one SMALL_MATH_*.  Errors as small_conv2d; SHAPE
 * also when the convolution's output has fewer than 2 rows or columns. */
int small_conv_maxpool2d(small_ctx *ctx, const float *in, const float *w_blk, const float *bias, float *out, float *scratch,
                         int N, int C, int K, int H, int W, int FH, int FW, int stride,
                         int pad_t, int pad_b, int pad_l, int pad_r, unsigned flags, void *stream);
/* 1 if small_conv_maxpool2d runs this shape as one fused kernel, else 0. */
int small_conv_maxpool_fused(int N, int C, int K, int H, int W, int FH, int FW, int stride, int pad_t, int pad_b, int pad_l, int pad_r);
/* 1 if small_conv2d would run this shape on the tensor cores under SMALL_MATH_TF32 (automatic path), else 0. */
int small_conv2d_uses_tensor_cores(int N, int C, int K, int H, int W, int FH, int FW, int stride,
                                   int pad_t, int pad_b, int pad_l, int pad_r);

/* Single channel reduction with weights (Section 3.2 item 2; Table 1: F_C = 1, K = 1, G = I_C):
 * depthwise convolution, one FH x FW filter per channel, + bias[c], optional ReLU.
 * flags: SMALL_RELU (a math mode is accepted and ignored: FP32 FMA; the layer is bandwidth-bound). */
int small_dwconv2d(small_ctx *ctx, const float *in, const float *w_blk, const float *bias, float *out,
                   int N, int C, int H, int W, int FH, int FW, int stride,
                   int pad_t, int pad_b, int pad_l, int pad_r, unsigned flags, void *stream);

/* Single channel reduction without weights: max or average pooling (Section 3.2 item 2; Table 2).
 * Padded positions are ignored (never the max; excluded from the mean's sum and count).
 * Max: the window is scanned row by row and the first maximum wins; idx (NULL, or a blocked int32 tensor
 * of the output's shape, max mode only) receives ih*W + iw of the winner.  Pad lanes: value 0, index 0. */
int small_pool2d(small_ctx *ctx, const float *in, float *out, int32_t *idx,
                 int N, int C, int H, int W, int FH, int FW, int stride,
                 int pad_t, int pad_b, int pad_l, int pad_r, int mode, void *stream);

/* Single element reduction (Section 3.2 item 1; Table 2: ReLU = Max): out = in > 0 ? in : +0.
 * out may equal in (in place); any other overlap is an error. */
int small_relu(small_ctx *ctx, const float *in, float *out, int N, int C, int H, int W, void *stream);

/* Batch normalisation at inference (Table 2: a single element layer whose operation is FMA):
 *   out[n,c,h,w] = scale[c] * in[n,c,h,w] + shift[c]   (then max(., 0) with SMALL_RELU)
 * scale, shift: device, C floats each (gamma / sqrt(var + eps) and beta - mean * that, folded by the caller).
 * in, out: blocked [N][C][H][W]; out may be the same buffer as in; pad lanes are written as +0. */
int small_scale_shift(small_ctx *ctx, const float *in, const float *scale, const float *shift, float *out,
                      int N, int C, int H, int W, unsigned flags, void *stream);
/* Upsample (Table 2: nearest neighbour interpolation) by an integer factor in both plane dimensions:
 *   out[n,c,oh,ow] = in[n,c,oh / factor,ow / factor];  out: blocked [N][C][H*factor][W*factor].  Bit-exact move. */
int small_upsample_nearest(small_ctx *ctx, const float *in, float *out, int N, int C, int H, int W, int factor, void *stream);
/* Single element reduction "addition" (Section 3.2 item 1): out = a + b, then ReLU if SMALL_RELU.
 * out may equal a or b. */
int small_add(small_ctx *ctx, const float *a, const float *b, float *out, int N, int C, int H, int W,
              unsigned flags, void *stream);

/* Full reduction (Section 3.2 item 5; Table 1 row 5): out[n,k] = bias[k] + sum_j in[n,j] * w[k,j].
 * in: blocked [N][J][1][1]; out: blocked [N][K][1][1].  (A full reduction over an H x W plane is
 * small_conv2d with FH = H, FW = W, as long as that window fits the kernel's shared-memory tile.)
 * flags: SMALL_RELU | one SMALL_MATH_*.  Under a tensor-core math mode (with filters packed for it) a layer of 4 MFLOP
 * or more runs on the tensor-core kernel as a 1x1 convolution whose pixels are the images; smaller ones (classifier
 * heads) and SMALL_MATH_FP32 run FP32 FMAs on the CUDA cores. */
int small_fc(small_ctx *ctx, const float *in, const float *w_blk, const float *bias, float *out,
             int N, int J, int K, unsigned flags, void *stream);

/* Abstract fused layer (Section 6, "abstract fused layer"): a global average pool - the single channel reduction of
 * Section 3.2 item 2 over the whole H x W plane, Average in place of Max - and the full reduction (item 5) behind
 * it, the classifier head of the paper's networks, as one kernel:
 *   out[n,k] = bias[k] + sum_c w[k,c] * mean_{h,w} in[n,c,h,w]      (the mean rounded to float as the pooling layer stores it)
 * in: blocked [N][C][H][W]; w_blk: small_pack_fc_weights(J = C, K); out: blocked [N][K][1][1]; flags: SMALL_RELU | one
 * SMALL_MATH_* (FP32 FMAs on the CUDA cores in every mode: a classifier head is far below the size at which small_fc
 * takes the tensor cores).  Where small_gap_fc_fused says 0 (a full reduction large enough for the tensor-core route)
 * the two layers run one after the other through `scratch`, a blocked [N][C][1][1] tensor the caller provides (NULL:
 * UNSUPPORTED for such shapes).  Errors: NOT_INIT, INVALID_ARG, SHAPE, ALIGN, OVERLAP, UNSUPPORTED. */
int small_gap_fc(small_ctx *ctx, const float *in, const float *w_blk, const float *bias, float *out, float *scratch,
                 int N, int C, int H, int W, int K, unsigned flags, void *stream);
/* 1 if small_gap_fc runs this shape as one fused kernel, else 0. */
int small_gap_fc_fused(int N, int C, int K, unsigned math);

/* ---- quantised inference (Section 5.1: "quantized to integer (unsigned 8 bit)"; Section 5.3: uint8 values, int32
 * accumulation; Section 5.5) -------------------------------------------------------------------------------------
 * The same blocked layout with one byte per channel: uint8[N][ceil(C/32)][H][W][32], pad lanes 0.  A tensor's real
 * value is scale * (q - zero_point), one (scale, zero_point) per tensor; the paper fixes only the types, the affine
 * form and the rounding below are this library's reading.  A weighted layer is exact integer arithmetic:
 *     acc   = bias[k] + sum (q_in - z_in) * (q_w - z_w)                      (int32; padding = real zeros = z_in)
 *     q_out = clamp(z_out + floor((acc * mult + 2^(shift-1)) / 2^shift), lo, 255)        (64-bit product, one rounding)
 * mult / 2^shift (0 <= mult < 2^31, 1 <= shift <= 62) stands for scale_in * scale_w / scale_out; bias: int32 in
 * units of scale_in * scale_w, or NULL; lo = z_out with SMALL_RELU (the only flag), else 0.  C * FH * FW must not
 * exceed 33000 so that the sums stay inside 32 bits (SMALL_ERR_SHAPE).  Results are bit-exact against that
 * definition.  Errors otherwise as the float layers. */
size_t small_q_packed_bytes(int N, int C, int H, int W);      /* bytes of a blocked uint8 tensor */
/* NCHW uint8[N][C][H][W] <-> blocked; byte moves. */
int small_q_pack(small_ctx *ctx, const uint8_t *nchw, uint8_t *blk, int N, int C, int H, int W, void *stream);
int small_q_unpack(small_ctx *ctx, const uint8_t *blk, uint8_t *nchw, int N, int C, int H, int W, void *stream);
size_t small_q_conv_weight_bytes(int C, int K, int FH, int FW);
/* w_kcrs: device uint8[K][C][FH][FW]; w_blk: device, 16-byte aligned, small_q_conv_weight_bytes bytes (private layout). */
int small_q_pack_conv_weights(small_ctx *ctx, const uint8_t *w_kcrs, void *w_blk, int C, int K, int FH, int FW, void *stream);
/* Full channel reduction on uint8 (Table 1 row 4): standard and 1x1 convolution; with H = W = FH = FW = 1 a fully
 * connected layer.  Windows 1 or 3 wide of any height, stride 1 or 2, any padding (else SMALL_ERR_UNSUPPORTED). */
int small_q_conv2d(small_ctx *ctx, const uint8_t *in, const void *w_blk, const int32_t *bias, uint8_t *out,
                   int N, int C, int K, int H, int W, int FH, int FW, int stride,
                   int pad_t, int pad_b, int pad_l, int pad_r,
                   int z_in, int z_w, int z_out, int mult, int shift, unsigned flags, void *stream);
size_t small_q_dw_weight_bytes(int C, int FH, int FW);
/* w_crs: device uint8[C][FH][FW]. */
int small_q_pack_dw_weights(small_ctx *ctx, const uint8_t *w_crs, uint8_t *w_blk, int C, int FH, int FW, void *stream);
/* Single channel reduction with weights on uint8 (Table 1 row 2): depthwise convolution, any window and stride. */
int small_q_dwconv2d(small_ctx *ctx, const uint8_t *in, const uint8_t *w_blk, const int32_t *bias, uint8_t *out,
                     int N, int C, int H, int W, int FH, int FW, int stride,
                     int pad_t, int pad_b, int pad_l, int pad_r,
                     int z_in, int z_w, int z_out, int mult, int shift, unsigned flags, void *stream);
/* Max pooling on uint8 (Table 2: Max): the maximum of the bytes (the affine map keeps order); padded positions are
 * ignored, a window wholly in the padding gives z (the tensor's zero point). */
int small_q_maxpool2d(small_ctx *ctx, const uint8_t *in, uint8_t *out, int N, int C, int H, int W, int FH, int FW,
                      int stride, int pad_t, int pad_b, int pad_l, int pad_r, int z, void *stream);
/* ReLU on uint8 (Table 2: Max with zero): out = max(in, z), real zero being the zero point z.  out may equal in. */
int small_q_relu(small_ctx *ctx, const uint8_t *in, uint8_t *out, int N, int C, int H, int W, int z, void *stream);

/* Abstract fused layer (Section 6) for a chain of full reductions, out = f_L(... f_1(in)), f_i(x) = act_i(W_i x + b_i):
 * widths[0 .. L] are the channel counts (layer i maps widths[i] to widths[i+1]); w_blk[i] from small_pack_fc_weights(widths[i],
 * widths[i+1], math); bias: NULL or L pointers (each NULL or widths[i+1] floats); relu[i] != 0 applies max(., 0) after layer i.
 * in: blocked [N][widths[0]][1][1]; out: blocked [N][widths[L]][1][1], 32-byte aligned for the fused kernel.  flags: one
 * SMALL_MATH_*.  Chains small_fc_chain_fused accepts (2 to 12 layers; widths[1 .. L-1] at most 128, widths[0] at most 8192,
 * widths[L] at most 1024; a tensor-core math mode) run as ONE kernel: a thread block keeps a tile of images' activations in shared
 * memory as the tensor cores' operand from the first layer to the last, streams the filters (and the first layer's input
 * where it is wider than 128), and writes only the final result.  Any other chain runs small_fc layer by layer
 * through `scratch` (device, 2 * small_packed_elems(N, widest inner width, 1, 1) floats; may be NULL when the fused kernel runs
 * or L == 1 - SMALL_ERR_WORKSPACE if it is needed and NULL).  All arrays are HOST arrays.  Errors as small_fc. */
int small_fc_chain(small_ctx *ctx, const float *in, const float *const *w_blk, const float *const *bias, const int *widths,
                   const int *relu, float *out, float *scratch, int L, int N, unsigned flags, void *stream);
/* Images per thread block of the fused kernel: 0 (default) chooses by batch size - 32 while that gives every SM at most
 * one tile, then 64, then 128 (larger tiles stream the filters fewer times, smaller ones occupy more SMs); 32, 64 or 128
 * force one (a tile whose shared memory does not fit - a wide first layer with the larger tiles - is halved).
 * SMALL_ERR_INVALID_ARG for any other value.  Results do not depend on the choice. */
int small_set_fc_chain_tile(small_ctx *ctx, int images);
/* 1 if small_fc_chain runs this chain as one fused kernel under the given math mode, else 0. */
int small_fc_chain_fused(const int *widths, int L, unsigned math);
/* 1 if small_fc runs this layer on the tensor cores under the given math mode, else 0. */
int small_fc_uses_tensor_cores(int N, int J, int K, unsigned math);

/* ---- networks (Section 5.3: layers share intermediate buffers; Section 5.4: end-to-end inference) -- */

enum { SMALL_OP_CONV = 0, SMALL_OP_DWCONV = 1, SMALL_OP_POOL = 2, SMALL_OP_RELU = 3, SMALL_OP_ADD = 4, SMALL_OP_FC = 5,
       SMALL_OP_DWPW = 6,     /* depthwise 3x3 then 1x1 convolution as one fused layer (small_dwpw_conv2d) */
       SMALL_OP_CONVPOOL = 7 }; /* convolution then 2x2 stride-2 max pool as one fused layer (small_conv_maxpool2d); the shape
                                 * must be one small_conv_maxpool_fused accepts */
enum { SMALL_SLOT_INPUT = -1, SMALL_SLOT_OUTPUT = -2 }; /* the caller's in_blk / out_blk */

typedef struct small_layer {
    int op;                 /* SMALL_OP_* */
    int C, K;               /* input / output channels (K ignored for DWCONV, POOL, RELU, ADD; C = J for FC) */
    int H, W;               /* input plane (1 x 1 for FC) */
    int FH, FW, stride;     /* window and stride (CONV, DWCONV, POOL) */
    int pad_t, pad_b, pad_l, pad_r;
    unsigned flags;         /* SMALL_RELU | SMALL_ACCUMULATE | SMALL_MATH_* as the op allows; DWPW: RELU, RELU_MID and a
                             * tensor-core math mode - the shape must be one small_dwpw_fused accepts */
    int pool_mode;          /* SMALL_POOL_* */
    const float *w_blk;     /* packed filters (device) or NULL */
    const float *bias;      /* device or NULL */
    int src, dst;           /* slot ids >= 0, or SMALL_SLOT_INPUT / SMALL_SLOT_OUTPUT */
    int src2;               /* second operand of ADD; ignored otherwise */
    const float *w_blk2;    /* DWPW: packed 1x1 filters (w_blk, bias are the depthwise layer's); else ignored */
    const float *bias2;     /* DWPW: bias of the 1x1 convolution or NULL */
} small_layer;

/* Abstract fused layers (Section 6) inside small_run_net.  The caller describes plain layers; the runner itself runs
 * two neighbouring layers as one fused layer when the first one's result is read by the second one only (no later layer
 * reads that slot before it is written again), the pair's output slot differs from its input slot, and the fused kernel
 * takes the shape: a depthwise 3x3 and the 1x1 convolution behind it under a tensor-core math mode (SMALL_FUSE_DWPW: only
 * where the intermediate tensor is at most 24 MB, where fusing was measured to pay; SMALL_FUSE_DWPW_ALWAYS: wherever the
 * kernel takes the shape), a convolution and the 2x2 stride-2 max pool behind it (SMALL_FUSE_CONVPOOL), and a run of 2 to 12
 * full reductions whose inner widths are at most 128 under a tensor-core math mode (SMALL_FUSE_FC_CHAIN, see small_fc_chain), and
 * a global average pool with the full reduction behind it, in every math mode (SMALL_FUSE_POOLFC, see small_gap_fc).  The skipped
 * intermediate tensors are then not written.  Default: all four (without DWPW_ALWAYS); 0 runs every layer on its own.
 * Results stay within each math mode's tolerance either way. */
enum { SMALL_FUSE_DWPW = 1u, SMALL_FUSE_DWPW_ALWAYS = 2u, SMALL_FUSE_CONVPOOL = 4u, SMALL_FUSE_FC_CHAIN = 8u,
       SMALL_FUSE_POOLFC = 16u };   /* a global average pool and the full reduction behind it (small_gap_fc) */
int small_set_net_fusion(small_ctx *ctx, unsigned mask);
/* Number of kernel launches small_run_net makes for these layers at batch N under the context's fusion setting (one per
 * layer or fused pair); -1 for invalid arguments. */
int small_net_launches(small_ctx *ctx, const small_layer *layers, int n_layers, int N);
/* Bytes of workspace for `layers` at batch N: slot s is as large as the largest tensor any layer reads
 * from or writes to it, rounded up to 256 bytes; slots are laid out back to back.  0 on invalid input. */
size_t small_net_workspace_bytes(const small_layer *layers, int n_layers, int N);
/* Runs the layers in order on `stream`.  layers: HOST array.  in_blk: blocked network input (read by
 * layers whose src is SMALL_SLOT_INPUT); out_blk: receives what is written to SMALL_SLOT_OUTPUT.
 * workspace: device, 256-byte aligned.  No data is reformatted between layers.  Every layer is
 * validated before the first launch. */
int small_run_net(small_ctx *ctx, const small_layer *layers, int n_layers, int N,
                  const float *in_blk, float *out_blk, void *workspace, size_t workspace_bytes, void *stream);

/* Extra device bytes small_run_net_host needs beyond small_net_workspace_bytes: staging for the NCHW
 * input (twice) and output and their blocked forms. */
size_t small_net_host_staging_bytes(int N, int C, int H, int W, int outC, int outH, int outW);
/* End-to-end convenience: in_nchw_host (HOST, float[N][C][H][W]) is copied to the device, packed, run
 * through the layers, unpacked and copied to out_nchw_host (HOST, float[N][outC][outH][outW]).  Pinned
 * host memory makes the copies asynchronous.  workspace: device, 256-byte aligned, at least
 * small_net_workspace_bytes + small_net_host_staging_bytes.  Returns after enqueuing; synchronise
 * `stream` before reading the result, and keep in_nchw_host unchanged until then.
 * The input copy runs on a stream of the context's own into one of two staging areas of the workspace, so that with
 * back-to-back calls on one workspace the copy of a call's input overlaps the layers of the call before it; the caller's
 * stream waits for the copy by an event.  (While `stream` is being captured the copy stays on `stream`.) */
int small_run_net_host(small_ctx *ctx, const small_layer *layers, int n_layers, int N,
                       const float *in_nchw_host, int C, int H, int W,
                       float *out_nchw_host, int outC, int outH, int outW,
                       void *workspace, size_t workspace_bytes, void *stream);

/* ---- for callers that cannot allocate device memory (the paper has no counterpart to this entry point) ---- */

/* Size in bytes (32 MiB) of the workspace array built into the library image.  A GPU holds that much device memory
 * from small_init on that device (which loads the library's device code and looks the array up) until the process
 * exits. */
size_t small_static_workspace_bytes(void);
/* small_run_net with the intermediate buffers taken from that built-in array instead of a caller workspace, for
 * callers that have no device memory to give and may not allocate any: a process whose device memory is handed
 * to another allocator after start-up, or a request path on which an allocation's possible device-wide
 * synchronisation is not acceptable.  The call allocates nothing (no cudaMalloc / cudaFree, no allocating library
 * routine); the array's memory is taken earlier, when small_init loads the library on the device, so create the
 * context before the device's memory is given away, and before any stream capture.  (The first launch of a kernel
 * variant may still make the driver load that kernel's code; run the network once through either entry point
 * beforehand if even that must stay off the request path.)  The caller still passes the blocked input and output.
 * Arguments, validation and results are those of small_run_net.  Extra errors: SMALL_ERR_WORKSPACE when
 * small_net_workspace_bytes(layers, n_layers, N) exceeds small_static_workspace_bytes() (nothing is launched; use
 * small_run_net with your own workspace, or a smaller batch); SMALL_ERR_INVALID_ARG when the current CUDA device
 * is not the context's device.
 * Sharing: all calls on a device use the same array, and it keeps what the last call left there.  No call
 * depends on that content (each layer overwrites its whole output before it is read), but two calls whose work
 * overlaps on the GPU - different streams, or one stream per thread - race on the array: order them, e.g. by
 * issuing them on one stream. */
int small_run_net_static(small_ctx *ctx, const small_layer *layers, int n_layers, int N,
                         const float *in_blk, float *out_blk, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SMALL_H */
