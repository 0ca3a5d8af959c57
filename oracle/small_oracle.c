/*
 * CPU oracle for the SMaLL layer definitions (arXiv 2303.04769).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what each
 * layer computes.  It is used by the tests, by the smoke check and by the
 * benchmark's CPU-baseline leg, and by nothing else; the CUDA library neither
 * includes nor links it and shares no code with it.
 *
 * Conventions: tensors are dense NCHW float32 (the "natural" layout, before the
 * paper's blocked layout of Section 4.4 is applied); filters are [K][C][FH][FW];
 * every sum is carried in double and rounded to float once; bias is added in
 * double before that rounding; ReLU follows the rounding.  Padding (which the
 * paper leaves to "code surrounding the kernels", Section 4.2.1) is read as
 * zero padding for the FMA layers and as "ignored positions" for pooling.
 *
 * Two independent statements of the arithmetic live here on purpose:
 *   - so_conv2d / so_dwconv2d / so_pool2d / so_relu / so_scale_shift / so_upsample_nearest / so_fc: the per-output
 *     definitions of Section 3.2 (classes of layers);
 *   - so_abstract_layer: the abstract layer of Section 3.1 itself, element by element, for any
 *     (F_H, F_W, F_C, S_H, S_W, S_C, K, G) - the one definition that Table 1 specialises into the classes.
 * The tests check each against the other, and both against brute force,
 * library routines and closed forms.
 *
 *   - so_q_*: the quantised (uint8 data, int32 accumulation) forms of the same definitions; the requantisation
 *     step is a reading of this build (the paper fixes only the types), stated above so_requantize.
 *
 * Parity unpinned: nothing (every exported routine has at least one pin in
 * tests/test_oracle_*.py).  Accuracy of trained networks is not computed here.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define SO_EXPORT __attribute__((visibility("default")))

/* ---- Section 3.1.2: output extent of a sliding window, with floor division and explicit pads.
 * With both pads zero this is the paper's O = (I - F) / S + 1. */
SO_EXPORT int so_out_size(int I, int F, int S, int pad_before, int pad_after) {
    int span = I + pad_before + pad_after - F;
    if (I < 1 || F < 1 || S < 1 || span < 0) return 0;
    return span / S + 1;
}

/* "same" padding: O = ceil(I / S); the total pad is what the last window needs, the smaller half first. */
SO_EXPORT void so_same_pad(int I, int F, int S, int *O, int *before, int *after) {
    int o = (I + S - 1) / S;
    int total = (o - 1) * S + F - I;
    if (total < 0) total = 0;
    *O = o;
    *before = total / 2;
    *after = total - total / 2;
}

/* Section 3.1.2: number of groups produced by sliding the window over channels, and O_C = K * G. */
SO_EXPORT int so_groups(int I_C, int F_C, int S_C) { return (I_C - F_C) / S_C + 1; }
SO_EXPORT int so_out_channels(int K, int G) { return K * G; }

/* Section 5.3: float model memory = 4 bytes x (parameters + largest input/output buffer pair + model input). */
SO_EXPORT double so_model_memory_mib(long params, long largest_in_out_pair, long model_input) {
    return 4.0 * (double)(params + largest_in_out_pair + model_input) / 1048576.0;
}

/* ---- Section 4.4 / Figure 2: blocked layout.  Fastest to slowest: Cb channels, width, height,
 * channel blocks; the batch is the added outermost dimension (Section 3.1.1). */
SO_EXPORT long so_blk_index(int n, int c, int h, int w, int C, int H, int W, int Cb) {
    long blocks = (C + Cb - 1) / Cb;
    long blk = c / Cb, lane = c % Cb;
    return ((((long)n * blocks + blk) * H + h) * W + w) * Cb + lane;
}

SO_EXPORT long so_blk_elems(int N, int C, int H, int W, int Cb) {
    long blocks = (C + Cb - 1) / Cb;
    return (long)N * blocks * Cb * H * W;
}

SO_EXPORT void so_pack(const float *nchw, float *blk, int N, int C, int H, int W, int Cb) {
    long total = so_blk_elems(N, C, H, W, Cb);
    for (long i = 0; i < total; ++i) blk[i] = 0.0f; /* pad lanes hold +0 */
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w)
                    blk[so_blk_index(n, c, h, w, C, H, W, Cb)] = nchw[(((long)n * C + c) * H + h) * W + w];
}

SO_EXPORT void so_unpack(const float *blk, float *nchw, int N, int C, int H, int W, int Cb) {
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int h = 0; h < H; ++h)
                for (int w = 0; w < W; ++w)
                    nchw[(((long)n * C + c) * H + h) * W + w] = blk[so_blk_index(n, c, h, w, C, H, W, Cb)];
}

static inline float so_finish(double acc, int relu) {
    float r = (float)acc;
    if (relu) r = r > 0.0f ? r : 0.0f;
    return r;
}

/* ---- Full channel reduction (Section 3.2 item 4, Table 1 row 4): convolution, incl. 1x1.
 * out[n,k,oh,ow] = bias[k] + sum_{c,x,y} in[n,c,oh*S+x-pt,ow*S+y-pl] * w[k,c,x,y]  (no filter flip);
 * reads outside the plane are 0.  accumulate != 0 adds the previous content of out (the kernel's
 * LOAD phase of Algorithm 2 picking up an existing partial result). */
SO_EXPORT void so_conv2d(const float *in, const float *w, const float *bias, float *out,
                         int N, int C, int K, int H, int W, int FH, int FW, int S,
                         int pt, int pb, int pl, int pr, int relu, int accumulate) {
    int OH = so_out_size(H, FH, S, pt, pb), OW = so_out_size(W, FW, S, pl, pr);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k)
            for (int oh = 0; oh < OH; ++oh)
                for (int ow = 0; ow < OW; ++ow) {
                    double acc = bias ? (double)bias[k] : 0.0;
                    for (int c = 0; c < C; ++c)
                        for (int x = 0; x < FH; ++x) {
                            int ih = oh * S + x - pt;
                            if (ih < 0 || ih >= H) continue;
                            for (int y = 0; y < FW; ++y) {
                                int iw = ow * S + y - pl;
                                if (iw < 0 || iw >= W) continue;
                                acc += (double)in[(((long)n * C + c) * H + ih) * W + iw] *
                                       (double)w[(((long)k * C + c) * FH + x) * FW + y];
                            }
                        }
                    long o = (((long)n * K + k) * OH + oh) * OW + ow;
                    if (accumulate) acc += (double)out[o];
                    out[o] = so_finish(acc, relu);
                }
}

/* Same sums with a float accumulator, in the same loop order: only used to report a second CPU timing. */
SO_EXPORT void so_conv2d_f32acc(const float *in, const float *w, const float *bias, float *out,
                                int N, int C, int K, int H, int W, int FH, int FW, int S,
                                int pt, int pb, int pl, int pr, int relu, int accumulate) {
    int OH = so_out_size(H, FH, S, pt, pb), OW = so_out_size(W, FW, S, pl, pr);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k)
            for (int oh = 0; oh < OH; ++oh)
                for (int ow = 0; ow < OW; ++ow) {
                    float acc = bias ? bias[k] : 0.0f;
                    for (int c = 0; c < C; ++c)
                        for (int x = 0; x < FH; ++x) {
                            int ih = oh * S + x - pt;
                            if (ih < 0 || ih >= H) continue;
                            for (int y = 0; y < FW; ++y) {
                                int iw = ow * S + y - pl;
                                if (iw < 0 || iw >= W) continue;
                                acc += in[(((long)n * C + c) * H + ih) * W + iw] *
                                       w[(((long)k * C + c) * FH + x) * FW + y];
                            }
                        }
                    long o = (((long)n * K + k) * OH + oh) * OW + ow;
                    if (accumulate) acc += out[o];
                    out[o] = so_finish((double)acc, relu);
                }
}

/* ---- Single channel reduction with weights (Section 3.2 item 2; Table 1 row 2: F_C = 1, K = 1,
 * G = I_C): depthwise convolution, one FHxFW filter per channel, w is [C][FH][FW]. */
SO_EXPORT void so_dwconv2d(const float *in, const float *w, const float *bias, float *out,
                           int N, int C, int H, int W, int FH, int FW, int S,
                           int pt, int pb, int pl, int pr, int relu) {
    int OH = so_out_size(H, FH, S, pt, pb), OW = so_out_size(W, FW, S, pl, pr);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int oh = 0; oh < OH; ++oh)
                for (int ow = 0; ow < OW; ++ow) {
                    double acc = bias ? (double)bias[c] : 0.0;
                    for (int x = 0; x < FH; ++x) {
                        int ih = oh * S + x - pt;
                        if (ih < 0 || ih >= H) continue;
                        for (int y = 0; y < FW; ++y) {
                            int iw = ow * S + y - pl;
                            if (iw < 0 || iw >= W) continue;
                            acc += (double)in[(((long)n * C + c) * H + ih) * W + iw] *
                                   (double)w[((long)c * FH + x) * FW + y];
                        }
                    }
                    out[(((long)n * C + c) * OH + oh) * OW + ow] = so_finish(acc, relu);
                }
}

/* ---- Single channel reduction without weights: pooling.  mode 0 = max, 1 = average.
 * Max: the window is scanned row by row and a later element replaces the best only when strictly
 * greater, so the first maximum wins; idx (optional) receives ih*W+iw of the winner.  Padded
 * positions never take part: they cannot win the max and are left out of the mean's sum and count. */
SO_EXPORT void so_pool2d(const float *in, float *out, int32_t *idx,
                         int N, int C, int H, int W, int FH, int FW, int S,
                         int pt, int pb, int pl, int pr, int mode) {
    int OH = so_out_size(H, FH, S, pt, pb), OW = so_out_size(W, FW, S, pl, pr);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c) {
            const float *plane = in + ((long)n * C + c) * H * W;
            for (int oh = 0; oh < OH; ++oh)
                for (int ow = 0; ow < OW; ++ow) {
                    long o = (((long)n * C + c) * OH + oh) * OW + ow;
                    int have = 0, best_i = -1, count = 0;
                    float best = 0.0f;
                    double sum = 0.0;
                    for (int x = 0; x < FH; ++x) {
                        int ih = oh * S + x - pt;
                        if (ih < 0 || ih >= H) continue;
                        for (int y = 0; y < FW; ++y) {
                            int iw = ow * S + y - pl;
                            if (iw < 0 || iw >= W) continue;
                            float v = plane[(long)ih * W + iw];
                            if (!have || v > best) { best = v; best_i = ih * W + iw; have = 1; }
                            sum += (double)v;
                            ++count;
                        }
                    }
                    if (mode == 0) {
                        out[o] = have ? best : 0.0f;
                        if (idx) idx[o] = best_i;
                    } else {
                        out[o] = count ? (float)(sum / (double)count) : 0.0f;
                    }
                }
        }
}

/* ---- Single element reductions (Section 3.2 item 1): ReLU = Max with zero (Table 2); addition. */
SO_EXPORT void so_relu(const float *in, float *out, long n) {
    for (long i = 0; i < n; ++i) out[i] = in[i] > 0.0f ? in[i] : 0.0f;
}

SO_EXPORT void so_add(const float *a, const float *b, float *out, long n, int relu) {
    for (long i = 0; i < n; ++i) out[i] = so_finish((double)a[i] + (double)b[i], relu);
}

/* Batch normalisation at inference (Table 2: single element, FMA): one multiply-add per element with the channel's
 * scale and shift, out = scale[c] * in + shift[c].  NCHW. */
SO_EXPORT void so_scale_shift(const float *in, const float *scale, const float *shift, float *out,
                              int N, int C, int H, int W, int relu) {
    long plane = (long)H * W;
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (long i = 0; i < plane; ++i) {
                long at = ((long)n * C + c) * plane + i;
                out[at] = so_finish((double)scale[c] * (double)in[at] + (double)shift[c], relu);
            }
}

/* Upsample (Table 2: nearest neighbour interpolation): every input element is repeated f x f times,
 * out[n][c][oh][ow] = in[n][c][oh / f][ow / f], out is [N][C][H*f][W*f]. */
SO_EXPORT void so_upsample_nearest(const float *in, float *out, int N, int C, int H, int W, int f) {
    long OH = (long)H * f, OW = (long)W * f;
    for (long nc = 0; nc < (long)N * C; ++nc)
        for (long oh = 0; oh < OH; ++oh)
            for (long ow = 0; ow < OW; ++ow)
                out[(nc * OH + oh) * OW + ow] = in[(nc * H + oh / f) * W + ow / f];
}

/* ---- Full reduction (Section 3.2 item 5): the flattened input [N][J] times a J x K filter bank,
 * stored as w[K][J] with J in (c, h, w) order. */
SO_EXPORT void so_fc(const float *in, const float *w, const float *bias, float *out,
                     int N, int J, int K, int relu) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            double acc = bias ? (double)bias[k] : 0.0;
            for (int j = 0; j < J; ++j) acc += (double)in[(long)n * J + j] * (double)w[(long)k * J + j];
            out[(long)n * K + k] = so_finish(acc, relu);
        }
}

/* ---- The abstract layer of Section 3.1, for one image, element by element.
 *
 * Section 3.1.2: a window of F_H x F_W x F_C input elements slides with strides S_H, S_W over the plane and S_C over
 * the channels, which gives G = (I_C - F_C)/S_C + 1 channel positions ("groups") and O_H x O_W plane positions; at
 * every position K filters are applied, so O_C = K*G.  Output element (g*K + k, oh, ow) is the reduction of the input
 * window whose corner is (g*S_C, oh*S_H, ow*S_W) - with the matching elements of filter W[g][k] when the reduction
 * is a sum of products (Section 3.1.3: the filter tensor is F_H x F_W x F_C x K x G; stored here as
 * [G][K][F_C][F_H][F_W]).  Table 1 gives the layer classes as settings of (F_H, F_W, F_C, K, G) and Table 2 the
 * reduction of each layer: op 0 = sum of products (FMA), op 1 = maximum (W unused, may be NULL).  No padding: this is
 * the paper's definition as printed.  `init` is what the reduction starts from (0 for sums, -inf for max pooling, 0
 * for ReLU).  The sum is carried in double and rounded once. */
SO_EXPORT int so_abstract_layer(const float *in, const float *w, float *out,
                                int I_C, int I_H, int I_W,
                                int F_H, int F_W, int F_C, int S_H, int S_W, int S_C, int K,
                                int op, double init) {
    if (F_C < 1 || S_C < 1 || I_C < F_C || (I_C - F_C) % S_C != 0 || K < 1) return -1;
    int G = so_groups(I_C, F_C, S_C);
    int O_H = so_out_size(I_H, F_H, S_H, 0, 0), O_W = so_out_size(I_W, F_W, S_W, 0, 0);
    if (O_H < 1 || O_W < 1 || G < 1) return -1;
    if (op == 0 && !w) return -1;
    for (int g = 0; g < G; ++g)
        for (int k = 0; k < K; ++k)
            for (int oh = 0; oh < O_H; ++oh)
                for (int ow = 0; ow < O_W; ++ow) {
                    double r = init;
                    for (int c = 0; c < F_C; ++c)
                        for (int x = 0; x < F_H; ++x)
                            for (int y = 0; y < F_W; ++y) {
                                double v = (double)in[((long)(g * S_C + c) * I_H + (oh * S_H + x)) * I_W + (ow * S_W + y)];
                                if (op == 0) r += v * (double)w[((((long)g * K + k) * F_C + c) * F_H + x) * F_W + y];
                                else if (v > r) r = v;
                            }
                    out[((long)(g * K + k) * O_H + oh) * O_W + ow] = (float)r;
                }
    return 0;
}

/* ======================================================================================================
 * Quantised inference (Section 5.1: "quantized to integer (unsigned 8 bit)"; Section 5.3: "input and output values
 * are uint8, accumulations to the partial result are in int32"; Section 5.5).  The paper fixes the types and says
 * no more; the reading taken here is the usual affine one: a tensor's real value is scale * (q - zero_point), with
 * one (scale, zero_point) per tensor.  A layer then is exact integer arithmetic:
 *     acc  = bias[k] + sum (q_in - z_in) * (q_w - z_w)                       (int32; padded positions are real zeros,
 *                                                                             i.e. q_in = z_in: they add nothing)
 *     q_out = clamp(z_out + round_half_up(acc * mult / 2^shift), lo, 255)    (one rounding; 64-bit product)
 * where mult / 2^shift (0 <= mult < 2^31, 1 <= shift <= 62) stands for scale_in * scale_w / scale_out and bias is in
 * units of scale_in * scale_w; lo = z_out when ReLU is fused (real 0 maps to z_out), else 0.
 * round_half_up(a / 2^s) = floor((a + 2^(s-1)) / 2^s): an arithmetic right shift after the addition. */
SO_EXPORT int so_requantize(int acc, int mult, int shift, int z_out, int lo) {
    int64_t prod = (int64_t)acc * (int64_t)mult;
    int64_t r = (prod + ((int64_t)1 << (shift - 1))) >> shift;      /* >> of a negative value: arithmetic (gcc) */
    int64_t q = (int64_t)z_out + r;
    if (q < lo) q = lo;
    if (q > 255) q = 255;
    return (int)q;
}

/* Full channel reduction on uint8 (Table 1 row 4), NCHW, filters [K][C][FH][FW] uint8, bias int32 (or NULL). */
SO_EXPORT void so_q_conv2d(const uint8_t *in, const uint8_t *w, const int32_t *bias, uint8_t *out,
                           int N, int C, int K, int H, int W, int FH, int FW, int S,
                           int pt, int pb, int pl, int pr,
                           int z_in, int z_w, int z_out, int mult, int shift, int relu) {
    int OH = so_out_size(H, FH, S, pt, pb), OW = so_out_size(W, FW, S, pl, pr);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k)
            for (int oh = 0; oh < OH; ++oh)
                for (int ow = 0; ow < OW; ++ow) {
                    int32_t acc = bias ? bias[k] : 0;
                    for (int c = 0; c < C; ++c)
                        for (int x = 0; x < FH; ++x) {
                            int ih = oh * S + x - pt;
                            if (ih < 0 || ih >= H) continue;
                            for (int y = 0; y < FW; ++y) {
                                int iw = ow * S + y - pl;
                                if (iw < 0 || iw >= W) continue;
                                acc += ((int32_t)in[(((long)n * C + c) * H + ih) * W + iw] - z_in) *
                                       ((int32_t)w[(((long)k * C + c) * FH + x) * FW + y] - z_w);
                            }
                        }
                    out[(((long)n * K + k) * OH + oh) * OW + ow] = (uint8_t)so_requantize(acc, mult, shift, z_out, relu ? z_out : 0);
                }
}

/* Single channel reduction with weights on uint8 (Table 1 row 2): depthwise, filters [C][FH][FW]. */
SO_EXPORT void so_q_dwconv2d(const uint8_t *in, const uint8_t *w, const int32_t *bias, uint8_t *out,
                             int N, int C, int H, int W, int FH, int FW, int S,
                             int pt, int pb, int pl, int pr,
                             int z_in, int z_w, int z_out, int mult, int shift, int relu) {
    int OH = so_out_size(H, FH, S, pt, pb), OW = so_out_size(W, FW, S, pl, pr);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < C; ++c)
            for (int oh = 0; oh < OH; ++oh)
                for (int ow = 0; ow < OW; ++ow) {
                    int32_t acc = bias ? bias[c] : 0;
                    for (int x = 0; x < FH; ++x) {
                        int ih = oh * S + x - pt;
                        if (ih < 0 || ih >= H) continue;
                        for (int y = 0; y < FW; ++y) {
                            int iw = ow * S + y - pl;
                            if (iw < 0 || iw >= W) continue;
                            acc += ((int32_t)in[(((long)n * C + c) * H + ih) * W + iw] - z_in) *
                                   ((int32_t)w[((long)c * FH + x) * FW + y] - z_w);
                        }
                    }
                    out[(((long)n * C + c) * OH + oh) * OW + ow] = (uint8_t)so_requantize(acc, mult, shift, z_out, relu ? z_out : 0);
                }
}

/* Max pooling on uint8 (Table 2: Max): order-preserving under the affine map, so it is the maximum of the bytes;
 * padded positions are ignored; a window that lies wholly in the pad gives the zero point. */
SO_EXPORT void so_q_maxpool2d(const uint8_t *in, uint8_t *out, int N, int C, int H, int W, int FH, int FW, int S,
                              int pt, int pb, int pl, int pr, int z) {
    int OH = so_out_size(H, FH, S, pt, pb), OW = so_out_size(W, FW, S, pl, pr);
    for (long nc = 0; nc < (long)N * C; ++nc)
        for (int oh = 0; oh < OH; ++oh)
            for (int ow = 0; ow < OW; ++ow) {
                int best = -1;
                for (int x = 0; x < FH; ++x) {
                    int ih = oh * S + x - pt;
                    if (ih < 0 || ih >= H) continue;
                    for (int y = 0; y < FW; ++y) {
                        int iw = ow * S + y - pl;
                        if (iw < 0 || iw >= W) continue;
                        int v = in[(nc * H + ih) * W + iw];
                        if (v > best) best = v;
                    }
                }
                out[(nc * OH + oh) * OW + ow] = (uint8_t)(best < 0 ? z : best);
            }
}

/* ReLU on uint8 (Table 2: Max with zero): real 0 is the zero point. */
SO_EXPORT void so_q_relu(const uint8_t *in, uint8_t *out, long n, int z) {
    for (long i = 0; i < n; ++i) out[i] = in[i] > z ? in[i] : (uint8_t)z;
}

/* Section 5.3, quantised models: parameters + intermediates (one byte each) + 4 bytes x the largest H x W plane of
 * any intermediate (the int32 accumulators), in MiB. */
SO_EXPORT double so_model_memory_q_mib(long params, long intermediates, long largest_plane) {
    return ((double)params + (double)intermediates + 4.0 * (double)largest_plane) / 1048576.0;
}

SO_EXPORT int so_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
