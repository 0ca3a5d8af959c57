// Full channel reduction for layers with at most four input channels (paper Section 3.2 item 4 with a very small
// F_C: the first layer of a network, whose input is an image or a spectrogram).  Such a layer is not a dense
// contraction: its reduction is F_H x F_W x C = 27 or 40 terms, a 32-channel block of the layout holds one to four
// real channels, and a tensor-core K step would carry seven or more zeros for every real product.  It runs on the
// CUDA cores instead, specialised at compile time by (C, F_H, F_W, stride) the way the paper specialises its kernels
// by layer dimensions (Section 4.2):
//   * the filters of a thread's one or two output channels (lane = output channel, as in the other kernels) live in
//     registers for the whole kernel: C x F_H x F_W x KPT values;
//   * the real channels of the input tile are copied into shared memory as dense planes [image][channel][row][column]
//     (one 16-byte read per pixel instead of its 128-byte line), zero padded;
//   * a warp computes PIX adjacent output pixels of one row for its 32 (or 64) filters: per window row it reads the
//     (PIX - 1) S + F_W inputs it needs as 8-byte shared-memory broadcasts and issues PIX x F_W x KPT FMAs on them.
// Bias, accumulate (the residual join), ReLU and the zero pad lanes are handled as in the other convolution kernels.
#include "common.cuh"

namespace small {

namespace {

struct ThinArgs {
    const float *in; const float *w; const float *bias; float *out;
    int N, K, KB, H, W, OH, OW, pt, pl;
    int nb, TH, bands, groups, kgroups;      // images and output rows per tile; tiles per image; column groups; filter groups
    int rows, pitch, plane;                  // shared tile: rows x pitch floats per (image, channel); plane = rows * pitch
    long long tiles;
    bool relu, accumulate;
    bool nchw;                               // the input is the NCHW tensor float[N][C][H][W] itself (the network's edge)
    bool half;                               // at most 16 filters: the two halves of a warp take different items (see the kernel)
};

// Threads per block: four warps.  A block loads a tile, then computes on it, with nothing in flight meanwhile, so
// memory-level parallelism comes from many small blocks per SM being at different points of that cycle.
constexpr int kThinThreads = 128;

template <int C, int FH, int FW, int S, int PIX, int KPT>
__global__ void __launch_bounds__(kThinThreads) conv_thin_kernel(const ThinArgs a) {
    extern __shared__ __align__(16) float tile[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int SEG = (PIX - 1) * S + FW, SEG2 = (SEG + 1) / 2;

    // With at most 16 filters, lanes 16-31 would hold pad filters: the half-warps then hold the same 16 filters and work
    // on different items, `fl` being a lane's filter and `sub` its half (measured: 3 -> 16 stem at batch 256 21.9 us before).
    const int fl = a.half ? (lane & 15) : lane, sub = a.half ? (lane >> 4) : 0, halves = a.half ? 2 : 1;
    // filters of this lane's output channels (the filter group is fixed per CTA: blockIdx.y): [kb][0][x][y][ci][ko]
    const int kg = blockIdx.y;
    float wr[C][FH][FW][KPT];
#pragma unroll
    for (int kp = 0; kp < KPT; ++kp) {
        const int kb = kg * KPT + kp;
#pragma unroll
        for (int x = 0; x < FH; ++x)
#pragma unroll
            for (int y = 0; y < FW; ++y)
#pragma unroll
                for (int c = 0; c < C; ++c)
                    wr[c][x][y][kp] = kb < a.KB ? __ldg(a.w + ((((size_t)kb * FH + x) * FW + y) * 32 + c) * 32 + fl) : 0.0f;
    }
    float bv[KPT];
#pragma unroll
    for (int kp = 0; kp < KPT; ++kp) {
        const int k = (kg * KPT + kp) * 32 + fl;
        bv[kp] = (a.bias && k < a.K) ? a.bias[k] : 0.0f;
    }
    grid_dep_sync();       // filters and bias are the layer's own constants; the tensors come next
    grid_dep_trigger();

    for (long long t = blockIdx.x; t < a.tiles; t += gridDim.x) {
        const int band = (int)(t % a.bands);
        const int n0 = (int)(t / a.bands) * a.nb;
        const int imgs = min(a.nb, a.N - n0);
        const int oh0 = band * a.TH;
        const int th = min(a.TH, a.OH - oh0);
        const int ih0 = oh0 * S - a.pt;
        const int rows = (th - 1) * S + FH;
        __syncthreads();                       // the previous tile is no longer read
        // four pixels per thread and step: the loads are issued together, then stored, so that a thread has four
        // lines in flight instead of one
        const int total = imgs * rows * a.pitch;
        for (int e0 = threadIdx.x; e0 < total; e0 += 4 * kThinThreads) {
            float4 v[4];
            int at[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int e = e0 + u * kThinThreads;
                v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                at[u] = -1;
                if (e < total) {
                    const int img = e / (rows * a.pitch), rc = e - img * rows * a.pitch;
                    const int r = rc / a.pitch, c = rc - r * a.pitch;
                    const int gh = ih0 + r, gw = c - a.pl;
                    at[u] = img * C * a.plane + r * a.pitch + c;
                    if (gh >= 0 && gh < a.H && gw >= 0 && gw < a.W) {
                        if (a.nchw) {       // planes of the NCHW tensor: the same values land at the same places of the tile
                            const size_t hw = (size_t)a.H * a.W;
                            const float *p = a.in + ((size_t)(n0 + img) * C * a.H + gh) * a.W + gw;
                            v[u].x = __ldg(p);
                            if (C > 1) v[u].y = __ldg(p + hw);
                            if (C > 2) v[u].z = __ldg(p + 2 * hw);
                            if (C > 3) v[u].w = __ldg(p + 3 * hw);
                        } else {
                            const float *p = a.in + (((size_t)(n0 + img) * a.H + gh) * a.W + gw) * 32;    // one channel block
                            if (C == 1) v[u].x = __ldg(p); else v[u] = __ldg(reinterpret_cast<const float4 *>(p));
                        }
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (at[u] < 0) continue;
                float *dst = tile + at[u];
                dst[0] = v[u].x;
                if (C > 1) dst[a.plane] = v[u].y;
                if (C > 2) dst[2 * a.plane] = v[u].z;
                if (C > 3) dst[3 * a.plane] = v[u].w;
            }
        }
        __syncthreads();
        const int items = imgs * th * a.groups;              // (image, output row, column group)
        for (int it = warp * halves + sub; it < items; it += halves * (kThinThreads / 32)) {
            const int img = it / (th * a.groups), rg = it - img * th * a.groups;
            const int r = rg / a.groups, cg = rg - r * a.groups;
            float acc[PIX][KPT];
#pragma unroll
            for (int p = 0; p < PIX; ++p)
#pragma unroll
                for (int kp = 0; kp < KPT; ++kp) acc[p][kp] = 0.0f;
#pragma unroll
            for (int c = 0; c < C; ++c) {
#pragma unroll
                for (int x = 0; x < FH; ++x) {
                    // (PIX - 1) S + FW inputs of this window row; the start is an even number of floats by construction
                    const float2 *rowp = reinterpret_cast<const float2 *>(tile + ((size_t)img * C + c) * a.plane + (r * S + x) * a.pitch + cg * PIX * S);
                    float seg[2 * SEG2];
#pragma unroll
                    for (int i = 0; i < SEG2; ++i) { const float2 v = rowp[i]; seg[2 * i] = v.x; seg[2 * i + 1] = v.y; }
#pragma unroll
                    for (int y = 0; y < FW; ++y)
#pragma unroll
                        for (int p = 0; p < PIX; ++p)
#pragma unroll
                            for (int kp = 0; kp < KPT; ++kp) acc[p][kp] = fmaf(seg[p * S + y], wr[c][x][y][kp], acc[p][kp]);
                }
            }
            const int oh = oh0 + r, ow0 = cg * PIX;
#pragma unroll
            for (int kp = 0; kp < KPT; ++kp) {
                const int kb = kg * KPT + kp;
                if (kb >= a.KB) break;
                const bool real = kb * 32 + fl < a.K;             // pad lanes of the last filter block stay +0
                float *dst = a.out + ((((size_t)(n0 + img) * a.KB + kb) * a.OH + oh) * a.OW + ow0) * 32 + fl;
#pragma unroll
                for (int p = 0; p < PIX; ++p) {
                    if (ow0 + p < a.OW) {
                        float v = acc[p][kp] + bv[kp];
                        if (a.accumulate) v += dst[p * 32];
                        if (a.relu) v = v > 0.f ? v : 0.f;
                        dst[p * 32] = real ? v : 0.0f;
                        if (a.half) dst[p * 32 + 16] = 0.0f;      // the line's other 16 lanes
                    }
                }
            }
        }
    }
}

typedef void (*ThinKernel)(const ThinArgs);

template <int C, int FH, int FW, int S, int PIX>
ThinKernel pick_kpt(int kpt) { return kpt == 1 ? conv_thin_kernel<C, FH, FW, S, PIX, 1> : conv_thin_kernel<C, FH, FW, S, PIX, 2>; }

template <int FH, int FW, int S, int PIX>
ThinKernel pick_c(int C, int kpt) {
    switch (C) {
        case 1: return pick_kpt<1, FH, FW, S, PIX>(kpt);
        case 2: return pick_kpt<2, FH, FW, S, PIX>(kpt);
        case 3: return pick_kpt<3, FH, FW, S, PIX>(kpt);
        case 4: return pick_kpt<4, FH, FW, S, PIX>(kpt);
        default: return nullptr;
    }
}

// The compiled specialisations: 3 x 3 windows at strides 1 and 2 for one to four channels, and the 10 x 4 stride-2
// window of a one-channel spectrogram.  PIX = 5 serves planes five outputs wide (stride 2 keeps its reads aligned).
ThinKernel pick_thin(const Geom &g, int pix, int kpt) {
    if (g.FH == 3 && g.FW == 3 && g.S == 1 && pix == 8) return pick_c<3, 3, 1, 8>(g.C, kpt);
    if (g.FH == 3 && g.FW == 3 && g.S == 2 && pix == 8) return pick_c<3, 3, 2, 8>(g.C, kpt);
    if (g.FH == 10 && g.FW == 4 && g.S == 2 && g.C == 1) return pix == 5 ? pick_kpt<1, 10, 4, 2, 5>(kpt) : pick_kpt<1, 10, 4, 2, 8>(kpt);
    return nullptr;
}

int thin_pix(const Geom &g) {
    // five outputs per warp when that wastes fewer lanes of work than eight (stride 2 only: 8-byte aligned reads)
    if (g.S == 2 && g.FH == 10 && ceil_div(g.OW, 5) * 5 < ceil_div(g.OW, 8) * 8) return 5;
    return 8;
}

}  // namespace

bool conv_thin_supported(const Geom &g) {
    if (g.C > 4 || g.CB != 1) return false;
    if (!pick_thin(g, thin_pix(g), 1)) return false;
    const int pix = thin_pix(g), groups = ceil_div(g.OW, pix);
    const int seg2 = ((pix - 1) * g.S + g.FW + 1) / 2;
    int pitch = (groups - 1) * pix * g.S + 2 * seg2;
    if (pitch < g.W + g.pl) pitch = g.W + g.pl;
    pitch = (pitch + 1) & ~1;
    // at least one output row of one image must fit the shared tile
    return (size_t)g.C * g.FH * pitch * sizeof(float) <= 40 * 1024;
}

int launch_conv_thin(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, const Geom &g,
                     bool relu, bool accumulate, cudaStream_t st, bool nchw_in) {
    if (!conv_thin_supported(g)) return SMALL_ERR_UNSUPPORTED;
    ThinArgs a{};
    a.in = in; a.w = w; a.bias = bias; a.out = out;
    a.N = g.N; a.K = g.K; a.KB = g.KB; a.H = g.H; a.W = g.W; a.OH = g.OH; a.OW = g.OW; a.pt = g.pt; a.pl = g.pl;
    a.relu = relu; a.accumulate = accumulate; a.nchw = nchw_in;
    a.half = g.K <= 16;
    const int pix = thin_pix(g);
    const int kpt = g.KB >= 2 ? 2 : 1;
    a.groups = ceil_div(g.OW, pix);
    a.kgroups = ceil_div(g.KB, kpt);
    const int seg2 = ((pix - 1) * g.S + g.FW + 1) / 2;
    a.pitch = (a.groups - 1) * pix * g.S + 2 * seg2;          // the last column group's reads stay inside the row
    if (a.pitch < g.W + g.pl) a.pitch = g.W + g.pl;
    a.pitch = (a.pitch + 1) & ~1;
    const ThinKernel kern = pick_thin(g, pix, kpt);
    if (!kern) return SMALL_ERR_UNSUPPORTED;
    const size_t budget = 40 * 1024;
    auto tile_bytes = [&](int nb, int th) { return (size_t)nb * g.C * ((th - 1) * g.S + g.FH) * a.pitch * sizeof(float); };
    // CTAs that run at once: the grid is that many (or fewer), each walking the tile list
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThinThreads, budget / 2) != cudaSuccess || per_sm < 1) per_sm = 1;
    const long long cap = (long long)per_sm * ctx->sm_count;
    // output rows per tile: the whole plane if it fits, halved while that leaves the GPU short of tiles
    a.TH = g.OH;
    while (a.TH > 1 && tile_bytes(1, a.TH) > budget) a.TH = ceil_div(a.TH, 2);
    while (a.TH > 8 && (long long)g.N * ceil_div(g.OH, a.TH) * a.kgroups < 4 * cap) a.TH = ceil_div(a.TH, 2);
    a.bands = ceil_div(g.OH, a.TH);
    // small planes: several images per tile, the count that needs the fewest image-rounds on the busiest CTA
    a.nb = 1;
    if (a.bands == 1) {
        double best = 0.0;
        for (int nb = 1; nb <= g.N && nb <= 64 && tile_bytes(nb, a.TH) <= budget; ++nb) {
            const long long tiles = (long long)ceil_div(g.N, nb) * a.kgroups;
            const double rounds = (double)((tiles + cap - 1) / cap);
            const double cost = rounds * (nb + 0.25);
            if (nb == 1 || cost < best) { best = cost; a.nb = nb; }
        }
    }
    a.rows = (a.TH - 1) * g.S + g.FH;
    a.plane = a.rows * a.pitch;
    a.tiles = (long long)ceil_div(g.N, a.nb) * a.bands;
    const size_t smem = tile_bytes(a.nb, a.TH);
    long long gx_ll = cap / a.kgroups;
    if (gx_ll < 1) gx_ll = 1;
    const unsigned gx = (unsigned)(a.tiles < gx_ll ? a.tiles : gx_ll);
    launch_kernel(ctx, kern, dim3(gx, (unsigned)a.kgroups), dim3(kThinThreads), smem, st, a);
    return check_launch(ctx);
}

}  // namespace small
