// Full channel reduction on CUDA cores with a register tile per thread (paper Section 3.2 item 4; Algorithm 2:
// LOAD hoisted out of the window loops, an FMA tile, STORE), FP32 FMA, windows 1 or 3 wide of any height, strides 1
// and 2, any padding.  It is the path of SMALL_MATH_FP32 for these windows, and of the tensor-core modes for layers
// whose few channels leave an MMA mostly empty (FP32 FMAs meet every mode's tolerance).
//
// Mapping of the paper's loop nest (Algorithm 1):
//   O_wb x K_b kernel tile          -> 8 adjacent output pixels of a row x 8 filters in the registers of one thread
//   k block loop ("in parallel")    -> warps of a thread block side by side over the filters (KT = 8 x filter warps)
//   j, l loops over the output      -> lanes of a warp: 8 rows x 1, 2 or 4 column groups of 8 pixels (small planes:
//                                      several images per warp); one such "unit" per row warp of the block
//   i loop over F_C in F_Cb steps   -> stages of 8 or 16 input channels: TMA copies the halo box of each unit and the
//                                      filter box of the stage into shared memory, ring of up to 3 stages
//   x, y, ii kernel loops           -> per 4 channels and filter row: one 16-byte read per input pixel of the run
//                                      (8 S + FW - S pixels), then 4 x FW x 64 FMAs against filter values that the
//                                      whole warp reads as broadcasts
// The input box keeps the blocked layout's [pixel][channel] order: nothing is transposed and no thread computes a
// load address or a bounds check - pixels outside the plane are TMA's zero fill, which is the padding.  Bank
// conflicts are avoided by the copy's swizzle (16-byte chunk j of pixel p lies at chunk j ^ f(p)) together with an
// odd box width: the 8 lanes that share a shared-memory wavefront hold 8 consecutive rows, so their pixel indices
// differ in the low three bits.
#include <cuda.h>

#include <type_traits>

#include "common.cuh"
#include "sm100.cuh"

namespace small {

namespace {

constexpr int kPW = 8;          // output pixels per thread (adjacent in a row)
constexpr int kKQ = 8;          // filters per thread
constexpr int kMaxStages = 3;
constexpr int kMaxThreads = 256;
constexpr int kMaxRegs = 168;     // 12 resident warps per SM

struct DirectArgs {
    const void *bias; void *out; int *status;     // float (quantised form: int32 bias, uint8 output)
    int N, C, K, OH, OW, CB, KB, FH, pt, pl;
    int H, W;                   // input plane (the quantised epilogue needs the taps that fall inside it)
    const int *q_tab;           // quantised form: per filter and tap the sum of its weight bytes [K][T], then per filter [K]
    int zx, zw, zo, mult, shift;   // quantised form: zero points of input, weights and output; requantisation multiplier / 2^shift
    int cpb;                    // stages per 32-channel block (32 / cch; the quantised form takes a whole block per stage)
    int gw, gw_shift;           // column groups (of 8 pixels) of a unit: 1, 2 or 4
    int TH, NI;                 // output rows per image in a unit, images per unit
    int bands, tiles_w, units;  // row bands per image, column tiles per row, all units of the layer
    int th_in, cols_box;        // input box of a unit: rows per image, columns (odd)
    int cch;                    // channels per stage: 8 (32-byte swizzle) or 16 (64-byte swizzle)
    int sw_shift, sw_mask;      // chunk j of pixel p lies at chunk j ^ ((p >> sw_shift) & sw_mask)
    int KT, k_tiles, pwarps;    // filters per block, filter tiles, units (row warps) per block
    int stages;
    int cs, es;                 // stride of the box origin in the tensor; TMA element stride (2: a 1 x 1 stride-2 layer's
                                // box holds every other pixel and the kernel runs its stride-1 form on it)
    uint32_t unit_bytes, in_box_bytes, w_bytes, w_box_bytes, stage_bytes;
    int span, Kg, S_C;          // group convolution: channel blocks a filter block reads, filters per group, channel step
    int relu, accumulate;
    uint32_t wait_iters;        // limit of the bounded waits (polls)
    int pool;                   // fused 2 x 2 stride-2 max pool behind the layer (float form): out is [N][K][OH/2][OW/2]
};

__device__ __forceinline__ void lds128(uint32_t addr, uint32_t *v) {
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(addr));
}

// Q: the quantised form of the same loop nest (Section 5.5).  A pixel of a channel block is 32 bytes = 8 words of 4
// channels, so the shared-memory geometry is that of the float form with 8 channels per stage; a word of the input
// meets a word of 4 channel bytes of a filter in one 4-way dot product with 32-bit accumulation (dp4a) instead of an
// FMA.  Accumulated are the raw sums of byte products and, per pixel, the sum of the input bytes; the zero points enter
// in the STORE phase:  sum (x - zx)(w - zw) = sum x w - zw sum x - zx sum_{taps inside the plane} w + taps C zx zw,
// where pixels outside the plane (TMA's zero fill) take no part, which makes them real zeros.
template <int FW, int S, bool Q>
__global__ void __maxnreg__(kMaxRegs)
conv_direct_kernel(const __grid_constant__ CUtensorMap map_in, const __grid_constant__ CUtensorMap map_w, const DirectArgs a) {
    constexpr int PXH = S == 1 ? 8 : 4;           // pixels per pass over the registers (stride 2: two passes of 4)
    constexpr int NPASS = kPW / PXH;
    constexpr int NINH = (PXH - 1) * S + FW;      // input pixels a pass reads per filter row
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (sm100::smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) unsigned long long bars[kMaxStages];
    __shared__ int failed;
    const uint32_t bar0 = sm100::smem_u32(&bars[0]);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pw = warp % a.pwarps, kw = warp / a.pwarps;
    const int kt = blockIdx.x % a.k_tiles, ublock = blockIdx.x / a.k_tiles;
    const int k0 = kt * a.KT, kb0 = k0 >> 5;

    // unit u of the layer -> (image group, row band, column tile)
    auto unit_origin = [&](int u, int &n0, int &oh0, int &ow0) {
        if (u >= a.units) u = a.units - 1;        // a block's spare row warps repeat the last unit and store nothing
        const int wt = u % a.tiles_w; u /= a.tiles_w;
        const int band = u % a.bands;
        n0 = (u / a.bands) * a.NI; oh0 = band * a.TH; ow0 = wt * a.gw * kPW;
    };
    int n0, oh0, ow0;
    unit_origin(ublock * a.pwarps + pw, n0, oh0, ow0);
    // this thread's outputs: 8 pixels from column ow0 + 8 g of row oh0 + row of image n0 + img, filters k0 + 8 kw ..
    const int rest = lane >> 3;
    const int g = rest & (a.gw - 1);
    const int rslot = (rest >> a.gw_shift) * 8 + (lane & 7);
    const int img = rslot / a.TH, row = rslot - img * a.TH;
    const bool valid = ublock * a.pwarps + pw < a.units && img < a.NI && n0 + img < a.N && oh0 + row < a.OH && ow0 + g * kPW < a.OW;

    // channel blocks this filter tile reduces over (all of them; a group convolution's filter block reads `span`)
    const int cb0 = a.Kg > 0 ? ((kb0 * 32) / a.Kg * a.S_C) / 32 : 0;
    const int blocks = min(a.span, a.CB - cb0);
    const int cpb = a.cpb;
    const int last_n = min(32, a.C - (cb0 + blocks - 1) * 32);
    const int n_chunks = Q ? blocks : (blocks - 1) * cpb + (last_n + a.cch - 1) / a.cch;

    auto issue = [&](int q, int s) {       // one thread: arm the stage's barrier, start its copies
        const int cbj = q / cpb, c0 = (q - cbj * cpb) * a.cch;
        const uint32_t bar = bar0 + 8 * s, dst = base + s * a.stage_bytes;
        sm100::mbar_expect_tx(bar, a.pwarps * a.in_box_bytes + a.w_bytes);
        for (int u = 0; u < a.pwarps; ++u) {
            int un0, uoh0, uow0;
            unit_origin(ublock * a.pwarps + u, un0, uoh0, uow0);
            sm100::tma_load_5d(dst + u * a.unit_bytes, &map_in, bar, c0, uow0 * a.cs - a.pl, uoh0 * a.cs - a.pt, cb0 + cbj, un0);
        }
        const uint32_t wdst = dst + a.pwarps * a.unit_bytes;
        for (int h = 0; h * 32 < a.KT; ++h)       // 32 filters per box: [tap][channel][32 or fewer filters]
            sm100::tma_load_4d(wdst + h * a.w_box_bytes, &map_w, bar, k0 & 31, c0, 0, (kb0 + h) * a.span + cbj);
    };
    if (threadIdx.x == 0) {
        for (int s = 0; s < a.stages; ++s) sm100::mbar_init(bar0 + 8 * s, 1);
        sm100::mbar_fence_init();
        failed = 0;
    }
    __syncthreads();
    grid_dep_sync();
    if (threadIdx.x == 0)
        for (int q = 0; q < a.stages - 1 && q < n_chunks; ++q) issue(q, q);

    typedef typename std::conditional<Q, uint32_t, float>::type AccT;
    AccT acc[kPW][kKQ];
    uint32_t sx[Q ? kPW : 1];                     // quantised form: sum of the input bytes each pixel's window has seen
#pragma unroll
    for (int p = 0; p < kPW; ++p) {
        if (Q) sx[Q ? p : 0] = 0u;
#pragma unroll
        for (int k = 0; k < kKQ; ++k) acc[p][k] = AccT(0);
    }

    // idle lanes read the box's first run: in bounds, never stored
    const int p_base = img < a.NI ? (img * a.th_in + row * S) * a.cols_box + g * kPW * S : 0;
    const int pix_shift = a.cch == 16 ? 6 : 5;                    // bytes per pixel of the box: 64 or 32
    const int KTb = a.KT < 32 ? a.KT : 32;                        // filters per filter box
    const uint32_t w_off = a.pwarps * a.unit_bytes + ((kw * kKQ) >> 5) * a.w_box_bytes + ((kw * kKQ) & 31) * 4;

    int s = 0, phase = 0;
    for (int q = 0; q < n_chunks; ++q) {
        if (threadIdx.x == 0 && q + a.stages - 1 < n_chunks) {
            int sn = s + a.stages - 1;
            if (sn >= a.stages) sn -= a.stages;
            issue(q + a.stages - 1, sn);          // the stage read in the previous iteration, released by its __syncthreads
        }
        int ok = 1;
        if (lane == 0) ok = sm100::mbar_wait(bar0 + 8 * s, phase, a.wait_iters) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) { failed = 1; atomicExch(a.status, (int)SMALL_ERR_TIMEOUT); }
        __syncwarp();
        if (ok) {
            const int cbj = q / cpb, c0 = (q - cbj * cpb) * a.cch;
            // 16-byte chunks of a pixel that hold real channels: 4 floats, or 16 channel bytes, each
            const int lanes_n = min(32, a.C - (cb0 + cbj) * 32);
            const int c4_n = Q ? (lanes_n + 15) >> 4 : (min(a.cch, lanes_n - c0) + 3) >> 2;
            const uint32_t in_u = base + s * a.stage_bytes + pw * a.unit_bytes;       // shared-window addresses
            const uint32_t w_s = base + s * a.stage_bytes + w_off;
            for (int x = 0; x < a.FH; ++x) {
#pragma unroll
                for (int pass = 0; pass < NPASS; ++pass) {
                    // swizzled address of chunk 0 of each pixel of the run; chunk j then lies at that address ^ (j << 4)
                    // (the chunk field of the address is XORed with bits of the pixel index: see the file header)
                    const int p0 = p_base + x * a.cols_box + pass * PXH * S;
                    uint32_t pa[NINH];
#pragma unroll
                    for (int i = 0; i < NINH; ++i) {
                        const int p = p0 + i;
                        pa[i] = in_u + ((uint32_t)p << pix_shift) + (((uint32_t)(p >> a.sw_shift) & a.sw_mask) << 4);
                    }
                    for (int j = 0; j < c4_n; ++j) {
                        uint32_t v[NINH * 4];
#pragma unroll
                        for (int i = 0; i < NINH; ++i) lds128(pa[i] ^ ((uint32_t)j << 4), &v[4 * i]);
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
#pragma unroll
                            for (int y = 0; y < FW; ++y) {
                                uint32_t w[8];
                                const uint32_t wa = w_s + (uint32_t)(((x * FW + y) * a.cch + 4 * j + cc) * KTb) * 4u;
                                lds128(wa, &w[0]);
                                lds128(wa + 16, &w[4]);
#pragma unroll
                                for (int p = 0; p < PXH; ++p) {
                                    const uint32_t xv = v[(p * S + y) * 4 + cc];
                                    AccT *ac = acc[pass * PXH + p];
                                    if (Q) {
                                        sx[Q ? pass * PXH + p : 0] = __dp4a(xv, 0x01010101u, sx[Q ? pass * PXH + p : 0]);
#pragma unroll
                                        for (int k = 0; k < kKQ; ++k) ac[k] = (AccT)__dp4a(xv, w[k], (uint32_t)ac[k]);
                                    } else {
#pragma unroll
                                        for (int k = 0; k < kKQ; ++k) ac[k] = (AccT)fmaf(__uint_as_float(xv), __uint_as_float(w[k]), (float)ac[k]);
                                    }
                                }
                            }
                        }
                    }
                }
            }
        }
        __syncthreads();                          // everyone is done with stage s (and sees `failed`)
        if (failed) break;
        if (++s == a.stages) { s = 0; phase ^= 1; }
    }
    if (failed) {     // a wait ran out: give copies that may still be in flight a bounded grace period, store nothing
        if (threadIdx.x == 0)
            for (uint32_t k = 0; k < (1u << 14); ++k) __nanosleep(200);
        return;
    }

    // STORE phase.  Lanes of the last filter block beyond K stay zero: the thread holding the launch's last filter group
    // writes them.
    const int kq0 = k0 + kw * kKQ;
    const int kb = kq0 >> 5, kl = kq0 & 31;
    if (kb >= a.KB) return;                       // the same for a whole warp
    const int n = n0 + img, oh = oh0 + row;
    const bool last_group = kq0 + kKQ == a.k_tiles * a.KT;
    if (!Q && a.pool) {
        // Abstract fused layer (Section 6): the 2 x 2 stride-2 max pool behind the convolution is taken in the STORE
        // phase.  A thread holds 8 adjacent columns of one row: column pairs are reduced in its registers; rows 2i and
        // 2i + 1 sit in neighbouring lanes (a unit has an even number of rows per image), so the row pair is one
        // shuffle; the even row's lane stores 4 pooled pixels.  All lanes take part in the shuffles.
        const float *bias = static_cast<const float *>(a.bias);
        float bv[kKQ];
#pragma unroll
        for (int k = 0; k < kKQ; ++k) bv[k] = (bias && kq0 + k < a.K) ? bias[kq0 + k] : 0.0f;
        const int PH = a.OH >> 1, PW = a.OW >> 1;
        const int prow = oh >> 1, pcol0 = (ow0 + g * kPW) >> 1;
        const bool store_lane = valid && !(oh & 1) && prow < PH;
        float *dst = static_cast<float *>(a.out) + ((((size_t)(valid ? n : 0) * a.KB + kb) * PH + (store_lane ? prow : 0)) * PW + pcol0) * 32 + kl;
#pragma unroll
        for (int pp = 0; pp < kPW / 2; ++pp) {
            float m[kKQ];
#pragma unroll
            for (int k = 0; k < kKQ; ++k) {
                float r0 = (float)acc[2 * pp][k] + bv[k], r1 = (float)acc[2 * pp + 1][k] + bv[k];
                if (a.relu) { r0 = fmaxf(r0, 0.0f); r1 = fmaxf(r1, 0.0f); }
                m[k] = fmaxf(r0, r1);
                m[k] = fmaxf(m[k], __shfl_xor_sync(0xffffffffu, m[k], 1));
                if (kq0 + k >= a.K) m[k] = 0.0f;
            }
            if (store_lane && pcol0 + pp < PW) {
                float4 *d4 = reinterpret_cast<float4 *>(dst + pp * 32);
                d4[0] = make_float4(m[0], m[1], m[2], m[3]);
                d4[1] = make_float4(m[4], m[5], m[6], m[7]);
                if (last_group)
                    for (int z = kl + kKQ; z < 32; z += 4) *reinterpret_cast<float4 *>(dst + pp * 32 - kl + z) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        return;
    }
    if (!valid) return;
    if constexpr (Q) {
        // zero points, bias, one requantisation (round half up of the 64-bit product), clamp, 8 bytes per pixel and thread
        const int T = a.FH * FW;
        const int *bias = static_cast<const int *>(a.bias);
        int bv[kKQ], wall[kKQ];
#pragma unroll
        for (int k = 0; k < kKQ; ++k) {
            const bool real = kq0 + k < a.K;
            bv[k] = (bias && real) ? bias[kq0 + k] : 0;
            wall[k] = real ? a.q_tab[a.K * T + kq0 + k] : 0;
        }
        const int ih0 = oh * a.cs - a.pt;
        const int x0 = max(0, -ih0), x1 = min(a.FH, a.H - ih0);
        const int lo = a.relu ? a.zo : 0;
        uint8_t *dst = static_cast<uint8_t *>(a.out) + ((((size_t)n * a.KB + kb) * a.OH + oh) * a.OW + ow0 + g * kPW) * 32 + kl;
#pragma unroll
        for (int p = 0; p < kPW; ++p) {
            const int ow = ow0 + g * kPW + p;
            if (ow >= a.OW) break;
            const int iw0 = ow * a.cs - a.pl;
            const int y0 = max(0, -iw0), y1 = min(FW, a.W - iw0);
            const int nv = (x1 - x0) * (y1 - y0);                 // taps of this pixel's window that lie inside the plane
            uint32_t packed[2] = {0u, 0u};
#pragma unroll
            for (int k = 0; k < kKQ; ++k) {
                int q = 0;
                if (kq0 + k < a.K) {
                    int sw = wall[k];
                    if (nv != T) {                                // a border pixel: only the taps inside count
                        sw = 0;
                        for (int x = x0; x < x1; ++x)
                            for (int y = y0; y < y1; ++y) sw += a.q_tab[(kq0 + k) * T + x * FW + y];
                    }
                    const long long t = (long long)acc[p][k] - (long long)a.zw * (long long)sx[Q ? p : 0] - (long long)a.zx * sw +
                                        (long long)nv * a.C * a.zx * a.zw + bv[k];
                    const long long r = (t * (long long)a.mult + (1ll << (a.shift - 1))) >> a.shift;
                    const long long z = (long long)a.zo + r;
                    q = (int)(z < lo ? lo : z > 255 ? 255 : z);
                }
                packed[k >> 2] |= (uint32_t)q << (8 * (k & 3));
            }
            *reinterpret_cast<uint2 *>(dst + p * 32) = make_uint2(packed[0], packed[1]);
            if (last_group)
                for (int z = kl + kKQ; z < 32; z += 8) *reinterpret_cast<uint2 *>(dst + p * 32 - kl + z) = make_uint2(0u, 0u);
        }
    } else {
        // + bias, + the tensor already in `out` (accumulate), ReLU; 32 bytes per pixel and thread
        const float *bias = static_cast<const float *>(a.bias);
        float bv[kKQ];
#pragma unroll
        for (int k = 0; k < kKQ; ++k) bv[k] = (bias && kq0 + k < a.K) ? bias[kq0 + k] : 0.0f;
        float *dst = static_cast<float *>(a.out) + ((((size_t)n * a.KB + kb) * a.OH + oh) * a.OW + ow0 + g * kPW) * 32 + kl;
#pragma unroll
        for (int p = 0; p < kPW; ++p) {
            if (ow0 + g * kPW + p >= a.OW) break;
            float4 *d4 = reinterpret_cast<float4 *>(dst + p * 32);
            float r[kKQ];
#pragma unroll
            for (int k = 0; k < kKQ; ++k) r[k] = (float)acc[p][k] + bv[k];
            if (a.accumulate) {
                const float4 o0 = d4[0], o1 = d4[1];
                r[0] += o0.x; r[1] += o0.y; r[2] += o0.z; r[3] += o0.w;
                r[4] += o1.x; r[5] += o1.y; r[6] += o1.z; r[7] += o1.w;
            }
            if (a.relu) {
#pragma unroll
                for (int k = 0; k < kKQ; ++k) r[k] = fmaxf(r[k], 0.0f);
            }
            if (kq0 + kKQ > a.K) {
#pragma unroll
                for (int k = 0; k < kKQ; ++k) if (kq0 + k >= a.K) r[k] = 0.0f;
            }
            d4[0] = make_float4(r[0], r[1], r[2], r[3]);
            d4[1] = make_float4(r[4], r[5], r[6], r[7]);
            if (last_group)
                for (int z = kl + kKQ; z < 32; z += 4) *reinterpret_cast<float4 *>(dst + p * 32 - kl + z) = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
}

struct DirectPlan { DirectArgs a; size_t smem; int threads; long long blocks; bool ok; };

size_t round1k(size_t b) { return (b + 1023) & ~(size_t)1023; }

// Tile shapes.  The unit of a row warp follows from the plane's width; what is chosen is the number of channels per
// stage (8 or 16) and of units per block: the smallest blocks (finest work granularity over the SMs) that still keep
// 12 or more warps resident per SM within shared memory.
DirectPlan plan_direct(const Geom &g, int span, int Kg, int S_C, size_t max_smem, bool quant = false, bool pool = false) {
    DirectPlan best{};
    best.ok = false;
    if ((g.FW != 1 && g.FW != 3) || (g.S != 1 && g.S != 2) || g.FH * g.FW > 256) return best;
    DirectArgs a{};
    a.N = g.N; a.C = g.C; a.K = g.K; a.OH = g.OH; a.OW = g.OW; a.CB = g.CB; a.KB = g.KB; a.FH = g.FH; a.pt = g.pt; a.pl = g.pl;
    a.H = g.H; a.W = g.W;
    a.span = span > 0 ? span : g.CB; a.Kg = span > 0 ? Kg : 0; a.S_C = S_C;
    a.gw = g.OW <= 8 ? 1 : g.OW <= 16 ? 2 : 4;
    a.gw_shift = a.gw == 1 ? 0 : a.gw == 2 ? 1 : 2;
    a.tiles_w = ceil_div(g.OW, a.gw * kPW);
    const int rows_u = 32 / a.gw;
    if (g.OH <= rows_u) { a.TH = g.OH; a.NI = rows_u / g.OH; a.bands = 1; if (a.NI > g.N) a.NI = g.N; }
    else { a.TH = rows_u; a.NI = 1; a.bands = ceil_div(g.OH, rows_u); }
    if (pool && ((a.TH & 1) || g.OH < 2 || g.OW < 2 || quant || span > 0)) return best;   // row pairs must share a unit
    a.pool = pool ? 1 : 0;
    const long long units = (long long)ceil_div(g.N, a.NI) * a.bands * a.tiles_w;
    if (units > 0x3fffffffLL) return best;
    a.units = (int)units;
    a.cs = g.S;
    a.es = (g.FH == 1 && g.FW == 1) ? g.S : 1;      // 1 x 1 windows: the copy itself skips the pixels a stride leaves out
    const int S = g.S / a.es;                       // stride the kernel sees in shared memory
    a.th_in = (a.TH - 1) * S + g.FH;
    a.cols_box = ((a.gw * kPW - 1) * S + g.FW) | 1;
    if (a.th_in * a.es > 256 || a.cols_box * a.es > 256 || a.NI > 256) return best;
    a.KT = g.K <= 8 ? 8 : g.K <= 16 ? 16 : (g.K <= 32 || span > 0) ? 32 : 64;
    a.k_tiles = ceil_div(g.K, a.KT);
    const int kwarps = a.KT / kKQ;
    const int T = g.FH * g.FW;
    const int last_n = g.C - (g.CB - 1) * 32;
    int best_warps = 0;
    // (the quantised form has one geometry: a stage is a whole 32-channel block, 8 words of 4 channel bytes per pixel)
    for (int cch = quant ? 8 : 16; cch >= 8; cch -= 8) {
        const int n_chunks = quant ? g.CB : ((span > 0 ? span : g.CB) - 1) * (32 / cch) + ceil_div(last_n, cch);
        for (int pwarps = 1; pwarps * kwarps * 32 <= kMaxThreads; ++pwarps) {
            if (pwarps * kwarps < 2) continue;
            DirectArgs c = a;
            c.cch = cch; c.pwarps = pwarps; c.cpb = quant ? 1 : 32 / cch;
            c.sw_shift = cch == 16 ? 1 : 2; c.sw_mask = cch == 16 ? 3 : 1;
            c.in_box_bytes = (uint32_t)((size_t)a.NI * a.th_in * a.cols_box * cch * 4);
            c.unit_bytes = (uint32_t)round1k(c.in_box_bytes);
            const int KTb = a.KT < 32 ? a.KT : 32;
            c.w_box_bytes = (uint32_t)((size_t)T * cch * KTb * 4);
            c.w_bytes = c.w_box_bytes * (uint32_t)ceil_div(a.KT, 32);
            c.stage_bytes = (uint32_t)round1k((size_t)pwarps * c.unit_bytes + c.w_bytes);
            c.stages = n_chunks < kMaxStages ? n_chunks : kMaxStages;
            size_t smem = (size_t)c.stages * c.stage_bytes + 1024;
            while (smem > 110 * 1024 && c.stages > 2) { --c.stages; smem = (size_t)c.stages * c.stage_bytes + 1024; }
            if (smem > max_smem) continue;
            const int warps = pwarps * kwarps;
            int per_sm = (int)((225 * 1024) / (smem + 1024));
            if (per_sm * warps > 12) per_sm = 12 / warps;             // registers: kMaxRegs allows 12 warps per SM
            const int resident = per_sm * warps > 12 ? 12 : per_sm * warps;   // beyond 12 warps per SM nothing is gained
            if (resident > best_warps) {
                best_warps = resident;
                best.a = c; best.smem = smem; best.threads = 32 * warps;
                best.blocks = (long long)ceil_div(a.units, pwarps) * a.k_tiles;
                best.ok = best.blocks <= 0x7fffffffLL;
            }
        }
    }
    return best;
}

using sm100::EncodeTiledFn;

}  // namespace

bool conv_direct_supported(const Geom &g, int span, int Kg, int S_C) {
    return plan_direct(g, span, Kg, S_C, 227 * 1024).ok;
}

long long conv_direct_blocks(const Geom &g) {
    const DirectPlan p = plan_direct(g, 0, 0, 0, 227 * 1024);
    return p.ok ? p.blocks : 0;
}

namespace {

// Tensor maps and launch shared by the float and the quantised form.  esize: bytes per channel of the activation
// tensor (4 or 1); the filter tensor is [KB][span][FH*FW][32][32] 4-byte words in both forms (floats [ci][ko], or
// words of 4 channel bytes [c4][ko] in the first 8 of the 32 rows' worth - see pack_q_conv_w_kernel).
int launch_direct(small_ctx *ctx, DirectPlan &p, const Geom &g, const void *in, const void *w, bool quant, cudaStream_t st) {
    DirectArgs &a = p.a;
    a.wait_iters = ctx->wait_iters;
    EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    CUtensorMap map_in, map_w;
    {   // activations [N][CB][H][W][32]: box = one stage's channels x cols_box x th_in x 1 block x NI images, swizzled
        const cuuint64_t px = quant ? 32 : 128;      // bytes per pixel and channel block
        cuuint64_t dims[5] = {32, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.CB, (cuuint64_t)g.N};
        cuuint64_t strides[4] = {px, (cuuint64_t)g.W * px, (cuuint64_t)g.H * g.W * px, (cuuint64_t)g.CB * g.H * g.W * px};
        const cuuint32_t es = (cuuint32_t)a.es;     // element stride 2: a box of 2 cols x 2 rows elements lands as cols x rows pixels
        cuuint32_t box[5] = {(cuuint32_t)(quant ? 32 : a.cch), (cuuint32_t)a.cols_box * es, (cuuint32_t)a.th_in * es, 1, (cuuint32_t)a.NI};
        cuuint32_t estr[5] = {1, es, es, 1, 1};
        CUresult r = encode(&map_in, quant ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<void *>(in), dims,
                            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            a.cch == 16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    {   // packed filters: box = up to 32 filters x one stage's channel rows x all taps
        const int T = g.FH * g.FW;
        const cuuint64_t rows = quant ? 8 : 32;      // words per filter, tap and channel block
        cuuint64_t dims[4] = {32, rows, (cuuint64_t)T, (cuuint64_t)g.KB * a.span};
        cuuint64_t strides[3] = {128, rows * 128, (cuuint64_t)T * rows * 128};
        cuuint32_t box[4] = {(cuuint32_t)(a.KT < 32 ? a.KT : 32), (cuuint32_t)a.cch, (cuuint32_t)T, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        CUresult r = encode(&map_w, quant ? CU_TENSOR_MAP_DATA_TYPE_INT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void *>(w), dims,
                            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    const int S = g.S / a.es;
    void (*kern)(const CUtensorMap, const CUtensorMap, const DirectArgs);
    if (quant) kern = g.FW == 1 ? (S == 1 ? conv_direct_kernel<1, 1, true> : conv_direct_kernel<1, 2, true>)
                                : (S == 1 ? conv_direct_kernel<3, 1, true> : conv_direct_kernel<3, 2, true>);
    else kern = g.FW == 1 ? (S == 1 ? conv_direct_kernel<1, 1, false> : conv_direct_kernel<1, 2, false>)
                          : (S == 1 ? conv_direct_kernel<3, 1, false> : conv_direct_kernel<3, 2, false>);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    // an ordinary launch whose successor starts only as its blocks leave, like the general FP32 kernel
    const int dependent = ctx->dependent;
    ctx->dependent = 0;
    launch_kernel(ctx, kern, dim3((unsigned)p.blocks), dim3(p.threads), p.smem, st, map_in, map_w, a);
    ctx->dependent = dependent;
    return check_launch(ctx);
}

}  // namespace

int launch_conv_direct(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, const Geom &g,
                       bool relu, bool accumulate, cudaStream_t st, int span, int Kg, int S_C) {
    DirectPlan p = plan_direct(g, span, Kg, S_C, ctx->max_smem_optin);
    if (!p.ok) return SMALL_ERR_UNSUPPORTED;
    DirectArgs &a = p.a;
    a.bias = bias; a.out = out; a.status = ctx->dev_status; a.relu = relu; a.accumulate = accumulate;
    return launch_direct(ctx, p, g, in, w, false, st);
}

bool conv_direct_pool_supported(const Geom &g) { return plan_direct(g, 0, 0, 0, 227 * 1024, false, true).ok; }

int launch_conv_direct_pool(small_ctx *ctx, const float *in, const float *w, const float *bias, float *out, const Geom &g,
                            bool relu, cudaStream_t st) {
    DirectPlan p = plan_direct(g, 0, 0, 0, ctx->max_smem_optin, false, true);
    if (!p.ok) return SMALL_ERR_UNSUPPORTED;
    DirectArgs &a = p.a;
    a.bias = bias; a.out = out; a.status = ctx->dev_status; a.relu = relu; a.accumulate = 0;
    return launch_direct(ctx, p, g, in, w, false, st);
}

bool q_conv_supported(const Geom &g) { return plan_direct(g, 0, 0, 0, 227 * 1024, true).ok; }

int launch_q_conv(small_ctx *ctx, const uint8_t *in, const uint32_t *w_words, const int *tables, const int *bias, uint8_t *out,
                  const Geom &g, bool relu, int zx, int zw, int zo, int mult, int shift, cudaStream_t st) {
    DirectPlan p = plan_direct(g, 0, 0, 0, ctx->max_smem_optin, true);
    if (!p.ok) return SMALL_ERR_UNSUPPORTED;
    DirectArgs &a = p.a;
    a.bias = bias; a.out = out; a.status = ctx->dev_status; a.relu = relu; a.accumulate = 0;
    a.q_tab = tables; a.zx = zx; a.zw = zw; a.zo = zo; a.mult = mult; a.shift = shift;
    return launch_direct(ctx, p, g, in, w_words, true, st);
}

}  // namespace small
