// Kernel of the warp-level tensor-core convolution (see conv_mma.cu for the design); a header so that its template
// instances can be compiled in several translation units side by side.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "sm100.cuh"

namespace small {
namespace mma_conv {

struct MmaArgs {
    const float *bias; float *out; int *status;
    int N, K, OH, OW, KB, FH, FW, pt, pl;
    int fwd_shift;             // a fragment is (16 >> fwd_shift) rows x (1 << fwd_shift) columns of one image
    int TH, TWd, NI;           // output rows, columns and images of a tile
    int Ht, Wt;                // halo box: rows and columns per image
    int tiles_w, tiles_h, n_tiles;
    int frags_w, frags_img, frags_tile;   // fragments per fragment row, per image of a tile, per tile (the rest idle)
    int mf_warp;               // fragments per warp actually used (<= MF)
    int vert;                  // a warp's fragments are mf_warp consecutive rows of one column block (see VERT)
    int cs;                    // stride of the box origin in the tensor (S of the kernel = stride between the box's pixels:
                               // 1 when a 1 x 1 window's copy itself skips the pixels a stride leaves out)
    int k_tiles;               // filter tiles of 32 (= KB): thread block b computes tile b % k_tiles of its pixel tiles
    uint32_t in_box_bytes, stage_bytes;
    uint32_t w_box_bytes, w_half_bytes;   // bytes of one filter box (TF32 part or residual) and its 1 KB-rounded place
    int relu, accumulate;
    uint32_t wait_iters;
};

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16 pixels x 8 filters, FP32) += A (16 pixels x 8 channels) * B (8 channels x 8 filters), TF32 operands
__device__ __forceinline__ void mma_16x8x8(float (&c)[4], const uint32_t *a, const uint32_t *b) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
// NF: fragments of 8 filters; MF: fragments of 16 pixels per warp; CW: channels per shared-memory row (16: 64-byte
// rows and swizzle, layers of at most 16 channels; 32: 128-byte rows); S: stride; X3: 3xTF32; FWT: width of the window
// (1 or 3; 0: any, at run time).  The halo box is a multiple of 8 pixels wide, so a step down the window leaves a
// pixel's swizzle phase alone and each lane keeps one ready-made address per window column and fragment.
// VERT (3 x 3 windows at stride 1, fragments of one row): a warp's fragments are consecutive output rows of one column
// block, so input row r of that block serves the window rows of up to three of them: each input fragment is loaded
// (and, for 3xTF32, split) once per window column instead of once per tap - half the operand loads and splits.
template <int NF, int MF, int CW, int S, bool X3, int FWT, bool VERT = false>
__global__ void __launch_bounds__(256)
conv_mma_kernel(const __grid_constant__ CUtensorMap map_in, const __grid_constant__ CUtensorMap map_w,
                const __grid_constant__ CUtensorMap map_w_lo, const MmaArgs a) {
    constexpr uint32_t RB = CW * 4;                 // bytes per pixel / filter row
    constexpr int RSH = CW == 16 ? 6 : 7;
    constexpr int PAIRS = CW / 16;
    constexpr int GM = NF >= 4 ? 2 : 4;   // pixel fragments whose MMAs are interleaved
    constexpr int FWU = FWT ? FWT : 1;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (sm100::smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) unsigned long long bars[3];
    __shared__ int failed;
    const uint32_t bar_w = sm100::smem_u32(&bars[0]), bar_in = sm100::smem_u32(&bars[1]);
    const uint32_t w_hi_s = base, w_lo_s = base + a.w_half_bytes;
    const uint32_t in_s = base + (X3 ? 2u : 1u) * a.w_half_bytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = a.FH * a.FW;
    // filter tile of this block, and its walk over the pixel tiles
    const int kt = a.k_tiles > 1 ? (int)(blockIdx.x % (unsigned)a.k_tiles) : 0;
    const int t_first = a.k_tiles > 1 ? (int)(blockIdx.x / (unsigned)a.k_tiles) : (int)blockIdx.x;
    const int t_step = a.k_tiles > 1 ? (int)(gridDim.x / (unsigned)a.k_tiles) : (int)gridDim.x;

    auto tile_origin = [&](int t, int &n0, int &oh0, int &ow0) {
        const int wt = t % a.tiles_w; t /= a.tiles_w;
        const int band = t % a.tiles_h;
        n0 = (t / a.tiles_h) * a.NI; oh0 = band * a.TH; ow0 = wt * a.TWd;
    };
    auto issue = [&](int t, int s) {
        int n0, oh0, ow0;
        tile_origin(t, n0, oh0, ow0);
        sm100::mbar_expect_tx(bar_in + 8 * s, a.in_box_bytes);
        sm100::tma_load_5d(in_s + s * a.stage_bytes, &map_in, bar_in + 8 * s, 0, ow0 * a.cs - a.pl, oh0 * a.cs - a.pt, 0, n0);
    };

    if (threadIdx.x == 0) {
        sm100::mbar_init(bar_w, 1); sm100::mbar_init(bar_in, 1); sm100::mbar_init(bar_in + 8, 1);
        sm100::mbar_fence_init();
        failed = 0;
    }
    __syncthreads();
    if (threadIdx.x == 0) {       // the filters are the layer's own constants: no earlier kernel of the stream writes them
        sm100::mbar_expect_tx(bar_w, a.w_box_bytes * (X3 ? 2u : 1u));
        sm100::tma_load_4d(w_hi_s, &map_w, bar_w, 0, kt * 32, 0, 0);
        if (X3) sm100::tma_load_4d(w_lo_s, &map_w_lo, bar_w, 0, kt * 32, 0, 0);
    }
    grid_dep_sync();
    grid_dep_trigger();
    if (threadIdx.x == 0 && t_first < a.n_tiles) issue(t_first, 0);

    // this lane's part in the loads: row (lane & 7) of matrix (lane >> 3)
    // A: matrices 0 / 1 = pixels 0-7 / 8-15 of the fragment at the K step's first 4 channels, 2 / 3 = the next 4
    // B: matrices 0 .. 3 = 16-byte chunks 0 .. 3 of a pair of K steps, rows = the fragment's 8 filters
    const int FWD = 1 << a.fwd_shift;
    const int jl = (lane & 7) | (((lane >> 3) & 1) << 3);          // pixel of the fragment this lane addresses
    const int a_chunk = lane >> 4;
    // fragment m of this warp: image, fragment row and fragment column within the tile; false for an idle one
    auto frag_of = [&](int m, int &img, int &frow, int &fcol) {
        if (a.vert) {       // consecutive rows of one column block (one image per tile)
            img = 0; fcol = warp % a.frags_w; frow = (warp / a.frags_w) * a.mf_warp + m;
            return m < a.mf_warp && frow * a.frags_w + fcol < a.frags_tile;
        }
        const int f = warp * a.mf_warp + m;
        img = f / a.frags_img;
        const int rem = f - img * a.frags_img;
        frow = rem / a.frags_w; fcol = rem - frow * a.frags_w;
        return m < a.mf_warp && f < a.frags_tile;
    };
    int p_lane[MF];                                                // its pixel index in the halo box at tap (0, 0)
    uint32_t pre[FWU][MF];                                         // byte offset of its 16 bytes at window column y, row 0
#pragma unroll
    for (int m = 0; m < MF; ++m) {
        int img, frow, fcol;
        if (!frag_of(m, img, frow, fcol)) {                        // idle fragments read in bounds and store nothing
            img = 0; fcol = 0;
            if (!a.vert) frow = 0;                                 // (a vertical warp's rows stay consecutive: all inside the box)
        }
        const int row = frow * (16 >> a.fwd_shift) + (jl >> a.fwd_shift), col = fcol * FWD + (jl & (FWD - 1));
        p_lane[m] = (img * a.Ht + row * S) * a.Wt + col * S;
#pragma unroll
        for (int y = 0; y < FWU; ++y) {
            const uint32_t p = (uint32_t)(p_lane[m] + y);
            pre[y][m] = (p << RSH) + ((((uint32_t)a_chunk) ^ (CW == 16 ? (p >> 1) & 3u : p & 7u)) << 4);
        }
    }
    // filter rows: row r of a tap lies at r * RB, chunk j at j ^ (swizzle of r); r & 7 = lane & 7 for every fragment
    const uint32_t w_sw = CW == 16 ? (uint32_t)((lane & 7) >> 1) & 3u : (uint32_t)(lane & 7);
    const uint32_t w_lane = (uint32_t)(lane & 7) * RB + ((((uint32_t)lane >> 3) ^ w_sw) << 4);

    float bv[NF][2];
    uint32_t k_real = 0;                                           // bit 2 n + e: filter 8 n + 2 (lane & 3) + e exists
#pragma unroll
    for (int n = 0; n < NF; ++n)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int k = kt * 32 + 8 * n + 2 * (lane & 3) + e;
            bv[n][e] = (a.bias && k < a.K) ? a.bias[k] : 0.0f;
            if (k < a.K) k_real |= 1u << (2 * n + e);
        }
    // the pixels this lane stores (accumulator rows lane >> 2 and + 8 of each fragment): (image, row, column) within a
    // tile, packed 12 + 10 + 10 bits, and the offset in floats from the tile's first output pixel; the same for every tile
    uint32_t st_pix[MF][2];
    int st_off[MF][2];
#pragma unroll
    for (int m = 0; m < MF; ++m) {
        int img, frow, fcol;
        const bool used = frag_of(m, img, frow, fcol);
        if (!used) { img = 0; frow = 0; fcol = 0; }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int j = (lane >> 2) + 8 * h;
            const int row = frow * (16 >> a.fwd_shift) + (j >> a.fwd_shift), col = fcol * FWD + (j & (FWD - 1));
            st_pix[m][h] = used ? ((uint32_t)img << 20) | ((uint32_t)row << 10) | (uint32_t)col : 0xffffffffu;
            st_off[m][h] = ((img * a.KB * a.OH + row) * a.OW + col) * 32 + 2 * (lane & 3);
        }
    }

    bool w_ready = false;
    int it = 0;
    for (int t = t_first; t < a.n_tiles; t += t_step, ++it) {
        const int s = it & 1;
        // the other stage was last read before the block-wide barrier that ended the previous tile
        if (threadIdx.x == 0 && t + t_step < a.n_tiles) issue(t + t_step, s ^ 1);
        int ok = 1;
        if (lane == 0) {
            if (!w_ready) ok = sm100::mbar_wait(bar_w, 0, a.wait_iters) ? 1 : 0;
            if (ok) ok = sm100::mbar_wait(bar_in + 8 * s, (it >> 1) & 1, a.wait_iters) ? 1 : 0;
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        w_ready = true;
        if (!ok) { failed = 1; atomicExch(a.status, (int)SMALL_ERR_TIMEOUT); }
        __syncwarp();

        float acc[MF][NF][4];
#pragma unroll
        for (int m = 0; m < MF; ++m)
#pragma unroll
            for (int n = 0; n < NF; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[m][n][e] = 0.0f;

        if (ok) {
            const uint32_t in_t = in_s + s * a.stage_bytes;
            // one window position: filter fragments of the tap, then the pixel fragments GM at a time, so that four
            // independent accumulators take turns (an MMA that adds to the accumulator of the one before it waits out
            // that one's whole latency)
            auto tap_step = [&](const int tap, const uint32_t row_base, const int y, const int tapoff) {
                const uint32_t w_tap = (uint32_t)(tap * NF * 8) * RB + w_lane;
#pragma unroll
                for (int pr = 0; pr < PAIRS; ++pr) {
                    uint32_t bh[NF][4], bl[X3 ? NF : 1][4];
#pragma unroll
                    for (int n = 0; n < NF; ++n) {
                        const uint32_t wa = (w_tap + (uint32_t)(n * 8) * RB) ^ ((uint32_t)pr << 6);
                        ldsm4(w_hi_s + wa, bh[n]);
                        if (X3) ldsm4(w_lo_s + wa, bl[X3 ? n : 0]);
                    }
#pragma unroll
                    for (int m0 = 0; m0 < MF; m0 += GM) {
                        if (m0 >= a.mf_warp) break;
                        uint32_t ah[GM][2][4], al[X3 ? GM : 1][2][4];
#pragma unroll
                        for (int g = 0; g < GM; ++g) {
                            uint32_t addr;
                            if (FWT) {
                                addr = row_base + pre[FWT ? y : 0][m0 + g];
                            } else {
                                const uint32_t p = (uint32_t)(p_lane[m0 + g] + tapoff);
                                addr = in_t + (p << RSH) + ((((uint32_t)a_chunk) ^ (CW == 16 ? (p >> 1) & 3u : p & 7u)) << 4);
                            }
#pragma unroll
                            for (int ks = 0; ks < 2; ++ks) {
                                uint32_t av[4];
                                ldsm4(addr ^ ((uint32_t)(4 * pr + 2 * ks) << 4), av);
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    // TF32: the MMA reads the leading 11 bits of the raw word.  3xTF32: those bits and the
                                    // exact residual, of which the MMA again reads the leading 11 bits.
                                    ah[g][ks][e] = X3 ? av[e] & 0xffffe000u : av[e];
                                    if (X3) al[X3 ? g : 0][ks][e] = __float_as_uint(__uint_as_float(av[e]) - __uint_as_float(ah[g][ks][e]));
                                }
                            }
                        }
#pragma unroll
                        for (int ks = 0; ks < 2; ++ks) {
                            if (X3) {                                  // small terms first
#pragma unroll
                                for (int g = 0; g < GM; ++g)
#pragma unroll
                                    for (int n = 0; n < NF; ++n) mma_16x8x8(acc[m0 + g][n], al[X3 ? g : 0][ks], &bh[n][2 * ks]);
#pragma unroll
                                for (int g = 0; g < GM; ++g)
#pragma unroll
                                    for (int n = 0; n < NF; ++n) mma_16x8x8(acc[m0 + g][n], ah[g][ks], &bl[X3 ? n : 0][2 * ks]);
                            }
#pragma unroll
                            for (int g = 0; g < GM; ++g)
#pragma unroll
                                for (int n = 0; n < NF; ++n) mma_16x8x8(acc[m0 + g][n], ah[g][ks], &bh[n][2 * ks]);
                        }
                    }
                }
            };
            if constexpr (VERT) {
                // window column y: the filter fragments of its three taps, then one pass down the MF + 2 input rows
#pragma unroll
                for (int pr = 0; pr < PAIRS; ++pr) {
#pragma unroll
                    for (int y = 0; y < 3; ++y) {
                        uint32_t bh[3][NF][4], bl[X3 ? 3 : 1][X3 ? NF : 1][4];
#pragma unroll
                        for (int x = 0; x < 3; ++x)
#pragma unroll
                            for (int n = 0; n < NF; ++n) {
                                const uint32_t wa = ((uint32_t)((x * 3 + y) * NF * 8 + n * 8) * RB + w_lane) ^ ((uint32_t)pr << 6);
                                ldsm4(w_hi_s + wa, bh[x][n]);
                                if (X3) ldsm4(w_lo_s + wa, bl[X3 ? x : 0][X3 ? n : 0]);
                            }
#pragma unroll
                        for (int ir = 0; ir < MF + 2; ++ir) {
                            if (ir >= a.mf_warp + 2) break;
                            const uint32_t addr = in_t + (uint32_t)(ir * a.Wt) * RB + pre[y][0];
                            uint32_t ah[2][4], al[2][4];
#pragma unroll
                            for (int ks = 0; ks < 2; ++ks) {
                                uint32_t av[4];
                                ldsm4(addr ^ ((uint32_t)(4 * pr + 2 * ks) << 4), av);
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    ah[ks][e] = X3 ? av[e] & 0xffffe000u : av[e];
                                    if (X3) al[ks][e] = __float_as_uint(__uint_as_float(av[e]) - __uint_as_float(ah[ks][e]));
                                }
                            }
                            // input row ir is window row x of output row ir - x
#pragma unroll
                            for (int ks = 0; ks < 2; ++ks) {
                                if (X3) {
#pragma unroll
                                    for (int x = 0; x < 3; ++x)
                                        if (ir - x >= 0 && ir - x < MF && ir - x < a.mf_warp)
#pragma unroll
                                            for (int n = 0; n < NF; ++n) mma_16x8x8(acc[ir - x < 0 ? 0 : ir - x >= MF ? 0 : ir - x][n], al[ks], &bh[x][n][2 * ks]);
#pragma unroll
                                    for (int x = 0; x < 3; ++x)
                                        if (ir - x >= 0 && ir - x < MF && ir - x < a.mf_warp)
#pragma unroll
                                            for (int n = 0; n < NF; ++n) mma_16x8x8(acc[ir - x < 0 ? 0 : ir - x >= MF ? 0 : ir - x][n], ah[ks], &bl[X3 ? x : 0][X3 ? n : 0][2 * ks]);
                                }
#pragma unroll
                                for (int x = 0; x < 3; ++x)
                                    if (ir - x >= 0 && ir - x < MF && ir - x < a.mf_warp)
#pragma unroll
                                        for (int n = 0; n < NF; ++n) mma_16x8x8(acc[ir - x < 0 ? 0 : ir - x >= MF ? 0 : ir - x][n], ah[ks], &bh[x][n][2 * ks]);
                            }
                        }
                    }
                }
            } else if (FWT) {
                for (int dy = 0; dy < a.FH; ++dy) {
                    const uint32_t row_base = in_t + (uint32_t)(dy * a.Wt) * RB;
#pragma unroll
                    for (int y = 0; y < FWU; ++y) tap_step(dy * FWU + y, row_base, y, 0);
                }
            } else {
                int dy = 0, dx = 0;
                for (int tap = 0; tap < T; ++tap) {
                    tap_step(tap, 0u, 0, dy * a.Wt + dx);
                    if (++dx == a.FW) { dx = 0; ++dy; }
                }
            }

            // STORE phase: accumulator rows lane >> 2 and + 8 are pixels, columns 2 (lane & 3), + 1 of each filter fragment
            int n0, oh0, ow0;
            tile_origin(t, n0, oh0, ow0);
            float *tile_out = a.out + ((((size_t)n0 * a.KB + kt) * a.OH + oh0) * a.OW + ow0) * 32;
            const int n_left = a.N - n0, oh_left = a.OH - oh0, ow_left = a.OW - ow0;
            uint32_t vmask = 0;                                     // bit 2 m + h: this lane stores that pixel
#pragma unroll
            for (int m = 0; m < MF; ++m)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t pk = st_pix[m][h];               // image, row, column of this pixel within the tile
                    if (pk != 0xffffffffu && (int)(pk >> 20) < n_left && (int)((pk >> 10) & 1023u) < oh_left && (int)(pk & 1023u) < ow_left)
                        vmask |= 1u << (2 * m + h);
                }
            if (a.accumulate) {
                // the residual join: all loads of the tensor already in `out` first, so that their latencies overlap
                // (between stores the compiler has to keep them in program order)
                float2 res[MF][2][NF];
#pragma unroll
                for (int m = 0; m < MF; ++m)
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int nf = 0; nf < NF; ++nf)
                            res[m][h][nf] = (vmask >> (2 * m + h) & 1u) ? *reinterpret_cast<const float2 *>(tile_out + st_off[m][h] + 8 * nf)
                                                                        : make_float2(0.0f, 0.0f);
#pragma unroll
                for (int m = 0; m < MF; ++m)
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int nf = 0; nf < NF; ++nf) { acc[m][nf][2 * h] += res[m][h][nf].x; acc[m][nf][2 * h + 1] += res[m][h][nf].y; }
            }
#pragma unroll
            for (int m = 0; m < MF; ++m) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (!(vmask >> (2 * m + h) & 1u)) continue;
                    float *dst = tile_out + st_off[m][h];
#pragma unroll
                    for (int nf = 0; nf < NF; ++nf) {
                        float2 r = make_float2(acc[m][nf][2 * h] + bv[nf][0], acc[m][nf][2 * h + 1] + bv[nf][1]);
                        if (a.relu) { r.x = fmaxf(r.x, 0.0f); r.y = fmaxf(r.y, 0.0f); }
                        if (!(k_real >> (2 * nf) & 1u)) r.x = 0.0f;      // pad lanes stay +0
                        if (!(k_real >> (2 * nf + 1) & 1u)) r.y = 0.0f;
                        *reinterpret_cast<float2 *>(dst + 8 * nf) = r;
                    }
#pragma unroll
                    for (int z = 8 * NF; z < 32; z += 8) *reinterpret_cast<float2 *>(dst + z) = make_float2(0.0f, 0.0f);
                }
            }
        }
        __syncthreads();                    // everyone is done with stage s (and sees `failed`)
        if (failed) break;
    }
    if (failed) {     // a wait ran out: give copies that may still be in flight a bounded grace period
        if (threadIdx.x == 0)
            for (uint32_t k = 0; k < (1u << 14); ++k) __nanosleep(200);
    }
}

typedef void (*MmaKernel)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const MmaArgs);

// One function per (shared-memory row width, math mode), each in its own translation unit (conv_mma_inst*.cu)
MmaKernel pick_mma_16_tf32(int NF, int FW, int S, bool vert);
MmaKernel pick_mma_16_x3(int NF, int FW, int S, bool vert);
MmaKernel pick_mma_32_tf32(int NF, int FW, int S, bool vert);
MmaKernel pick_mma_32_x3(int NF, int FW, int S, bool vert);

template <int NF, int CW, bool X3, int FWT>
MmaKernel pick_mma_s(int S) { return S == 1 ? conv_mma_kernel<NF, 4, CW, 1, X3, FWT> : conv_mma_kernel<NF, 4, CW, 2, X3, FWT>; }
template <int NF, int CW, bool X3>
MmaKernel pick_mma_fw(int FW, int S, bool vert) {
    if (vert && NF <= 2) return conv_mma_kernel<NF <= 2 ? NF : 2, 4, CW, 1, X3, 3, true>;
    return FW == 1 ? pick_mma_s<NF, CW, X3, 1>(S) : FW == 3 ? pick_mma_s<NF, CW, X3, 3>(S) : pick_mma_s<NF, CW, X3, 0>(S);
}
template <int CW, bool X3>
MmaKernel pick_mma_nf(int NF, int FW, int S, bool vert) {
    return NF == 1 ? pick_mma_fw<1, CW, X3>(FW, S, vert) : NF == 2 ? pick_mma_fw<2, CW, X3>(FW, S, vert) : pick_mma_fw<4, CW, X3>(FW, S, vert);
}

}  // namespace mma_conv
}  // namespace small
