// Full channel reduction for layers with few channels and few filters (at most 32 of each) on the warp-level tensor
// core instruction (paper Section 3.2 item 4; Algorithms 1 and 2), TF32 and 3xTF32, strides 1 and 2, any window.
//
// Why a second tensor-core kernel.  The block-level MMA of conv_tc.cu works on 128 rows and reads both operands from
// shared memory: whatever its N, one 128 x N x 8 step costs the pipe 40 to 52 cycles, so a layer with 16 filters fills
// an eighth of what it pays for.  The warp-level m16n8k8 MMA has no such floor - 16 pixels x 8 filters x 8 channels is
// the whole instruction - and runs at 512 multiply-adds per clock and SM (measured), all of them useful here.
//
// Mapping of the paper's loop nest (Algorithm 1):
//   O_wb x K_b kernel tile          -> a warp's MF fragments of 16 output pixels x all filters of the layer (NF
//                                      fragments of 8), accumulators in registers
//   j, l loops over the output      -> tiles of (images x rows x columns) walked by persistent thread blocks; a tile's
//                                      fragments are dealt to the block's warps
//   x, y kernel loops               -> taps: the SAME halo tile in shared memory is read again at a shifted pixel
//   ii loop                         -> K steps of 8 channels, two per ldmatrix of a filter fragment
//   LOAD / STORE phases             -> bias, (+ previous output), ReLU, 8-byte stores straight from the accumulators
// The halo tile keeps the blocked layout's [pixel][channel] order (TMA box, swizzled; pixels outside the plane are
// TMA's zero fill = the padding) and so do the filters ([tap][filter][channel], the tensor-core section of the packed
// filter buffer), which makes both operands plain ldmatrix reads: a matrix row is one pixel's (or filter's) 16 bytes
// of four channels.  The swizzle makes eight consecutive rows fall into eight different bank groups.
// 3xTF32: x = x_hi + x_lo split in registers after the load, filters arrive split; x_lo w_hi + x_hi w_lo + x_hi w_hi.
#include <cuda.h>

#include "common.cuh"
#include "sm100.cuh"

namespace small {

namespace {

struct MmaArgs {
    const float *bias; float *out; int *status;
    int N, K, OH, OW, KB, FH, FW, pt, pl;
    int fwd_shift;             // a fragment is (16 >> fwd_shift) rows x (1 << fwd_shift) columns of one image
    int TH, TWd, NI;           // output rows, columns and images of a tile
    int Ht, Wt;                // halo box: rows and columns per image
    int tiles_w, tiles_h, n_tiles;
    int frags_w, frags_img, frags_tile;   // fragments per fragment row, per image of a tile, per tile (the rest idle)
    int mf_warp;               // fragments per warp actually used (<= MF)
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
template <int NF, int MF, int CW, int S, bool X3, int FWT>
__global__ void __launch_bounds__(256)
conv_mma_kernel(const __grid_constant__ CUtensorMap map_in, const __grid_constant__ CUtensorMap map_w,
                const __grid_constant__ CUtensorMap map_w_lo, const MmaArgs a) {
    constexpr uint32_t RB = CW * 4;                 // bytes per pixel / filter row
    constexpr int RSH = CW == 16 ? 6 : 7;
    constexpr int PAIRS = CW / 16;
    constexpr int GM = NF >= 4 ? 1 : NF == 2 ? 2 : 4;   // pixel fragments whose MMAs are interleaved
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

    auto tile_origin = [&](int t, int &n0, int &oh0, int &ow0) {
        const int wt = t % a.tiles_w; t /= a.tiles_w;
        const int band = t % a.tiles_h;
        n0 = (t / a.tiles_h) * a.NI; oh0 = band * a.TH; ow0 = wt * a.TWd;
    };
    auto issue = [&](int t, int s) {
        int n0, oh0, ow0;
        tile_origin(t, n0, oh0, ow0);
        sm100::mbar_expect_tx(bar_in + 8 * s, a.in_box_bytes);
        sm100::tma_load_5d(in_s + s * a.stage_bytes, &map_in, bar_in + 8 * s, 0, ow0 * S - a.pl, oh0 * S - a.pt, 0, n0);
    };

    if (threadIdx.x == 0) {
        sm100::mbar_init(bar_w, 1); sm100::mbar_init(bar_in, 1); sm100::mbar_init(bar_in + 8, 1);
        sm100::mbar_fence_init();
        failed = 0;
    }
    __syncthreads();
    if (threadIdx.x == 0) {       // the filters are the layer's own constants: no earlier kernel of the stream writes them
        sm100::mbar_expect_tx(bar_w, a.w_box_bytes * (X3 ? 2u : 1u));
        sm100::tma_load_4d(w_hi_s, &map_w, bar_w, 0, 0, 0, 0);
        if (X3) sm100::tma_load_4d(w_lo_s, &map_w_lo, bar_w, 0, 0, 0, 0);
    }
    grid_dep_sync();
    grid_dep_trigger();
    if (threadIdx.x == 0 && (int)blockIdx.x < a.n_tiles) issue(blockIdx.x, 0);

    // this lane's part in the loads: row (lane & 7) of matrix (lane >> 3)
    // A: matrices 0 / 1 = pixels 0-7 / 8-15 of the fragment at the K step's first 4 channels, 2 / 3 = the next 4
    // B: matrices 0 .. 3 = 16-byte chunks 0 .. 3 of a pair of K steps, rows = the fragment's 8 filters
    const int FWD = 1 << a.fwd_shift;
    const int jl = (lane & 7) | (((lane >> 3) & 1) << 3);          // pixel of the fragment this lane addresses
    const int a_chunk = lane >> 4;
    int p_lane[MF];                                                // its pixel index in the halo box at tap (0, 0)
    uint32_t pre[FWU][MF];                                         // byte offset of its 16 bytes at window column y, row 0
#pragma unroll
    for (int m = 0; m < MF; ++m) {
        int f = warp * a.mf_warp + m;
        if (m >= a.mf_warp || f >= a.frags_tile) f = 0;            // idle fragments read in bounds and store nothing
        const int img = f / a.frags_img, rem = f - img * a.frags_img;
        const int frow = rem / a.frags_w, fcol = rem - frow * a.frags_w;
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
            const int k = 8 * n + 2 * (lane & 3) + e;
            bv[n][e] = (a.bias && k < a.K) ? a.bias[k] : 0.0f;
            if (k < a.K) k_real |= 1u << (2 * n + e);
        }
    // the pixels this lane stores (accumulator rows lane >> 2 and + 8 of each fragment): (image, row, column) within a
    // tile, packed 12 + 10 + 10 bits, and the offset in floats from the tile's first output pixel; the same for every tile
    uint32_t st_pix[MF][2];
    int st_off[MF][2];
#pragma unroll
    for (int m = 0; m < MF; ++m) {
        const int f = warp * a.mf_warp + m;
        const bool used = m < a.mf_warp && f < a.frags_tile;
        const int ff = used ? f : 0;
        const int img = ff / a.frags_img, rem = ff - img * a.frags_img;
        const int frow = rem / a.frags_w, fcol = rem - frow * a.frags_w;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int j = (lane >> 2) + 8 * h;
            const int row = frow * (16 >> a.fwd_shift) + (j >> a.fwd_shift), col = fcol * FWD + (j & (FWD - 1));
            st_pix[m][h] = used ? ((uint32_t)img << 20) | ((uint32_t)row << 10) | (uint32_t)col : 0xffffffffu;
            st_off[m][h] = ((img * a.OH + row) * a.OW + col) * 32 + 2 * (lane & 3);
        }
    }

    bool w_ready = false;
    int it = 0;
    for (int t = blockIdx.x; t < a.n_tiles; t += gridDim.x, ++it) {
        const int s = it & 1;
        // the other stage was last read before the block-wide barrier that ended the previous tile
        if (threadIdx.x == 0 && t + (int)gridDim.x < a.n_tiles) issue(t + gridDim.x, s ^ 1);
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
            if (FWT) {
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
            float *tile_out = a.out + ((((size_t)n0 * a.OH) + oh0) * a.OW + ow0) * 32;
            const int n_left = a.N - n0, oh_left = a.OH - oh0, ow_left = a.OW - ow0;
#pragma unroll
            for (int m = 0; m < MF; ++m) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t pk = st_pix[m][h];               // image, row, column of this pixel within the tile
                    if (pk == 0xffffffffu || (int)(pk >> 20) >= n_left || (int)((pk >> 10) & 1023u) >= oh_left || (int)(pk & 1023u) >= ow_left) continue;
                    float *dst = tile_out + st_off[m][h];
#pragma unroll
                    for (int nf = 0; nf < NF; ++nf) {
                        float2 r = make_float2(acc[m][nf][2 * h] + bv[nf][0], acc[m][nf][2 * h + 1] + bv[nf][1]);
                        float2 *d2 = reinterpret_cast<float2 *>(dst + 8 * nf);
                        if (a.accumulate) { const float2 o = *d2; r.x += o.x; r.y += o.y; }
                        if (a.relu) { r.x = fmaxf(r.x, 0.0f); r.y = fmaxf(r.y, 0.0f); }
                        if (!(k_real >> (2 * nf) & 1u)) r.x = 0.0f;      // pad lanes stay +0
                        if (!(k_real >> (2 * nf + 1) & 1u)) r.y = 0.0f;
                        *d2 = r;
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

struct MmaPlan { MmaArgs a; int NF, MF, CW, warps; size_t smem; int per_sm; bool ok; };

size_t round1k(size_t b) { return (b + 1023) & ~(size_t)1023; }

MmaPlan plan_mma(const Geom &g, bool x3, size_t max_smem) {
    MmaPlan p{};
    p.ok = false;
    if (g.CB != 1 || g.KB != 1 || (g.S != 1 && g.S != 2) || g.FH * g.FW > 49) return p;
    MmaArgs &a = p.a;
    a.N = g.N; a.K = g.K; a.OH = g.OH; a.OW = g.OW; a.KB = g.KB; a.FH = g.FH; a.FW = g.FW; a.pt = g.pt; a.pl = g.pl;
    p.NF = g.K <= 8 ? 1 : g.K <= 16 ? 2 : 4;
    p.CW = g.C <= 16 ? 16 : 32;
    p.MF = 4;
    a.fwd_shift = g.OW >= 12 ? 4 : g.OW >= 6 ? 3 : 2;
    const int FWD = 1 << a.fwd_shift, frag_h = 16 >> a.fwd_shift;
    const int fw_total = ceil_div(g.OW, FWD), fh_total = ceil_div(g.OH, frag_h);
    a.frags_w = fw_total <= 4 ? fw_total : 2;
    a.tiles_w = ceil_div(fw_total, a.frags_w);
    a.TWd = a.frags_w * FWD;
    const int RB = p.CW * 4;
    const int T = g.FH * g.FW;
    a.w_box_bytes = (uint32_t)((size_t)T * p.NF * 8 * RB);
    a.w_half_bytes = (uint32_t)round1k(a.w_box_bytes);
    // fragments per tile: 4 warps x 4, or 8 warps x 4 where the halo tiles stay small; a tile is a band of fragment
    // rows of one image, or several whole images
    MmaPlan best{};
    best.ok = false;
    double best_score = 0.0;
    const int GM = p.NF >= 4 ? 1 : p.NF == 2 ? 2 : 4;      // the kernel computes fragments in groups of GM
    for (int warps = 2; warps <= 8; warps *= 2)
    for (int mfw = p.MF; mfw >= GM; mfw /= 2) {
        const int F = warps * mfw;
        MmaArgs c = a;
        int rows_f;
        if (fh_total * a.frags_w <= F) {
            rows_f = fh_total; c.NI = F / (rows_f * a.frags_w); c.tiles_h = 1;
            if (c.NI > g.N) c.NI = g.N;
            if (c.NI > 256) c.NI = 256;
        } else {
            rows_f = F / a.frags_w; if (rows_f < 1) continue;
            c.tiles_h = ceil_div(fh_total, rows_f);
            rows_f = ceil_div(fh_total, c.tiles_h);       // balanced bands
            c.NI = 1;
        }
        c.frags_img = rows_f * a.frags_w;
        c.frags_tile = c.frags_img * c.NI;
        c.mf_warp = ceil_div(ceil_div(c.frags_tile, warps), GM) * GM;
        if (c.mf_warp > p.MF) continue;
        c.TH = rows_f * frag_h;
        c.Ht = (c.TH - 1) * g.S + g.FH;
        c.Wt = ((c.TWd - 1) * g.S + g.FW + 7) & ~7;      // a multiple of 8: see the kernel's ready-made addresses
        if (c.Ht > 256 || c.Wt > 256) continue;
        c.in_box_bytes = (uint32_t)((size_t)c.NI * c.Ht * c.Wt * RB);
        c.stage_bytes = (uint32_t)round1k(c.in_box_bytes);
        const long long tiles = (long long)ceil_div(g.N, c.NI) * c.tiles_h * c.tiles_w;
        if (tiles > 0x3fffffffLL) continue;
        c.n_tiles = (int)tiles;
        const size_t smem = 1024 + (size_t)c.w_half_bytes * (x3 ? 2 : 1) + 2 * (size_t)c.stage_bytes;
        if (smem + 1024 > max_smem) continue;
        int per_sm = (int)((225 * 1024) / (smem + 1024));
        const int reg_warps = p.NF == 4 ? 12 : 16;         // registers: up to 140 (32 filters) or 100 per thread
        if (per_sm * warps > reg_warps) per_sm = reg_warps / warps;
        if (per_sm < 1) per_sm = 1;
        // resident warps count; idle fragments and few tiles per block cost
        const double fill = (double)c.frags_tile / (warps * c.mf_warp);
        // (more fragments per warp share a tap's filter fragments among more MMAs: worth a little)
        const double score = (double)(per_sm * warps > 12 ? 12 : per_sm * warps) * fill * (1.0 + 0.02 * c.mf_warp);
        if (!best.ok || score > best_score) {
            best = p; best.a = c; best.warps = warps; best.smem = smem; best.per_sm = per_sm; best.ok = true;
            best_score = score;
        }
    }
    return best;
}

typedef void (*MmaKernel)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const MmaArgs);

template <int NF, int CW, int FWT>
MmaKernel pick_mma3(int S, bool x3) {
    if (S == 1) return x3 ? conv_mma_kernel<NF, 4, CW, 1, true, FWT> : conv_mma_kernel<NF, 4, CW, 1, false, FWT>;
    return x3 ? conv_mma_kernel<NF, 4, CW, 2, true, FWT> : conv_mma_kernel<NF, 4, CW, 2, false, FWT>;
}
template <int NF, int CW>
MmaKernel pick_mma2(int FW, int S, bool x3) {
    return FW == 1 ? pick_mma3<NF, CW, 1>(S, x3) : FW == 3 ? pick_mma3<NF, CW, 3>(S, x3) : pick_mma3<NF, CW, 0>(S, x3);
}
MmaKernel pick_mma(int NF, int CW, int FW, int S, bool x3) {
    if (CW == 16) return NF == 1 ? pick_mma2<1, 16>(FW, S, x3) : NF == 2 ? pick_mma2<2, 16>(FW, S, x3) : pick_mma2<4, 16>(FW, S, x3);
    return NF == 1 ? pick_mma2<1, 32>(FW, S, x3) : NF == 2 ? pick_mma2<2, 32>(FW, S, x3) : pick_mma2<4, 32>(FW, S, x3);
}

}  // namespace

bool conv_mma_supported(const Geom &g, bool x3) { return plan_mma(g, x3, 227 * 1024).ok; }

int launch_conv_mma(small_ctx *ctx, const float *in, const float *w_hi, const float *w_lo, const float *bias, float *out,
                    const Geom &g, bool relu, bool accumulate, unsigned mode, cudaStream_t st) {
    const bool x3 = mode == SMALL_MATH_3XTF32;
    if (x3 && !w_lo) return SMALL_ERR_INVALID_ARG;
    MmaPlan p = plan_mma(g, x3, ctx->max_smem_optin);
    if (!p.ok) return SMALL_ERR_UNSUPPORTED;
    MmaArgs &a = p.a;
    a.bias = bias; a.out = out; a.status = ctx->dev_status; a.relu = relu; a.accumulate = accumulate; a.wait_iters = ctx->wait_iters;
    sm100::EncodeTiledFn encode = reinterpret_cast<sm100::EncodeTiledFn>(ctx->encode_tiled);
    const CUtensorMapSwizzle swz = p.CW == 16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
    CUtensorMap map_in, map_w, map_w_lo;
    {   // activations [N][1][H][W][32]: box = CW channels x Wt x Ht x 1 x NI images; outside the tensor reads as zero
        cuuint64_t dims[5] = {32, (cuuint64_t)g.W, (cuuint64_t)g.H, 1, (cuuint64_t)g.N};
        cuuint64_t strides[4] = {128, (cuuint64_t)g.W * 128, (cuuint64_t)g.H * g.W * 128, (cuuint64_t)g.H * g.W * 128};
        cuuint32_t box[5] = {(cuuint32_t)p.CW, (cuuint32_t)a.Wt, (cuuint32_t)a.Ht, 1, (cuuint32_t)a.NI};
        cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        CUresult r = encode(&map_in, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<float *>(in), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    for (int half = 0; half < (x3 ? 2 : 1); ++half) {   // filters [1][FH*FW][32 filters][32 ci]: box = CW x 8 NF rows x all taps
        const int T = g.FH * g.FW;
        cuuint64_t dims[4] = {32, 32, (cuuint64_t)T, 1};
        cuuint64_t strides[3] = {128, 32 * 128, (cuuint64_t)T * 32 * 128};
        cuuint32_t box[4] = {(cuuint32_t)p.CW, (cuuint32_t)(8 * p.NF), (cuuint32_t)T, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        CUresult r = encode(half ? &map_w_lo : &map_w, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float *>(half ? w_lo : w_hi), dims,
                            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    if (!x3) map_w_lo = map_w;
    const MmaKernel kern = pick_mma(p.NF, p.CW, g.FW, g.S, x3);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->max_smem_optin - 1024);   // the kernel has static shared memory too
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    const long long slots = (long long)ctx->sm_count * p.per_sm;
    const unsigned grid = (unsigned)(a.n_tiles < slots ? a.n_tiles : slots);
    launch_kernel(ctx, kern, dim3(grid), dim3(32 * p.warps), p.smem, st, map_in, map_w, map_w_lo, a);
    return check_launch(ctx);
}

}  // namespace small
