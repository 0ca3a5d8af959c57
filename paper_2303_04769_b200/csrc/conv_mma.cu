// Full channel reduction for layers with few channels (one channel block, C <= 32; filters in tiles of 32) on the
// warp-level tensor core instruction (paper Section 3.2 item 4; Algorithms 1 and 2), TF32 and 3xTF32, strides 1 and 2, any window.
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

#include <string>
#include <unordered_map>

#include "conv_mma.cuh"

namespace small {

using namespace mma_conv;

namespace {

struct MmaPlan { MmaArgs a; int NF, MF, CW, warps, es; size_t smem; int per_sm; bool ok; };

size_t round1k(size_t b) { return (b + 1023) & ~(size_t)1023; }

MmaPlan plan_mma(const Geom &g, bool x3, size_t max_smem) {
    MmaPlan p{};
    p.ok = false;
    if (g.CB != 1 || g.KB > 8 || (g.S != 1 && g.S != 2) || g.FH * g.FW > 49) return p;
    MmaArgs &a = p.a;
    a.N = g.N; a.K = g.K; a.OH = g.OH; a.OW = g.OW; a.KB = g.KB; a.FH = g.FH; a.FW = g.FW; a.pt = g.pt; a.pl = g.pl;
    p.NF = g.K <= 8 ? 1 : g.K <= 16 ? 2 : 4;            // several filter tiles: 32 filters each
    a.k_tiles = g.KB;
    a.cs = g.S;
    p.es = (g.FH == 1 && g.FW == 1) ? g.S : 1;       // TMA element stride: a 1 x 1 window fetches only the pixels it uses
    const int S = g.S / p.es;                        // stride between the pixels of the box
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
    const int GM = p.NF >= 4 ? 2 : 4;      // the kernel computes fragments in groups of GM
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
        // rows shared down the window (see VERT in the kernel): fragments of one row, a 3 x 3 window at stride 1, the
        // tile's rows dealt to the warps in whole groups of mf_warp, and at most 16 filters (with 32 the filter
        // fragments of three taps take 96 registers more: 32 -> 32 on 16x16 planes 31.9 us against 23.1 without)
        c.vert = (p.NF <= 2 && a.fwd_shift == 4 && g.FH == 3 && g.FW == 3 && g.S == 1 && c.NI == 1 && rows_f % c.mf_warp == 0 &&
                  (rows_f / c.mf_warp) * a.frags_w == warps) ? 1 : 0;
        c.TH = rows_f * frag_h;
        c.Ht = (c.TH - 1) * S + g.FH;
        c.Wt = ((c.TWd - 1) * S + g.FW + 7) & ~7;      // a multiple of 8: see the kernel's ready-made addresses
        if (c.Ht * p.es > 256 || c.Wt * p.es > 256) continue;
        c.in_box_bytes = (uint32_t)((size_t)c.NI * c.Ht * c.Wt * RB);
        c.stage_bytes = (uint32_t)round1k(c.in_box_bytes);
        const long long tiles = (long long)ceil_div(g.N, c.NI) * c.tiles_h * c.tiles_w;
        if (tiles > 0x3fffffffLL) continue;
        c.n_tiles = (int)tiles;
        const size_t smem = 1024 + (size_t)c.w_half_bytes * (x3 ? 2 : 1) + 2 * (size_t)c.stage_bytes;
        if (smem + 1024 > max_smem) continue;
        int per_sm = (int)((225 * 1024) / (smem + 1024));
        const int reg_warps = p.NF == 4 ? 12 : 16;   // registers per thread: up to 155 (32 filters), else up to 128
        if (per_sm * warps > reg_warps) per_sm = reg_warps / warps;
        if (per_sm < 1) per_sm = 1;
        // resident warps count; idle fragments and few tiles per block cost
        const double fill = (double)c.frags_tile / (warps * c.mf_warp);
        // (more fragments per warp share a tap's filter fragments among more MMAs: worth a little; beyond 12 resident
        // warps nothing is gained - measured on the 16 -> 16 layer: 2 blocks of 8 warps 28.7 us, 3 blocks of 4 warps 26.8)
        const double score = (double)(per_sm * warps > 12 ? 12 : per_sm * warps) * fill * (1.0 + 0.02 * c.mf_warp);
        if (!best.ok || score > best_score) {
            best = p; best.a = c; best.warps = warps; best.smem = smem; best.per_sm = per_sm; best.ok = true;
            best_score = score;
        }
    }
    return best;
}

}  // namespace

bool conv_mma_supported(const Geom &g, bool x3) { return plan_mma(g, x3, 227 * 1024).ok; }

// A finished launch - plan, tensor maps, arguments, kernel - is kept per context by (shape, mode, flags, tensors), so that
// a repeated call (a network step) only launches.
namespace {
struct MmaLaunch { CUtensorMap map_in, map_w, map_w_lo; MmaArgs a; MmaKernel kern; unsigned grid, threads; size_t smem; };
typedef std::unordered_map<std::string, MmaLaunch> MmaCache;
}  // namespace

void free_mma_cache(small_ctx *ctx) {
    delete static_cast<MmaCache *>(ctx->mma_cache);
    ctx->mma_cache = nullptr;
}

int launch_conv_mma(small_ctx *ctx, const float *in, const float *w_hi, const float *w_lo, const float *bias, float *out,
                    const Geom &g, bool relu, bool accumulate, unsigned mode, cudaStream_t st) {
    const bool x3 = mode == SMALL_MATH_3XTF32;
    if (x3 && !w_lo) return SMALL_ERR_INVALID_ARG;
    std::string key;
    {
        const int f[] = {g.N, g.C, g.K, g.H, g.W, g.FH, g.FW, g.S, g.pt, g.pb, g.pl, g.pr, x3 ? 1 : 0, relu ? 1 : 0, accumulate ? 1 : 0, (int)ctx->wait_iters};
        const void *ptrs[] = {in, w_hi, w_lo, bias, out};
        key.append(reinterpret_cast<const char *>(f), sizeof(f));
        key.append(reinterpret_cast<const char *>(ptrs), sizeof(ptrs));
    }
    if (!ctx->mma_cache) ctx->mma_cache = new MmaCache();
    MmaCache &cache = *static_cast<MmaCache *>(ctx->mma_cache);
    {
        auto it = cache.find(key);
        if (it != cache.end()) {
            const MmaLaunch &L = it->second;
            launch_kernel(ctx, L.kern, dim3(L.grid), dim3(L.threads), L.smem, st, L.map_in, L.map_w, L.map_w_lo, L.a);
            return check_launch(ctx);
        }
    }
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
        const cuuint32_t es = (cuuint32_t)p.es;     // element stride 2: a box of 2 Wt x 2 Ht elements lands as Wt x Ht pixels
        cuuint32_t box[5] = {(cuuint32_t)p.CW, (cuuint32_t)a.Wt * es, (cuuint32_t)a.Ht * es, 1, (cuuint32_t)a.NI};
        cuuint32_t estr[5] = {1, es, es, 1, 1};
        CUresult r = encode(&map_in, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<float *>(in), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    for (int half = 0; half < (x3 ? 2 : 1); ++half) {   // filters [1][FH*FW][32 filters][32 ci]: box = CW x 8 NF rows x all taps
        const int T = g.FH * g.FW;
        const cuuint64_t Kp = (cuuint64_t)g.KB * 32;
        cuuint64_t dims[4] = {32, Kp, (cuuint64_t)T, 1};
        cuuint64_t strides[3] = {128, Kp * 128, (cuuint64_t)T * Kp * 128};
        cuuint32_t box[4] = {(cuuint32_t)p.CW, (cuuint32_t)(8 * p.NF), (cuuint32_t)T, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        CUresult r = encode(half ? &map_w_lo : &map_w, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float *>(half ? w_lo : w_hi), dims,
                            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    if (!x3) map_w_lo = map_w;
    const MmaKernel kern = p.CW == 16 ? (x3 ? pick_mma_16_x3(p.NF, g.FW, g.S / p.es, a.vert) : pick_mma_16_tf32(p.NF, g.FW, g.S / p.es, a.vert))
                                        : (x3 ? pick_mma_32_x3(p.NF, g.FW, g.S / p.es, a.vert) : pick_mma_32_tf32(p.NF, g.FW, g.S / p.es, a.vert));
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->max_smem_optin - 1024);   // the kernel has static shared memory too
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    // persistent blocks: as many as are resident at once (a multiple of the filter tiles), or one per (pixel, filter) tile
    long long slots = (long long)ctx->sm_count * p.per_sm / a.k_tiles;
    if (slots < 1) slots = 1;
    const unsigned grid = (unsigned)((a.n_tiles < slots ? a.n_tiles : slots) * a.k_tiles);
    if (cache.size() >= 4096) cache.clear();
    cache[key] = MmaLaunch{map_in, map_w, map_w_lo, a, kern, grid, (unsigned)(32 * p.warps), p.smem};
    launch_kernel(ctx, kern, dim3(grid), dim3(32 * p.warps), p.smem, st, map_in, map_w, map_w_lo, a);
    return check_launch(ctx);
}

}  // namespace small
