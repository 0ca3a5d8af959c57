// Full channel reduction on the tensor cores (paper Section 3.2 item 4; Algorithms 1 and 2), strides 1 and 2: an
// implicit GEMM straight from the blocked layout, with no im2col buffer and no reformatting (Section 4.4).
//
//   D[k, pixel] = sum over (channel block cb, tap (x,y), 32 channels ci)  W[k, ci] * X[pixel + shift(x,y), ci]
//
// How the paper's loop nest maps onto the SM:
//   k block loop (parallel)        -> filter tiles, one tile = (pixel tile, filter tile); groups = filter tiles too
//   i loop over F_C in F_Cb steps  -> cb loop over 32-channel blocks: one TMA box of the input per block
//   x, y kernel loops              -> taps: the SAME shared-memory strip is re-read with a shifted start address
//   ii loop                        -> up to four K=8 TF32 MMAs per 32-channel block (tcgen05.mma kind::tf32)
//   O_wb x K_b register tile       -> accumulator slots in tensor memory (2 slots x 256 columns x 128 lanes)
//   LOAD / STORE phases            -> epilogue: tensor memory -> registers, + bias, (+ previous output), ReLU, store
//
// Two orientations, chosen per layer by the host's cost model.  Filters on the MMA's M axis: 128 filters x up to 256
// pixels per slot; the accumulator comes out as [filter][pixel], a warp holds 32 consecutive filters of one pixel =
// one 128-byte line of the blocked output, so its 4-byte stores are fully coalesced.  Pixels on M: 128-pixel chunks x
// up to 256 filters; a thread holds 32 filters of its pixel and stores the line as four 32-byte vectors - the choice for
// layers with few filters, where M = 128 filters would be mostly padding.  The pipe needs N / 2 cycles per 128 x N x 8
// MMA for N >= 128 and 40 to 52 cycles below that, whatever M is (measured with this library's issue probe).
//
// The strip.  A blocked input plane is [H][W][32 floats]: one pixel and channel block = one 128-byte row, the K-major
// operand row of a TF32 MMA with the 128-byte swizzle.  TMA copies a box of Rs rows x Wq pixels (starting at column
// -pad_l, row -pad_t of the tile, out-of-range elements filled with zeros = the padding) densely into shared memory.
// With the row pitch Wq = W + max(pad_l, pad_r), the right padding of one row and the left padding of the next are the
// same zero pixels, so the strip is the zero-padded image flattened to one pixel sequence, and output pixel q (also
// numbered with pitch Wq) needs strip pixel q + x*Wq + y for tap (x, y).  Any run of consecutive q is a valid MMA
// operand: rows 128 bytes apart, start address (q + x*Wq + y) * 128.  Columns ow >= OW of each row are computed and
// dropped.  Small planes put several whole images in one strip the same way (image pitch Hq = H + max(pad_t, pad_b)).
// Stride 2 is a stride-1 window over the input's phase planes (see Virt); 3xTF32 and the fused depthwise layer put a
// transform between the copy and the MMAs (see the X3 and DW template flags).
//
// Persistent CTAs (one per SM) walk the tile list with stride gridDim.x.  Roles: warp 0 = TMA producer for input
// strips, warp 2 = TMA producer for filter tiles, warps 1 and 3 = MMA issuers (one thread each; a tile's chains are
// split between them), warps 4-7 = epilogue, warps 8 and up = strip transform where there is one.  The producers run
// ahead across tiles; accumulator slots are handed back to the issuers as soon as the epilogue has read them out of
// tensor memory, so the next tile's MMAs overlap the current tile's stores (one-slot tiles alternate between the two
// slots).  Every mbarrier wait is bounded; on expiry the kernel records SMALL_ERR_TIMEOUT in the context's status
// word, lets its in-flight copies land, frees tensor memory and returns.
#include <cuda.h>

#include <mutex>
#include <string>
#include <type_traits>
#include <unordered_map>

#include "common.cuh"
#include "sm100.cuh"

namespace small {

namespace {

using namespace sm100;

constexpr int kThreads = 256;            // roles of the TF32 kernel; the 3xTF32 kernel adds four splitting warps
constexpr int kThreadsX3 = 384;
constexpr int kThreadsDW = 512;          // fused depthwise: eight warps compute the strips
constexpr int kSlots = 2;              // accumulator slots of 256 tensor-memory columns
constexpr int kSlotPx = 256;           // pixels per slot = the MMA's largest N
constexpr int kFilterTile = 128;       // filters per tile = the MMA's M
constexpr int kMaxAStages = 6;         // input strips in flight (at least 2; as many as shared memory allows)
constexpr int kMaxBStages = 8;
constexpr int kRawStages = 2;           // fused depthwise: halo tiles in flight
constexpr int kCtrlBarrierBytes = 24 * kMaxAStages + 16 * kMaxBStages + 16 * kSlots + 16 * kRawStages;   // all mbarriers
constexpr int kTapTabEntries = 4 * 64;   // original tap of every (phase plane, view tap), -1 where the view tap has none

struct TcPlan {
    int OH, OW, Wq, Hq;
    int nn;              // images per strip (1: runs of pixels of one image)
    int px_tile;         // pixels per tile (multiple of 16, at most kSlots * kSlotPx)
    int px_img;          // nn == 1: pixels of one image in the flattened padded numbering (OH * Wq)
    int tiles_img;       // nn == 1: tiles per image
    int m_tiles;         // pixel tiles in the grid
    int Rs;              // box rows (per image)
    int strip_px, tail_px, stage_px;
    int n_tiles;         // filter tiles
    int w_rows;          // rows of the filter box (min(128, padded filters))
    int a_stages, b_stages;
    int pixel_m;         // 1: pixels are the MMA's M rows (128 per chunk) and filters its N; 0: the other way round
    int w_tile;          // filters per tile: 128 (filters on M) or up to 256 (filters on N)
    int cps;             // pixel_m: 128-pixel chunks per accumulator slot (4, 2 or 1 for up to 64, 128 or 256 filters)
    int b_resident;      // all filter tiles of the layer stay in shared memory for the whole kernel
    int racc;            // accumulators per slot, 256 / racc tensor-memory columns apart (bounds the accumulation chains)
    uint32_t raw_stage_bytes; int dw_Hb, dw_Wb, dw_rows;   // fused depthwise: halo tile per (tile, channel block)
    int x_packed;        // 3xTF32 with one channel block of <= 16 channels: hi in lanes [0, h), lo in [h, 2h) of each row
    int x3;              // 3xTF32: stages hold both halves, three MMAs per K step
    int x3_wide;         // 3xTF32, pixels on M, at most 64 filters: two MMAs per K step, the first over both filter halves
    double taps_eff;     // taps per block that exist (a stride-2 view has empty ones)
    int ks_last;         // K steps (8 channels each) of the last channel block that hold real channels
    uint32_t a_stage_bytes, b_stage_bytes, smem_bytes;
    uint32_t a_half, b_half;   // 3xTF32: each stage holds the TF32 part and, a_half / b_half bytes on, the residual
    bool ok;
};

struct TcArgs {
    const float *bias; float *out; int *status;
    int N, K, KB, CB, OH, OW, Wq, Hq, FH, FW, pt, pl;   // CB, FH, FW, pt, pl: the stride-1 view (see Virt)
    int S, n_phase, CBr, phase_bits, FHo, FWo, pto, plo;  // stride, phase planes, real channel blocks, original window
    int nn, px_tile, px_img, tiles_img, m_tiles, n_tiles, strip_px, tail_px, w_rows;
    int a_stages, b_stages, pixel_m, w_tile, cps, b_resident, ks_last;
    int rows_tile;       // whole rows per tile when every tile starts at a row start, else 0
    int cb_group;        // group convolution: channel blocks per group (filter tile g reads blocks g * cb_group ..), else 0
    int slots, n_slot;   // accumulator slots per tile and pixels per slot: the same for every tile of the layer
    uint32_t a_stage_bytes, b_stage_bytes, a_box_bytes;
    uint32_t a_half, b_half;   // 3xTF32: byte offset of the residual half of a strip stage / filter stage
    int racc;                  // accumulators per slot that the channel blocks rotate over (filters on M only)
    // fused depthwise 3x3 in front of a 1x1 convolution: the strips are computed in shared memory from halo tiles
    const float *dw_w; const float *dw_bias;   // depthwise filters [CB][9][32] and bias (C floats or null)
    int dw_s, dw_Wb, dw_Hb, dw_pt, dw_pl, dw_relu, dw_rows, dw_C;   // stride, halo box, pads, ReLU, strip rows per image
    uint32_t raw_stage_bytes, raw_box_bytes;
    int x_packed;              // 3xTF32, at most 16 channels: the residual sits in the unused lanes of the same row
    int x3_wide;               // 3xTF32, pixels on M: x_hi meets [w_hi; w_lo] in one MMA of twice the filters (see the issue loop)
    int alt_tiles;             // one chain per tile: the two MMA threads take alternate tiles (else warp 1 issues everything)
    uint32_t x_lo_off;         // 3xTF32: 16-byte units from a strip's TF32 part to its residual
    int relu, accumulate;
    uint32_t wait_iters;       // limit of every bounded wait (polls)
};

// ---------------------------------------------------------------------------------------------- kernel
// One tile: `px` pixels starting at flattened index q0 of image n0 (nn == 1) or of the strip of images n0.. (nn > 1),
// split over `slots` accumulator slots of `n_slot` pixels each (a multiple of 16), and filter tile n_tile.
struct Tile { int n_tile, n0, q0, row0, a0, px, slots, n_slot; };

__device__ __forceinline__ Tile decode_tile(const TcArgs &a, int t) {
    Tile r;
    // the common shapes (one filter tile, one tile per image, row-aligned tiles) need no division at all
    int m_tile = t;
    r.n_tile = 0;
    if (a.n_tiles > 1) { m_tile = (int)((unsigned)t / (unsigned)a.n_tiles); r.n_tile = t - m_tile * a.n_tiles; }
    if (a.nn == 1) {
        r.n0 = a.tiles_img > 1 ? (int)((unsigned)m_tile / (unsigned)a.tiles_img) : m_tile;
        const int ti = m_tile - r.n0 * a.tiles_img;
        r.q0 = ti * a.px_tile;
        r.px = min(a.px_tile, a.px_img - r.q0);
        if (a.rows_tile > 0) { r.row0 = ti * a.rows_tile; r.a0 = 0; }
        else { r.row0 = (int)((unsigned)r.q0 / (unsigned)a.Wq); r.a0 = r.q0 - r.row0 * a.Wq; }
    } else {
        r.n0 = m_tile * a.nn;
        r.q0 = 0; r.row0 = 0; r.a0 = 0;
        r.px = a.px_tile;
    }
    // every tile takes the slots of a full tile; a ragged last tile leaves the tail of them unused
    r.slots = a.slots;
    r.n_slot = a.n_slot;
    return r;
}

// CH: MMA chains per tile (accumulator slots with filters on M, 128-pixel chunks with pixels on M); KS_LAST: K steps
// of the last channel block that hold real channels (1, 2 or 4); PM: pixels on the MMA's M axis;
// MASKED: some view taps do not exist (stride-2 layers).  They are template
// parameters so that the single issuing thread runs straight-line code: with run-time chain and K-step counts every
// MMA costs it about 100 cycles of branches and selects, more than a small MMA occupies the pipe (measured).
// X3: 3xTF32.  Every FP32 operand is split into its TF32 part and the residual (x = x_hi + x_lo, w = w_hi + w_lo) and
// each K step issues x_lo*w_hi, x_hi*w_lo and x_hi*w_hi into the same FP32 accumulator (x_lo*w_lo is below FP32
// resolution).  Filters arrive split (packed so); the activations are split in shared memory by four extra warps as
// each strip lands: hi = the top 19 bits, in place; lo = x - hi, exact, in the second half of the stage.
// DW: a depthwise 3x3 (+ bias, ReLU) is computed in front of this 1x1 convolution: TMA loads halo tiles of the layer's
// input, warps 8-11 compute the depthwise result straight into the strip the MMAs read (and split it for 3xTF32),
// so the depthwise output never goes to global memory.
template <int CH, int KS_LAST, bool PM, bool MASKED, bool X3, bool DW>
__global__ void __launch_bounds__(DW ? kThreadsDW : X3 ? kThreadsX3 : kThreads, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_b_lo, const TcArgs a) {
    constexpr int kNT = DW ? kThreadsDW : X3 ? kThreadsX3 : kThreads;
    constexpr int kXform = DW ? 256 : 128;     // threads that split (3xTF32) or compute (fused depthwise) the strips
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t a_base = base;
    const int kAStages = a.a_stages;
    const uint32_t b_base = a_base + kAStages * a.a_stage_bytes;
    const uint32_t kBStageBytes = a.b_stage_bytes;
    const uint32_t raw_base = b_base + a.b_stages * kBStageBytes;          // fused depthwise: halo tiles (no swizzle)
    const uint32_t ctrl = raw_base + (DW ? kRawStages * a.raw_stage_bytes : 0u);
    uint8_t *ctrl_ptr = base_ptr + (ctrl - base);
    // control block: barriers (8 bytes each), tensor-memory address, abort flag, bias for all filters
    const uint32_t bar_a_full = ctrl, bar_a_empty = ctrl + 8 * kMaxAStages;
    const uint32_t bar_a_split = ctrl + 16 * kMaxAStages;      // 3xTF32: strip split into hi and lo
    const uint32_t bar_b_full = ctrl + 24 * kMaxAStages, bar_b_empty = bar_b_full + 8 * kMaxBStages;
    const uint32_t bar_slot_full = bar_b_empty + 8 * kMaxBStages, bar_slot_free = bar_slot_full + 8 * kSlots;
    const uint32_t bar_raw_full = bar_slot_free + 8 * kSlots, bar_raw_empty = bar_raw_full + 8 * kRawStages;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(ctrl_ptr + kCtrlBarrierBytes);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(ctrl_ptr + kCtrlBarrierBytes + 4);
    float *bias_s = reinterpret_cast<float *>(ctrl_ptr + kCtrlBarrierBytes + 16);
    volatile short *tap_tab = reinterpret_cast<volatile short *>(ctrl_ptr + kCtrlBarrierBytes + 16 + (size_t)a.KB * 32 * 4);
    float *dw_s_w = reinterpret_cast<float *>(ctrl_ptr + kCtrlBarrierBytes + 16 + (size_t)a.KB * 32 * 4 + kTapTabEntries * sizeof(short));   // [CB][10][32]: 9 taps + bias

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Two issuing threads (warps 1 and 3, on different schedulers): issuing a small MMA costs a thread about twice the
    // cycles the pipe needs to run it.  A tile's MMA chains are split between them; an odd number of chains is split the
    // other way round on odd tiles (chains [0, kSplit) and [kSplit, CH) on even tiles, [0, CH - kSplit) and the rest on
    // odd ones), so that both issue the same number of MMAs over two tiles.  With one chain per tile the two threads take
    // alternate tiles where the MMAs are small enough to be issue-bound (alt_tiles; measured: the 32 -> 32 layer of the
    // residual CNN 32.4 -> 26.6 us in 3xTF32; the host side leaves it off today, see there), else warp 1 issues alone: a second thread that only walks the barriers
    // cost the TF32 step 6 us.  Both threads walk every tile and every barrier; only the chains they issue for differ.
    // (TF32 kernels keep the fixed split and the single thread: alternating measured 7 us slower per step there.)
    const int kIssuers = (CH >= 2 || (X3 && a.alt_tiles)) ? 2 : 1;
    constexpr int kSplit = (CH + 1) / 2, kOddSplit = X3 ? CH - kSplit : kSplit;      // chains of warp 1 on even / odd tiles
    const int T = a.FH * a.FW;
    const int total_tiles = a.m_tiles * a.n_tiles;

    if (threadIdx.x == 0) {
        // every MMA issuer commits to the stage-empty and slot-full barriers; 4 epilogue warps free a slot
        for (int s = 0; s < kAStages; ++s) { mbar_init(bar_a_full + 8 * s, 1); mbar_init(bar_a_empty + 8 * s, kIssuers); mbar_init(bar_a_split + 8 * s, kXform); }
        for (int s = 0; s < a.b_stages; ++s) { mbar_init(bar_b_full + 8 * s, 1); mbar_init(bar_b_empty + 8 * s, kIssuers); }
        for (int s = 0; s < kSlots; ++s) { mbar_init(bar_slot_full + 8 * s, kIssuers); mbar_init(bar_slot_free + 8 * s, 4); }
        for (int s = 0; s < kRawStages; ++s) { mbar_init(bar_raw_full + 8 * s, 1); mbar_init(bar_raw_empty + 8 * s, kXform); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // zero tail behind each strip: the padding pixels a row (or image) wrap runs into after the last strip row
    for (int s = 0; s < kAStages; ++s) {
        float4 *tail = reinterpret_cast<float4 *>(base_ptr + (size_t)s * a.a_stage_bytes + (size_t)a.strip_px * 128);
        for (int i = threadIdx.x; i < a.tail_px * 8; i += kNT) tail[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // filter rows the TMA box does not cover (fewer than 128 filters in the layer) stay zero for the whole kernel
    if (!PM && a.w_rows < kFilterTile)
        for (int s = 0; s < a.b_stages; ++s) {
            float4 *rest = reinterpret_cast<float4 *>(base_ptr + (b_base - base) + (size_t)s * kBStageBytes + (size_t)a.w_rows * 128);
            for (int i = threadIdx.x; i < (kFilterTile - a.w_rows) * 8; i += kNT) {
                rest[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (X3) rest[i + a.b_half / 16] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    for (int i = threadIdx.x; i < a.KB * 32; i += kNT) bias_s[i] = (a.bias && i < a.K) ? a.bias[i] : 0.0f;
    if (DW)
        for (int i = threadIdx.x; i < a.CBr * 10 * 32; i += kNT) {
            const int cb = i / 320, rest = i - cb * 320, tap = rest >> 5, c = rest & 31;
            dw_s_w[i] = tap < 9 ? a.dw_w[(cb * 9 + tap) * 32 + c] : (a.dw_bias && cb * 32 + c < a.dw_C ? a.dw_bias[cb * 32 + c] : 0.0f);
        }
    // view tap (x', y') of phase plane (ph, pw) is the original tap x = S (x' - pt') + ph + pt, y likewise, if it exists
    for (int i = threadIdx.x; i < a.n_phase * T; i += kNT) {
        const int p = i / T, tv = i - p * T, xv = tv / a.FW, yv = tv - xv * a.FW;
        const int x = a.S * (xv - a.pt) + ((a.phase_bits >> (2 * p)) & 1) + a.pto;
        const int y = a.S * (yv - a.pl) + ((a.phase_bits >> (2 * p + 1)) & 1) + a.plo;
        tap_tab[i] = (short)((x >= 0 && x < a.FHo && y >= 0 && y < a.FWo) ? x * a.FWo + y : -1);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy zeros visible to the tensor core
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), (uint32_t)(kSlots * kSlotPx));
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // everything above touched only shared memory, tensor memory and the layer's own constants (bias, depthwise
    // filters); from here on the roles read the input tensor and write the output tensor
    grid_dep_sync();
    grid_dep_trigger();

    // Stages a producer has armed and the parity of each stage's latest fill, kept past the role loops: if any role
    // gave up, the producers wait (bounded) for their copies in flight before the CTA may exit.
    uint32_t armed_mask = 0, armed_parity = 0;
    uint32_t drain_bar = 0;

    // The three single-thread roles below keep their loops free of divisions: stage indices, phase bits and tap
    // offsets advance incrementally, because every scalar instruction of the one issuing thread is a few cycles that
    // the tensor pipe may have to wait for.
    if (warp == 0 && lane == 0) {
        // ---- input strips: one box per (tile, channel block)
        drain_bar = DW ? bar_raw_full : bar_a_full;
        bool alive = true, wrapped = false;
        uint32_t s = 0, phase = 0;
        if (DW) {
            // fused depthwise: one halo box of the layer's input per (tile, channel block), into the raw-tile ring
            for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x) {
                const Tile tl = decode_tile(a, t);
                for (int cb = 0; cb < a.CBr; ++cb) {
                    if (wrapped) alive = mbar_wait(bar_raw_empty + 8 * s, phase ^ 1u, abort_flag, a.status, a.wait_iters);
                    if (!alive) break;
                    mbar_expect_tx(bar_raw_full + 8 * s, a.raw_box_bytes);
                    tma_load_5d(raw_base + s * a.raw_stage_bytes, &map_a, bar_raw_full + 8 * s, 0, -a.dw_pl, tl.row0 * a.dw_s - a.dw_pt, cb, tl.n0);
                    armed_mask |= 1u << s;
                    armed_parity = (armed_parity & ~(1u << s)) | (phase << s);
                    if (++s == (uint32_t)kRawStages) { s = 0; phase ^= 1u; wrapped = true; }
                }
            }
        } else
        for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x) {
            const Tile tl = decode_tile(a, t);
            // one box per (phase plane, real channel block); with stride 2 the map's element strides pick every
            // other row and column, starting at the plane's parity
            const int c1 = a.S * (-a.pl), c2 = a.S * (tl.row0 - a.pt);
            for (int p = 0; p < a.n_phase && alive; ++p) {
                const int ph = (a.phase_bits >> (2 * p)) & 1, pw = (a.phase_bits >> (2 * p + 1)) & 1;
                for (int cb = 0; cb < a.CBr; ++cb) {
                    if (wrapped) alive = mbar_wait(bar_a_empty + 8 * s, phase ^ 1u, abort_flag, a.status, a.wait_iters);
                    if (!alive) break;
                    mbar_expect_tx(bar_a_full + 8 * s, a.a_box_bytes);
                    tma_load_5d(a_base + s * a.a_stage_bytes, &map_a, bar_a_full + 8 * s, 0, c1 + pw, c2 + ph, cb + tl.n_tile * a.cb_group, tl.n0);
                    armed_mask |= 1u << s;
                    armed_parity = (armed_parity & ~(1u << s)) | (phase << s);
                    if (++s == (uint32_t)kAStages) { s = 0; phase ^= 1u; wrapped = true; }
                }
            }
        }
    } else if (warp == 2 && lane == 0) {
        // ---- filter tiles: w_rows x 128 bytes per (channel block, tap).  Resident: all of them once, on one barrier.
        drain_bar = bar_b_full;
        const uint32_t box_bytes = (uint32_t)a.w_rows * 128u;
        if (a.b_resident) {
            int boxes = 0;
            for (int i = 0; i < a.n_phase * T; ++i) boxes += tap_tab[i] >= 0 ? 1 : 0;
            mbar_expect_tx(bar_b_full, box_bytes * (uint32_t)(boxes * a.CBr) * (X3 ? 2u : 1u));
            uint32_t dst = b_base;
            for (int p = 0; p < a.n_phase; ++p)
                for (int cb = 0; cb < a.CBr; ++cb)
                    for (int tap = 0; tap < T; ++tap, dst += kBStageBytes) {
                        const int orig = tap_tab[p * T + tap];
                        if (orig >= 0) {
                            tma_load_4d(dst, &map_b, bar_b_full, 0, 0, orig, cb);
                            if (X3) tma_load_4d(dst + a.b_half, &map_b_lo, bar_b_full, 0, 0, orig, cb);
                        }
                    }
            armed_mask = 1u;
        } else {
            bool alive = true, wrapped = false;
            uint32_t s = 0, phase = 0;
            for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x) {
                const int row = (t % a.n_tiles) * a.w_tile;
                for (int p = 0; p < a.n_phase && alive; ++p)
                    for (int cb = 0; cb < a.CBr && alive; ++cb)
                        for (int tap = 0; tap < T; ++tap) {
                            const int orig = tap_tab[p * T + tap];
                            if (orig < 0) continue;
                            if (wrapped) alive = mbar_wait(bar_b_empty + 8 * s, phase ^ 1u, abort_flag, a.status, a.wait_iters);
                            if (!alive) break;
                            mbar_expect_tx(bar_b_full + 8 * s, X3 ? 2u * box_bytes : box_bytes);
                            tma_load_4d(b_base + s * kBStageBytes, &map_b, bar_b_full + 8 * s, 0, row, orig, cb);
                            if (X3) tma_load_4d(b_base + s * kBStageBytes + a.b_half, &map_b_lo, bar_b_full + 8 * s, 0, row, orig, cb);
                            armed_mask |= 1u << s;
                            armed_parity = (armed_parity & ~(1u << s)) | (phase << s);
                            if (++s == (uint32_t)a.b_stages) { s = 0; phase ^= 1u; wrapped = true; }
                        }
            }
        }
    } else if ((warp == 1 || (kIssuers == 2 && warp == 3)) && lane == 0) {
        // ---- MMA issue: this thread's chains are [C0, C1)
        auto mma_role = [&](auto c0_tag, auto c1_tag, auto d0_tag, auto d1_tag) {
        constexpr int C0 = decltype(c0_tag)::value, C1 = decltype(c1_tag)::value;       // chains on even tiles
        constexpr int D0 = decltype(d0_tag)::value, D1 = decltype(d1_tag)::value;       // chains on odd tiles
        bool alive = true;
        uint32_t sa = 0, pa = 0, sb = 0, pb = 0;
        uint32_t slot_uses = 0;                   // slots taken so far; slot j of a tile is (slot_uses + j) % 2
        const uint32_t b_step = kBStageBytes >> 4;
        const uint32_t x_half = a.x_lo_off, w_half = a.b_half >> 4;
        const uint32_t row_wrap = (uint32_t)(a.Wq - a.FW + 1) * 8u;     // tap offset step from the end of a window row
        // N of the MMA: pixels of a slot (filters on M), or the filters of the tile (pixels on M)
        const uint32_t idesc = instr_desc(PM ? a.w_rows : a.n_slot);
        const uint32_t idesc_wide = instr_desc(PM ? 2 * a.w_rows : a.n_slot);   // x3_wide: both filter halves on N
        const bool wide = X3 && PM && a.x3_wide;
        // strip offset (in 16-byte units) of each MMA chain of a tile: one per slot or one per 128-pixel chunk
        uint32_t xo[CH];
#pragma unroll
        for (int c = 0; c < CH; ++c) xo[c] = (uint32_t)(c * (PM ? 128 : a.n_slot)) * 8u;
        if (a.b_resident) alive = mbar_wait(bar_b_full, 0, abort_flag, a.status, a.wait_iters);

        // all taps of one channel block with KS K-steps each; straight-line MMA issue
        // bit t set: view tap t of the phase plane exists (all of them for stride 1); kept in a register so that the
        // tap loop reads no memory
        auto load_mask = [&](int p) {
            unsigned long long m = 0;
            for (int tv = 0; tv < T; ++tv) m |= (unsigned long long)(tap_tab[p * T + tv] >= 0 ? 1 : 0) << tv;
            return m;
        };
        const unsigned long long mask0 = MASKED ? load_mask(0) : ~0ull;

        auto issue_block = [&](auto ks_tag, auto lo_tag, auto hi_tag, const uint32_t x_stage, const uint32_t (&acc)[CH], const unsigned long long taps, const uint32_t r_sel, uint32_t &started, uint32_t &w_res) {
            const uint32_t r_col = r_sel * (uint32_t)(kSlotPx / a.racc);   // this block's accumulator within each slot
            constexpr int KS = decltype(ks_tag)::value, CL = decltype(lo_tag)::value, CU = decltype(hi_tag)::value;
            uint32_t off = 0;
            int y = 0;
            for (int tap = 0; tap < T; ++tap) {
                uint32_t w_lo;
                if (MASKED && !((taps >> tap) & 1ull)) {   // the view has no such tap in this phase plane
                    if (a.b_resident) w_res += b_step;
                    if (++y == a.FW) { y = 0; off += row_wrap; } else off += 8u;
                    continue;
                }
                if (a.b_resident) {
                    w_lo = w_res; w_res += b_step;
                } else {
                    alive = mbar_wait(bar_b_full + 8 * sb, pb, abort_flag, a.status, a.wait_iters);
                    if (!alive) return;
                    w_lo = smem_desc_lo(b_base + sb * kBStageBytes);
                }
                const uint32_t x_lo = x_stage + off;
                const uint32_t first = (started >> r_sel) & 1u;   // 0 for an accumulator's first MMAs of the tile: they overwrite
                started |= 1u << r_sel;
#pragma unroll
                for (int c = CL; c < CU; ++c) {
                    const uint32_t xs = x_lo + xo[c];
                    const uint32_t da = PM ? xs : w_lo, db = PM ? w_lo : xs;
                    if (!X3) {
                        mma_tf32(acc[c] + r_col, da, db, kDescHi, idesc, first);
                        if (KS > 1) mma_tf32(acc[c] + r_col, da + 2u, db + 2u, kDescHi, idesc, 1u);        // K steps of 32 bytes
                        if (KS > 2) mma_tf32(acc[c] + r_col, da + 4u, db + 4u, kDescHi, idesc, 1u);
                        if (KS > 3) mma_tf32(acc[c] + r_col, da + 6u, db + 6u, kDescHi, idesc, 1u);
                    } else {
                        // the residual halves sit x_half / w_half (16-byte units) behind the TF32 halves
                        const uint32_t da_lo = da + (PM ? x_half : w_half), db_lo = db + (PM ? w_half : x_half);
                        if (PM && wide) {
                            // columns [0, w) of the chunk: x_hi w_hi + x_lo w_hi; columns [w, 2w): x_hi w_lo
#pragma unroll
                            for (int k = 0; k < KS; ++k) {
                                mma_tf32(acc[c] + r_col, da + 2u * k, db + 2u * k, kDescHi, idesc_wide, k == 0 ? first : 1u);
                                mma_tf32(acc[c] + r_col, da_lo + 2u * k, db + 2u * k, kDescHi, idesc, 1u);
                            }
                        } else
#pragma unroll
                        for (int k = 0; k < KS; ++k) {
                            mma_tf32(acc[c] + r_col, da_lo + 2u * k, db + 2u * k, kDescHi, idesc, k == 0 ? first : 1u);   // small terms first
                            mma_tf32(acc[c] + r_col, da + 2u * k, db_lo + 2u * k, kDescHi, idesc, 1u);
                            mma_tf32(acc[c] + r_col, da + 2u * k, db + 2u * k, kDescHi, idesc, 1u);
                        }
                    }
                }
                if (!a.b_resident) {
                    mma_commit(bar_b_empty + 8 * sb);                // filter stage reusable once these MMAs have read it
                    if (++sb == (uint32_t)a.b_stages) { sb = 0; pb ^= 1u; }
                }
                if (++y == a.FW) { y = 0; off += row_wrap; } else off += 8u;
            }
        };

        bool odd_tile = false;
        for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x, odd_tile = !odd_tile) {
            const Tile tl = decode_tile(a, t);
            // the previous content of the slots this tile takes must have left tensor memory
            for (int j = 0; j < a.slots && alive; ++j) {
                const uint32_t u = slot_uses + j;
                if (u >= kSlots) alive = mbar_wait(bar_slot_free + 8 * (u % kSlots), (u / kSlots - 1) & 1, abort_flag, a.status, a.wait_iters);
            }
            if (!alive) break;
            tc_fence_after();
            uint32_t acc[CH];                     // accumulator address of each chain
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                if (PM) {
                    const int j = c / a.cps;
                    acc[c] = tmem + ((slot_uses + j) % kSlots) * kSlotPx + (uint32_t)(c - j * a.cps) * (256u / (uint32_t)a.cps);
                } else {
                    acc[c] = tmem + ((slot_uses + c) % kSlots) * kSlotPx;
                }
            }
            uint32_t w_res = smem_desc_lo(b_base), started = 0, r_sel = 0;
            int cb = 0, plane = 0;
            unsigned long long taps = mask0;
            for (int blk = 0; blk < a.CB && alive; ++blk) {       // blocks = phase planes x real channel blocks
                alive = mbar_wait(((X3 || DW) ? bar_a_split : bar_a_full) + 8 * sa, pa, abort_flag, a.status, a.wait_iters);   // once split / computed
                if (!alive) break;
                const uint32_t x_stage = smem_desc_lo(a_base + sa * a.a_stage_bytes) + (uint32_t)tl.a0 * 8u;   // 128 bytes per pixel, >> 4
                if (odd_tile && (D0 != C0 || D1 != C1)) {
                    if (cb == a.CBr - 1) issue_block(std::integral_constant<int, KS_LAST>{}, d0_tag, d1_tag, x_stage, acc, taps, r_sel, started, w_res);
                    else issue_block(std::integral_constant<int, 4>{}, d0_tag, d1_tag, x_stage, acc, taps, r_sel, started, w_res);
                } else {
                    if (cb == a.CBr - 1) issue_block(std::integral_constant<int, KS_LAST>{}, c0_tag, c1_tag, x_stage, acc, taps, r_sel, started, w_res);
                    else issue_block(std::integral_constant<int, 4>{}, c0_tag, c1_tag, x_stage, acc, taps, r_sel, started, w_res);
                }
                if (++r_sel == (uint32_t)a.racc) r_sel = 0;
                if (alive) mma_commit(bar_a_empty + 8 * sa);
                if (++sa == (uint32_t)kAStages) { sa = 0; pa ^= 1u; }
                if (++cb == a.CBr) { cb = 0; if (MASKED && ++plane < a.n_phase) taps = load_mask(plane); }
            }
            if (alive)
                for (int j = 0; j < a.slots; ++j) mma_commit(bar_slot_full + 8 * ((slot_uses + j) % kSlots));
            slot_uses += a.slots;
        }
        };
        if (CH == 1 && kIssuers == 1) mma_role(std::integral_constant<int, 0>{}, std::integral_constant<int, CH>{},
                                               std::integral_constant<int, 0>{}, std::integral_constant<int, CH>{});
        else if (warp == 1) mma_role(std::integral_constant<int, 0>{}, std::integral_constant<int, kSplit>{},
                                     std::integral_constant<int, 0>{}, std::integral_constant<int, kOddSplit>{});
        else mma_role(std::integral_constant<int, kSplit>{}, std::integral_constant<int, CH>{},
                      std::integral_constant<int, kOddSplit>{}, std::integral_constant<int, CH>{});
    } else if (DW && warp >= 8) {
        // ---- fused depthwise 3x3: halo tile -> strip (FMAs, bias, ReLU, 16-byte stores at the swizzled places of the
        // K-major strip the MMAs read).
        const int tid = threadIdx.x - 256;
        bool alive = true, wrapped = false;
        uint32_t r = 0, pr = 0, s = 0, ps = 0;
        const int px_img = a.dw_rows * a.OW;                     // strip pixels per image (row pitch = OW: a 1x1 view)
        for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x)
            for (int cb = 0; cb < a.CBr; ++cb) {
                alive = mbar_wait_warp(bar_raw_full + 8 * r, pr, abort_flag, a.status, a.wait_iters);
                if (alive && wrapped) alive = mbar_wait_warp(bar_a_empty + 8 * s, ps ^ 1u, abort_flag, a.status, a.wait_iters);
                if (!alive) break;
                const float4 *raw = reinterpret_cast<const float4 *>(base_ptr + (raw_base - base) + (size_t)r * a.raw_stage_bytes);
                float4 *hi = reinterpret_cast<float4 *>(base_ptr + (size_t)s * a.a_stage_bytes);
                float4 *lo = reinterpret_cast<float4 *>(base_ptr + (size_t)s * a.a_stage_bytes + a.a_half);
                const float4 *w4 = reinterpret_cast<const float4 *>(dw_s_w + cb * 320);
                // One unit = 4 channels (chunk j) of one output column of one image; the thread walks down the column
                // with the 3x3 window in registers, so each output costs three (stride 2: six) 16-byte loads.  j is
                // the same for all units of a thread (128 threads, 8 chunks), so its nine filter vectors load once.
                const int j = tid & 7;                                  // (256 threads: 32 column groups in flight)
                float4 wv[9];
#pragma unroll
                for (int k = 0; k < 9; ++k) wv[k] = w4[k * 8 + j];
                const float4 bias4 = w4[9 * 8 + j];
                const int units = a.nn * a.OW;                       // (image, column) pairs; this thread takes every 16th
                for (int u = tid >> 3; u < units; u += kXform / 8) {
                    const int img = u / a.OW, ow = u - img * a.OW;
                    const float4 *col = raw + ((size_t)img * a.dw_Hb * a.dw_Wb + ow * a.dw_s) * 8 + j;
                    const int q0 = img * px_img + ow;
                    float4 win[3][3];
                    // rows 0 .. (3 - stride) - 1 of the first window; the loop loads the remaining `stride` rows per output
                    if (a.dw_s == 1) {
#pragma unroll
                        for (int y = 0; y < 3; ++y) { win[1][y] = col[y * 8]; win[2][y] = col[(a.dw_Wb + y) * 8]; }
                    } else {
#pragma unroll
                        for (int y = 0; y < 3; ++y) win[2][y] = col[y * 8];
                    }
                    for (int rr = 0; rr < a.dw_rows; ++rr) {
                        if (a.dw_s == 1) {
                            const float4 *row = col + (size_t)(rr + 2) * a.dw_Wb * 8;
#pragma unroll
                            for (int y = 0; y < 3; ++y) { win[0][y] = win[1][y]; win[1][y] = win[2][y]; win[2][y] = row[y * 8]; }
                        } else {
                            const float4 *row = col + (size_t)(2 * rr + 1) * a.dw_Wb * 8;
#pragma unroll
                            for (int y = 0; y < 3; ++y) { win[0][y] = win[2][y]; win[1][y] = row[y * 8]; win[2][y] = row[(a.dw_Wb + y) * 8]; }
                        }
                        float4 acc = bias4;
#pragma unroll
                        for (int x = 0; x < 3; ++x)
#pragma unroll
                            for (int y = 0; y < 3; ++y) {
                                const float4 v = win[x][y], w = wv[x * 3 + y];
                                acc.x = fmaf(v.x, w.x, acc.x); acc.y = fmaf(v.y, w.y, acc.y);
                                acc.z = fmaf(v.z, w.z, acc.z); acc.w = fmaf(v.w, w.w, acc.w);
                            }
                        if (a.dw_relu) { acc.x = fmaxf(acc.x, 0.f); acc.y = fmaxf(acc.y, 0.f); acc.z = fmaxf(acc.z, 0.f); acc.w = fmaxf(acc.w, 0.f); }
                        const int q = q0 + rr * a.OW;
                        const int at = q * 8 + (j ^ (q & 7));                      // 128-byte swizzle of the K-major strip
                        if (X3) {
                            const float4 h = make_float4(__uint_as_float(__float_as_uint(acc.x) & 0xffffe000u), __uint_as_float(__float_as_uint(acc.y) & 0xffffe000u),
                                                         __uint_as_float(__float_as_uint(acc.z) & 0xffffe000u), __uint_as_float(__float_as_uint(acc.w) & 0xffffe000u));
                            hi[at] = h;
                            lo[at] = make_float4(acc.x - h.x, acc.y - h.y, acc.z - h.z, acc.w - h.w);
                        } else {
                            hi[at] = acc;
                        }
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // these writes are read by the tensor core
                mbar_arrive(bar_a_split + 8 * s);
                mbar_arrive(bar_raw_empty + 8 * r);
                if (++r == (uint32_t)kRawStages) { r = 0; pr ^= 1u; }
                if (++s == (uint32_t)kAStages) { s = 0; ps ^= 1u; wrapped = true; }
            }
    } else if (X3 && warp >= 8) {
        // ---- 3xTF32: split each strip as it lands.  Elementwise at equal offsets, so the swizzled layout carries over.
        const int tid = threadIdx.x - 256;
        bool alive = true;
        uint32_t s = 0, phase = 0;
        const int n4 = (a.strip_px + a.tail_px) * 8;          // 16-byte vectors of the strip and its zero tail
        for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x)
            for (int blk = 0; blk < a.CB; ++blk) {
                alive = mbar_wait_warp(bar_a_full + 8 * s, phase, abort_flag, a.status, a.wait_iters);
                if (!alive) break;
                uint4 *hi = reinterpret_cast<uint4 *>(base_ptr + (size_t)s * a.a_stage_bytes);
                float4 *lo = reinterpret_cast<float4 *>(base_ptr + (size_t)s * a.a_stage_bytes + a.a_half);
                if (a.x_packed) {
                    // at most 16 channels: lanes [h, 2h) of every row are pad lanes (zero), and the residual goes
                    // there instead of into a second half-stage.  A row's 16-byte chunk j sits at chunk j ^ (row & 7)
                    // (128-byte swizzle; stages start on 1024-byte boundaries).
                    const int hc = (int)a.x_lo_off >> 0;              // chunks per half: 2 (h = 8) or 4 (h = 16)
                    const int rows = a.strip_px + a.tail_px;
                    for (int i = tid; i < rows * hc; i += 128) {
                        const int r = i / hc, j = i - r * hc;
                        const int sw7 = r & 7;
                        uint4 *src = hi + r * 8 + (j ^ sw7);
                        const uint4 v = *src;
                        const uint4 h = make_uint4(v.x & 0xffffe000u, v.y & 0xffffe000u, v.z & 0xffffe000u, v.w & 0xffffe000u);
                        reinterpret_cast<float4 *>(hi)[r * 8 + ((j + hc) ^ sw7)] =
                            make_float4(__uint_as_float(v.x) - __uint_as_float(h.x), __uint_as_float(v.y) - __uint_as_float(h.y),
                                        __uint_as_float(v.z) - __uint_as_float(h.z), __uint_as_float(v.w) - __uint_as_float(h.w));
                        *src = h;
                    }
                } else
                {
                    // four vectors per step, loads first: one warp per scheduler has nothing else to hide their latency
                    auto split1 = [&](int i, const uint4 v) {
                        const uint4 h = make_uint4(v.x & 0xffffe000u, v.y & 0xffffe000u, v.z & 0xffffe000u, v.w & 0xffffe000u);
                        lo[i] = make_float4(__uint_as_float(v.x) - __uint_as_float(h.x), __uint_as_float(v.y) - __uint_as_float(h.y),
                                            __uint_as_float(v.z) - __uint_as_float(h.z), __uint_as_float(v.w) - __uint_as_float(h.w));
                        hi[i] = h;
                    };
                    int i = tid;
                    for (; i + 3 * 128 < n4; i += 4 * 128) {
                        const uint4 v0 = hi[i], v1 = hi[i + 128], v2 = hi[i + 256], v3 = hi[i + 384];
                        split1(i, v0); split1(i + 128, v1); split1(i + 256, v2); split1(i + 384, v3);
                    }
                    for (; i < n4; i += 128) split1(i, hi[i]);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // these writes are read by the tensor core
                mbar_arrive(bar_a_split + 8 * s);
                if (++s == (uint32_t)kAStages) { s = 0; phase ^= 1u; }
            }
    } else if (warp >= 4 && warp < 8) {
        // ---- epilogue: warp q owns tensor-memory lanes 32q.. = filters 32q.. of the tile; lane = filter, column = pixel
        const int quarter = warp & 3;
        bool alive = true;
        uint32_t slot_uses = 0;
        const int pv = a.Hq * a.Wq;
        for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x) {
            const Tile tl = decode_tile(a, t);
            const int kb = tl.n_tile * (a.w_tile / 32) + quarter;        // quarters past the tile's filters have nothing to store
            const int k = kb * 32 + lane;
            const float bv = kb < a.KB ? bias_s[k] : 0.0f;
            const bool lane_real = k < a.K;
            for (int j = 0; j < tl.slots && alive; ++j) {
                const uint32_t u = slot_uses + j, s = u % kSlots;
                alive = mbar_wait_warp(bar_slot_full + 8 * s, (u / kSlots) & 1, abort_flag, a.status, a.wait_iters);
                if (!alive) break;
                tc_fence_after();
                const int px_here = min(tl.n_slot, tl.px - j * tl.n_slot);      // real pixels in this slot
                if (PM) {
                    // pixels on M: this thread owns one pixel of each 128-pixel chunk (tensor-memory lane = pixel) and
                    // reads 32 filters at a time = one whole 128-byte output line, stored as four 32-byte vectors
                    const uint32_t sw = 256u / (uint32_t)a.cps;
                    const int kb_tile = tl.n_tile * (a.w_tile / 32);
                    for (int c = 0; c * 128 < px_here; ++c) {
                        const int p = c * 128 + quarter * 32 + lane;            // pixel within the slot
                        int q = tl.q0 + j * tl.n_slot + p, img = 0;
                        if (a.nn > 1) { img = q / pv; q -= img * pv; }
                        const int oh = q / a.Wq, ow = q - oh * a.Wq;
                        const int n = tl.n0 + img;
                        const bool ok = p < px_here && ow < a.OW && oh < a.OH && img < a.nn && n < a.N;
                        for (int jj = 0; jj * 32 < a.w_rows; ++jj) {
                            float v[32];
                            tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(s * kSlotPx) + (uint32_t)c * sw + jj * 32u, v);
                            if (X3 && a.x3_wide) {     // the x_hi w_lo products of the same filters, w_rows columns on
                                float v2[32];
                                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(s * kSlotPx) + (uint32_t)c * sw + (uint32_t)a.w_rows + jj * 32u, v2);
#pragma unroll
                                for (int e = 0; e < 32; ++e) v[e] += v2[e];
                            }
                            const int kbj = kb_tile + jj;
                            if (!ok || kbj >= a.KB) continue;
                            float *dst = a.out + ((((size_t)n * a.KB + kbj) * a.OH + oh) * a.OW + ow) * 32;
                            const float4 *bs = reinterpret_cast<const float4 *>(bias_s + kbj * 32);   // 16-byte aligned: two loads per eight filters
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                float r[8];
                                const float4 b0 = bs[2 * i], b1 = bs[2 * i + 1];
                                r[0] = v[8 * i + 0] + b0.x; r[1] = v[8 * i + 1] + b0.y; r[2] = v[8 * i + 2] + b0.z; r[3] = v[8 * i + 3] + b0.w;
                                r[4] = v[8 * i + 4] + b1.x; r[5] = v[8 * i + 5] + b1.y; r[6] = v[8 * i + 6] + b1.z; r[7] = v[8 * i + 7] + b1.w;
                                if (a.accumulate) {
                                    float o[8];
                                    ld_global_v8(dst + 8 * i, o);
#pragma unroll
                                    for (int e = 0; e < 8; ++e) r[e] += o[e];
                                }
                                if (a.relu) {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) r[e] = fmaxf(r[e], 0.f);
                                }
                                const int k0 = kbj * 32 + 8 * i;               // pad lanes of the last filter block stay +0
                                if (k0 + 7 >= a.K) {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) if (k0 + e >= a.K) r[e] = 0.f;
                                }
                                st_global_v8(dst + 8 * i, r);
                            }
                        }
                    }
                } else if (kb < a.KB && quarter * 32 < a.w_rows) {
                    // All lanes hold the same 32 pixels (columns) of different filters.  The pixel -> output line
                    // mapping is therefore computed once per group with one pixel per lane (divisions in parallel)
                    // and handed round by shuffle; the stores themselves are straight-line predicated code.
                    const size_t plane = (size_t)a.OH * a.OW * 32;
                    const uint32_t image = (uint32_t)(plane * a.KB);
                    float *base_out = a.out + (size_t)tl.n0 * image + kb * plane + lane;
                    const int q_slot = tl.q0 + j * tl.n_slot;
                    const int imgs_here = min(a.nn, a.N - tl.n0);
                    for (int g = 0; g < px_here; g += 32) {
                        float v[32];
                        tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(s * kSlotPx + g), v);
                        for (int r = 1; r < a.racc; ++r) {       // channel blocks rotated over several accumulators: add them up
                            float v2[32];
                            tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(s * kSlotPx + r * (kSlotPx / a.racc) + g), v2);
#pragma unroll
                            for (int e = 0; e < 32; ++e) v[e] += v2[e];
                        }
                        int q = q_slot + g + lane, img = 0;
                        if (a.nn > 1) { img = q / pv; q -= img * pv; }
                        const int oh = q / a.Wq, ow = q - oh * a.Wq;
                        const bool ok = g + lane < px_here && ow < a.OW && oh < a.OH && img < imgs_here;
                        const uint32_t my_off = (uint32_t)img * image + (uint32_t)(oh * a.OW + ow) * 32u;   // floats from base_out
                        const uint32_t mask = __ballot_sync(0xffffffffu, ok);
                        // straight-line code: 32 independent shuffles, then 32 predicated stores (no branches, so the
                        // single warp per scheduler can keep them all in flight)
                        uint32_t off[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) off[e] = __shfl_sync(0xffffffffu, my_off, e);
                        if (a.accumulate) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) v[e] += ld_global_if(base_out + off[e], mask >> e & 1u);
                        }
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            float r = v[e] + bv;
                            if (a.relu) r = fmaxf(r, 0.f);
                            st_global_if(base_out + off[e], lane_real ? r : 0.0f, mask >> e & 1u);   // pad lanes stay +0
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_slot_free + 8 * s);
            }
            slot_uses += tl.slots;
        }
        tc_fence_before();
    }
    __syncthreads();
    if (*abort_flag && armed_mask) {   // a role gave up: let the copies that are still in flight land before the CTA exits
        for (int st = 0; st < 32; ++st)
            if (armed_mask >> st & 1u)
                for (uint32_t it = 0; it < a.wait_iters && !mbar_try_wait(drain_bar + 8 * st, armed_parity >> st & 1u); ++it) __nanosleep(200);
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, (uint32_t)(kSlots * kSlotPx));
    }
}

// ---------------------------------------------------------------------------------------------- host side
size_t ctrl_bytes(int KB) { return kCtrlBarrierBytes + 16 + (size_t)KB * 32 * 4 + kTapTabEntries * sizeof(short); }

// Plan with at most `max_px` pixels per tile in the given orientation; ok = false when it does not fit.
TcPlan make_plan_with(const Geom &g, size_t max_smem, int max_px, int pixel_m, int S, double taps_eff, bool x3, int racc, bool pack_ok, int group_k, const DwFuse *dw) {
    TcPlan p{};
    p.ok = false;
    if (g.S != 1) return p;                      // g is the stride-1 view; S scales the TMA box of the real tensor
    p.taps_eff = taps_eff;
    p.OH = g.OH; p.OW = g.OW;
    const int padw = g.pl > g.pr ? g.pl : g.pr, padh = g.pt > g.pb ? g.pt : g.pb;
    const int minw = g.pl < g.pr ? g.pl : g.pr, minh = g.pt < g.pb ? g.pt : g.pb;
    p.Wq = g.W + padw;
    p.Hq = g.H + padh;
    if (p.Wq * S > 256 || g.FH * g.FW > 64) return p;
    const int Kp = g.KB * 32;
    p.pixel_m = pixel_m;
    p.w_tile = pixel_m ? 256 : kFilterTile;
    p.n_tiles = ceil_div(Kp, p.w_tile);
    p.w_rows = Kp < p.w_tile ? Kp : p.w_tile;
    if (group_k > 0) {                           // group convolution: one filter tile per group
        if (group_k > p.w_tile) return p;
        p.w_tile = group_k; p.w_rows = group_k; p.n_tiles = Kp / group_k;
    }
    // 3xTF32 with pixels on M and few filters: the residual filter rows lie directly behind the TF32 rows in a stage, so
    // one MMA of N = 2 x filters forms x_hi w_hi and x_hi w_lo side by side in tensor memory (an MMA below N = 128 costs
    // the pipe the same 50 cycles whatever N is); a second MMA adds x_lo w_hi, and the epilogue adds the two column
    // groups.  Two MMAs per K step instead of three.
    p.x3_wide = (x3 && pixel_m && p.w_rows <= 64) ? 1 : 0;
    const int acc_cols = p.x3_wide ? 2 * p.w_rows : p.w_rows;      // tensor-memory columns of one 128-pixel chunk
    p.cps = !pixel_m ? 1 : acc_cols <= 64 ? 4 : acc_cols <= 128 ? 2 : 1;
    p.ks_last = (g.C - (g.CB - 1) * 32 + 7) / 8;
    if (pixel_m && max_px > kSlots * p.cps * 128) return p;       // more pixels than the accumulator slots hold
    p.racc = racc;
    if (racc > 1 && (pixel_m || max_px > kSlots * (kSlotPx / racc))) return p;   // each slot holds racc accumulators
    const long long pv = (long long)p.Hq * p.Wq;
    int a0max, slot_reach;
    if (pv <= max_px && p.Hq * S <= 256) {
        // whole images per strip: as many as fill the tile (at least one)
        p.nn = (int)(max_px / pv);
        if (p.nn > 256) p.nn = 256;
        if (p.nn > g.N) p.nn = g.N;
        p.px_tile = (int)(p.nn * pv);
        p.px_img = p.px_tile; p.tiles_img = 1;
        p.Rs = p.Hq;
        p.m_tiles = ceil_div(g.N, p.nn);
        p.tail_px = minh * p.Wq + minw;
        p.strip_px = p.nn * p.Rs * p.Wq;
        a0max = 0;   // with one image per strip the kernel's run-of-pixels formulas describe the same geometry (q0 = 0)
    } else {
        // runs of pixels of one image in the flattened padded numbering, balanced over the tiles
        p.nn = 1;
        p.px_img = g.OH * p.Wq;
        const int tiles = ceil_div(p.px_img, max_px);
        p.px_tile = ((ceil_div(p.px_img, tiles) + 31) / 32) * 32;    // two slots of a multiple of 16
        if (pixel_m) p.px_tile = ((p.px_tile + 127) / 128) * 128;    // whole 128-pixel chunks
        if (p.px_tile > max_px) p.px_tile = max_px;
        // whole rows per tile when at least two fit: the strip then needs no partial rows at either end
        if (p.Wq <= p.px_tile && (g.FH == 1 || 2 * p.Wq <= p.px_tile)) p.px_tile = (p.px_tile / p.Wq) * p.Wq;
        p.tiles_img = ceil_div(p.px_img, p.px_tile);
        const bool row_aligned = p.px_tile % p.Wq == 0;             // every tile starts at a row start
        p.Rs = row_aligned ? p.px_tile / p.Wq + g.FH - 1 : (p.Wq - 1 + p.px_tile - 1) / p.Wq + 1 + g.FH - 1;
        if (p.Rs * S > 256) return p;
        p.m_tiles = g.N * p.tiles_img;
        p.tail_px = minw;
        p.strip_px = p.Rs * p.Wq;
        a0max = row_aligned ? 0 : p.Wq - 1;
    }
    // every pixel an MMA can touch lies inside the stage: strip + zero tail, and the furthest shifted slot
    if (pixel_m) {
        slot_reach = ceil_div(p.px_tile, 128) * 128;
    } else {
        const int slots = p.px_tile > kSlotPx / racc ? 2 : 1;
        const int n_slot = ((p.px_tile + slots - 1) / slots + 15) & ~15;
        slot_reach = slots * n_slot;
    }
    const int reach = a0max + slot_reach + (g.FH - 1) * p.Wq + g.FW - 1;
    p.stage_px = p.strip_px + p.tail_px > reach ? p.strip_px + p.tail_px : reach;
    p.a_half = (uint32_t)(((size_t)p.stage_px * 128 + 1023) & ~(size_t)1023);
    p.b_half = (uint32_t)(((size_t)(pixel_m ? p.w_rows : kFilterTile) * 128 + 1023) & ~(size_t)1023);
    p.x3 = x3 ? 1 : 0;
    p.x_packed = (x3 && pack_ok) ? 1 : 0;
    p.a_stage_bytes = p.a_half * ((x3 && !p.x_packed) ? 2u : 1u);   // 3xTF32: TF32 part and residual side by side
    const size_t b_stage = (size_t)p.b_half * (x3 ? 2 : 1);
    p.b_stage_bytes = (uint32_t)b_stage;
    // shared memory.  When one filter tile covers the layer and all its (channel block, tap) boxes fit beside enough
    // strips, the filters are loaded once and stay; otherwise at least two strips and two filter boxes, and the rest
    // shared out as described below.
    size_t dw_extra = 0;
    if (dw) {
        // the depthwise result of whole output rows (or whole images) is computed from one halo box of the input
        if (p.nn == 1 && p.px_tile % p.Wq != 0) return p;
        p.dw_rows = p.nn == 1 ? p.px_tile / p.Wq : p.Hq;
        p.dw_Hb = (p.dw_rows - 1) * dw->s + 3;
        p.dw_Wb = (g.OW - 1) * dw->s + 3;
        if (p.dw_Hb > 256 || p.dw_Wb > 256) return p;
        p.raw_stage_bytes = (uint32_t)(((size_t)p.nn * p.dw_Hb * p.dw_Wb * 128 + 1023) & ~(size_t)1023);
        dw_extra = (size_t)kRawStages * p.raw_stage_bytes + (size_t)g.CB * 320 * sizeof(float);
    }
    const size_t fixed = 1024 + ctrl_bytes(g.KB) + dw_extra;
    const size_t all_b = (size_t)g.CB * g.FH * g.FW * b_stage;
    p.b_resident = 0;
    if (p.n_tiles == 1 && fixed + all_b + 2 * (size_t)p.a_stage_bytes <= max_smem) {
        size_t fit = (max_smem - fixed - all_b) / p.a_stage_bytes;
        if (fit > (size_t)kMaxAStages) fit = kMaxAStages;
        const size_t want = g.CB + 1 < 4 ? g.CB + 1 : 4;
        if (fit >= want) { p.b_resident = 1; p.a_stages = (int)fit; p.b_stages = g.CB * g.FH * g.FW; }
    }
    if (!p.b_resident) {
        if (fixed + 2 * (size_t)p.a_stage_bytes + 2 * b_stage > max_smem) return p;
        size_t room = max_smem - fixed - 2 * (size_t)p.a_stage_bytes - 2 * b_stage;
        p.a_stages = 2; p.b_stages = 2;
        // Both streams are latency bound (a stage is refilled only after its MMAs have finished), so what counts is
        // how many channel-block steps of MMA work the stages in flight cover: a strip covers one, a filter box 1/taps.
        // Grow whichever side covers less until nothing more fits.
        const int taps = g.FH * g.FW;
        for (;;) {
            const bool can_a = p.a_stages < kMaxAStages && room >= p.a_stage_bytes;
            const bool can_b = p.b_stages < kMaxBStages && room >= b_stage;
            if (!can_a && !can_b) break;
            const bool b_behind = (double)p.b_stages / taps <= (double)p.a_stages;
            if (can_b && (b_behind || !can_a)) { ++p.b_stages; room -= b_stage; }
            else { ++p.a_stages; room -= p.a_stage_bytes; }
        }
    }
    p.smem_bytes = (uint32_t)(fixed + (size_t)p.a_stages * p.a_stage_bytes + (size_t)p.b_stages * b_stage);
    if ((long long)p.m_tiles * p.n_tiles > 0x7fffffffLL) return p;
    p.ok = true;
    return p;
}

// The tensor core adds each K step's products to its FP32 accumulator with truncation, an error that grows with the
// number of accumulation steps (measured: about 5e-8 relative per K step of 8 channels).  TF32's own tolerance absorbs
// it; 3xTF32 promises 1e-5, which holds up to about 180 steps per accumulator.
constexpr int kMaxKStepsX3 = 160;

// Estimated cycles of the whole layer under a plan, from measured rates.  A 128 x N x 8 TF32 MMA occupies the pipe
// for N / 2 cycles, with a floor of about 48; each tap costs the issuing thread some tens of cycles more (waiting for
// and releasing a filter stage when the filters stream).  The epilogue's stores run at memory speed in either
// orientation; what differs is how many of the four epilogue warps have filters to store (filters on M: one warp per
// 32 filters of the tile) and the instructions per pixel (about 20 cycles per pixel and warp with 4-byte stores, about
// 1.2 per pixel and 32 filters with 32-byte vector stores).  A tile that takes one accumulator slot overlaps its
// epilogue with the next tile's MMAs (the slots alternate); a tile that takes both cannot.  Per tile the slowest of
// MMA issue, epilogue and L2 -> shared-memory traffic counts, plus a hand-over cost and, when the strips of two tiles
// do not fit in the stages, the exposed load of one tile; times the tiles the busiest SM gets.
double plan_cost(const TcPlan &p, const Geom &g, int sms) {
    const double taps = p.taps_eff;
    const double ksteps = (g.CB - 1) * 4.0 + p.ks_last;
    const double avg_px = p.nn == 1 ? (double)p.px_img / p.tiles_img : (double)p.px_tile;
    double mma, epi;
    int slots;
    if (p.pixel_m) {
        const double chunks = (double)(long long)((avg_px + 127.0) / 128.0);
        slots = p.px_tile > p.cps * 128 ? 2 : 1;
        mma = taps * ksteps * chunks * (p.w_rows / 2.0 > 48.0 ? p.w_rows / 2.0 : 48.0);
        if (p.x3_wide) mma = taps * ksteps * chunks * ((p.w_rows > 48.0 ? p.w_rows : 48.0) + 48.0) / 3.0;   // x 3 below
        epi = avg_px * 1.2 * (p.w_rows / 32.0) + 300.0 * chunks;
    } else {
        slots = p.px_tile > kSlotPx / p.racc ? 2 : 1;
        const double n_slot = avg_px / slots;
        mma = taps * ksteps * slots * (n_slot / 2.0 > 48.0 ? n_slot / 2.0 : 48.0);
        const double warps = p.w_rows >= 128 ? 4.0 : p.w_rows / 32.0;
        epi = avg_px * 20.0 * 4.0 / warps;
    }
    if (p.x3) mma *= 3.0;
    mma += taps * g.CB * (p.b_resident ? 40.0 : 120.0);
    // fused depthwise: what is loaded is the halo tile, and eight warps compute the strip from it (about 6 cycles per
    // pixel and channel block, measured)
    const double strip_bytes = p.raw_stage_bytes ? (double)g.CB * p.nn * p.dw_Hb * p.dw_Wb * 128.0 : (double)g.CB * p.strip_px * 128.0;
    const double bytes = strip_bytes + (p.b_resident ? 0.0 : taps * g.CB * p.w_rows * 128.0 * (p.x3 ? 2.0 : 1.0)) + avg_px * 128.0 * (p.w_rows / 32.0);
    const double mem = bytes / 30.0;                 // bytes per clock one SM can expect when all SMs pull
    double tile = mma > mem ? mma : mem;
    if (p.raw_stage_bytes && g.CB * avg_px * 6.0 > tile) tile = g.CB * avg_px * 6.0;
    if (slots == 2) tile += epi;
    else if (epi > tile) tile = epi;
    if (p.raw_stage_bytes && !p.x3 && p.a_stages < 3) tile *= 1.25;   // measured: two strips starve the load -> compute -> MMA chain
    tile += p.raw_stage_bytes ? 8000.0 : 1500.0;     // hand-over per tile; the fused depthwise adds a load -> compute -> MMA chain
    if (p.a_stages < 2 * g.CB) tile += strip_bytes / 30.0 * 0.5;     // the next tile's strips cannot all be in flight
    const double tiles = (double)p.m_tiles * p.n_tiles;
    const double per_sm = tiles <= sms ? 1.0 : tiles / sms;
    const double waves = per_sm < 4.0 ? (double)(long long)(per_sm + 0.999) : per_sm;   // few tiles per SM: whole waves
    return waves * tile + (p.b_resident ? g.CB * taps * p.w_rows * 128.0 / 30.0 : 0.0);
}

// The cheapest plan over both orientations and the tile sizes that fit (wide rows or tall windows leave room for
// fewer pixels per tile).  The pixels-on-M orientation stores 32-byte vectors and needs `out` aligned to 32 bytes.
TcPlan make_plan(const Geom &g, size_t max_smem, int sms, bool out_aligned32, int S, double taps_eff, bool x3, bool pack_ok, int group_k = 0, const DwFuse *dw = nullptr) {
    // 3xTF32 keeps every accumulation chain within kMaxKStepsX3 K steps by rotating the channel blocks over 2 or 4
    // accumulators (added up in the epilogue); TF32's tolerance needs none of that
    int racc = 1;
    if (x3) {
        const int ksteps = g.CB * 4 * g.FH * g.FW;
        racc = ksteps <= kMaxKStepsX3 ? 1 : ksteps <= 2 * kMaxKStepsX3 ? 2 : 4;
        if (ksteps > 4 * kMaxKStepsX3) return TcPlan{};
    }
    TcPlan best{};
    double best_cost = 0.0;
    for (int pixel_m = 0; pixel_m <= (out_aligned32 ? 1 : 0); ++pixel_m)
        for (int px = kSlots * kSlotPx; px >= 64; px -= 64) {
            TcPlan p = make_plan_with(g, max_smem, px, pixel_m, S, taps_eff, x3, racc, pack_ok, group_k, dw);
            if (!p.ok) continue;
            const double c = plan_cost(p, g, sms);
            if (!best.ok || c < best_cost) { best = p; best_cost = c; }
        }
    return best;
}

typedef void (*TcKernel)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const TcArgs);

template <int CH, int KS, bool PM>
TcKernel pick_flags(bool masked, bool x3, bool dw) {
    if (dw) return masked ? nullptr : x3 ? conv_tc_kernel<CH, KS, PM, false, true, true> : conv_tc_kernel<CH, KS, PM, false, false, true>;
    if (x3) return masked ? conv_tc_kernel<CH, KS, PM, true, true, false> : conv_tc_kernel<CH, KS, PM, false, true, false>;
    return masked ? conv_tc_kernel<CH, KS, PM, true, false, false> : conv_tc_kernel<CH, KS, PM, false, false, false>;
}
template <int CH, bool PM>
TcKernel pick_ks(int ks, bool masked, bool x3, bool dw) {
    switch (ks) {
        case 1: return pick_flags<CH, 1, PM>(masked, x3, dw);
        case 2: return pick_flags<CH, 2, PM>(masked, x3, dw);
        case 4: return pick_flags<CH, 4, PM>(masked, x3, dw);
        default: return nullptr;
    }
}
// Filters on M: one chain per accumulator slot (1 or 2); pixels on M: one per 128-pixel chunk (1 to 4).
TcKernel pick_kernel(int chains, int ks, bool pixel_m, bool masked, bool x3, bool dw) {
    if (!pixel_m) return chains == 1 ? pick_ks<1, false>(ks, masked, x3, dw) : chains == 2 ? pick_ks<2, false>(ks, masked, x3, dw) : nullptr;
    switch (chains) {
        case 1: return pick_ks<1, true>(ks, masked, x3, dw);
        case 2: return pick_ks<2, true>(ks, masked, x3, dw);
        case 3: return pick_ks<3, true>(ks, masked, x3, dw);
        case 4: return pick_ks<4, true>(ks, masked, x3, dw);
        default: return nullptr;
    }
}

}  // namespace

// A 1x1 window without padding never looks at a neighbour, so the plane may be viewed with any row length that
// divides H*W: the longest one that still fits a TMA box makes every tile a run of whole rows and every strip exactly
// the pixels the tile needs.
static Geom flatten_pointwise(const Geom &g) {
    if (g.FH != 1 || g.FW != 1 || g.S != 1 || (g.pt | g.pb | g.pl | g.pr)) return g;
    const long long hw = (long long)g.H * g.W;
    int best = 0;
    for (int w = 256; w >= 1; --w)
        if (hw % w == 0) { best = w; break; }
    if (best <= g.W) return g;
    Geom f = g;
    f.W = f.OW = best;
    f.H = f.OH = (int)(hw / best);
    return f;
}

// The stride-1 view of a layer.  A stride-2 window over X is a stride-1 window over X's four phase planes
// P(ph,pw)[i][j] = X[2i+ph][2j+pw]: tap x of the original window reads row 2 oh + x - pt = 2 (oh + dh) + ph with
// ph = (x - pt) mod 2 and dh = floor((x - pt) / 2), i.e. row oh + dh of plane ph.  So the layer becomes a stride-1
// convolution with window (dh_max - dh_min + 1), top pad -dh_min, and n_phase x CB "channel blocks", one per (phase
// plane, real block); view taps that no original tap maps to are skipped.  TMA reads a phase plane straight from the
// blocked tensor with element strides 2, so nothing is reformatted.  (Stride 1: the view is the layer itself.)
struct Virt { Geom g; int S, n_phase, CBr, phase_bits, FHo, FWo, pto, plo; double taps_eff; };

static int floor_half(int v) { return v >= 0 ? v / 2 : -((1 - v) / 2); }

static bool make_virt(const Geom &g_in, Virt &v, bool keep_rows = false) {
    v.S = g_in.S; v.FHo = g_in.FH; v.FWo = g_in.FW; v.pto = g_in.pt; v.plo = g_in.pl; v.CBr = g_in.CB;
    if (g_in.S == 1) {
        v.g = keep_rows ? g_in : flatten_pointwise(g_in);
        v.n_phase = 1; v.phase_bits = 0; v.taps_eff = (double)g_in.FH * g_in.FW;
        return true;
    }
    if (g_in.S != 2) return false;
    const int dh0 = floor_half(-g_in.pt), dh1 = floor_half(g_in.FH - 1 - g_in.pt);
    const int dw0 = floor_half(-g_in.pl), dw1 = floor_half(g_in.FW - 1 - g_in.pl);
    bool has_h[2] = {false, false}, has_w[2] = {false, false};
    for (int x = 0; x < g_in.FH; ++x) has_h[(x - g_in.pt) & 1] = true;
    for (int y = 0; y < g_in.FW; ++y) has_w[(y - g_in.pl) & 1] = true;
    v.n_phase = 0; v.phase_bits = 0;
    for (int ph = 0; ph < 2; ++ph)
        for (int pw = 0; pw < 2; ++pw)
            if (has_h[ph] && has_w[pw]) { v.phase_bits |= (ph | (pw << 1)) << (2 * v.n_phase); ++v.n_phase; }
    Geom g = g_in;
    g.S = 1;
    g.FH = dh1 - dh0 + 1; g.FW = dw1 - dw0 + 1;
    g.pt = -dh0; g.pl = -dw0; g.pb = 0; g.pr = 0;
    g.H = g_in.OH + g.FH - 1 - g.pt; g.W = g_in.OW + g.FW - 1 - g.pl;     // rows and columns of a plane that outputs reach
    if (g.H < 1 || g.W < 1 || g.pt < 0 || g.pl < 0) return false;
    g.CB = v.n_phase * g_in.CB;
    g.C = (g.CB - 1) * 32 + (g_in.C - (g_in.CB - 1) * 32);                  // keeps the K steps of the last real block
    v.g = g;
    v.taps_eff = (double)g_in.FH * g_in.FW / v.n_phase;
    return g.FH * g.FW <= 64;
}

// groups > 1: g describes one group's channels (C = F_C) and all the filters (K = groups * filters per group)
static bool conv_tc_supported_uncached(const Geom &g, bool x3, int groups, const DwFuse *dw) {
    Virt v;
    if (!make_virt(g, v, dw != nullptr)) return false;
    if (dw) return groups == 1 && make_plan(v.g, 227 * 1024, 148, false, v.S, v.taps_eff, x3, false, 0, dw).ok;
    if (groups > 1) return (g.C % 32 == 0) && (g.K % (32 * groups) == 0) &&
                           make_plan(v.g, 227 * 1024, 148, false, v.S, v.taps_eff, x3, false, g.K / groups).ok;
    return make_plan(v.g, 227 * 1024, 148, false, v.S, v.taps_eff, x3, v.CBr == 1 && g.C <= 16).ok;
}

// Planning a layer walks two orientations x eight tile sizes; its answers depend on the shape alone, so they are kept:
// whether the kernel takes a shape (process-wide), and per context the finished launch of a (shape, mode, pointers)
// combination - plan, tensor maps, arguments, kernel - so that a repeated call only launches.
namespace {

template <typename T>
void key_add(std::string &k, const T &v) { k.append(reinterpret_cast<const char *>(&v), sizeof(T)); }

std::string shape_key(const Geom &g, bool x3, int groups, const DwFuse *dw) {
    std::string k;
    const int f[] = {g.N, g.C, g.K, g.H, g.W, g.FH, g.FW, g.S, g.pt, g.pb, g.pl, g.pr, x3 ? 1 : 0, groups, dw ? 1 : 0,
                     dw ? dw->C : 0, dw ? dw->H : 0, dw ? dw->W : 0, dw ? dw->s : 0, dw ? dw->pt : 0, dw ? dw->pl : 0};
    key_add(k, f);
    return k;
}

struct TcLaunch {
    CUtensorMap map_a, map_b, map_b_lo;
    TcArgs a;
    TcKernel kern;
    unsigned grid, threads;
    uint32_t smem;
};
typedef std::unordered_map<std::string, TcLaunch> TcCache;

}  // namespace

bool conv_tc_supported(const Geom &g, bool x3, int groups, const DwFuse *dw) {
    static std::mutex mu;
    static std::unordered_map<std::string, bool> known;
    const std::string key = shape_key(g, x3, groups, dw);
    {
        std::lock_guard<std::mutex> lock(mu);
        auto it = known.find(key);
        if (it != known.end()) return it->second;
    }
    const bool ok = conv_tc_supported_uncached(g, x3, groups, dw);
    std::lock_guard<std::mutex> lock(mu);
    if (known.size() > 65536) known.clear();
    known[key] = ok;
    return ok;
}

void free_tc_cache(small_ctx *ctx) {
    delete static_cast<TcCache *>(ctx->tc_cache);
    ctx->tc_cache = nullptr;
}

int launch_conv_tc(small_ctx *ctx, const float *in, const float *w_hi, const float *w_lo, const float *bias, float *out,
                   const Geom &g_in, bool relu, bool accumulate, unsigned mode, cudaStream_t st, int groups, const DwFuse *dw) {
    const bool x3 = mode == SMALL_MATH_3XTF32;
    if (x3 && !w_lo) return SMALL_ERR_INVALID_ARG;
    // a launch seen before (same shape, mode, flags and tensors): everything is ready
    std::string key = shape_key(g_in, x3, groups, dw);
    {
        const void *ptrs[] = {in, w_hi, w_lo, bias, out, dw ? dw->w : nullptr, dw ? dw->bias : nullptr};
        const unsigned misc[] = {relu ? 1u : 0u, accumulate ? 1u : 0u, mode, dw ? (unsigned)dw->relu : 0u, ctx->wait_iters};
        key_add(key, ptrs);
        key_add(key, misc);
    }
    if (!ctx->tc_cache) ctx->tc_cache = new TcCache();
    TcCache &cache = *static_cast<TcCache *>(ctx->tc_cache);
    {
        auto it = cache.find(key);
        if (it != cache.end()) {
            const TcLaunch &L = it->second;
            launch_kernel(ctx, L.kern, dim3(L.grid), dim3(L.threads), L.smem, st, L.map_a, L.map_b, L.map_b_lo, L.a);
            return check_launch(ctx);
        }
    }
    Virt v;
    if (!make_virt(g_in, v, dw != nullptr)) return SMALL_ERR_UNSUPPORTED;
    const Geom &g = v.g;
    TcPlan p = make_plan(g, ctx->max_smem_optin < 227 * 1024 ? ctx->max_smem_optin : 227 * 1024, ctx->sm_count,
                         (reinterpret_cast<uintptr_t>(out) & 31u) == 0, v.S, v.taps_eff, x3, groups == 1 && !dw && v.CBr == 1 && g_in.C <= 16,
                         groups > 1 ? g_in.K / groups : 0, dw);
    if (!p.ok) return SMALL_ERR_UNSUPPORTED;
    EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    CUtensorMap map_a, map_b, map_b_lo;
    if (dw) {   // fused depthwise: halo boxes of the depthwise layer's input, read by CUDA threads (no swizzle)
        cuuint64_t dims[5] = {32, (cuuint64_t)dw->W, (cuuint64_t)dw->H, (cuuint64_t)v.CBr, (cuuint64_t)g.N};
        cuuint64_t strides[4] = {128, (cuuint64_t)dw->W * 128, (cuuint64_t)dw->H * dw->W * 128, (cuuint64_t)v.CBr * dw->H * dw->W * 128};
        cuuint32_t box[5] = {32, (cuuint32_t)p.dw_Wb, (cuuint32_t)p.dw_Hb, 1, (cuuint32_t)p.nn};
        cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        CUresult r = encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<float *>(in), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    } else {   // activations: [N][CB][H][W][32 floats]; box = 32 x Wq x Rs x 1 x nn, out-of-range elements read as zero
        // the real tensor (for stride 1 possibly with a 1x1 layer's rows re-cut); with stride 2 the box spans 2 Wq x 2 Rs
        // elements and the element strides keep every other one, so shared memory receives Wq x Rs pixels either way
        const int Hr = v.S == 1 ? g.H : g_in.H, Wr = v.S == 1 ? g.W : g_in.W;
        const cuuint32_t es = (cuuint32_t)v.S;
        const cuuint64_t cb_all = (cuuint64_t)v.CBr * groups;      // a group's tiles address their blocks inside the whole tensor
        cuuint64_t dims[5] = {32, (cuuint64_t)Wr, (cuuint64_t)Hr, cb_all, (cuuint64_t)g.N};
        cuuint64_t strides[4] = {128, (cuuint64_t)Wr * 128, (cuuint64_t)Hr * Wr * 128, cb_all * Hr * Wr * 128};
        cuuint32_t box[5] = {32, (cuuint32_t)p.Wq * es, (cuuint32_t)p.Rs * es, 1, (cuuint32_t)p.nn};
        cuuint32_t estr[5] = {1, es, es, 1, 1};
        CUresult r = encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<float *>(in), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    for (int half = 0; half < (x3 ? 2 : 1); ++half) {   // filters: [CB][FH*FW][KB*32][32 floats], TF32 part and (3xTF32) residual
        const int T = v.FHo * v.FWo, Kp = g.KB * 32;
        cuuint64_t dims[4] = {32, (cuuint64_t)Kp, (cuuint64_t)T, (cuuint64_t)v.CBr};
        cuuint64_t strides[3] = {128, (cuuint64_t)Kp * 128, (cuuint64_t)T * Kp * 128};
        cuuint32_t box[4] = {32, (cuuint32_t)p.w_rows, 1, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        CUresult r = encode(half ? &map_b_lo : &map_b, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float *>(half ? w_lo : w_hi), dims, strides,
                            box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    if (!x3) map_b_lo = map_b;
    TcArgs a{};
    a.bias = bias; a.out = out; a.status = ctx->dev_status;
    a.N = g.N; a.K = g.K; a.KB = g.KB; a.CB = g.CB; a.OH = g.OH; a.OW = g.OW; a.Wq = p.Wq; a.Hq = p.Hq;
    a.FH = g.FH; a.FW = g.FW; a.pt = g.pt; a.pl = g.pl;
    a.S = v.S; a.n_phase = v.n_phase; a.CBr = v.CBr; a.phase_bits = v.phase_bits;
    a.FHo = v.FHo; a.FWo = v.FWo; a.pto = v.S == 1 ? g.pt : v.pto; a.plo = v.S == 1 ? g.pl : v.plo;
    a.nn = p.nn; a.px_tile = p.px_tile; a.px_img = p.px_img; a.tiles_img = p.tiles_img; a.m_tiles = p.m_tiles; a.n_tiles = p.n_tiles;
    a.strip_px = p.strip_px; a.tail_px = p.tail_px; a.w_rows = p.w_rows; a.b_stages = p.b_stages;
    a.a_stages = p.a_stages; a.pixel_m = p.pixel_m; a.w_tile = p.w_tile; a.cps = p.cps; a.b_stage_bytes = p.b_stage_bytes;
    a.a_stage_bytes = p.a_stage_bytes; a.a_half = p.a_half; a.b_half = p.b_half; a.racc = p.racc;
    a.x_packed = p.x_packed;
    a.x3_wide = p.x3_wide;
    a.x_lo_off = p.x_packed ? 2u * (uint32_t)p.ks_last : (p.a_half >> 4);   // packed: the residual starts h = 8 ks_last lanes on
    a.a_box_bytes = (uint32_t)p.strip_px * 128u;
    a.b_resident = p.b_resident; a.ks_last = p.ks_last;
    a.rows_tile = (p.nn == 1 && p.px_tile % p.Wq == 0) ? p.px_tile / p.Wq : 0;
    a.cb_group = groups > 1 ? v.CBr : 0;
    if (dw) {
        a.dw_w = dw->w; a.dw_bias = dw->bias; a.dw_C = dw->C; a.dw_s = dw->s; a.dw_pt = dw->pt; a.dw_pl = dw->pl; a.dw_relu = dw->relu;
        a.dw_Wb = p.dw_Wb; a.dw_Hb = p.dw_Hb; a.dw_rows = p.dw_rows; a.raw_stage_bytes = p.raw_stage_bytes;
        a.raw_box_bytes = (uint32_t)((size_t)p.nn * p.dw_Hb * p.dw_Wb * 128);
    }
    int chains;
    if (p.pixel_m) {
        a.n_slot = p.cps * 128;
        a.slots = p.px_tile > a.n_slot ? 2 : 1;
        chains = ceil_div(p.px_tile, 128);
    } else {
        a.slots = p.px_tile > kSlotPx / p.racc ? 2 : 1;
        a.n_slot = ((p.px_tile + a.slots - 1) / a.slots + 15) & ~15;
        chains = a.slots;
    }
    // the MMA's N: filters of the tile (twice that for x3_wide) or pixels of a slot; up to 128 columns an MMA is issue-bound
    // Off: alternating paid on the residual CNN's 32 -> 32 layer, which the warp-level kernel has taken since, and cost
    // the 64 -> 64 pointwise layers of the keyword-spotting and depthwise-separable networks 2-3 % of their step
    // (219 -> 213 us and 213 -> 209 us with it off).
    a.alt_tiles = 0;
    const int ks = p.ks_last == 3 ? 4 : p.ks_last;     // a K step of zero channels more is harmless
    a.relu = relu; a.accumulate = accumulate; a.wait_iters = ctx->wait_iters;
    const TcKernel kern = pick_kernel(chains, ks, p.pixel_m != 0, v.S != 1, x3, dw != nullptr);
    if (!kern) return SMALL_ERR_UNSUPPORTED;
    // the attribute belongs to the kernel instance, which other layers share: always the device's limit, so that a
    // launch kept in the cache never finds it lowered by a later layer with a smaller tile
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->max_smem_optin);
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    const long long tiles = (long long)p.m_tiles * p.n_tiles;
    const unsigned grid = (unsigned)(tiles < ctx->sm_count ? tiles : ctx->sm_count);   // persistent: one CTA per SM
    const unsigned threads = dw ? kThreadsDW : x3 ? kThreadsX3 : kThreads;
    if (cache.size() >= 4096) cache.clear();
    cache[key] = TcLaunch{map_a, map_b, map_b_lo, a, kern, grid, threads, p.smem_bytes};
    launch_kernel(ctx, kern, dim3(grid), dim3(threads), p.smem_bytes, st, map_a, map_b, map_b_lo, a);
    return check_launch(ctx);
}

}  // namespace small
