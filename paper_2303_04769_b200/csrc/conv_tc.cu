// Full channel reduction on the tensor cores (paper Section 3.2 item 4; Algorithms 1 and 2) for stride-1 windows:
// an implicit GEMM straight from the blocked layout, with no im2col buffer and no reformatting (Section 4.4).
//
//   D[pixel, k] = sum over (channel block cb, tap (x,y), 32 channels ci)  A[pixel + shift(x,y), ci] * B[k, ci]
//
// How the paper's loop nest maps onto the SM:
//   k block loop (parallel)        -> N tiles of BN filters, one CTA per (pixel tile, N tile)
//   i loop over F_C in F_Cb steps  -> cb loop over 32-channel blocks: one TMA box of the input per block
//   x, y kernel loops              -> taps: the SAME shared-memory strip is re-read with a shifted start address
//   ii loop                        -> four K=8 TF32 MMAs per 32-channel block (tcgen05.mma kind::tf32)
//   O_wb x K_b register tile       -> 128-pixel x BN accumulator chunks in tensor memory (up to 4 per CTA)
//   LOAD / STORE phases            -> epilogue: tensor memory -> registers, + bias, (+ previous output), ReLU, store
//
// The strip.  A blocked input plane is [H][W][32 floats]: one pixel and channel block = one 128-byte row, the K-major
// operand row of a TF32 MMA with the 128-byte swizzle.  TMA copies a box of Rs rows x Wq pixels (starting at column
// -pad_l, row -pad_t of the tile, out-of-range elements filled with zeros = the padding) densely into shared memory.
// With the row pitch Wq = W + max(pad_l, pad_r), the right padding of one row and the left padding of the next are the
// same zero pixels, so the strip is the zero-padded image flattened to one pixel sequence, and output pixel q (also
// numbered with pitch Wq) needs strip pixel q + x*Wq + y for tap (x, y).  Any 128 consecutive q form a valid MMA A
// operand: rows 128 bytes apart, start address (q + x*Wq + y) * 128.  Columns ow >= OW of each row are computed and
// dropped.  Small planes put several whole images in one strip the same way (image pitch Hq = H + max(pad_t, pad_b)).
//
// Persistent CTAs (one per SM) walk the tile list with stride gridDim.x.  Roles: warp 0 = TMA producer for input
// strips, warp 2 = TMA producer for filter tiles, warp 1 = MMA issuer (one elected thread each), warps 4-7 = epilogue.
// The producers run ahead across tiles; the epilogue hands each 128-pixel accumulator chunk back to the MMA issuer as
// soon as it has been read out of tensor memory, so the next tile's MMAs overlap the current tile's stores.
// Every mbarrier wait is bounded; on expiry the kernel records SMALL_ERR_TIMEOUT in the context's status word, lets
// its in-flight copies land, frees tensor memory and returns.
#include <cuda.h>

#include "common.cuh"

namespace small {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxChunks = 4;          // 128-pixel accumulator chunks per CTA
constexpr int kAStages = 2;
constexpr int kMaxBStages = 8;
constexpr uint32_t kWaitIters = 1u << 24;   // bounded spin: try_wait itself suspends for a while per call
constexpr int kCtrlBarrierBytes = 16 * kAStages + 16 * kMaxBStages + 8 + 8 * kMaxChunks;   // all mbarriers

struct TcPlan {
    int OH, OW, Wq, Hq;
    int nn;              // images per strip (1: row tiles of one image)
    int chunks;          // accumulator chunks per tile (<= kMaxChunks)
    int total_chunks;    // row-tile mode: chunks per image
    int tiles_img;       // row-tile mode: tiles per image
    int m_tiles;         // pixel tiles in the grid
    int Rs;              // box rows (per image)
    int strip_px, tail_px, stage_px;
    int BN, n_tiles;     // filters per N tile, N tiles
    int tmem_cols;
    int b_stages;
    uint32_t a_stage_bytes, b_stage_bytes, smem_bytes;
    bool ok;
};

struct TcArgs {
    const float *bias; float *out; int *status;
    int N, K, KB, CB, OH, OW, Wq, Hq, FH, FW, pt, pl;
    int nn, chunks, total_chunks, tiles_img, m_tiles, n_tiles, BN, Rs, strip_px, tail_px;
    int tmem_cols, b_stages;
    uint32_t a_stage_bytes, b_stage_bytes, a_box_bytes;
    int relu, accumulate;
};

// ---------------------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out or another role already gave up (abort flag set).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status) {
    for (uint32_t it = 0; it < kWaitIters; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(status, (int)SMALL_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2, int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, TF32 inputs, FP32 accumulate, M = 128, N from the instruction descriptor, K = 8.
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier receives one arrival when every MMA issued so far by this thread has finished.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows 128 bytes apart, groups of 8 rows 1024
// bytes apart.  `addr` is the 128-byte-aligned row start plus the 32-byte K step.  The tensor core, like TMA, takes
// the swizzle phase from the absolute shared-memory address (bits 7-9 select the XOR applied to the 16-byte chunk
// index), so a start that is not on a 1024-byte boundary - every shifted tap - reads the strip exactly as TMA wrote
// it and the descriptor's base-offset field stays 0 (checked on the device: a non-zero value permutes the chunks).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);            // start address
    d |= (uint64_t)1 << 16;                              // leading byte offset (unused with this swizzle)
    d |= (uint64_t)(1024u >> 4) << 32;                   // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                              // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                              // 128-byte swizzle
    return d;
}

// Instruction descriptor: FP32 accumulator, TF32 A and B, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc(int n) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// ---------------------------------------------------------------------------------------------- kernel
struct Tile { int n_tile, n0, q0, row0, a0, chunks; };

__device__ __forceinline__ Tile decode_tile(const TcArgs &a, int t) {
    Tile r;
    r.n_tile = t % a.n_tiles;
    const int m_tile = t / a.n_tiles;
    if (a.nn == 1) {
        r.n0 = m_tile / a.tiles_img;
        const int ti = m_tile - r.n0 * a.tiles_img;
        const int c0 = ti * a.chunks;
        r.chunks = min(a.chunks, a.total_chunks - c0);
        r.q0 = c0 * 128;
        r.row0 = r.q0 / a.Wq;
        r.a0 = r.q0 - r.row0 * a.Wq;
    } else {
        r.n0 = m_tile * a.nn;
        r.q0 = 0; r.row0 = 0; r.a0 = 0;
        r.chunks = a.chunks;
    }
    return r;
}

__device__ __forceinline__ void st_global_v8(float *p, const float *v) {
    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
}
__device__ __forceinline__ void ld_global_v8(const float *p, float *v) {
    asm volatile("ld.global.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]) : "l"(p) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const TcArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t a_base = base;
    const uint32_t b_base = a_base + kAStages * a.a_stage_bytes;
    const uint32_t ctrl = b_base + a.b_stages * a.b_stage_bytes;
    uint8_t *ctrl_ptr = base_ptr + (ctrl - base);
    // control block: barriers (8 bytes each), tensor-memory address, abort flag, bias for all filters
    const uint32_t bar_a_full = ctrl, bar_a_empty = ctrl + 8 * kAStages;
    const uint32_t bar_b_full = ctrl + 16 * kAStages, bar_b_empty = bar_b_full + 8 * kMaxBStages;
    const uint32_t bar_acc = bar_b_empty + 8 * kMaxBStages;
    const uint32_t bar_chunk_free = bar_acc + 8;                 // kMaxChunks barriers
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(ctrl_ptr + kCtrlBarrierBytes);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(ctrl_ptr + kCtrlBarrierBytes + 4);
    float *bias_s = reinterpret_cast<float *>(ctrl_ptr + kCtrlBarrierBytes + 16);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = a.FH * a.FW;
    const int total_tiles = a.m_tiles * a.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kAStages; ++s) { mbar_init(bar_a_full + 8 * s, 1); mbar_init(bar_a_empty + 8 * s, 1); }
        for (int s = 0; s < a.b_stages; ++s) { mbar_init(bar_b_full + 8 * s, 1); mbar_init(bar_b_empty + 8 * s, 1); }
        mbar_init(bar_acc, 1);
        for (int c = 0; c < kMaxChunks; ++c) mbar_init(bar_chunk_free + 8 * c, 4);   // one arrival per epilogue warp
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // zero tail behind each strip: the padding pixels a row (or image) wrap runs into after the last strip row
    for (int s = 0; s < kAStages; ++s) {
        float4 *tail = reinterpret_cast<float4 *>(base_ptr + (size_t)s * a.a_stage_bytes + (size_t)a.strip_px * 128);
        for (int i = threadIdx.x; i < a.tail_px * 8; i += kThreads) tail[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int i = threadIdx.x; i < a.KB * 32; i += kThreads) bias_s[i] = (a.bias && i < a.K) ? a.bias[i] : 0.0f;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy zeros visible to the tensor core
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), (uint32_t)a.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0 && lane == 0) {
        // ---- input strips: one box per (tile, channel block)
        uint32_t armed_mask = 0, last_parity[kAStages] = {0, 0};
        bool alive = true;
        uint32_t ia = 0;
        for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x) {
            const Tile tl = decode_tile(a, t);
            for (int cb = 0; cb < a.CB && alive; ++cb, ++ia) {
                const int s = ia % kAStages;
                const uint32_t use = ia / kAStages;
                if (use > 0) alive = mbar_wait(bar_a_empty + 8 * s, (use - 1) & 1, abort_flag, a.status);
                if (!alive) break;
                mbar_expect_tx(bar_a_full + 8 * s, a.a_box_bytes);
                tma_load_5d(a_base + s * a.a_stage_bytes, &map_a, bar_a_full + 8 * s, 0, -a.pl, tl.row0 - a.pt, cb, tl.n0);
                armed_mask |= 1u << s;
                last_parity[s] = use & 1;
            }
        }
        if (!alive)   // let copies that are still in flight land before the CTA exits
            for (int s = 0; s < kAStages; ++s)
                if (armed_mask >> s & 1) for (uint32_t it = 0; it < kWaitIters && !mbar_try_wait(bar_a_full + 8 * s, last_parity[s]); ++it) {}
    } else if (warp == 2 && lane == 0) {
        // ---- filter tiles: BN rows x 128 bytes per (tile, channel block, tap)
        uint32_t armed_mask = 0, last_parity[kMaxBStages] = {};
        bool alive = true;
        uint32_t ib = 0;
        const int per_tile = a.CB * T;
        for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x) {
            const int n_tile = t % a.n_tiles;
            for (int i = 0; i < per_tile && alive; ++i, ++ib) {
                const int s = ib % a.b_stages;
                const uint32_t use = ib / a.b_stages;
                if (use > 0) alive = mbar_wait(bar_b_empty + 8 * s, (use - 1) & 1, abort_flag, a.status);
                if (!alive) break;
                mbar_expect_tx(bar_b_full + 8 * s, a.b_stage_bytes);
                tma_load_4d(b_base + s * a.b_stage_bytes, &map_b, bar_b_full + 8 * s, 0, n_tile * a.BN, i % T, i / T);
                armed_mask |= 1u << s;
                last_parity[s] = use & 1;
            }
        }
        if (!alive)
            for (int s = 0; s < a.b_stages; ++s)
                if (armed_mask >> s & 1) for (uint32_t it = 0; it < kWaitIters && !mbar_try_wait(bar_b_full + 8 * s, last_parity[s]); ++it) {}
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issue
        const uint32_t idesc = instr_desc(a.BN);
        bool alive = true;
        uint32_t ia = 0, ib = 0, it = 0;
        for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x, ++it) {
            const Tile tl = decode_tile(a, t);
            for (int cb = 0; cb < a.CB && alive; ++cb, ++ia) {
                const int sa = ia % kAStages;
                alive = mbar_wait(bar_a_full + 8 * sa, (ia / kAStages) & 1, abort_flag, a.status);
                if (!alive) break;
                const uint32_t a_stage = a_base + sa * a.a_stage_bytes;
                for (int tap = 0; tap < T && alive; ++tap, ++ib) {
                    const int sb = ib % a.b_stages;
                    alive = mbar_wait(bar_b_full + 8 * sb, (ib / a.b_stages) & 1, abort_flag, a.status);
                    if (!alive) break;
                    tc_fence_after();
                    const int x = tap / a.FW, y = tap - x * a.FW;
                    const uint32_t a_tap = a_stage + (uint32_t)(tl.a0 + x * a.Wq + y) * 128u;
                    const uint32_t b_stage = b_base + sb * a.b_stage_bytes;
                    for (int c = 0; c < tl.chunks && alive; ++c) {
                        if (it > 0 && cb == 0 && tap == 0) {   // the previous tile's values of this chunk must have left tensor memory
                            alive = mbar_wait(bar_chunk_free + 8 * c, (it - 1) & 1, abort_flag, a.status);
                            if (!alive) break;
                            tc_fence_after();
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            mma_tf32(tmem + (uint32_t)(c * a.BN), smem_desc(a_tap + (uint32_t)c * (128u * 128u) + k * 32u),
                                     smem_desc(b_stage + k * 32u), idesc, (cb | tap | k) != 0);
                        }
                    }
                    if (alive) mma_commit(bar_b_empty + 8 * sb);     // filter stage reusable once these MMAs have read it
                }
                if (alive) mma_commit(bar_a_empty + 8 * sa);
            }
            if (alive) mma_commit(bar_acc);
        }
    } else if (warp >= 4) {
        // ---- epilogue: each warp owns the 32 tensor-memory lanes of its quarter; thread = one pixel of a chunk
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        bool alive = true;
        uint32_t it = 0;
        for (int t = blockIdx.x; t < total_tiles && alive; t += gridDim.x, ++it) {
            const Tile tl = decode_tile(a, t);
            alive = mbar_wait(bar_acc, it & 1, abort_flag, a.status);
            if (!alive) break;
            tc_fence_after();
            const int kb0 = tl.n_tile * (a.BN / 32);
            // every chunk slot is handed back each tile (also the ones this tile did not use), so that the MMA issuer's
            // wait on a slot always refers to the previous tile
            for (int c = 0; c < kMaxChunks; ++c) {
                if (c >= tl.chunks) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_chunk_free + 8 * c);
                    continue;
                }
                const int q = c * 128 + row;
                bool valid;
                int n, oh, ow;
                if (a.nn == 1) {
                    const int qq = tl.q0 + q;
                    oh = qq / a.Wq; ow = qq - oh * a.Wq; n = tl.n0;
                    valid = oh < a.OH && ow < a.OW;
                } else {
                    const int pv = a.Hq * a.Wq;
                    const int img = q / pv, rem = q - img * pv;
                    oh = rem / a.Wq; ow = rem - oh * a.Wq; n = tl.n0 + img;
                    valid = img < a.nn && n < a.N && oh < a.OH && ow < a.OW;
                }
                const int nj = a.BN / 32;
                for (int j = 0; j < nj; ++j) {
                    float v[32];
                    tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * a.BN + j * 32), v);
                    if (j == nj - 1) {   // the chunk's values are in registers: give the slot back before storing
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_chunk_free + 8 * c);
                    }
                    const int kb = kb0 + j;
                    if (!valid || kb >= a.KB) continue;
                    float *dst = a.out + ((((size_t)n * a.KB + kb) * a.OH + oh) * a.OW + ow) * 32;
                    const float *bs = bias_s + kb * 32;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float r[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) r[e] = v[8 * i + e] + bs[8 * i + e];
                        if (a.accumulate) {
                            float p[8];
                            ld_global_v8(dst + 8 * i, p);
#pragma unroll
                            for (int e = 0; e < 8; ++e) r[e] += p[e];
                        }
                        if (a.relu) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) r[e] = fmaxf(r[e], 0.f);
                        }
                        const int k = kb * 32 + 8 * i;   // pad lanes of the last filter block stay +0
                        if (k + 7 >= a.K) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) if (k + e >= a.K) r[e] = 0.f;
                        }
                        st_global_v8(dst + 8 * i, r);
                    }
                }
            }
        }
        tc_fence_before();
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------------- host side
size_t ctrl_bytes(int KB) { return kCtrlBarrierBytes + 16 + (size_t)KB * 32 * 4; }

// Plan for at most `max_chunks` accumulator chunks per tile and filter tiles of `BN`; ok = false when it does not fit.
TcPlan make_plan_with(const Geom &g, size_t max_smem, int max_chunks, int BN) {
    TcPlan p{};
    p.ok = false;
    if (g.S != 1) return p;
    p.OH = g.OH; p.OW = g.OW;
    const int padw = g.pl > g.pr ? g.pl : g.pr, padh = g.pt > g.pb ? g.pt : g.pb;
    const int minw = g.pl < g.pr ? g.pl : g.pr, minh = g.pt < g.pb ? g.pt : g.pb;
    p.Wq = g.W + padw;
    p.Hq = g.H + padh;
    if (p.Wq > 256 || g.FH * g.FW > 64) return p;
    const int Kp = g.KB * 32;
    p.BN = BN < Kp ? BN : Kp;
    p.n_tiles = ceil_div(Kp, p.BN);
    const long long pv = (long long)p.Hq * p.Wq;
    int a0max;
    if (pv <= max_chunks * 128 && p.Hq <= 256) {
        // whole images per strip: as many as fill the chunks (at least one)
        p.nn = (int)((max_chunks * 128) / pv);
        if (p.nn > 256) p.nn = 256;
        if (p.nn > g.N) p.nn = g.N;
        p.chunks = ceil_div((int)(p.nn * pv), 128);
        p.total_chunks = p.chunks; p.tiles_img = 1;
        p.Rs = p.Hq;
        p.m_tiles = ceil_div(g.N, p.nn);
        p.tail_px = minh * p.Wq + minw;
        p.strip_px = p.nn * p.Rs * p.Wq;
        a0max = 0;   // with one image per strip the kernel's row-tile formulas describe the same geometry (q0 = 0)
    } else {
        // row tiles of one image: runs of chunks * 128 pixels of the flattened padded plane
        p.nn = 1;
        p.total_chunks = ceil_div(g.OH * p.Wq, 128);
        const int tiles = ceil_div(p.total_chunks, max_chunks);
        p.chunks = ceil_div(p.total_chunks, tiles);              // balanced: 7 chunks -> 4 + 3, not 4 + 4 slots
        p.tiles_img = ceil_div(p.total_chunks, p.chunks);
        p.Rs = (p.Wq - 1 + p.chunks * 128 - 1) / p.Wq + 1 + g.FH - 1;
        if (p.Rs > 256) return p;
        p.m_tiles = g.N * p.tiles_img;
        p.tail_px = minw;
        p.strip_px = p.Rs * p.Wq;
        a0max = p.Wq - 1;
    }
    // every pixel an MMA can touch lies inside the stage: strip + zero tail, and the furthest shifted chunk
    const int reach = a0max + p.chunks * 128 + (g.FH - 1) * p.Wq + g.FW - 1;
    p.stage_px = p.strip_px + p.tail_px > reach ? p.strip_px + p.tail_px : reach;
    p.a_stage_bytes = (uint32_t)(((size_t)p.stage_px * 128 + 1023) & ~(size_t)1023);
    p.b_stage_bytes = (uint32_t)p.BN * 128u;
    int cols = p.chunks * p.BN;
    p.tmem_cols = 32;
    while (p.tmem_cols < cols) p.tmem_cols <<= 1;
    if (p.tmem_cols > 512) return p;
    const size_t fixed = 1024 + (size_t)kAStages * p.a_stage_bytes + ctrl_bytes(g.KB);
    if (fixed + 2 * (size_t)p.b_stage_bytes > max_smem) return p;
    size_t room = (max_smem - fixed) / p.b_stage_bytes;
    p.b_stages = (int)(room < (size_t)kMaxBStages ? room : kMaxBStages);
    p.smem_bytes = (uint32_t)(fixed + (size_t)p.b_stages * p.b_stage_bytes);
    if ((long long)p.m_tiles * p.n_tiles > 0x7fffffffLL) return p;
    p.ok = true;
    return p;
}

// Estimated cycles of the whole layer under a plan: the slower of MMA issue and L2 -> shared-memory traffic per tile,
// plus a fixed hand-over cost, times the tiles the busiest SM gets.
double plan_cost(const TcPlan &p, const Geom &g, int sms) {
    const double steps = (double)g.CB * g.FH * g.FW;
    const double avg_chunks = p.nn == 1 ? (double)p.total_chunks / p.tiles_img : (double)p.chunks;
    const double mma = avg_chunks * steps * 4.0 * (p.BN / 2.0 < 16.0 ? 16.0 : p.BN / 2.0);
    const double bytes = (double)g.CB * p.strip_px * 128.0 + steps * p.b_stage_bytes + avg_chunks * 128.0 * p.BN * 4.0;
    const double mem = bytes / 24.0;                 // bytes per clock one SM can expect from L2 when all SMs pull
    const double starve = p.b_stages < 4 ? 1.15 : 1.0;   // few filter stages in flight: the MMA issuer waits on L2 latency
    const double tile = (mma > mem ? mma : mem) * starve + 2500.0;
    const double tiles = (double)p.m_tiles * p.n_tiles;
    const double per_sm = tiles <= sms ? 1.0 : tiles / sms;
    const double waves = per_sm < 4.0 ? (double)(long long)(per_sm + 0.999) : per_sm;   // few tiles per SM: whole waves
    return waves * tile;
}

// The cheapest plan over the tile shapes that fit (wide rows or tall windows leave room for fewer chunks).
TcPlan make_plan(const Geom &g, size_t max_smem, int sms) {
    TcPlan best{};
    double best_cost = 0.0;
    const int bns[3] = {128, 64, 32};
    for (int chunks = kMaxChunks; chunks >= 1; --chunks)
        for (int b = 0; b < 3; ++b) {
            if (b > 0 && bns[b] >= g.KB * 32) continue;      // same as the previous candidate
            TcPlan p = make_plan_with(g, max_smem, chunks, bns[b]);
            if (!p.ok) continue;
            const double c = plan_cost(p, g, sms);
            if (!best.ok || c < best_cost) { best = p; best_cost = c; }
        }
    return best;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

bool conv_tc_supported(const Geom &g) {
    return make_plan(g, 227 * 1024, 148).ok;
}

int launch_conv_tc(small_ctx *ctx, const float *in, const float *w_hi, const float *w_lo, const float *bias, float *out,
                   const Geom &g, bool relu, bool accumulate, unsigned mode, cudaStream_t st) {
    (void)w_lo; (void)mode;
    TcPlan p = make_plan(g, ctx->max_smem_optin < 227 * 1024 ? ctx->max_smem_optin : 227 * 1024, ctx->sm_count);
    if (!p.ok) return SMALL_ERR_UNSUPPORTED;
    EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    CUtensorMap map_a, map_b;
    {   // activations: [N][CB][H][W][32 floats]; box = 32 x Wq x Rs x 1 x nn, out-of-range elements read as zero
        cuuint64_t dims[5] = {32, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.CB, (cuuint64_t)g.N};
        cuuint64_t strides[4] = {128, (cuuint64_t)g.W * 128, (cuuint64_t)g.H * g.W * 128, (cuuint64_t)g.CB * g.H * g.W * 128};
        cuuint32_t box[5] = {32, (cuuint32_t)p.Wq, (cuuint32_t)p.Rs, 1, (cuuint32_t)p.nn};
        cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        CUresult r = encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<float *>(in), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    {   // filters: [CB][FH*FW][KB*32][32 floats]; box = 32 x BN rows
        const int T = g.FH * g.FW, Kp = g.KB * 32;
        cuuint64_t dims[4] = {32, (cuuint64_t)Kp, (cuuint64_t)T, (cuuint64_t)g.CB};
        cuuint64_t strides[3] = {128, (cuuint64_t)Kp * 128, (cuuint64_t)T * Kp * 128};
        cuuint32_t box[4] = {32, (cuuint32_t)p.BN, 1, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        CUresult r = encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float *>(w_hi), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    TcArgs a{};
    a.bias = bias; a.out = out; a.status = ctx->dev_status;
    a.N = g.N; a.K = g.K; a.KB = g.KB; a.CB = g.CB; a.OH = g.OH; a.OW = g.OW; a.Wq = p.Wq; a.Hq = p.Hq;
    a.FH = g.FH; a.FW = g.FW; a.pt = g.pt; a.pl = g.pl;
    a.nn = p.nn; a.chunks = p.chunks; a.total_chunks = p.total_chunks; a.tiles_img = p.tiles_img; a.m_tiles = p.m_tiles; a.n_tiles = p.n_tiles;
    a.BN = p.BN; a.Rs = p.Rs; a.strip_px = p.strip_px; a.tail_px = p.tail_px; a.tmem_cols = p.tmem_cols; a.b_stages = p.b_stages;
    a.a_stage_bytes = p.a_stage_bytes; a.b_stage_bytes = p.b_stage_bytes;
    a.a_box_bytes = (uint32_t)p.strip_px * 128u;
    a.relu = relu; a.accumulate = accumulate;
    cudaError_t e = cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes);
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    const long long tiles = (long long)p.m_tiles * p.n_tiles;
    const unsigned grid = (unsigned)(tiles < ctx->sm_count ? tiles : ctx->sm_count);   // persistent: one CTA per SM
    conv_tc_kernel<<<grid, kThreads, p.smem_bytes, st>>>(map_a, map_b, a);
    return check_launch(ctx);
}

}  // namespace small
