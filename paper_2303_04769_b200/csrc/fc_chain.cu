// A chain of full reductions (paper Section 3.2 item 5; Section 6: the abstract fused layer) as ONE kernel on the tensor
// cores: out = f_L(... f_2(f_1(in))), f_i(x) = act(W_i x + b_i), every width at most 128.  A thread block keeps a tile of
// 128 images for the whole chain: the activations never leave the SM between layers.
//
//   A operand   = the tile's activations [128 images][J], K-major with the 128-byte swizzle, one 16 KB block per 32
//                 channels, resident in shared memory (3xTF32: the TF32 part and, 64 KB on, the residual)
//   B operand   = the layer's filters [K rows][32 channels] per channel block, streamed by TMA through a small ring
//   accumulator = 128 lanes (images) x up to 128 columns (outputs) of tensor memory
//   epilogue    = tensor memory -> registers, + bias, ReLU, and the result is written straight back into the A buffer as
//                 the next layer's operand (swizzled 16-byte chunks, split into TF32 part and residual for 3xTF32); the
//                 last layer's result goes to global memory as blocked [N][K] lines
// Roles: warp 0 streams filters, one thread of warp 1 loads the tile's input and issues the MMAs, warps 4-7 (one thread
// per image = tensor-memory lane) run the epilogue.  A layer's MMAs wait for the epilogue of the layer before it (which
// has then also finished reading the accumulator), and the in-place rewrite of the A buffer waits for the layer's MMAs to
// complete.  Every wait is bounded; on expiry the kernel records SMALL_ERR_TIMEOUT, lets its copies land, frees its
// tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "sm100.cuh"

namespace small {

namespace {

using namespace sm100;

constexpr int kChainMax = 12;          // layers per launch
constexpr int kTile = 128;             // images per tile = the MMA's M
constexpr int kBlockBytes = 16 * 1024; // 128 rows x 128 bytes: one 32-channel block of the A operand or of a filter box
constexpr int kAHalf = 4 * kBlockBytes;
constexpr int kChainThreads = 256;
constexpr uint32_t kSpin = 4096;       // polls without back-off for the roles on the layer-to-layer critical path
constexpr int kChainCtrl = 192;        // barriers, tensor-memory address, abort flag; the bias table follows

struct ChainArgs {
    CUtensorMap map_in;                 // [N][JB0][32] activations of the first layer
    CUtensorMap map_w[kChainMax];       // TF32 filters of layer i: [CB][K rows][32]
    CUtensorMap map_w_lo[kChainMax];    // their residuals (3xTF32)
    const float *bias[kChainMax];
    int J[kChainMax], K[kChainMax], relu[kChainMax];
    int box_rows[kChainMax];            // filter rows per box: the layer's rows, 128 for a last layer wider than that
    float *out; int *status;
    int L, N, tiles, b_stages;
    uint32_t wait_iters;
};


// Shared memory: [A: 4 slots of 16 KB, 3xTF32 twice that][filter ring: b_stages x (16 KB, 3xTF32 32 KB)][control block].
// The first layer may be wider than 128 channels: its input blocks stream through the four A slots (slot = block & 3, a
// slot refilled once the MMAs that read it have completed), the epilogue warps splitting each block for 3xTF32 as it
// lands.  From the second layer on the operand is what the epilogue of the layer before wrote into slots 0 .. 3.
template <bool X3>
__global__ void __launch_bounds__(kChainThreads, 1) fc_chain_kernel(const __grid_constant__ ChainArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    constexpr uint32_t kABytes = X3 ? 2 * kAHalf : kAHalf;
    constexpr uint32_t kBStage = X3 ? 2 * kBlockBytes : kBlockBytes;
    const uint32_t a_base = base, b_base = base + kABytes;
    const uint32_t ctrl = b_base + a.b_stages * kBStage;
    uint8_t *ctrl_ptr = base_ptr + (ctrl - base);
    // barriers: filter stages full / empty, input block landed / split / its slot free again (four each), operand ready
    // (= epilogue of the layer before done), accumulator complete
    const uint32_t bar_b_full = ctrl, bar_b_empty = ctrl + 32, bar_in = ctrl + 64, bar_split = ctrl + 96, bar_slot_free = ctrl + 128;
    const uint32_t bar_a_ready = ctrl + 160, bar_acc = ctrl + 168;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(ctrl_ptr + 176);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(ctrl_ptr + 180);
    float *bias_s = reinterpret_cast<float *>(ctrl_ptr + kChainCtrl);            // [L - 1][128], then the last layer's

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int JB0 = (a.J[0] + 31) >> 5;
    // the last layer may have more than 128 filters: it runs as chunks of 128, each one more pass over the same operand
    const int last_chunks = (a.K[a.L - 1] + 127) >> 7, steps_per_tile = a.L - 1 + last_chunks;
    if (threadIdx.x == 0) {
        for (int s = 0; s < 4; ++s) {
            mbar_init(bar_b_full + 8 * s, 1); mbar_init(bar_b_empty + 8 * s, 1);
            mbar_init(bar_in + 8 * s, 1); mbar_init(bar_split + 8 * s, 4); mbar_init(bar_slot_free + 8 * s, 1);
        }
        mbar_init(bar_a_ready, 4);        // one arrival per epilogue warp
        mbar_init(bar_acc, 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    for (int i = threadIdx.x; i < steps_per_tile * 128; i += kChainThreads) {
        const int l = min(i >> 7, a.L - 1), k = i - l * 128;
        bias_s[i] = (a.bias[l] && k < a.K[l]) ? a.bias[l][k] : 0.0f;
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), 128u);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    grid_dep_sync();
    grid_dep_trigger();

    // copies a producer started and the parity of each barrier's latest one, kept for the drain after an abort
    uint32_t armed_mask = 0, armed_parity = 0, in_mask = 0, in_par = 0;

    if (warp == 0 && lane == 0) {
        // ---- first layer: its input blocks; every layer: one filter box (K rows x 128 bytes; 3xTF32: two) per channel block
        bool alive = true, wrapped = false;
        uint32_t s = 0, phase = 0, tile_k = 0;
        uint32_t loads[4] = {0, 0, 0, 0};              // input blocks loaded into each slot so far
        for (int t = blockIdx.x; t < a.tiles && alive; t += gridDim.x, ++tile_k)
            for (int l = 0; l < a.L && alive; ++l) {
                const int JB = (a.J[l] + 31) >> 5, chunks = l == a.L - 1 ? last_chunks : 1;
                for (int i = 0; i < chunks * JB; ++i) {
                    const int ch = i / JB, cb = i - ch * JB;
                    if (l == 0) {
                        const int slot = cb & 3;
                        // the slot's previous content: this tile's block cb - 4, or the previous tile's activations
                        if (cb >= 4) alive = mbar_wait(bar_slot_free + 8 * slot, (loads[slot] - 1) & 1u, abort_flag, a.status, a.wait_iters);
                        else if (tile_k > 0) alive = mbar_wait(bar_acc, (tile_k * (uint32_t)steps_per_tile - 1) & 1u, abort_flag, a.status, a.wait_iters);
                        if (!alive) break;
                        mbar_expect_tx(bar_in + 8 * slot, kBlockBytes);
                        tma_load_3d(a_base + slot * kBlockBytes, &a.map_in, bar_in + 8 * slot, 0, cb, t * kTile);
                        in_mask |= 1u << slot;
                        in_par = (in_par & ~(1u << slot)) | ((loads[slot] & 1u) << slot);
                        ++loads[slot];
                    }
                    if (wrapped) alive = mbar_wait(bar_b_empty + 8 * s, phase ^ 1u, abort_flag, a.status, a.wait_iters);
                    if (!alive) break;
                    mbar_expect_tx(bar_b_full + 8 * s, (uint32_t)a.box_rows[l] * 128u * (X3 ? 2u : 1u));
                    tma_load_3d(b_base + s * kBStage, &a.map_w[l], bar_b_full + 8 * s, 0, ch * 128, cb);
                    if (X3) tma_load_3d(b_base + s * kBStage + kBlockBytes, &a.map_w_lo[l], bar_b_full + 8 * s, 0, ch * 128, cb);
                    armed_mask |= 1u << s;
                    armed_parity = (armed_parity & ~(1u << s)) | (phase << s);
                    if (++s == (uint32_t)a.b_stages) { s = 0; phase ^= 1u; wrapped = true; }
                }
            }
    } else if (warp == 1 && lane == 0) {
        // ---- the MMAs of every layer
        bool alive = true, first_layer_ever = true;
        uint32_t sb = 0, pb = 0, n_ready = 0;
        uint32_t used[4] = {0, 0, 0, 0};               // input blocks consumed from each slot so far
        for (int t = blockIdx.x; t < a.tiles && alive; t += gridDim.x) {
            for (int st = 0; st < steps_per_tile && alive; ++st) {
                const int l = min(st, a.L - 1), ch = st - l;
                // the epilogue of the layer before (the last layer of the tile before) is done: the accumulator has been
                // read out and, from the second layer on, the operand is in place
                if (!first_layer_ever) {
                    alive = mbar_wait<kSpin>(bar_a_ready, n_ready & 1u, abort_flag, a.status, a.wait_iters);
                    ++n_ready;
                    if (!alive) break;
                }
                first_layer_ever = false;
                tc_fence_after();
                const int JB = (a.J[l] + 31) >> 5, rows = min(((a.K[l] + 31) >> 5) * 32 - ch * 128, 128);
                const uint32_t idesc = instr_desc(rows);
                uint32_t started = 0;
                for (int cb = 0; cb < JB && alive; ++cb) {
                    const int slot = l == 0 ? (cb & 3) : cb;
                    if (l == 0) {
                        alive = mbar_wait<kSpin>((X3 ? bar_split : bar_in) + 8 * slot, used[slot] & 1u, abort_flag, a.status, a.wait_iters);
                        ++used[slot];
                        if (!alive) break;
                    }
                    alive = mbar_wait<kSpin>(bar_b_full + 8 * sb, pb, abort_flag, a.status, a.wait_iters);
                    if (!alive) break;
                    tc_fence_after();
                    const int ks = cb == JB - 1 ? (a.J[l] - cb * 32 + 7) >> 3 : 4;      // K steps with real channels
                    const uint32_t xa = smem_desc_lo(a_base + slot * kBlockBytes), wb = smem_desc_lo(b_base + sb * kBStage);
                    for (int k = 0; k < ks; ++k) {
                        if (X3) {
                            mma_tf32(tmem, xa + (kAHalf >> 4) + 2u * k, wb + 2u * k, kDescHi, idesc, started);          // x_lo w_hi
                            mma_tf32(tmem, xa + 2u * k, wb + (kBlockBytes >> 4) + 2u * k, kDescHi, idesc, 1u);          // x_hi w_lo
                            mma_tf32(tmem, xa + 2u * k, wb + 2u * k, kDescHi, idesc, 1u);                               // x_hi w_hi
                        } else {
                            mma_tf32(tmem, xa + 2u * k, wb + 2u * k, kDescHi, idesc, started);
                        }
                        started = 1u;
                    }
                    if (l == 0) mma_commit(bar_slot_free + 8 * slot);
                    mma_commit(bar_b_empty + 8 * sb);
                    if (++sb == (uint32_t)a.b_stages) { sb = 0; pb ^= 1u; }
                }
                if (alive) mma_commit(bar_acc);
            }
        }
    } else if (warp >= 4) {
        // ---- epilogue: thread = image = tensor-memory lane; also splits the first layer's input blocks for 3xTF32
        const int quarter = warp & 3, r = quarter * 32 + lane;
        uint8_t *a_row = base_ptr + (size_t)r * 128;                 // this image's row in every 16 KB slot
        const int sw = r & 7;                                         // 16-byte chunk c of the row lies at chunk c ^ sw
        bool alive = true;
        uint32_t n_acc = 0;
        uint32_t seen[4] = {0, 0, 0, 0};
        auto put = [&](int blk, int c, const float4 v) {              // 4 channels of this image into the A operand
            uint8_t *dst = a_row + (size_t)blk * kBlockBytes + ((c ^ sw) << 4);
            if (X3) {
                const float4 h = make_float4(__uint_as_float(__float_as_uint(v.x) & 0xffffe000u), __uint_as_float(__float_as_uint(v.y) & 0xffffe000u),
                                             __uint_as_float(__float_as_uint(v.z) & 0xffffe000u), __uint_as_float(__float_as_uint(v.w) & 0xffffe000u));
                *reinterpret_cast<float4 *>(dst) = h;
                *reinterpret_cast<float4 *>(dst + kAHalf) = make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w);
            } else {
                *reinterpret_cast<float4 *>(dst) = v;
            }
        };
        for (int t = blockIdx.x; t < a.tiles && alive; t += gridDim.x) {
            if (X3)
                for (int cb = 0; cb < JB0 && alive; ++cb) {
                    const int slot = cb & 3;
                    alive = mbar_wait_warp<kSpin>(bar_in + 8 * slot, seen[slot] & 1u, abort_flag, a.status, a.wait_iters);
                    ++seen[slot];
                    if (!alive) break;
#pragma unroll
                    for (int c = 0; c < 8; ++c) put(slot, c, *reinterpret_cast<const float4 *>(a_row + (size_t)slot * kBlockBytes + ((c ^ sw) << 4)));
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_split + 8 * slot);
                }
            const long long n = (long long)t * kTile + r;
            for (int st = 0; st < steps_per_tile && alive; ++st) {
                const int l = min(st, a.L - 1), ch = st - l;
                alive = mbar_wait_warp<kSpin>(bar_acc, n_acc & 1u, abort_flag, a.status, a.wait_iters);
                ++n_acc;
                if (!alive) break;
                tc_fence_after();
                const int K = a.K[l] - ch * 128, KB = min((K + 31) >> 5, 4), KB_all = (a.K[l] + 31) >> 5;
                const bool last = l == a.L - 1;
                for (int kb = 0; kb < KB; ++kb) {
                    float v[32];
                    tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)kb * 32u, v);
                    const float *bs = bias_s + st * 128 + kb * 32;
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        float x = v[e] + bs[e];
                        if (a.relu[l]) x = fmaxf(x, 0.0f);
                        v[e] = kb * 32 + e < K ? x : 0.0f;            // pad lanes stay +0
                    }
                    if (!last) {
#pragma unroll
                        for (int c = 0; c < 8; ++c) put(kb, c, make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]));
                    } else if (n < a.N) {
                        float *dst = a.out + ((size_t)n * KB_all + ch * 4 + kb) * 32;
#pragma unroll
                        for (int c = 0; c < 4; ++c) st_global_v8(dst + 8 * c, v + 8 * c);
                    }
                }
                tc_fence_before();
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_a_ready);
            }
        }
    }
    __syncthreads();
    if (*abort_flag && warp == 0 && lane == 0) {     // a role gave up: let the copies still in flight land before the block exits
        for (int st = 0; st < 4; ++st) {
            if (armed_mask >> st & 1u)
                for (uint32_t it = 0; it < a.wait_iters && !mbar_try_wait(bar_b_full + 8 * st, armed_parity >> st & 1u); ++it) __nanosleep(200);
            if (in_mask >> st & 1u)
                for (uint32_t it = 0; it < a.wait_iters && !mbar_try_wait(bar_in + 8 * st, in_par >> st & 1u); ++it) __nanosleep(200);
        }
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, 128u);
    }
}

}  // namespace

// A run of full reductions that the fused kernel takes: 2 to 12 layers, every width between two layers at most 128 (the
// first layer's input and the last layer's output may be wider), a tensor-core math mode.
bool fc_chain_supported(const int *widths, int L, unsigned math) {
    if (L < 2 || L > kChainMax || (math != SMALL_MATH_TF32 && math != SMALL_MATH_3XTF32)) return false;
    if (widths[0] < 1 || widths[0] > 8192) return false;        // the first layer's input streams: it may be wide
    for (int i = 1; i < L; ++i)
        if (widths[i] < 1 || widths[i] > 128) return false;
    return widths[L] >= 1 && widths[L] <= 1024;                 // the last layer runs in chunks of 128 filters
}

int launch_fc_chain(small_ctx *ctx, const float *in, const float *const *w_blk, const float *const *bias, const int *widths,
                    const int *relu, float *out, int L, int N, unsigned math, cudaStream_t st) {
    if (!fc_chain_supported(widths, L, math)) return SMALL_ERR_UNSUPPORTED;
    const bool x3 = math == SMALL_MATH_3XTF32;
    EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    ChainArgs a{};
    a.L = L; a.N = N; a.tiles = ceil_div(N, kTile); a.out = out; a.status = ctx->dev_status; a.wait_iters = ctx->wait_iters;
    a.b_stages = x3 ? 2 : 4;
    {   // the first layer's input, blocked [N][JB][32]: one box = 128 images x one 32-channel block
        const int JB = blocks_of(widths[0]);
        cuuint64_t dims[3] = {32, (cuuint64_t)JB, (cuuint64_t)N};
        cuuint64_t strides[2] = {128, (cuuint64_t)JB * 128};
        cuuint32_t box[3] = {32, 1, (cuuint32_t)kTile};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = encode(&a.map_in, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(in), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    for (int l = 0; l < L; ++l) {
        const int J = widths[l], K = widths[l + 1], CB = blocks_of(J), Kp = blocks_of(K) * 32;
        a.J[l] = J; a.K[l] = K; a.box_rows[l] = Kp < 128 ? Kp : 128; a.relu[l] = relu[l] ? 1 : 0; a.bias[l] = bias ? bias[l] : nullptr;
        // the tensor-core sections of the layer's packed filters: [CB][K rows][32], TF32 part then residual
        const float *w_hi = w_blk[l] + conv_w_fp32_elems(J, K, 1, 1);
        const float *w_lo = w_hi + conv_w_tc_elems(J, K, 1, 1);
        for (int half = 0; half < (x3 ? 2 : 1); ++half) {
            cuuint64_t dims[3] = {32, (cuuint64_t)Kp, (cuuint64_t)CB};
            cuuint64_t strides[2] = {128, (cuuint64_t)Kp * 128};
            cuuint32_t box[3] = {32, (cuuint32_t)(Kp < 128 ? Kp : 128), 1};
            cuuint32_t estr[3] = {1, 1, 1};
            CUresult r = encode(half ? &a.map_w_lo[l] : &a.map_w[l], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(half ? w_lo : w_hi),
                                dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
        }
        if (!x3) a.map_w_lo[l] = a.map_w[l];
    }
    for (int l = L; l < kChainMax; ++l) { a.map_w[l] = a.map_w[0]; a.map_w_lo[l] = a.map_w_lo[0]; }
    const size_t smem = 1024 + (x3 ? 2 : 1) * (size_t)kAHalf + (size_t)a.b_stages * (x3 ? 2 : 1) * kBlockBytes + kChainCtrl + ((size_t)L - 1 + ceil_div(widths[L], 128)) * 128 * sizeof(float);
    void (*kern)(const ChainArgs) = x3 ? fc_chain_kernel<true> : fc_chain_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->max_smem_optin);
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    if (smem > ctx->max_smem_optin) return SMALL_ERR_UNSUPPORTED;
    const unsigned grid = (unsigned)(a.tiles < ctx->sm_count ? a.tiles : ctx->sm_count);
    launch_kernel(ctx, kern, dim3(grid), dim3(kChainThreads), smem, st, a);
    return check_launch(ctx);
}

}  // namespace small
