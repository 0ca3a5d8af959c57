// A chain of full reductions (paper Section 3.2 item 5; Section 6: the abstract fused layer) as ONE kernel on the tensor
// cores: out = f_L(... f_2(f_1(in))), f_i(x) = act(W_i x + b_i), every width between two layers at most 128.  A thread
// block keeps a tile of nt images (32, 64 or 128) for the whole chain: the activations never leave the SM between layers.
// The filters sit on the MMA's M side, the images on its N side, so a small batch still spreads over many SMs:
//
//   A operand   = the layer's filters [128 rows][32 channels] per channel block (K-major, 128-byte swizzle), streamed by
//                 TMA through a ring of stages (3xTF32: the TF32 part and, 16 KB on, the residual); rows past the layer's
//                 filter count hold whatever the stage held before and only feed accumulator lanes nobody reads
//   B operand   = the tile's activations [nt images][32 channels] per channel block, K-major with the 128-byte swizzle,
//                 resident in shared memory slots 0 .. 3 (3xTF32: each block's residual rows right behind its TF32 rows);
//                 the first layer's input, which may be wider than 128 channels, streams through all the slots
//   accumulator = 128 lanes (filters) x nt columns (images) of tensor memory, 256 / nt of them in rotation, so that a
//                 last layer wider than 128 filters runs its chunks of 128 back to back while the epilogue drains them.
//                 3xTF32 takes two MMAs per K step for its three products: w_hi against the 2 nt rows [x_hi; x_lo]
//                 (columns [0, nt) and [nt, 2 nt) of a 2 nt wide accumulator), then w_lo against x_hi into columns
//                 [0, nt); the epilogue adds the two halves
//   epilogue    = thread = filter: tensor memory -> registers, + bias, ReLU, and the filter's nt values go straight back
//                 into the B slots as the next layer's operand (for 3xTF32 split into TF32 part and residual); the last
//                 layer's values go to global memory, a warp writing one image's 32-channel line per store
// Roles: one thread of warp 0 issues the MMAs; the first lanes of warp 1 stream the first layer's input and every layer's
// filters, each lane its own loads in lockstep with the others; warps 4 .. (four per 32 images) run the epilogue.
//
// The chain is latency-bound, so the design follows what one thread's instructions were measured to cost: a poll of an
// mbarrier that is already complete takes a hundred cycles or more, arming a barrier and starting a copy several hundred,
// and a tcgen05.commit stalls the issuing thread for about 450 cycles - each more than the four MMAs of a channel block.
// Hence: several producer lanes; the MMA thread starts the polls of up to four blocks together; filter stages are handed
// back in groups (one commit per group, not per stage), operand slots of a wide first layer in groups of four, and only
// where a later block reuses them.
//
// A layer's MMAs wait for the epilogue of the layer before it, the rewrite of the slots waits for the MMAs that read them
// (the accumulator's barrier), and an accumulator is reused only after its epilogue.  A barrier's phase is only ever
// awaited by a thread that has itself seen the phase before (stages, slots and their groups have fixed owners among the
// producer lanes); what a latecomer may read is a counter (steps_done).  Every wait is bounded; on expiry the kernel
// records SMALL_ERR_TIMEOUT, lets its copies land, frees its tensor memory and returns.
#include <cuda.h>

#include <algorithm>

#include "common.cuh"
#include "sm100.cuh"

namespace small {

namespace {

using namespace sm100;

constexpr int kChainMax = 12;          // layers per launch
constexpr int kWBlock = 16 * 1024;     // one filter box: 128 rows x 128 bytes
constexpr int kTmemCols = 256;
constexpr uint32_t kSpin = 1u << 15;      // polls without back-off for the roles on the layer-to-layer critical path
constexpr int kMaxThreads = 128 + 16 * 32;
// control block: barriers (8 bytes each), then the tensor-memory address, the abort flag and the step counter; the bias
// table follows
constexpr int kOffWFull = 0, kOffWEmpty = 64, kOffInFull = 128, kOffSplit = 256, kOffSlotFree = 384, kOffAccFull = 512,
              kOffEpiDone = 576, kOffTmem = 640, kOffAbort = 644, kOffStepsDone = 648, kCtrl = 704;

struct ChainArgs {
    CUtensorMap map_in;                 // [N][JB0][32] activations of the first layer; box = nt images x one channel block
    CUtensorMap map_w[kChainMax];       // TF32 filters of layer i: [CB][K rows][32]
    CUtensorMap map_w_lo[kChainMax];    // their residuals (3xTF32)
    const float *bias[kChainMax];
    int J[kChainMax], K[kChainMax], relu[kChainMax];
    int box_rows[kChainMax];            // filter rows per box: the layer's rows, 128 for a last layer wider than that
    int first_load[kChainMax + 1];      // loads (one per channel block and chunk) of a tile before layer i; [L] = per tile
    float *out; int *status;
    int L, N, tiles;
    int nt, n_slots, w_stages;          // images per tile, operand slots, filter stages
    int release;                        // stages handed back per commit; divides w_stages
    int lanes;                          // producer lanes (4, or 2); divides w_stages, and n_slots where slots are reused
    uint32_t wait_iters;
};

// Bounded wait for a counter in shared memory to reach `need` (a count, unlike a barrier's phase parity, can be read
// however late the reader comes).
__device__ __forceinline__ bool counter_wait(volatile uint32_t *counter, uint32_t need, volatile int *abort_flag, int *status, uint32_t limit) {
    for (uint32_t it = 0; it < limit; ++it) {
        if (*counter >= need) { __threadfence_block(); return true; }
        if (it >= kSpin) __nanosleep(100);
        if ((it & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(status, (int)SMALL_ERR_TIMEOUT);
    return false;
}

template <bool X3>
__global__ void __launch_bounds__(kMaxThreads, 1) fc_chain_kernel(const __grid_constant__ ChainArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    constexpr uint32_t kWStage = X3 ? 2 * kWBlock : kWBlock;
    const int nt = a.nt, n_slots = a.n_slots;
    // a slot: the tile's nt rows of one channel block; 3xTF32: the residuals' nt rows right behind them, so that one
    // descriptor of 2 nt rows covers both
    const uint32_t slot_bytes = (uint32_t)nt * 128u, slot_pitch = X3 ? 2u * slot_bytes : slot_bytes;
    const uint32_t x_base = base, w_base = base + (uint32_t)n_slots * slot_pitch;
    const uint32_t ctrl = w_base + (uint32_t)a.w_stages * kWStage;
    uint8_t *ctrl_ptr = base_ptr + (ctrl - base);
    const uint32_t bar_w_full = ctrl + kOffWFull, bar_w_empty = ctrl + kOffWEmpty, bar_in = ctrl + kOffInFull, bar_split = ctrl + kOffSplit,
                   bar_slot_free = ctrl + kOffSlotFree, bar_acc = ctrl + kOffAccFull, bar_epi = ctrl + kOffEpiDone;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(ctrl_ptr + kOffTmem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(ctrl_ptr + kOffAbort);
    volatile uint32_t *steps_done = reinterpret_cast<volatile uint32_t *>(ctrl_ptr + kOffStepsDone);   // steps whose MMAs have all completed
    float *bias_s = reinterpret_cast<float *>(ctrl_ptr + kCtrl);                // [L - 1][128], then the last layer's

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_epi_warps = nt >> 3;                     // four warps (one per 32 tensor-memory lanes) per 32 images
    const int JB0 = (a.J[0] + 31) >> 5;
    // the last layer may have more than 128 filters: it runs as chunks of 128, each one more pass over the same operand
    const int last_chunks = (a.K[a.L - 1] + 127) >> 7, steps_per_tile = a.L - 1 + last_chunks;
    // accumulators in rotation: 256 columns / (nt, or 2 nt for 3xTF32, whose x_lo products land in a second set of columns)
    const uint32_t acc_cols = X3 ? 2u * (uint32_t)nt : (uint32_t)nt;
    const uint32_t nacc_log2 = (nt == 32 ? 3u : nt == 64 ? 2u : 1u) - (X3 ? 1u : 0u), nacc = 1u << nacc_log2;
    // slots, stages and stages per commit are powers of two
    const int ns_log2 = 31 - __clz(n_slots);
    const uint32_t ws_log2 = 31 - __clz(a.w_stages), rel_log2 = 31 - __clz(a.release);
    // The first layer's channel block cb lies in slot cb mod n_slots, its `cb / n_slots`-th use in the tile.  Slots are
    // handed back for reuse in groups of four (group = slot / 4), once per use that another use in the same tile follows.
    auto slot_uses = [&](int slot) -> uint32_t { return slot < JB0 ? (uint32_t)((JB0 - 1 - slot) >> ns_log2) + 1u : 0u; };
    auto group_uses = [&](int sg) -> uint32_t { return 4 * sg < JB0 ? (uint32_t)((JB0 - 1 - 4 * sg) >> ns_log2) + 1u : 0u; };

    // Set-up.  TF32: in two halves that meet at named barrier 1 - warp 1 initialises the barriers, arrives and goes straight
    // to its loads; the other warps fill the bias table, allocate tensor memory and wait there for the barriers to exist
    // (measured on the ten-layer chain: 39.6 -> 37.8 us).  3xTF32 keeps one block-wide barrier after the set-up: the same
    // change measured slower there (52.5 -> 57.8 us).
    if (threadIdx.x == 32) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(bar_w_full + 8 * s, 1); mbar_init(bar_w_empty + 8 * s, 1);
            mbar_init(bar_acc + 8 * s, 1); mbar_init(bar_epi + 8 * s, n_epi_warps);
        }
        for (int s = 0; s < 16; ++s) {
            mbar_init(bar_in + 8 * s, 1); mbar_init(bar_split + 8 * s, n_epi_warps); mbar_init(bar_slot_free + 8 * s, 1);
        }
        *abort_flag = 0;
        *steps_done = 0;
        mbar_fence_init();
    }
    uint32_t tmem = 0;
    if (warp == 1 && !X3) {
        __syncwarp();
        asm volatile("bar.arrive 1, %0;" ::"r"(blockDim.x) : "memory");
    } else {
        // filters and biases are no layer's output: they are read ahead of the wait on the launch before this one
        const int fillers = X3 ? blockDim.x : blockDim.x - 32;            // every thread, or every thread but warp 1's
        for (int i = threadIdx.x - (!X3 && warp > 1 ? 32 : 0); i < steps_per_tile * 128; i += fillers) {
            const int l = min(i >> 7, a.L - 1), k = i - l * 128;
            bias_s[i] = (a.bias[l] && k < a.K[l]) ? a.bias[l][k] : 0.0f;
        }
        if (warp == 0) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), (uint32_t)kTmemCols);
        tc_fence_before();
        if (X3) __syncthreads();
        else asm volatile("bar.sync 1, %0;" ::"r"(blockDim.x) : "memory");
        tc_fence_after();
        tmem = *tmem_slot;
    }
    grid_dep_trigger();

    // copies a producer lane started and the parity of each barrier's latest one, kept for the drain after an abort
    uint32_t armed_mask = 0, armed_parity = 0, in_mask = 0, in_par = 0;

    if (warp == 1 && lane < a.lanes) {
        // ---- first layer: its input blocks; every layer: one filter box (rows x 128 bytes; 3xTF32: two) per channel block.
        // Lane j takes the loads q = j, j + lanes, ...: stage q mod w_stages is always its own.  The position of a load in
        // the chain is advanced, not divided out: an integer division costs a lone thread a hundred cycles or more.
        const uint32_t per_tile = (uint32_t)a.first_load[a.L];
        const uint32_t my_tiles = blockIdx.x < (uint32_t)a.tiles ? ((uint32_t)a.tiles - blockIdx.x + gridDim.x - 1u) / gridDim.x : 0u;
        const uint32_t total = my_tiles * per_tile;
        const uint32_t lanes_mask = (1u << a.lanes) - 1u;
        bool alive = true, synced = false;
        uint32_t tile_k = 0, r = (uint32_t)lane;             // this lane's load: tile of this block, position in the tile
        int l = 0;
        for (uint32_t q0 = 0; q0 < total; q0 += (uint32_t)a.lanes) {       // every lane runs every round (they meet in it)
            const uint32_t q = q0 + (uint32_t)lane;
            const bool mine = q < total;
            while (r >= per_tile) { r -= per_tile; ++tile_k; l = 0; }
            while (l + 1 < a.L && (int)r >= a.first_load[l + 1]) ++l;
            const int JB = (a.J[l] + 31) >> 5;
            int cb = (int)r - a.first_load[l], ch = 0;
            while (cb >= JB) { cb -= JB; ++ch; }             // chunks: the last layer only
            const int t = (int)(blockIdx.x + tile_k * gridDim.x);
            const uint32_t s = q & (uint32_t)(a.w_stages - 1), turn = q >> ws_log2;           // turn: loads into this stage before
            // A tile's first loads wait for the tile before to complete, and that needs its last loads, which another lane
            // may hold in this very round: the lanes that wait for nothing of this round go first.
            const bool gated = l == 0 && cb < n_slots && tile_k > 0;
            auto load = [&]() {
                if (l == 0) {
                    const int slot = cb & (n_slots - 1), sg = slot >> 2, o = cb >> ns_log2;
                    const uint32_t use = tile_k * slot_uses(slot) + (uint32_t)o;
                    // the slot's previous content: this tile's block cb - n_slots, or the previous tile's activations
                    // (a group's barrier completes once per use that another use of the same tile follows)
                    if (o > 0)
                        alive = mbar_wait<kSpin>(bar_slot_free + 8 * sg, (tile_k * (group_uses(sg) - 1u) + (uint32_t)o - 1u) & 1u, abort_flag, a.status, a.wait_iters);
                    else if (tile_k > 0)
                        alive = counter_wait(steps_done, tile_k * (uint32_t)steps_per_tile, abort_flag, a.status, a.wait_iters);
                    if (!alive) return;
                    if (!synced) { grid_dep_sync(); synced = true; }
                    mbar_expect_tx(bar_in + 8 * slot, slot_bytes);
                    tma_load_3d(x_base + slot * slot_pitch, &a.map_in, bar_in + 8 * slot, 0, cb, t * nt);
                    in_mask |= 1u << slot;
                    in_par = (in_par & ~(1u << slot)) | ((use & 1u) << slot);
                }
                if (turn > 0) alive = mbar_wait<kSpin>(bar_w_empty + 8 * (s >> rel_log2), (turn - 1u) & 1u, abort_flag, a.status, a.wait_iters);
                if (!alive) return;
                mbar_expect_tx(bar_w_full + 8 * s, (uint32_t)a.box_rows[l] * 128u * (X3 ? 2u : 1u));
                tma_load_3d(w_base + s * kWStage, &a.map_w[l], bar_w_full + 8 * s, 0, ch * 128, cb);
                if (X3) tma_load_3d(w_base + s * kWStage + kWBlock, &a.map_w_lo[l], bar_w_full + 8 * s, 0, ch * 128, cb);
                armed_mask |= 1u << s;
                armed_parity = (armed_parity & ~(1u << s)) | ((turn & 1u) << s);
            };
            if (mine && alive && !gated) load();
            __syncwarp(lanes_mask);
            if (mine && alive && gated) load();
            r += (uint32_t)a.lanes;
        }
    } else if (warp == 0 && lane == 0) {
        // ---- the MMAs of every step (a layer, or a chunk of 128 filters of the last layer).  This thread's instruction
        // count is the chain's critical path: descriptors and counters advance by addition, a layer's polls start together.
        bool alive = true;
        uint32_t g = 0, tile_k = 0;                        // g: steps so far; accumulator and its barriers = g mod nacc
        const uint32_t idesc = instr_desc(nt), idesc_wide = instr_desc(2 * nt);
        const uint32_t w_desc0 = smem_desc_lo(w_base), x_desc0 = smem_desc_lo(x_base);
        const uint32_t w_step = kWStage >> 4, x_step = slot_pitch >> 4, w_lo = kWBlock >> 4;
        uint32_t sw = 0, pw = 0, wa = w_desc0;             // filter stage in turn, its parity, its descriptor
        uint32_t rel_left = (uint32_t)a.release, rel_bar = bar_w_empty;        // stages until the group in turn goes back
        const int group = min(4, a.w_stages);              // channel blocks whose barriers are polled together
        auto issue = [&](uint32_t acc, uint32_t xb, int ks, uint32_t &started) {      // the MMAs of one channel block
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k < ks) {
                    if (X3) {
                        // columns [0, nt): w_hi x_hi + w_lo x_hi; columns [nt, 2 nt): w_hi x_lo - two MMAs for three products
                        mma_tf32(acc, wa + 2u * k, xb + 2u * k, kDescHi, idesc_wide, started);
                        mma_tf32(acc, wa + w_lo + 2u * k, xb + 2u * k, kDescHi, idesc, 1u);
                    } else {
                        mma_tf32(acc, wa + 2u * k, xb + 2u * k, kDescHi, idesc, started);
                    }
                    started = 1u;
                }
        };
        auto next_stage = [&]() {                          // the filter stages go back in groups of `release`
            if (--rel_left == 0) {
                mma_commit(rel_bar);
                rel_left = (uint32_t)a.release;
                rel_bar += 8;
            }
            wa += w_step;
            if (++sw == (uint32_t)a.w_stages) { sw = 0; pw ^= 1u; wa = w_desc0; rel_bar = bar_w_empty; }
        };
        for (int t = blockIdx.x; t < a.tiles && alive; t += gridDim.x, ++tile_k) {
            for (int st = 0; st < steps_per_tile && alive; ++st, ++g) {
                const int l = min(st, a.L - 1), ch = st - l;
                const uint32_t ga = g & (nacc - 1u);
                const int JB = (a.J[l] + 31) >> 5, ks_last = (a.J[l] - (JB - 1) * 32 + 7) >> 3;      // K steps with real channels
                const uint32_t acc = tmem + ga * acc_cols;
                uint32_t started = 0;
                for (int cb0 = 0; cb0 < JB && alive; cb0 += group) {
                    const int nb = min(group, JB - cb0);
                    // start the group's polls together, then wait properly for whatever was not there yet
                    auto poll_group = [&]() {
                        uint32_t ready = 0;
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (j < nb) {
                                uint32_t sj = sw + j, pj = pw;
                                if (sj >= (uint32_t)a.w_stages) { sj -= a.w_stages; pj ^= 1u; }
                                bool ok = mbar_test_wait(bar_w_full + 8 * sj, pj);
                                if (l == 0) {
                                    const int slot = (cb0 + j) & (n_slots - 1);
                                    const uint32_t use = tile_k * slot_uses(slot) + (uint32_t)((cb0 + j) >> ns_log2);
                                    ok = mbar_test_wait((X3 ? bar_split : bar_in) + 8 * slot, use & 1u) && ok;
                                }
                                ready |= (ok ? 1u : 0u) << j;
                            }
                        return ready;
                    };
                    uint32_t ready = poll_group();
                    if (cb0 == 0) {
                        // Only now (the filters' polls are behind us) wait for the epilogue: the accumulator's previous
                        // step has been read out, and a new layer's operand is what the epilogue of the step before wrote
                        // (epilogues finish in order: the second wait covers the first).
                        if (st > 0 && ch == 0)
                            alive = mbar_wait<kSpin>(bar_epi + 8 * ((g - 1u) & (nacc - 1u)), ((g - 1u) >> nacc_log2) & 1u, abort_flag, a.status, a.wait_iters);
                        else if (g >= nacc)
                            alive = mbar_wait<kSpin>(bar_epi + 8 * ga, ((g >> nacc_log2) - 1u) & 1u, abort_flag, a.status, a.wait_iters);
                        if (!alive) break;
                        tc_fence_after();                  // once per step: orders the MMAs after the epilogue's reads of the accumulator
                    }
                    if (l > 0) {
                        uint32_t xb = x_desc0 + (uint32_t)cb0 * x_step;
                        for (int j = 0; j < nb; ++j, xb += x_step) {
                            if (!(ready >> j & 1u)) {
                                alive = mbar_wait<kSpin>(bar_w_full + 8 * sw, pw, abort_flag, a.status, a.wait_iters);
                                if (!alive) break;
                            }
                            issue(acc, xb, cb0 + j == JB - 1 ? ks_last : 4, started);
                            next_stage();
                        }
                    } else {
                        for (int j = 0; j < nb; ++j) {
                            const int cb = cb0 + j, slot = cb & (n_slots - 1);
                            if (!(ready >> j & 1u)) {
                                const uint32_t use = tile_k * slot_uses(slot) + (uint32_t)(cb >> ns_log2);
                                alive = mbar_wait<kSpin>((X3 ? bar_split : bar_in) + 8 * slot, use & 1u, abort_flag, a.status, a.wait_iters);
                                if (alive) alive = mbar_wait<kSpin>(bar_w_full + 8 * sw, pw, abort_flag, a.status, a.wait_iters);
                                if (!alive) break;
                            }
                            issue(acc, x_desc0 + (uint32_t)slot * x_step, cb == JB - 1 ? ks_last : 4, started);
                            // a group of four slots that a later block of this layer reuses: signal when its last block is done
                            if (((cb & 3) == 3 || cb == JB - 1) && (cb & ~3) + n_slots < JB) mma_commit(bar_slot_free + 8 * (slot >> 2));
                            next_stage();
                        }
                    }
                }
                if (alive) mma_commit(bar_acc + 8 * ga);
            }
        }
    } else if (warp >= 4 && warp < 4 + n_epi_warps) {
        // ---- epilogue: thread = filter = tensor-memory lane, 32 images per warp; also splits the first layer's input
        // blocks for 3xTF32
        const int quarter = warp & 3, cg = (warp - 4) >> 2;           // lanes 32 quarter .., columns (images) 32 cg ..
        const int tid_e = threadIdx.x - 128, n_epi = n_epi_warps * 32;
        uint8_t *x_ptr = base_ptr;
        bool alive = true;
        uint32_t g = 0, tile_k = 0;
        grid_dep_sync();                                              // before the first write to global memory
        for (int t = blockIdx.x; t < a.tiles && alive; t += gridDim.x, ++tile_k) {
            if (X3)
                for (int cb = 0; cb < JB0 && alive; ++cb) {
                    const int slot = cb & (n_slots - 1);
                    const uint32_t use = tile_k * slot_uses(slot) + (uint32_t)(cb >> ns_log2);
                    alive = mbar_wait_warp<kSpin>(bar_in + 8 * slot, use & 1u, abort_flag, a.status, a.wait_iters);
                    if (!alive) break;
                    for (int idx = tid_e; idx < nt * 8; idx += n_epi) {               // 16-byte chunks of the block
                        float4 *p = reinterpret_cast<float4 *>(x_ptr + (size_t)slot * slot_pitch + (size_t)idx * 16);
                        const float4 v = *p;
                        const float4 h = make_float4(__uint_as_float(__float_as_uint(v.x) & 0xffffe000u), __uint_as_float(__float_as_uint(v.y) & 0xffffe000u),
                                                     __uint_as_float(__float_as_uint(v.z) & 0xffffe000u), __uint_as_float(__float_as_uint(v.w) & 0xffffe000u));
                        *p = h;
                        *reinterpret_cast<float4 *>(reinterpret_cast<uint8_t *>(p) + slot_bytes) = make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_split + 8 * slot);
                }
            for (int st = 0; st < steps_per_tile && alive; ++st, ++g) {
                const int l = min(st, a.L - 1), ch = st - l;
                const uint32_t ga = g & (nacc - 1u);
                alive = mbar_wait_warp<kSpin>(bar_acc + 8 * ga, (g >> nacc_log2) & 1u, abort_flag, a.status, a.wait_iters);
                if (!alive) break;
                // the step's MMAs have completed: its filter stages, and after a tile's last step the slots, may be refilled
                if (warp == 4 && lane == 0) { __threadfence_block(); *steps_done = g + 1u; }
                tc_fence_after();
                const int K = a.K[l] - ch * 128, KB_all = (a.K[l] + 31) >> 5;       // filters of this step; blocks of the layer
                const bool last = l == a.L - 1;
                if (quarter * 32 < K) {                                               // else: no filter of this step in this warp
                    const int k = quarter * 32 + lane;
                    float v[32];
                    tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + ga * acc_cols + (uint32_t)cg * 32u, v);
                    if (X3) {                                                         // + the x_lo products
                        float u[32];
                        tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + ga * acc_cols + (uint32_t)nt + (uint32_t)cg * 32u, u);
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] += u[e];
                    }
                    const float b = bias_s[st * 128 + k];
                    const bool relu = a.relu[l] != 0, real = k < K;
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        float x = v[e] + b;
                        if (relu) x = fmaxf(x, 0.0f);
                        v[e] = real ? x : 0.0f;                                       // pad lanes stay +0
                    }
                    if (!last) {
                        // image cg*32 + e, channel k: block `quarter`, row = image, 16-byte chunk (lane / 4) ^ (row & 7)
                        uint8_t *blk = x_ptr + (size_t)quarter * slot_pitch + (size_t)(cg * 32) * 128 + (lane & 3) * 4;
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            float *dst = reinterpret_cast<float *>(blk + e * 128 + (((lane >> 2) ^ (e & 7)) << 4));
                            if (X3) {
                                const float h = __uint_as_float(__float_as_uint(v[e]) & 0xffffe000u);
                                *dst = h;
                                *reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(dst) + slot_bytes) = v[e] - h;
                            } else {
                                *dst = v[e];
                            }
                        }
                    } else {
                        const long long n0 = (long long)t * nt + cg * 32;
                        float *dst = a.out + ((size_t)n0 * KB_all + ch * 4 + quarter) * 32 + lane;
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (n0 + e < a.N) dst[(size_t)e * KB_all * 32] = v[e];
                    }
                }
                tc_fence_before();
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_epi + 8 * ga);
            }
        }
    }
    __syncthreads();
    if (*abort_flag && warp == 1 && lane < a.lanes) {     // a role gave up: each producer lane lets its copies still in flight land
        for (int st = 0; st < 16; ++st) {
            if (st < 8 && (armed_mask >> st & 1u))
                for (uint32_t it = 0; it < a.wait_iters && !mbar_try_wait(bar_w_full + 8 * st, armed_parity >> st & 1u); ++it) __nanosleep(200);
            if (in_mask >> st & 1u)
                for (uint32_t it = 0; it < a.wait_iters && !mbar_try_wait(bar_in + 8 * st, in_par >> st & 1u); ++it) __nanosleep(200);
        }
    }
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, (uint32_t)kTmemCols);
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
    // Images per tile: the smallest tile that still gives every SM at most one tile keeps the most SMs busy; beyond that
    // the larger tiles stream the filters fewer times.  A tile whose shared memory does not fit is halved.
    int nt = ctx->fc_chain_tile;
    if (nt == 0) nt = N <= 32 * ctx->sm_count ? 32 : N <= 64 * ctx->sm_count ? 64 : 128;
    const size_t bias_bytes = ((size_t)L - 1 + ceil_div(widths[L], 128)) * 128 * sizeof(float);
    const size_t stage_bytes = (size_t)kWBlock * (x3 ? 2 : 1);
    const bool wide = widths[0] > 128;
    int w_stages = 0, release = 0, lanes = 0, n_slots = 0;
    size_t smem = 0;
    for (;; nt /= 2) {
        if (nt < 32) return SMALL_ERR_UNSUPPORTED;
        const size_t slot_bytes = (size_t)nt * 128 * (x3 ? 2 : 1);
        // Filter stages and how many go back per commit: two layers' worth in halves (TF32), one layer's in halves
        // (3xTF32).  Operand slots: four hold 128 channels; more deepen the stream of a wider first layer, which needs at
        // least eight (slots go back in groups of four while the four producer lanes run four blocks ahead).
        w_stages = x3 ? 4 : 8; release = x3 ? 2 : 4; lanes = 4; n_slots = 4;                 // all powers of two
        while (n_slots < 16 && (size_t)(2 * n_slots) * slot_bytes <= 64 * 1024) n_slots *= 2;
        if (wide && n_slots < 8) n_slots = 8;
        const size_t fixed = 1024 + n_slots * slot_bytes + kCtrl + bias_bytes;
        if (fixed + w_stages * stage_bytes > ctx->max_smem_optin && !wide) { w_stages = 2; release = 1; lanes = 2; }
        smem = fixed + w_stages * stage_bytes;
        if (smem <= ctx->max_smem_optin) break;
    }
    a.L = L; a.N = N; a.tiles = ceil_div(N, nt); a.out = out; a.status = ctx->dev_status; a.wait_iters = ctx->wait_iters;
    a.nt = nt; a.n_slots = n_slots; a.w_stages = w_stages; a.release = release; a.lanes = lanes;
    {   // the first layer's input, blocked [N][JB][32]: one box = nt images x one 32-channel block
        const int JB = blocks_of(widths[0]);
        cuuint64_t dims[3] = {32, (cuuint64_t)JB, (cuuint64_t)N};
        cuuint64_t strides[2] = {128, (cuuint64_t)JB * 128};
        cuuint32_t box[3] = {32, 1, (cuuint32_t)nt};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = encode(&a.map_in, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(in), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { ctx->last_cuda = (int)r; return SMALL_ERR_CUDA; }
    }
    for (int l = 0, loads = 0; l <= L; ++l) {
        a.first_load[l] = loads;
        if (l < L) loads += blocks_of(widths[l]) * (l == L - 1 ? ceil_div(widths[L], 128) : 1);
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
    void (*kern)(const ChainArgs) = x3 ? fc_chain_kernel<true> : fc_chain_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ctx->max_smem_optin);
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    const unsigned grid = (unsigned)(a.tiles < ctx->sm_count ? a.tiles : ctx->sm_count);
    launch_kernel(ctx, kern, dim3(grid), dim3(128 + 4 * nt), smem, st, a);
    return check_launch(ctx);
}

}  // namespace small
