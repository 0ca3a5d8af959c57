// Networks: a list of layer descriptors run in order over caller-provided slots of one workspace (paper Section 5.3:
// layers share intermediate buffers; Section 4.4: every layer reads and writes the same layout, so nothing is
// reformatted between layers).
#include <vector>

#include "common.cuh"

namespace small {

struct SlotPlan {
    std::vector<size_t> bytes;    // per slot
    std::vector<size_t> offset;   // per slot, 256-byte aligned
    size_t total = 0;
};

static size_t round256(size_t b) { return (b + 255) & ~(size_t)255; }

// Output shape of a layer; false if the descriptor is malformed.
static bool layer_out_shape(const small_layer &L, int N, int &oc, int &oh, int &ow) {
    Geom g;
    switch (L.op) {
        case SMALL_OP_CONV:
            if (make_geom(g, N, L.C, L.K, L.H, L.W, L.FH, L.FW, L.stride, L.pad_t, L.pad_b, L.pad_l, L.pad_r)) return false;
            oc = L.K; oh = g.OH; ow = g.OW; return true;
        case SMALL_OP_DWCONV:
        case SMALL_OP_POOL:
            if (make_geom(g, N, L.C, L.C, L.H, L.W, L.FH, L.FW, L.stride, L.pad_t, L.pad_b, L.pad_l, L.pad_r)) return false;
            oc = L.C; oh = g.OH; ow = g.OW; return true;
        case SMALL_OP_RELU:
        case SMALL_OP_ADD:
            if (L.C < 1 || L.H < 1 || L.W < 1) return false;
            oc = L.C; oh = L.H; ow = L.W; return true;
        case SMALL_OP_FC:
            if (L.C < 1 || L.K < 1 || L.H != 1 || L.W != 1) return false;
            oc = L.K; oh = 1; ow = 1; return true;
        case SMALL_OP_DWPW:
            if (L.K < 1 || make_geom(g, N, L.C, L.C, L.H, L.W, 3, 3, L.stride, L.pad_t, L.pad_b, L.pad_l, L.pad_r)) return false;
            oc = L.K; oh = g.OH; ow = g.OW; return true;
        case SMALL_OP_CONVPOOL:
            if (make_geom(g, N, L.C, L.K, L.H, L.W, L.FH, L.FW, L.stride, L.pad_t, L.pad_b, L.pad_l, L.pad_r)) return false;
            if (g.OH < 2 || g.OW < 2) return false;
            oc = L.K; oh = g.OH / 2; ow = g.OW / 2; return true;
        default: return false;
    }
}

static bool plan_slots(const small_layer *layers, int n_layers, int N, SlotPlan &plan) {
    if (!layers || n_layers < 1 || N < 1) return false;
    auto need = [&](int slot, size_t bytes) {
        if (slot < 0) return slot == SMALL_SLOT_INPUT || slot == SMALL_SLOT_OUTPUT;
        if (slot > 4096) return false;
        if ((size_t)slot >= plan.bytes.size()) plan.bytes.resize(slot + 1, 0);
        if (plan.bytes[slot] < bytes) plan.bytes[slot] = bytes;
        return true;
    };
    for (int i = 0; i < n_layers; ++i) {
        const small_layer &L = layers[i];
        int oc, oh, ow;
        if (!layer_out_shape(L, N, oc, oh, ow)) return false;
        size_t in_b = sizeof(float) * packed_elems(N, L.C, L.H, L.W), out_b = sizeof(float) * packed_elems(N, oc, oh, ow);
        if (!need(L.src, in_b) || !need(L.dst, out_b)) return false;
        if (L.op == SMALL_OP_ADD && !need(L.src2, in_b)) return false;
        if (L.dst == SMALL_SLOT_INPUT) return false;
    }
    plan.offset.resize(plan.bytes.size());
    size_t off = 0;
    for (size_t s = 0; s < plan.bytes.size(); ++s) { plan.offset[s] = off; off += round256(plan.bytes[s]); }
    plan.total = off;
    return true;
}

// ---- abstract fused layers (Section 6) chosen by the runner itself: the caller describes plain layers.
// A layer's result may stay on chip when the next layer is its only reader: nothing after that reads the slot before
// it is written again, and the pair's output slot is not the pair's input slot.
static bool slot_dead_after(const small_layer *layers, int n_layers, int from, int slot) {
    for (int j = from; j < n_layers; ++j) {
        const small_layer &L = layers[j];
        if (L.src == slot || (L.op == SMALL_OP_ADD && L.src2 == slot)) return false;
        if (L.dst == slot) return !((L.flags & SMALL_ACCUMULATE) && L.op == SMALL_OP_CONV);
    }
    return true;
}

// Fusing a depthwise 3x3 with the 1x1 convolution behind it pays where the two separate launches are short (measured:
// a few percent on the depthwise-separable network at batch 64, a loss on large intermediate tensors, where the fused
// kernel's eight depthwise warps per SM cannot keep up with two full-size kernels); above this size of the
// intermediate tensor the pair runs as two layers unless SMALL_FUSE_DWPW_ALWAYS is set.
static const size_t kFuseDwpwMaxBytes = 24u << 20;

// Two layers may run at the same time when neither writes a tensor the other one reads or writes.
static bool independent(const small_layer &A, const small_layer &Bn) {
    auto reads = [](const small_layer &L, int slot) {
        return L.src == slot || (L.op == SMALL_OP_ADD && L.src2 == slot) || ((L.flags & SMALL_ACCUMULATE) && L.op == SMALL_OP_CONV && L.dst == slot);
    };
    if (A.dst == Bn.dst || reads(Bn, A.dst) || reads(A, Bn.dst)) return false;
    return A.dst != SMALL_SLOT_INPUT && Bn.dst != SMALL_SLOT_INPUT;
}

// 0: layer i runs on its own; SMALL_OP_DWPW / SMALL_OP_CONVPOOL / kFusedPoolFc: layers i and i + 1 run as that fused layer
static const int kFusedPoolFc = 1000;      // (no descriptor op of its own: only the runner forms this pair)
static int fused_pair(const small_ctx *ctx, const small_layer *layers, int n_layers, int i, int N) {
    if (i + 1 >= n_layers) return 0;
    const small_layer &A = layers[i], &Bn = layers[i + 1];
    if (A.dst < 0 || Bn.src != A.dst || Bn.dst == A.src || Bn.dst == A.dst) return 0;
    if (!slot_dead_after(layers, n_layers, i + 2, A.dst)) return 0;
    Geom g;
    if (A.op == SMALL_OP_DWCONV && Bn.op == SMALL_OP_CONV && (ctx->net_fusion & (SMALL_FUSE_DWPW | SMALL_FUSE_DWPW_ALWAYS))) {
        const unsigned math = Bn.flags & SMALL_MATH_MASK;
        if (A.FH != 3 || A.FW != 3 || Bn.FH != 1 || Bn.FW != 1 || Bn.stride != 1 || (Bn.pad_t | Bn.pad_b | Bn.pad_l | Bn.pad_r)) return 0;
        if ((Bn.flags & SMALL_ACCUMULATE) || Bn.C != A.C || math == SMALL_MATH_FP32) return 0;
        if (make_geom(g, N, A.C, A.C, A.H, A.W, 3, 3, A.stride, A.pad_t, A.pad_b, A.pad_l, A.pad_r)) return 0;
        if (Bn.H != g.OH || Bn.W != g.OW) return 0;
        if (!(ctx->net_fusion & SMALL_FUSE_DWPW_ALWAYS) && sizeof(float) * packed_elems(N, A.C, g.OH, g.OW) > kFuseDwpwMaxBytes) return 0;
        return small_dwpw_fused(N, A.C, Bn.K, A.H, A.W, A.stride, A.pad_t, A.pad_b, A.pad_l, A.pad_r, math) ? SMALL_OP_DWPW : 0;
    }
    if (A.op == SMALL_OP_CONV && Bn.op == SMALL_OP_POOL && (ctx->net_fusion & SMALL_FUSE_CONVPOOL)) {
        if ((A.flags & SMALL_ACCUMULATE) || Bn.pool_mode != SMALL_POOL_MAX || Bn.FH != 2 || Bn.FW != 2 || Bn.stride != 2 ||
            (Bn.pad_t | Bn.pad_b | Bn.pad_l | Bn.pad_r) || Bn.C != A.K)
            return 0;
        if (make_geom(g, N, A.C, A.K, A.H, A.W, A.FH, A.FW, A.stride, A.pad_t, A.pad_b, A.pad_l, A.pad_r)) return 0;
        if (Bn.H != g.OH || Bn.W != g.OW) return 0;
        return small_conv_maxpool_fused(N, A.C, A.K, A.H, A.W, A.FH, A.FW, A.stride, A.pad_t, A.pad_b, A.pad_l, A.pad_r) ? SMALL_OP_CONVPOOL : 0;
    }
    if (A.op == SMALL_OP_POOL && Bn.op == SMALL_OP_FC && (ctx->net_fusion & SMALL_FUSE_POOLFC)) {
        // a global average pool (window = plane, no padding) and the full reduction over its channels
        if (A.pool_mode != SMALL_POOL_AVG || A.FH != A.H || A.FW != A.W || (A.pad_t | A.pad_b | A.pad_l | A.pad_r) || Bn.C != A.C) return 0;
        return small_gap_fc_fused(N, A.C, Bn.K, Bn.flags & SMALL_MATH_MASK) ? kFusedPoolFc : 0;
    }
    return 0;
}

// Length of the run of full reductions starting at layer i that runs as one fused kernel (0: none): each layer reads what
// the one before it wrote, nothing else reads those intermediates, every width between two layers is at most 128, one
// tensor-core math mode.
static int fc_chain_len(const small_ctx *ctx, const small_layer *layers, int n_layers, int i, int N, int *widths) {
    if (!(ctx->net_fusion & SMALL_FUSE_FC_CHAIN) || layers[i].op != SMALL_OP_FC) return 0;
    const unsigned math = layers[i].flags & SMALL_MATH_MASK;
    if (math != SMALL_MATH_TF32 && math != SMALL_MATH_3XTF32) return 0;
    if (layers[i].C > 8192 || layers[i].K > 128) return 0;       // the first layer's input may be wide, and the last one's output
    int L = 1;
    widths[0] = layers[i].C; widths[1] = layers[i].K;
    while (i + L < n_layers && L < 12) {
        const small_layer &P = layers[i + L - 1], &Q = layers[i + L];
        if (Q.op != SMALL_OP_FC || Q.src != P.dst || P.dst < 0 || (Q.flags & SMALL_MATH_MASK) != math || Q.C != P.K || Q.K > 1024 || P.K > 128) break;
        if (!slot_dead_after(layers, n_layers, i + L + 1, P.dst)) break;
        if (Q.dst == layers[i].src) break;                      // the run's output must not land on its input
        widths[L + 1] = Q.K;
        ++L;
    }
    (void)N;
    return L >= 2 ? L : 0;
}

}  // namespace small

using namespace small;

SMALL_API int small_set_net_fusion(small_ctx *ctx, unsigned mask) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (mask & ~(unsigned)(SMALL_FUSE_DWPW | SMALL_FUSE_DWPW_ALWAYS | SMALL_FUSE_CONVPOOL | SMALL_FUSE_FC_CHAIN | SMALL_FUSE_POOLFC)) return SMALL_ERR_INVALID_ARG;
    ctx->net_fusion = mask;
    return SMALL_OK;
}

SMALL_API int small_net_launches(small_ctx *ctx, const small_layer *layers, int n_layers, int N) {
    if (!ctx || !layers || n_layers < 1 || N < 1) return -1;
    int launches = 0;
    for (int i = 0; i < n_layers; ++i, ++launches) {
        int widths[13];
        if (const int L = fc_chain_len(ctx, layers, n_layers, i, N, widths)) i += L - 1;
        else if (fused_pair(ctx, layers, n_layers, i, N)) ++i;
    }
    return launches;
}

SMALL_API size_t small_net_workspace_bytes(const small_layer *layers, int n_layers, int N) {
    SlotPlan plan;
    if (!plan_slots(layers, n_layers, N, plan)) return 0;
    return plan.total;
}

static int run_layers(small_ctx *ctx, const small_layer *layers, int n_layers, int from, int N,
                      const float *in_blk, float *out_blk, void *workspace, size_t workspace_bytes, void *stream);

SMALL_API int small_run_net(small_ctx *ctx, const small_layer *layers, int n_layers, int N,
                            const float *in_blk, float *out_blk, void *workspace, size_t workspace_bytes, void *stream) {
    return run_layers(ctx, layers, n_layers, 0, N, in_blk, out_blk, workspace, workspace_bytes, stream);
}

// Validates the whole list, then runs layers from .. n_layers - 1.
static int run_layers(small_ctx *ctx, const small_layer *layers, int n_layers, int from, int N,
                      const float *in_blk, float *out_blk, void *workspace, size_t workspace_bytes, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!layers || !in_blk || !out_blk) return SMALL_ERR_INVALID_ARG;
    if (!aligned16(in_blk) || !aligned16(out_blk) || (workspace && ((uintptr_t)workspace & 255u))) return SMALL_ERR_ALIGN;
    SlotPlan plan;
    if (!plan_slots(layers, n_layers, N, plan)) return SMALL_ERR_SHAPE;
    if (plan.total > workspace_bytes || (plan.total && !workspace)) return SMALL_ERR_WORKSPACE;
    char *base = static_cast<char *>(workspace);
    auto rd = [&](int slot) -> const float * {
        if (slot == SMALL_SLOT_INPUT) return in_blk;
        if (slot == SMALL_SLOT_OUTPUT) return out_blk;
        return reinterpret_cast<const float *>(base + plan.offset[slot]);
    };
    auto wr = [&](int slot) -> float * {
        if (slot == SMALL_SLOT_OUTPUT) return out_blk;
        return reinterpret_cast<float *>(base + plan.offset[slot]);
    };
    // validate every layer before the first launch: weights present where needed, flags known
    for (int i = 0; i < n_layers; ++i) {
        const small_layer &L = layers[i];
        bool weighted = L.op == SMALL_OP_CONV || L.op == SMALL_OP_DWCONV || L.op == SMALL_OP_FC || L.op == SMALL_OP_DWPW || L.op == SMALL_OP_CONVPOOL;
        if (L.op == SMALL_OP_CONVPOOL &&
            !small_conv_maxpool_fused(N, L.C, L.K, L.H, L.W, L.FH, L.FW, L.stride, L.pad_t, L.pad_b, L.pad_l, L.pad_r))
            return SMALL_ERR_UNSUPPORTED;         // a network has no scratch tensor for the unfused form
        if (L.op == SMALL_OP_DWPW) {
            if (!L.w_blk2 || !aligned16(L.w_blk2) || (L.bias2 && !aligned16(L.bias2))) return SMALL_ERR_INVALID_ARG;
            if (!small_dwpw_fused(N, L.C, L.K, L.H, L.W, L.stride, L.pad_t, L.pad_b, L.pad_l, L.pad_r, L.flags & SMALL_MATH_MASK))
                return SMALL_ERR_UNSUPPORTED;     // a network has no scratch tensor for the unfused form
        }
        if (weighted && !L.w_blk) return SMALL_ERR_INVALID_ARG;
        if (weighted && (!aligned16(L.w_blk) || (L.bias && !aligned16(L.bias)))) return SMALL_ERR_ALIGN;
        unsigned allowed = L.op == SMALL_OP_CONV ? (SMALL_RELU | SMALL_ACCUMULATE | SMALL_MATH_MASK)
                         : (L.op == SMALL_OP_DWCONV || L.op == SMALL_OP_FC) ? (SMALL_RELU | SMALL_MATH_MASK)
                         : L.op == SMALL_OP_DWPW ? (SMALL_RELU | SMALL_RELU_MID | SMALL_MATH_MASK)
                         : L.op == SMALL_OP_CONVPOOL ? (SMALL_RELU | SMALL_MATH_MASK)
                         : L.op == SMALL_OP_ADD ? SMALL_RELU : 0u;
        if (L.flags & ~allowed) return SMALL_ERR_INVALID_ARG;
        if ((L.flags & SMALL_MATH_MASK) == SMALL_MATH_MASK) return SMALL_ERR_INVALID_ARG;
        if (L.op == SMALL_OP_POOL && L.pool_mode != SMALL_POOL_MAX && L.pool_mode != SMALL_POOL_AVG) return SMALL_ERR_INVALID_ARG;
        if (L.src == L.dst && L.op != SMALL_OP_RELU && L.op != SMALL_OP_ADD) return SMALL_ERR_OVERLAP;
    }
    auto run_one = [&](const small_layer &L, void *strm) -> int {
        switch (L.op) {
            case SMALL_OP_CONV:
                return small_conv2d(ctx, rd(L.src), L.w_blk, L.bias, wr(L.dst), N, L.C, L.K, L.H, L.W, L.FH, L.FW, L.stride,
                                 L.pad_t, L.pad_b, L.pad_l, L.pad_r, L.flags, strm);
            case SMALL_OP_DWCONV:
                return small_dwconv2d(ctx, rd(L.src), L.w_blk, L.bias, wr(L.dst), N, L.C, L.H, L.W, L.FH, L.FW, L.stride,
                                   L.pad_t, L.pad_b, L.pad_l, L.pad_r, L.flags, strm);
            case SMALL_OP_POOL:
                return small_pool2d(ctx, rd(L.src), wr(L.dst), nullptr, N, L.C, L.H, L.W, L.FH, L.FW, L.stride,
                                 L.pad_t, L.pad_b, L.pad_l, L.pad_r, L.pool_mode, strm);
            case SMALL_OP_RELU:
                return small_relu(ctx, rd(L.src), wr(L.dst), N, L.C, L.H, L.W, strm);
            case SMALL_OP_ADD:
                return small_add(ctx, rd(L.src), rd(L.src2), wr(L.dst), N, L.C, L.H, L.W, L.flags, strm);
            case SMALL_OP_FC:
                return small_fc(ctx, rd(L.src), L.w_blk, L.bias, wr(L.dst), N, L.C, L.K, L.flags, strm);
            case SMALL_OP_CONVPOOL:
                return small_conv_maxpool2d(ctx, rd(L.src), L.w_blk, L.bias, wr(L.dst), nullptr, N, L.C, L.K, L.H, L.W, L.FH, L.FW, L.stride,
                                         L.pad_t, L.pad_b, L.pad_l, L.pad_r, L.flags, strm);
            case SMALL_OP_DWPW:
                return small_dwpw_conv2d(ctx, rd(L.src), L.w_blk, L.bias, L.w_blk2, L.bias2, wr(L.dst), nullptr, N, L.C, L.K, L.H, L.W,
                                      L.stride, L.pad_t, L.pad_b, L.pad_l, L.pad_r, L.flags, strm);
        }
        return SMALL_ERR_INVALID_ARG;
    };
    bool after_join = false;
    for (int i = from; i < n_layers; ++i) {
        const small_layer &L = layers[i];
        int s = SMALL_OK;
        // every layer behind the first may start its set-up while the layer in front of it drains (see launch_kernel)
        ctx->dependent = ctx->overlap && i > 0 && !after_join;
        after_join = false;
        {
            int widths[13];
            if (const int Lc = fc_chain_len(ctx, layers, n_layers, i, N, widths)) {
                const float *w[12], *b[12];
                int relu[12];
                for (int j = 0; j < Lc; ++j) { w[j] = layers[i + j].w_blk; b[j] = layers[i + j].bias; relu[j] = (layers[i + j].flags & SMALL_RELU) ? 1 : 0; }
                float *dst = wr(layers[i + Lc - 1].dst);
                if ((reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
                    s = launch_fc_chain(ctx, rd(L.src), w, b, widths, relu, dst, Lc, N, L.flags & SMALL_MATH_MASK, static_cast<cudaStream_t>(stream));
                    ctx->dependent = 0;
                    if (s != SMALL_OK) return s;
                    i += Lc - 1;
                    continue;
                }
            }
        }
        if (const int fused = fused_pair(ctx, layers, n_layers, i, N)) {
            const small_layer &Nx = layers[i + 1];
            if (fused == SMALL_OP_DWPW) {
                const unsigned fl = ((L.flags & SMALL_RELU) ? SMALL_RELU_MID : 0u) | (Nx.flags & (SMALL_RELU | SMALL_MATH_MASK));
                s = small_dwpw_conv2d(ctx, rd(L.src), L.w_blk, L.bias, Nx.w_blk, Nx.bias, wr(Nx.dst), nullptr, N, L.C, Nx.K, L.H, L.W,
                                      L.stride, L.pad_t, L.pad_b, L.pad_l, L.pad_r, fl, stream);
            } else if (fused == kFusedPoolFc) {
                s = small_gap_fc(ctx, rd(L.src), Nx.w_blk, Nx.bias, wr(Nx.dst), nullptr, N, L.C, L.H, L.W, Nx.K,
                                 Nx.flags & (SMALL_RELU | SMALL_MATH_MASK), stream);
            } else {
                s = small_conv_maxpool2d(ctx, rd(L.src), L.w_blk, L.bias, wr(Nx.dst), nullptr, N, L.C, L.K, L.H, L.W, L.FH, L.FW, L.stride,
                                         L.pad_t, L.pad_b, L.pad_l, L.pad_r, L.flags, stream);
            }
            ctx->dependent = 0;
            if (s != SMALL_OK) return s;
            ++i;
            continue;
        }
        // Two neighbouring layers that touch no common tensor except as readers (a residual stage's convolution and its
        // shortcut) run side by side: the second one on the context's side stream, forked from and joined to the caller's
        // stream by events, so that a short layer hides behind a long one.  Both are ordinary launches, and so is the
        // layer behind the join.
        if (ctx->branch_overlap && ctx->side_stream && i + 1 < n_layers && independent(L, layers[i + 1]) &&
            !fused_pair(ctx, layers, n_layers, i + 1, N)) {
            cudaStream_t main_st = static_cast<cudaStream_t>(stream), side = static_cast<cudaStream_t>(ctx->side_stream);
            cudaError_t e = cudaEventRecord(static_cast<cudaEvent_t>(ctx->ev_fork), main_st);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(side, static_cast<cudaEvent_t>(ctx->ev_fork), 0);
            if (e != cudaSuccess) { ctx->last_cuda = (int)e; ctx->dependent = 0; return SMALL_ERR_CUDA; }
            s = run_one(L, stream);
            ctx->dependent = 0;
            if (s == SMALL_OK) s = run_one(layers[i + 1], ctx->side_stream);
            e = cudaEventRecord(static_cast<cudaEvent_t>(ctx->ev_join), side);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(main_st, static_cast<cudaEvent_t>(ctx->ev_join), 0);
            if (s != SMALL_OK) return s;
            if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
            ++i;
            after_join = true;
            continue;
        }
        s = run_one(L, stream);
        ctx->dependent = 0;
        if (s != SMALL_OK) return s;
    }
    return SMALL_OK;
}

SMALL_API size_t small_net_host_staging_bytes(int N, int C, int H, int W, int outC, int outH, int outW) {
    if (N < 1 || C < 1 || H < 1 || W < 1 || outC < 1 || outH < 1 || outW < 1) return 0;
    return 2 * round256(sizeof(float) * (size_t)N * C * H * W) + round256(sizeof(float) * packed_elems(N, C, H, W)) +
           round256(sizeof(float) * packed_elems(N, outC, outH, outW)) + round256(sizeof(float) * (size_t)N * outC * outH * outW);
}

// The host-buffer call keeps the copy engine busy next to the SMs: the NCHW input goes to one of two staging areas on
// the context's copy stream, so the copy of call i + 1 runs while the layers of call i are still computing on the caller's
// stream; the caller's stream waits for its own input by an event, and a staging area is not overwritten before the
// pack that read it last has finished.  Everything else (pack, layers, unpack, the result's copy back) stays in order on
// the caller's stream.  While the caller's stream is being captured, the input copy stays on that stream.
SMALL_API int small_run_net_host(small_ctx *ctx, const small_layer *layers, int n_layers, int N,
                                 const float *in_host, int C, int H, int W,
                                 float *out_host, int outC, int outH, int outW,
                                 void *workspace, size_t workspace_bytes, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!layers || !in_host || !out_host || !workspace) return SMALL_ERR_INVALID_ARG;
    if ((uintptr_t)workspace & 255u) return SMALL_ERR_ALIGN;
    {   // the layer list must be well formed even when it needs no slot
        SlotPlan plan;
        if (!plan_slots(layers, n_layers, N, plan)) return SMALL_ERR_SHAPE;
    }
    size_t net_b = small_net_workspace_bytes(layers, n_layers, N);
    size_t stage_b = small_net_host_staging_bytes(N, C, H, W, outC, outH, outW);
    if (stage_b == 0) return SMALL_ERR_SHAPE;
    if (net_b + stage_b > workspace_bytes) return SMALL_ERR_WORKSPACE;
    // the last layer must produce the declared output shape
    int oc, oh, ow;
    if (!layer_out_shape(layers[n_layers - 1], N, oc, oh, ow) || oc != outC || oh != outH || ow != outW) return SMALL_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *p = static_cast<char *>(workspace) + net_b;
    size_t in_nchw_b = sizeof(float) * (size_t)N * C * H * W, out_nchw_b = sizeof(float) * (size_t)N * outC * outH * outW;
    float *d_in_nchw[2];
    d_in_nchw[0] = reinterpret_cast<float *>(p); p += round256(in_nchw_b);
    d_in_nchw[1] = reinterpret_cast<float *>(p); p += round256(in_nchw_b);
    float *d_in_blk = reinterpret_cast<float *>(p); p += round256(sizeof(float) * packed_elems(N, C, H, W));
    float *d_out_blk = reinterpret_cast<float *>(p); p += round256(sizeof(float) * packed_elems(N, outC, outH, outW));
    float *d_out_nchw = reinterpret_cast<float *>(p);
    cudaError_t e = cudaSuccess;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    cudaStreamIsCapturing(st, &cap);
    const bool piped = ctx->copy_stream && cap == cudaStreamCaptureStatusNone;
    int par = 0;
    if (piped) {
        if (ctx->host_ws != workspace) { ctx->host_ws = workspace; ctx->host_parity = 0; ctx->host_used[0] = ctx->host_used[1] = 0; }
        par = ctx->host_parity;
        cudaStream_t cs = static_cast<cudaStream_t>(ctx->copy_stream);
        if (ctx->host_used[par]) e = cudaStreamWaitEvent(cs, static_cast<cudaEvent_t>(ctx->ev_pack[par]), 0);
        if (e == cudaSuccess) e = cudaMemcpyAsync(d_in_nchw[par], in_host, in_nchw_b, cudaMemcpyHostToDevice, cs);
        if (e == cudaSuccess) e = cudaEventRecord(static_cast<cudaEvent_t>(ctx->ev_h2d[par]), cs);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, static_cast<cudaEvent_t>(ctx->ev_h2d[par]), 0);
    } else {
        e = cudaMemcpyAsync(d_in_nchw[0], in_host, in_nchw_b, cudaMemcpyHostToDevice, st);
    }
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    // A first layer with at most four input channels (an image, a spectrogram) reads the NCHW tensor itself: its kernel
    // gathers the real channels into shared memory either way, so the blocked copy of the input - 32 lanes for one to four
    // channels - is never made.  The values and their order of summation are those of the blocked path.
    int first = 0;
    {
        const small_layer &L0 = layers[0];
        Geom g0;
        bool later_reads_input = false;
        for (int i = 1; i < n_layers; ++i)
            if (layers[i].src == SMALL_SLOT_INPUT || (layers[i].op == SMALL_OP_ADD && layers[i].src2 == SMALL_SLOT_INPUT)) later_reads_input = true;
        if (L0.op == SMALL_OP_CONV && L0.src == SMALL_SLOT_INPUT && L0.dst >= 0 && !(L0.flags & SMALL_ACCUMULATE) && !later_reads_input &&
            n_layers > 1 && L0.C == C && L0.H == H && L0.W == W && L0.w_blk && aligned16(L0.w_blk) && (!L0.bias || aligned16(L0.bias)) &&
            !(L0.flags & ~(SMALL_RELU | SMALL_MATH_MASK)) && !fused_pair(ctx, layers, n_layers, 0, N) &&
            make_geom(g0, N, L0.C, L0.K, L0.H, L0.W, L0.FH, L0.FW, L0.stride, L0.pad_t, L0.pad_b, L0.pad_l, L0.pad_r) == SMALL_OK &&
            conv_thin_supported(g0)) {
            SlotPlan plan;
            plan_slots(layers, n_layers, N, plan);
            float *dst0 = reinterpret_cast<float *>(static_cast<char *>(workspace) + plan.offset[L0.dst]);
            if (int s = launch_conv_thin(ctx, d_in_nchw[par], L0.w_blk, L0.bias, dst0, g0, L0.flags & SMALL_RELU, false, st, true)) return s;
            first = 1;
        }
    }
    if (!first)
        if (int s = small_pack(ctx, d_in_nchw[par], d_in_blk, N, C, H, W, stream)) return s;
    if (piped) {
        e = cudaEventRecord(static_cast<cudaEvent_t>(ctx->ev_pack[par]), st);
        if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
        ctx->host_used[par] = 1;
        ctx->host_parity = par ^ 1;
    }
    if (first) {
        // the rest of the list over the same slots: its plan must be the whole list's (slot sizes come from all layers)
        if (int s = run_layers(ctx, layers, n_layers, 1, N, d_in_blk, d_out_blk, workspace, net_b, stream)) return s;
    } else if (int s = small_run_net(ctx, layers, n_layers, N, d_in_blk, d_out_blk, workspace, net_b, stream)) return s;
    if (int s = small_unpack(ctx, d_out_blk, d_out_nchw, N, outC, outH, outW, stream)) return s;
    e = cudaMemcpyAsync(out_host, d_out_nchw, out_nchw_b, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    return SMALL_OK;
}
