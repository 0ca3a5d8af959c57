// small_run_net_static: the network runner for callers that cannot allocate device memory.
//
// Who that is: a process that handed the whole device to another allocator at start-up (a serving runtime's memory
// pool, a second framework living in the same process), so cudaMalloc has nothing left to give; or a control loop
// with a latency budget, where an allocation - which may synchronise the whole device and take milliseconds - is not
// acceptable on the request path.  Such a caller still owns its input and output tensors, but has nowhere to take the
// network's intermediate buffers from.  Here they live in an array that is part of the library image itself.
//
// Cost: every GPU that loads this library holds SMALL_STATIC_WORKSPACE_BYTES of device memory until the process
// exits, whether or not this entry point is ever called.
#include "common.cuh"

#define SMALL_STATIC_WORKSPACE_BYTES (32u << 20)
#define SMALL_STATIC_MAX_DEVICES 64

// File-scope device array.  In host code this name is only a handle for the runtime's symbol calls, not a device
// address: the address is looked up once per device below and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_workspace[SMALL_STATIC_WORKSPACE_BYTES];

static void *g_static_ptr[SMALL_STATIC_MAX_DEVICES];   // per device: address of g_static_workspace, 0 = not looked up yet

// Looks up the array's address on ctx's device (first call on that device only), with that device current.
static int static_workspace_ptr(small_ctx *ctx, void **out) {
    if (ctx->device < 0 || ctx->device >= SMALL_STATIC_MAX_DEVICES) return SMALL_ERR_UNSUPPORTED;
    if (!g_static_ptr[ctx->device]) {
        int current = -1;
        cudaError_t e = cudaGetDevice(&current);
        if (e == cudaSuccess && current != ctx->device) e = cudaSetDevice(ctx->device);
        void *p = nullptr;
        if (e == cudaSuccess) e = cudaGetSymbolAddress(&p, g_static_workspace);
        if (current >= 0 && current != ctx->device) cudaSetDevice(current);
        if (e != cudaSuccess || !p) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
        g_static_ptr[ctx->device] = p;
    }
    *out = g_static_ptr[ctx->device];
    return SMALL_OK;
}

SMALL_API size_t small_static_workspace_bytes(void) { return SMALL_STATIC_WORKSPACE_BYTES; }

SMALL_API int small_run_net_static(small_ctx *ctx, const small_layer *layers, int n_layers, int N,
                                   const float *in_blk, float *out_blk, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!layers || n_layers < 1 || N < 1) return SMALL_ERR_INVALID_ARG;
    const size_t need = small_net_workspace_bytes(layers, n_layers, N);
    if (need > SMALL_STATIC_WORKSPACE_BYTES) return SMALL_ERR_WORKSPACE;   // the network at this batch needs more than the array holds
    void *ws = nullptr;
    if (int s = static_workspace_ptr(ctx, &ws)) return s;
    // Nothing has to be cleared: every layer writes its whole output tensor (pad lanes included) before any later
    // layer reads it, so what an earlier call left in the array is never read.
    return small_run_net(ctx, layers, n_layers, N, in_blk, out_blk, ws, SMALL_STATIC_WORKSPACE_BYTES, stream);
}
