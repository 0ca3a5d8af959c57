// small_run_net_static: the network runner for callers that cannot allocate device memory.
//
// Who that is: a process that handed the whole device to another allocator at start-up (a serving runtime's memory
// pool, a second framework living in the same process), so cudaMalloc has nothing left to give; or a control loop
// with a latency budget, where an allocation - which may synchronise the whole device and take milliseconds - is not
// acceptable on the request path.  Such a caller still owns its input and output tensors, but has nowhere to take the
// network's intermediate buffers from.  Here they live in an array that is part of the library image itself.
//
// Cost: a GPU holds SMALL_STATIC_WORKSPACE_BYTES of device memory for this array from the moment the library's device
// code is loaded on it - at the latest in small_init, which looks the array up - until the process exits, whether or
// not this entry point is ever called.  Creating the context is therefore the step that needs the memory to be
// there; the calls themselves allocate nothing.
#include "common.cuh"

#define SMALL_STATIC_WORKSPACE_BYTES (32u << 20)

// File-scope device array.  In host code this name is only a handle for the runtime's symbol calls, not a device
// address: the address is looked up once per context, with the context's device current, and that pointer is what
// the kernels receive.
static __device__ __align__(256) unsigned char g_static_workspace[SMALL_STATIC_WORKSPACE_BYTES];

namespace small {

// Called by small_init with ctx->device current: loads this module on the device if it is not loaded yet (which is
// when the array's memory is taken) and keeps the array's device address in the context.
int resolve_static_workspace(small_ctx *ctx) {
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_workspace);
    if (e != cudaSuccess || !p) { ctx->last_cuda = (int)e; return SMALL_ERR_CUDA; }
    ctx->static_workspace = p;
    return SMALL_OK;
}

}  // namespace small

SMALL_API size_t small_static_workspace_bytes(void) { return SMALL_STATIC_WORKSPACE_BYTES; }

SMALL_API int small_run_net_static(small_ctx *ctx, const small_layer *layers, int n_layers, int N,
                                   const float *in_blk, float *out_blk, void *stream) {
    if (!ctx) return SMALL_ERR_NOT_INIT;
    if (!layers || n_layers < 1 || N < 1) return SMALL_ERR_INVALID_ARG;
    // the kernels launch on the current device: it must be the one whose copy of the array the context holds
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess || current != ctx->device) return SMALL_ERR_INVALID_ARG;
    const size_t need = small_net_workspace_bytes(layers, n_layers, N);
    if (need > SMALL_STATIC_WORKSPACE_BYTES) return SMALL_ERR_WORKSPACE;   // the network at this batch needs more than the array holds
    if (!ctx->static_workspace) return SMALL_ERR_NOT_INIT;
    // Nothing has to be cleared: every layer writes its whole output tensor (pad lanes included) before any later
    // layer reads it, so what an earlier call - of this or of another network - left in the array is never read.
    return small_run_net(ctx, layers, n_layers, N, in_blk, out_blk, ctx->static_workspace, SMALL_STATIC_WORKSPACE_BYTES, stream);
}
