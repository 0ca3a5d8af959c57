"""ctypes binding of libsmall.so: the functions of include/small.h under the same names.

Argument marshalling only.  Tensors are torch CUDA tensors used as device memory (their data_ptr() is what
crosses the boundary); `stream` defaults to torch's current stream.  A non-zero status raises SmallError.
There is no fallback: if the library is missing or a call fails, the caller gets an exception.
"""
from __future__ import annotations

import ctypes
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsmall.so")

# mirrors of the header's enums
OK = 0
RELU, ACCUMULATE, RELU_MID = 1, 2, 4
MATH_FP32, MATH_TF32, MATH_3XTF32 = 0 << 4, 1 << 4, 2 << 4
POOL_MAX, POOL_AVG = 0, 1
OP_CONV, OP_DWCONV, OP_POOL, OP_RELU, OP_ADD, OP_FC, OP_DWPW, OP_CONVPOOL = range(8)
SLOT_INPUT, SLOT_OUTPUT = -1, -2
MATH = {"fp32": MATH_FP32, "tf32": MATH_TF32, "3xtf32": MATH_3XTF32}

EXPORTS = [
    "small_init", "small_shutdown", "small_channel_block", "small_packed_elems", "small_out_size", "small_strerror",
    "small_last_cuda_error", "small_set_layer_overlap", "small_set_conv_path", "small_set_branch_overlap", "small_conv2d_path", "small_set_wait_limit", "small_set_fc_chain_tile", "small_selftest_wait_timeout", "small_device_status", "small_measure_tf32_peak", "small_pack", "small_unpack", "small_conv_weight_elems",
    "small_pack_conv_weights", "small_group_count", "small_group_conv_weight_elems", "small_pack_group_conv_weights",
    "small_group_conv2d", "small_dwpw_conv2d", "small_dwpw_fused", "small_conv_maxpool2d", "small_conv_maxpool_fused", "small_dw_weight_elems", "small_pack_dw_weights", "small_fc_weight_elems",
    "small_pack_fc_weights", "small_fc_uses_tensor_cores", "small_fc_chain", "small_fc_chain_fused", "small_conv2d", "small_conv2d_uses_tensor_cores", "small_dwconv2d", "small_pool2d",
    "small_relu", "small_scale_shift", "small_upsample_nearest", "small_add", "small_fc", "small_gap_fc", "small_gap_fc_fused", "small_net_workspace_bytes", "small_run_net", "small_set_net_fusion", "small_net_launches",
    "small_net_host_staging_bytes", "small_run_net_host", "small_static_workspace_bytes", "small_run_net_static",
    "small_q_packed_bytes", "small_q_pack", "small_q_unpack", "small_q_conv_weight_bytes", "small_q_pack_conv_weights", "small_q_conv2d",
    "small_q_dw_weight_bytes", "small_q_pack_dw_weights", "small_q_dwconv2d", "small_q_maxpool2d", "small_q_relu",
]


class SmallError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: status {status} ({lib().small_strerror(status).decode()})")


class small_layer(ctypes.Structure):
    _fields_ = [("op", ctypes.c_int), ("C", ctypes.c_int), ("K", ctypes.c_int), ("H", ctypes.c_int), ("W", ctypes.c_int),
                ("FH", ctypes.c_int), ("FW", ctypes.c_int), ("stride", ctypes.c_int),
                ("pad_t", ctypes.c_int), ("pad_b", ctypes.c_int), ("pad_l", ctypes.c_int), ("pad_r", ctypes.c_int),
                ("flags", ctypes.c_uint), ("pool_mode", ctypes.c_int),
                ("w_blk", ctypes.c_void_p), ("bias", ctypes.c_void_p),
                ("src", ctypes.c_int), ("dst", ctypes.c_int), ("src2", ctypes.c_int),
                ("w_blk2", ctypes.c_void_p), ("bias2", ctypes.c_void_p)]


_lib = None


def lib():
    """Loads libsmall.so (built by paper_2303_04769_b200.build) and declares the prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2303_04769_b200.build` (there is no fallback path)")
    L = ctypes.CDLL(LIB_PATH)
    I, U, P, Z = ctypes.c_int, ctypes.c_uint, ctypes.c_void_p, ctypes.c_size_t
    L.small_init.argtypes = [I, ctypes.POINTER(P)]
    L.small_shutdown.argtypes = [P]
    L.small_channel_block.argtypes = []
    L.small_packed_elems.argtypes = [I] * 4
    L.small_packed_elems.restype = Z
    L.small_out_size.argtypes = [I] * 5
    L.small_strerror.argtypes = [I]
    L.small_strerror.restype = ctypes.c_char_p
    L.small_last_cuda_error.argtypes = [P]
    L.small_set_layer_overlap.argtypes = [P, I]
    L.small_device_status.argtypes = [P, ctypes.POINTER(I), P]
    L.small_set_conv_path.argtypes = [P, I]
    L.small_set_branch_overlap.argtypes = [P, I]
    L.small_set_wait_limit.argtypes = [P, U]
    L.small_set_fc_chain_tile.argtypes = [P, I]
    L.small_selftest_wait_timeout.argtypes = [P, P]
    L.small_conv2d_path.argtypes = [P] + [I] * 12 + [U]
    L.small_pack.argtypes = [P, P, P, I, I, I, I, P]
    L.small_unpack.argtypes = [P, P, P, I, I, I, I, P]
    L.small_conv_weight_elems.argtypes = [I, I, I, I, U]
    L.small_conv_weight_elems.restype = Z
    L.small_pack_conv_weights.argtypes = [P, P, P, I, I, I, I, U, P]
    L.small_group_count.argtypes = [I, I, I]
    L.small_group_conv_weight_elems.argtypes = [I] * 6
    L.small_group_conv_weight_elems.restype = Z
    L.small_pack_group_conv_weights.argtypes = [P, P, P] + [I] * 6 + [P]
    L.small_group_conv2d.argtypes = [P, P, P, P, P] + [I] * 14 + [U, P]
    L.small_dwpw_conv2d.argtypes = [P] * 8 + [I] * 10 + [U, P]
    L.small_dwpw_fused.argtypes = [I] * 10 + [U]
    L.small_conv_maxpool2d.argtypes = [P] * 6 + [I] * 12 + [U, P]
    L.small_conv_maxpool_fused.argtypes = [I] * 12
    L.small_dw_weight_elems.argtypes = [I, I, I]
    L.small_dw_weight_elems.restype = Z
    L.small_pack_dw_weights.argtypes = [P, P, P, I, I, I, P]
    L.small_fc_weight_elems.argtypes = [I, I, U]
    L.small_fc_weight_elems.restype = Z
    L.small_pack_fc_weights.argtypes = [P, P, P, I, I, U, P]
    L.small_fc_uses_tensor_cores.argtypes = [I, I, I, U]
    L.small_fc_chain.argtypes = [P, P, ctypes.POINTER(P), ctypes.POINTER(P), ctypes.POINTER(I), ctypes.POINTER(I), P, P, I, I, U, P]
    L.small_fc_chain_fused.argtypes = [ctypes.POINTER(I), I, U]
    L.small_conv2d.argtypes = [P, P, P, P, P] + [I] * 12 + [U, P]
    L.small_conv2d_uses_tensor_cores.argtypes = [I] * 12
    L.small_dwconv2d.argtypes = [P, P, P, P, P] + [I] * 11 + [U, P]
    L.small_pool2d.argtypes = [P, P, P, P] + [I] * 11 + [I, P]
    L.small_relu.argtypes = [P, P, P, I, I, I, I, P]
    L.small_add.argtypes = [P, P, P, P, I, I, I, I, U, P]
    L.small_scale_shift.argtypes = [P, P, P, P, P, I, I, I, I, U, P]
    L.small_upsample_nearest.argtypes = [P, P, P, I, I, I, I, I, P]
    L.small_fc.argtypes = [P, P, P, P, P, I, I, I, U, P]
    L.small_gap_fc.argtypes = [P, P, P, P, P, P, I, I, I, I, I, U, P]
    L.small_gap_fc_fused.argtypes = [I, I, I, U]
    L.small_net_workspace_bytes.argtypes = [ctypes.POINTER(small_layer), I, I]
    L.small_net_workspace_bytes.restype = Z
    L.small_run_net.argtypes = [P, ctypes.POINTER(small_layer), I, I, P, P, P, Z, P]
    L.small_set_net_fusion.argtypes = [P, U]
    L.small_net_launches.argtypes = [P, ctypes.POINTER(small_layer), I, I]
    L.small_net_host_staging_bytes.argtypes = [I] * 7
    L.small_net_host_staging_bytes.restype = Z
    L.small_run_net_host.argtypes = [P, ctypes.POINTER(small_layer), I, I, P, I, I, I, P, I, I, I, P, Z, P]
    L.small_measure_tf32_peak.argtypes = [P, I, I, P, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), P]
    L.small_static_workspace_bytes.argtypes = []
    L.small_static_workspace_bytes.restype = Z
    L.small_run_net_static.argtypes = [P, ctypes.POINTER(small_layer), I, I, P, P, P]
    L.small_q_packed_bytes.argtypes = [I] * 4
    L.small_q_packed_bytes.restype = Z
    L.small_q_pack.argtypes = [P, P, P, I, I, I, I, P]
    L.small_q_unpack.argtypes = [P, P, P, I, I, I, I, P]
    L.small_q_conv_weight_bytes.argtypes = [I] * 4
    L.small_q_conv_weight_bytes.restype = Z
    L.small_q_pack_conv_weights.argtypes = [P, P, P, I, I, I, I, P]
    L.small_q_conv2d.argtypes = [P, P, P, P, P] + [I] * 17 + [U, P]
    L.small_q_dw_weight_bytes.argtypes = [I] * 3
    L.small_q_dw_weight_bytes.restype = Z
    L.small_q_pack_dw_weights.argtypes = [P, P, P, I, I, I, P]
    L.small_q_dwconv2d.argtypes = [P, P, P, P, P] + [I] * 16 + [U, P]
    L.small_q_maxpool2d.argtypes = [P, P, P] + [I] * 12 + [P]
    L.small_q_relu.argtypes = [P, P, P, I, I, I, I, I, P]
    _lib = L
    return L


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(status, where):
    if status != OK:
        raise SmallError(status, where)


# ---- the header's functions, same names ----------------------------------------------------------

def small_init(device=0):
    ctx = ctypes.c_void_p()
    _check(lib().small_init(device, ctypes.byref(ctx)), "small_init")
    return ctx


def small_shutdown(ctx):
    _check(lib().small_shutdown(ctx), "small_shutdown")


def small_channel_block():
    return lib().small_channel_block()


def small_packed_elems(N, C, H, W):
    return lib().small_packed_elems(N, C, H, W)


def small_out_size(I, F, stride, pad_before=0, pad_after=0):
    return lib().small_out_size(I, F, stride, pad_before, pad_after)


def small_set_layer_overlap(ctx, on):
    _check(lib().small_set_layer_overlap(ctx, 1 if on else 0), "small_set_layer_overlap")


CONV_PATH = {"auto": 0, "tensor": 1, "cuda_cores": 2, "general": 3, "warp_mma": 4}
CONV_KERNEL = {0: "conv_thin", 1: "conv_direct", 2: "conv_fp32", 3: "conv_tc", 4: "conv_mma"}


def small_set_conv_path(ctx, path):
    _check(lib().small_set_conv_path(ctx, CONV_PATH[path] if isinstance(path, str) else path), "small_set_conv_path")


def small_set_branch_overlap(ctx, on):
    _check(lib().small_set_branch_overlap(ctx, 1 if on else 0), "small_set_branch_overlap")


def small_set_fc_chain_tile(ctx, images):
    _check(lib().small_set_fc_chain_tile(ctx, images), "small_set_fc_chain_tile")


def small_set_wait_limit(ctx, polls):
    _check(lib().small_set_wait_limit(ctx, polls), "small_set_wait_limit")


def small_selftest_wait_timeout(ctx, stream=None):
    _check(lib().small_selftest_wait_timeout(ctx, _stream(stream)), "small_selftest_wait_timeout")


def small_conv2d_path(ctx, N, C, K, H, W, FH, FW, stride, pad, math):
    pt, pb, pl, pr = pad
    return int(lib().small_conv2d_path(ctx, N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr, math))


def small_device_status(ctx, stream=None):
    st = ctypes.c_int(0)
    _check(lib().small_device_status(ctx, ctypes.byref(st), _stream(stream)), "small_device_status")
    return st.value


def small_pack(ctx, nchw, blk, N, C, H, W, stream=None):
    _check(lib().small_pack(ctx, _ptr(nchw), _ptr(blk), N, C, H, W, _stream(stream)), "small_pack")


def small_unpack(ctx, blk, nchw, N, C, H, W, stream=None):
    _check(lib().small_unpack(ctx, _ptr(blk), _ptr(nchw), N, C, H, W, _stream(stream)), "small_unpack")


def small_conv_weight_elems(C, K, FH, FW, math=MATH_FP32):
    return lib().small_conv_weight_elems(C, K, FH, FW, math)


def small_pack_conv_weights(ctx, w_kcrs, w_blk, C, K, FH, FW, math=MATH_FP32, stream=None):
    _check(lib().small_pack_conv_weights(ctx, _ptr(w_kcrs), _ptr(w_blk), C, K, FH, FW, math, _stream(stream)), "small_pack_conv_weights")


def small_dw_weight_elems(C, FH, FW):
    return lib().small_dw_weight_elems(C, FH, FW)


def small_pack_dw_weights(ctx, w_crs, w_blk, C, FH, FW, stream=None):
    _check(lib().small_pack_dw_weights(ctx, _ptr(w_crs), _ptr(w_blk), C, FH, FW, _stream(stream)), "small_pack_dw_weights")


def small_fc_weight_elems(J, K, math=MATH_FP32):
    return lib().small_fc_weight_elems(J, K, math)


def small_fc_chain(ctx, inp, w_blks, biases, widths, relu, out, scratch, N, flags=0, stream=None):
    L = len(w_blks)
    wp = (ctypes.c_void_p * L)(*[_ptr(w) for w in w_blks])
    bp = (ctypes.c_void_p * L)(*[_ptr(b) for b in biases]) if biases is not None else None
    wd = (ctypes.c_int * (L + 1))(*widths)
    rl = (ctypes.c_int * L)(*[1 if r else 0 for r in relu])
    _check(lib().small_fc_chain(ctx, _ptr(inp), wp, bp, wd, rl, _ptr(out), _ptr(scratch), L, N, flags, _stream(stream)), "small_fc_chain")


def small_fc_chain_fused(widths, math):
    wd = (ctypes.c_int * len(widths))(*widths)
    return bool(lib().small_fc_chain_fused(wd, len(widths) - 1, math))


def small_fc_uses_tensor_cores(N, J, K, math):
    return bool(lib().small_fc_uses_tensor_cores(N, J, K, math))


def small_pack_fc_weights(ctx, w_kj, w_blk, J, K, math=MATH_FP32, stream=None):
    _check(lib().small_pack_fc_weights(ctx, _ptr(w_kj), _ptr(w_blk), J, K, math, _stream(stream)), "small_pack_fc_weights")


def small_conv2d(ctx, inp, w_blk, bias, out, N, C, K, H, W, FH, FW, stride, pad, flags=0, stream=None):
    pt, pb, pl, pr = pad
    _check(lib().small_conv2d(ctx, _ptr(inp), _ptr(w_blk), _ptr(bias), _ptr(out), N, C, K, H, W, FH, FW, stride,
                              pt, pb, pl, pr, flags, _stream(stream)), "small_conv2d")


def small_group_count(C, F_C, S_C):
    return int(lib().small_group_count(C, F_C, S_C))


def small_group_conv_weight_elems(C, F_C, S_C, K, FH, FW):
    return int(lib().small_group_conv_weight_elems(C, F_C, S_C, K, FH, FW))


def small_pack_group_conv_weights(ctx, w_gkcrs, w_blk, C, F_C, S_C, K, FH, FW, stream=None):
    _check(lib().small_pack_group_conv_weights(ctx, _ptr(w_gkcrs), _ptr(w_blk), C, F_C, S_C, K, FH, FW, _stream(stream)),
           "small_pack_group_conv_weights")


def small_group_conv2d(ctx, inp, w_blk, bias, out, N, C, F_C, S_C, K, H, W, FH, FW, stride, pad, flags=0, stream=None):
    pt, pb, pl, pr = pad
    _check(lib().small_group_conv2d(ctx, _ptr(inp), _ptr(w_blk), _ptr(bias), _ptr(out), N, C, F_C, S_C, K, H, W, FH, FW, stride,
                                    pt, pb, pl, pr, flags, _stream(stream)), "small_group_conv2d")


def small_dwpw_conv2d(ctx, inp, dw_w_blk, dw_bias, pw_w_blk, pw_bias, out, scratch, N, C, K, H, W, stride, pad, flags=0, stream=None):
    pt, pb, pl, pr = pad
    _check(lib().small_dwpw_conv2d(ctx, _ptr(inp), _ptr(dw_w_blk), _ptr(dw_bias), _ptr(pw_w_blk), _ptr(pw_bias), _ptr(out), _ptr(scratch),
                                   N, C, K, H, W, stride, pt, pb, pl, pr, flags, _stream(stream)), "small_dwpw_conv2d")


def small_dwpw_fused(N, C, K, H, W, stride, pad, math):
    pt, pb, pl, pr = pad
    return bool(lib().small_dwpw_fused(N, C, K, H, W, stride, pt, pb, pl, pr, math))


def small_conv_maxpool2d(ctx, inp, w_blk, bias, out, scratch, N, C, K, H, W, FH, FW, stride, pad, flags=0, stream=None):
    pt, pb, pl, pr = pad
    _check(lib().small_conv_maxpool2d(ctx, _ptr(inp), _ptr(w_blk), _ptr(bias), _ptr(out), _ptr(scratch), N, C, K, H, W, FH, FW, stride,
                                      pt, pb, pl, pr, flags, _stream(stream)), "small_conv_maxpool2d")


def small_conv_maxpool_fused(N, C, K, H, W, FH, FW, stride, pad):
    pt, pb, pl, pr = pad
    return bool(lib().small_conv_maxpool_fused(N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr))


def small_conv2d_uses_tensor_cores(N, C, K, H, W, FH, FW, stride, pad):
    pt, pb, pl, pr = pad
    return bool(lib().small_conv2d_uses_tensor_cores(N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr))


def small_dwconv2d(ctx, inp, w_blk, bias, out, N, C, H, W, FH, FW, stride, pad, flags=0, stream=None):
    pt, pb, pl, pr = pad
    _check(lib().small_dwconv2d(ctx, _ptr(inp), _ptr(w_blk), _ptr(bias), _ptr(out), N, C, H, W, FH, FW, stride,
                                pt, pb, pl, pr, flags, _stream(stream)), "small_dwconv2d")


def small_pool2d(ctx, inp, out, idx, N, C, H, W, FH, FW, stride, pad, mode=POOL_MAX, stream=None):
    pt, pb, pl, pr = pad
    _check(lib().small_pool2d(ctx, _ptr(inp), _ptr(out), _ptr(idx), N, C, H, W, FH, FW, stride, pt, pb, pl, pr, mode,
                              _stream(stream)), "small_pool2d")


def small_relu(ctx, inp, out, N, C, H, W, stream=None):
    _check(lib().small_relu(ctx, _ptr(inp), _ptr(out), N, C, H, W, _stream(stream)), "small_relu")


def small_scale_shift(ctx, inp, scale, shift, out, N, C, H, W, flags=0, stream=None):
    _check(lib().small_scale_shift(ctx, _ptr(inp), _ptr(scale), _ptr(shift), _ptr(out), N, C, H, W, flags, _stream(stream)), "small_scale_shift")


def small_upsample_nearest(ctx, inp, out, N, C, H, W, factor, stream=None):
    _check(lib().small_upsample_nearest(ctx, _ptr(inp), _ptr(out), N, C, H, W, factor, _stream(stream)), "small_upsample_nearest")


def small_add(ctx, a, b, out, N, C, H, W, flags=0, stream=None):
    _check(lib().small_add(ctx, _ptr(a), _ptr(b), _ptr(out), N, C, H, W, flags, _stream(stream)), "small_add")


def small_fc(ctx, inp, w_blk, bias, out, N, J, K, flags=0, stream=None):
    _check(lib().small_fc(ctx, _ptr(inp), _ptr(w_blk), _ptr(bias), _ptr(out), N, J, K, flags, _stream(stream)), "small_fc")


def small_gap_fc(ctx, inp, w_blk, bias, out, scratch, N, C, H, W, K, flags=0, stream=None):
    _check(lib().small_gap_fc(ctx, _ptr(inp), _ptr(w_blk), _ptr(bias), _ptr(out), _ptr(scratch), N, C, H, W, K, flags, _stream(stream)),
           "small_gap_fc")


def small_gap_fc_fused(N, C, K, math):
    return bool(lib().small_gap_fc_fused(N, C, K, math))


FUSE_DWPW, FUSE_DWPW_ALWAYS, FUSE_CONVPOOL, FUSE_FC_CHAIN, FUSE_POOLFC = 1, 2, 4, 8, 16
FUSE_DEFAULT = FUSE_DWPW | FUSE_CONVPOOL | FUSE_FC_CHAIN | FUSE_POOLFC


def small_set_net_fusion(ctx, mask):
    _check(lib().small_set_net_fusion(ctx, mask), "small_set_net_fusion")


def small_net_launches(ctx, layers, N):
    return int(lib().small_net_launches(ctx, layers, len(layers), N))


def small_net_workspace_bytes(layers, N):
    return lib().small_net_workspace_bytes(layers, len(layers), N)


def small_run_net(ctx, layers, N, in_blk, out_blk, workspace, workspace_bytes, stream=None):
    _check(lib().small_run_net(ctx, layers, len(layers), N, _ptr(in_blk), _ptr(out_blk), _ptr(workspace), workspace_bytes,
                               _stream(stream)), "small_run_net")


def small_net_host_staging_bytes(N, C, H, W, outC, outH, outW):
    return lib().small_net_host_staging_bytes(N, C, H, W, outC, outH, outW)


def small_run_net_host(ctx, layers, N, in_host, C, H, W, out_host, outC, outH, outW, workspace, workspace_bytes, stream=None):
    """in_host / out_host: CPU tensors (pinned for asynchronous copies)."""
    _check(lib().small_run_net_host(ctx, layers, len(layers), N, _ptr(in_host), C, H, W, _ptr(out_host), outC, outH, outW,
                                    _ptr(workspace), workspace_bytes, _stream(stream)), "small_run_net_host")


def small_static_workspace_bytes():
    return lib().small_static_workspace_bytes()


def small_run_net_static(ctx, layers, N, in_blk, out_blk, stream=None):
    """small_run_net on the library's built-in workspace: no device allocation by the call (see include/small.h)."""
    _check(lib().small_run_net_static(ctx, layers, len(layers), N, _ptr(in_blk), _ptr(out_blk), _stream(stream)),
           "small_run_net_static")


def small_measure_tf32_peak(ctx, n=128, iters=4096, stream=None):
    """(TFLOP/s of the whole device, cycles per 128 x n x 8 MMA) from the library's issue-rate probe."""
    sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    cycles = torch.zeros(sms, dtype=torch.int64, device="cuda")
    tf, cpm = ctypes.c_double(0), ctypes.c_double(0)
    _check(lib().small_measure_tf32_peak(ctx, n, iters, _ptr(cycles), ctypes.byref(tf), ctypes.byref(cpm), _stream(stream)),
           "small_measure_tf32_peak")
    return tf.value, cpm.value


# ---- quantised layers (uint8 tensors; qp = (z_in, z_w, z_out, mult, shift)) ----

def small_q_packed_bytes(N, C, H, W):
    return lib().small_q_packed_bytes(N, C, H, W)


def small_q_pack(ctx, nchw, blk, N, C, H, W, stream=None):
    _check(lib().small_q_pack(ctx, _ptr(nchw), _ptr(blk), N, C, H, W, _stream(stream)), "small_q_pack")


def small_q_unpack(ctx, blk, nchw, N, C, H, W, stream=None):
    _check(lib().small_q_unpack(ctx, _ptr(blk), _ptr(nchw), N, C, H, W, _stream(stream)), "small_q_unpack")


def small_q_conv_weight_bytes(C, K, FH, FW):
    return lib().small_q_conv_weight_bytes(C, K, FH, FW)


def small_q_pack_conv_weights(ctx, w_kcrs, w_blk, C, K, FH, FW, stream=None):
    _check(lib().small_q_pack_conv_weights(ctx, _ptr(w_kcrs), _ptr(w_blk), C, K, FH, FW, _stream(stream)), "small_q_pack_conv_weights")


def small_q_conv2d(ctx, inp, w_blk, bias, out, N, C, K, H, W, FH, FW, stride, pad, qp, flags=0, stream=None):
    pt, pb, pl, pr = pad
    z_in, z_w, z_out, mult, shift = qp
    _check(lib().small_q_conv2d(ctx, _ptr(inp), _ptr(w_blk), _ptr(bias), _ptr(out), N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr,
                                z_in, z_w, z_out, mult, shift, flags, _stream(stream)), "small_q_conv2d")


def small_q_dw_weight_bytes(C, FH, FW):
    return lib().small_q_dw_weight_bytes(C, FH, FW)


def small_q_pack_dw_weights(ctx, w_crs, w_blk, C, FH, FW, stream=None):
    _check(lib().small_q_pack_dw_weights(ctx, _ptr(w_crs), _ptr(w_blk), C, FH, FW, _stream(stream)), "small_q_pack_dw_weights")


def small_q_dwconv2d(ctx, inp, w_blk, bias, out, N, C, H, W, FH, FW, stride, pad, qp, flags=0, stream=None):
    pt, pb, pl, pr = pad
    z_in, z_w, z_out, mult, shift = qp
    _check(lib().small_q_dwconv2d(ctx, _ptr(inp), _ptr(w_blk), _ptr(bias), _ptr(out), N, C, H, W, FH, FW, stride, pt, pb, pl, pr,
                                  z_in, z_w, z_out, mult, shift, flags, _stream(stream)), "small_q_dwconv2d")


def small_q_maxpool2d(ctx, inp, out, N, C, H, W, FH, FW, stride, pad, z, stream=None):
    pt, pb, pl, pr = pad
    _check(lib().small_q_maxpool2d(ctx, _ptr(inp), _ptr(out), N, C, H, W, FH, FW, stride, pt, pb, pl, pr, z, _stream(stream)), "small_q_maxpool2d")


def small_q_relu(ctx, inp, out, N, C, H, W, z, stream=None):
    _check(lib().small_q_relu(ctx, _ptr(inp), _ptr(out), N, C, H, W, z, _stream(stream)), "small_q_relu")
