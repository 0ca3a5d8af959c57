"""Python face of the CPU oracle (oracle/small_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA package never imports this module and
this module never imports the CUDA package.

All arrays are C-contiguous float32 numpy arrays in NCHW (filters [K][C][FH][FW],
depthwise filters [C][FH][FW], FC filters [K][J]).  Every function returns new arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "small_oracle.c")
_LIB = os.path.join(_HERE, "libsmall_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP, no fast-math: the sums keep their written order)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-fvisibility=hidden",
                               "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None
_f32p = ctypes.POINTER(ctypes.c_float)
_i32p = ctypes.POINTER(ctypes.c_int32)


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        I = ctypes.c_int
        L.so_out_size.argtypes = [I] * 5
        L.so_out_size.restype = I
        L.so_same_pad.argtypes = [I, I, I, ctypes.POINTER(I), ctypes.POINTER(I), ctypes.POINTER(I)]
        L.so_groups.argtypes = [I] * 3
        L.so_out_channels.argtypes = [I] * 2
        L.so_model_memory_mib.argtypes = [ctypes.c_long] * 3
        L.so_model_memory_mib.restype = ctypes.c_double
        L.so_blk_index.argtypes = [I] * 8
        L.so_blk_index.restype = ctypes.c_long
        L.so_blk_elems.argtypes = [I] * 5
        L.so_blk_elems.restype = ctypes.c_long
        L.so_pack.argtypes = [_f32p, _f32p] + [I] * 5
        L.so_unpack.argtypes = [_f32p, _f32p] + [I] * 5
        conv_args = [_f32p, _f32p, _f32p, _f32p] + [I] * 14
        L.so_conv2d.argtypes = conv_args
        L.so_conv2d_f32acc.argtypes = conv_args
        L.so_dwconv2d.argtypes = [_f32p, _f32p, _f32p, _f32p] + [I] * 12
        L.so_pool2d.argtypes = [_f32p, _f32p, _i32p] + [I] * 12
        L.so_relu.argtypes = [_f32p, _f32p, ctypes.c_long]
        L.so_add.argtypes = [_f32p, _f32p, _f32p, ctypes.c_long, I]
        L.so_scale_shift.argtypes = [_f32p, _f32p, _f32p, _f32p, I, I, I, I, I]
        L.so_upsample_nearest.argtypes = [_f32p, _f32p, I, I, I, I, I]
        L.so_fc.argtypes = [_f32p, _f32p, _f32p, _f32p] + [I] * 4
        L.so_abstract_layer.argtypes = [_f32p, _f32p, _f32p] + [I] * 11 + [ctypes.c_double]
        L.so_abstract_layer.restype = I
        L.so_num_threads.restype = I
        _u8p = ctypes.POINTER(ctypes.c_uint8)
        L.so_requantize.argtypes = [I] * 5
        L.so_requantize.restype = I
        L.so_q_conv2d.argtypes = [_u8p, _u8p, _i32p, _u8p] + [I] * 18
        L.so_q_dwconv2d.argtypes = [_u8p, _u8p, _i32p, _u8p] + [I] * 17
        L.so_q_maxpool2d.argtypes = [_u8p, _u8p] + [I] * 12
        L.so_q_relu.argtypes = [_u8p, _u8p, ctypes.c_long, I]
        L.so_model_memory_q_mib.argtypes = [ctypes.c_long] * 3
        L.so_model_memory_q_mib.restype = ctypes.c_double
        _lib = L
    return _lib


def _f(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(_f32p)


def _opt(a):
    if a is None:
        return None, None
    return _f(a)


def num_threads() -> int:
    return int(lib().so_num_threads())


def out_size(I, F, S, pad_before=0, pad_after=0) -> int:
    return int(lib().so_out_size(I, F, S, pad_before, pad_after))


def same_pad(I, F, S):
    o, b, a = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    lib().so_same_pad(I, F, S, ctypes.byref(o), ctypes.byref(b), ctypes.byref(a))
    return o.value, b.value, a.value


def groups(I_C, F_C, S_C) -> int:
    return int(lib().so_groups(I_C, F_C, S_C))


def out_channels(K, G) -> int:
    return int(lib().so_out_channels(K, G))


def model_memory_mib(params, largest_pair, model_input) -> float:
    return float(lib().so_model_memory_mib(params, largest_pair, model_input))


def blk_index(n, c, h, w, C, H, W, Cb) -> int:
    return int(lib().so_blk_index(n, c, h, w, C, H, W, Cb))


def blk_elems(N, C, H, W, Cb) -> int:
    return int(lib().so_blk_elems(N, C, H, W, Cb))


def pack(x, Cb):
    x, xp = _f(x)
    N, C, H, W = x.shape
    out = np.empty(blk_elems(N, C, H, W, Cb), dtype=np.float32)
    lib().so_pack(xp, out.ctypes.data_as(_f32p), N, C, H, W, Cb)
    return out


def unpack(blk, N, C, H, W, Cb):
    blk, bp = _f(blk)
    assert blk.size == blk_elems(N, C, H, W, Cb)
    out = np.empty((N, C, H, W), dtype=np.float32)
    lib().so_unpack(bp, out.ctypes.data_as(_f32p), N, C, H, W, Cb)
    return out


def conv2d(x, w, bias=None, stride=1, pad=(0, 0, 0, 0), relu=False, accumulate_into=None, f32acc=False):
    x, xp = _f(x)
    w, wp = _f(w)
    b, bp = _opt(bias)
    N, C, H, W = x.shape
    K, C2, FH, FW = w.shape
    assert C2 == C
    pt, pb, pl, pr = pad
    OH, OW = out_size(H, FH, stride, pt, pb), out_size(W, FW, stride, pl, pr)
    assert OH > 0 and OW > 0
    if accumulate_into is not None:
        out = np.array(accumulate_into, dtype=np.float32, order="C", copy=True)
        assert out.shape == (N, K, OH, OW)
    else:
        out = np.empty((N, K, OH, OW), dtype=np.float32)
    fn = lib().so_conv2d_f32acc if f32acc else lib().so_conv2d
    fn(xp, wp, bp, out.ctypes.data_as(_f32p), N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr,
       int(relu), int(accumulate_into is not None))
    return out


def dwconv2d(x, w, bias=None, stride=1, pad=(0, 0, 0, 0), relu=False):
    x, xp = _f(x)
    w, wp = _f(w)
    b, bp = _opt(bias)
    N, C, H, W = x.shape
    C2, FH, FW = w.shape
    assert C2 == C
    pt, pb, pl, pr = pad
    OH, OW = out_size(H, FH, stride, pt, pb), out_size(W, FW, stride, pl, pr)
    assert OH > 0 and OW > 0
    out = np.empty((N, C, OH, OW), dtype=np.float32)
    lib().so_dwconv2d(xp, wp, bp, out.ctypes.data_as(_f32p), N, C, H, W, FH, FW, stride, pt, pb, pl, pr, int(relu))
    return out


def pool2d(x, FH, FW, stride, pad=(0, 0, 0, 0), mode="max", with_indices=False):
    x, xp = _f(x)
    N, C, H, W = x.shape
    pt, pb, pl, pr = pad
    OH, OW = out_size(H, FH, stride, pt, pb), out_size(W, FW, stride, pl, pr)
    assert OH > 0 and OW > 0
    out = np.empty((N, C, OH, OW), dtype=np.float32)
    idx = np.empty((N, C, OH, OW), dtype=np.int32) if with_indices else None
    lib().so_pool2d(xp, out.ctypes.data_as(_f32p), idx.ctypes.data_as(_i32p) if with_indices else None,
                    N, C, H, W, FH, FW, stride, pt, pb, pl, pr, 0 if mode == "max" else 1)
    return (out, idx) if with_indices else out


def relu(x):
    x, xp = _f(x)
    out = np.empty_like(x)
    lib().so_relu(xp, out.ctypes.data_as(_f32p), x.size)
    return out


def scale_shift(x, scale, shift, relu=False):
    """Inference batch normalisation as the paper classes it (Table 2): out = scale[c] * x + shift[c]."""
    x, xp = _f(x)
    s, sp = _f(scale)
    t, tp = _f(shift)
    N, C, H, W = x.shape
    assert s.shape == (C,) and t.shape == (C,)
    out = np.empty_like(x)
    lib().so_scale_shift(xp, sp, tp, out.ctypes.data_as(_f32p), N, C, H, W, int(relu))
    return out


def upsample_nearest(x, f):
    """Nearest-neighbour upsampling by an integer factor (Table 2)."""
    x, xp = _f(x)
    N, C, H, W = x.shape
    out = np.empty((N, C, H * f, W * f), dtype=np.float32)
    lib().so_upsample_nearest(xp, out.ctypes.data_as(_f32p), N, C, H, W, int(f))
    return out


def add(a, b, relu=False):
    a, ap = _f(a)
    b, bp = _f(b)
    assert a.shape == b.shape
    out = np.empty_like(a)
    lib().so_add(ap, bp, out.ctypes.data_as(_f32p), a.size, int(relu))
    return out


def fc(x, w, bias=None, relu=False):
    x, xp = _f(x)
    w, wp = _f(w)
    b, bp = _opt(bias)
    N = x.shape[0]
    J = int(np.prod(x.shape[1:]))
    K, J2 = w.shape
    assert J2 == J
    out = np.empty((N, K), dtype=np.float32)
    lib().so_fc(xp, wp, bp, out.ctypes.data_as(_f32p), N, J, K, int(relu))
    return out


def abstract_layer(x, w, F_H, F_W, F_C, S_H, S_W, S_C, K, op="fma", init=0.0):
    """The abstract layer of Section 3.1 on one image x[C][H][W]; w is [G][K][F_C][F_H][F_W] or None (op='max')."""
    x, xp = _f(x)
    I_C, I_H, I_W = x.shape
    G = groups(I_C, F_C, S_C)
    O_H, O_W = out_size(I_H, F_H, S_H), out_size(I_W, F_W, S_W)
    wp = None
    if w is not None:
        w, wp = _f(w)
        assert w.shape == (G, K, F_C, F_H, F_W), (w.shape, (G, K, F_C, F_H, F_W))
    out = np.empty((out_channels(K, G), O_H, O_W), dtype=np.float32)
    rc = lib().so_abstract_layer(xp, wp, out.ctypes.data_as(_f32p), I_C, I_H, I_W, F_H, F_W, F_C,
                                 S_H, S_W, S_C, K, 0 if op == "fma" else 1, float(init))
    if rc != 0:
        raise ValueError(f"abstract layer rejected the parameters (code {rc})")
    return out


# ---- quantised layers: uint8 tensors (NCHW), int32 accumulation, one requantisation per output ----
_u8p = ctypes.POINTER(ctypes.c_uint8)


def _u8(a):
    a = np.ascontiguousarray(a, dtype=np.uint8)
    return a, a.ctypes.data_as(_u8p)


def requantize(acc, mult, shift, z_out, lo=0) -> int:
    """clamp(z_out + floor((acc * mult + 2^(shift-1)) / 2^shift), lo, 255)."""
    return int(lib().so_requantize(int(acc), int(mult), int(shift), int(z_out), int(lo)))


def q_conv2d(x, w, bias, stride, pad, z_in, z_w, z_out, mult, shift, relu=False):
    x, xp = _u8(x)
    w, wp = _u8(w)
    N, C, H, W = x.shape
    K, C2, FH, FW = w.shape
    assert C2 == C
    pt, pb, pl, pr = pad
    OH, OW = out_size(H, FH, stride, pt, pb), out_size(W, FW, stride, pl, pr)
    assert OH > 0 and OW > 0
    bp = None
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.int32)
        bp = bias.ctypes.data_as(_i32p)
    out = np.empty((N, K, OH, OW), dtype=np.uint8)
    lib().so_q_conv2d(xp, wp, bp, out.ctypes.data_as(_u8p), N, C, K, H, W, FH, FW, stride, pt, pb, pl, pr,
                      z_in, z_w, z_out, mult, shift, int(relu))
    return out


def q_dwconv2d(x, w, bias, stride, pad, z_in, z_w, z_out, mult, shift, relu=False):
    x, xp = _u8(x)
    w, wp = _u8(w)
    N, C, H, W = x.shape
    C2, FH, FW = w.shape
    assert C2 == C
    pt, pb, pl, pr = pad
    OH, OW = out_size(H, FH, stride, pt, pb), out_size(W, FW, stride, pl, pr)
    bp = None
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.int32)
        bp = bias.ctypes.data_as(_i32p)
    out = np.empty((N, C, OH, OW), dtype=np.uint8)
    lib().so_q_dwconv2d(xp, wp, bp, out.ctypes.data_as(_u8p), N, C, H, W, FH, FW, stride, pt, pb, pl, pr,
                        z_in, z_w, z_out, mult, shift, int(relu))
    return out


def q_maxpool2d(x, FH, FW, stride, pad=(0, 0, 0, 0), z=0):
    x, xp = _u8(x)
    N, C, H, W = x.shape
    pt, pb, pl, pr = pad
    OH, OW = out_size(H, FH, stride, pt, pb), out_size(W, FW, stride, pl, pr)
    out = np.empty((N, C, OH, OW), dtype=np.uint8)
    lib().so_q_maxpool2d(xp, out.ctypes.data_as(_u8p), N, C, H, W, FH, FW, stride, pt, pb, pl, pr, z)
    return out


def q_relu(x, z):
    x, xp = _u8(x)
    out = np.empty_like(x)
    lib().so_q_relu(xp, out.ctypes.data_as(_u8p), x.size, z)
    return out


def model_memory_q_mib(params, intermediates, largest_plane) -> float:
    return float(lib().so_model_memory_q_mib(params, intermediates, largest_plane))
