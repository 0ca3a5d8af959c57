"""Helpers for the GPU parity tests: device buffers through torch, every operation through the C ABI."""
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


def pad_lanes_are_zero(blk, N, C, H, W):
    """True if channels C.. of the last block hold +0 everywhere."""
    cb = (C + 31) // 32
    v = blk.view(N, cb, H, W, 32)[:, -1, :, :, C - (cb - 1) * 32:]
    if v.numel() == 0:
        return True
    bits = v.contiguous().view(torch.int32)
    return bool((bits == 0).all().item())
