"""GPU parity of the warp-level tensor-core convolution (one channel block; filters in tiles of 32) against the CPU
oracle, through small_conv2d: TF32 at 2e-3, 3xTF32 at 1e-5, each on the relative L2 error and on every element."""
import numpy as np
import pytest
import torch

import oracle
import synth
from paper_2303_04769_b200 import binding as B
from gpu_util import ctx, dev, to_blk, from_blk, new_blk, rel_err, pad_lanes_are_zero, conv_path

pytestmark = pytest.mark.gpu
TOL = {"tf32": 2e-3, "3xtf32": 1e-5}
WARP_MMA = 4


def rnd(shape, tid, lo=-1.0, hi=1.0):
    return synth.uniform(shape, lo, hi, tid, seed=777)


# (N, C, K, H, W, FH, FW, stride, pads t b l r): the residual network's layers, every fragment shape (planes 12 and more,
# 6 to 11, under 6 columns wide), ragged widths and heights, several images per tile, bands and column tiles, both row
# widths of the shared-memory tiles (C <= 16 and C <= 32), 8 / 16 / 32 filters, several filter tiles and ragged filter counts, strides 1 and 2,
# windows 1x1, 3x3, 5x5, 1x3 and 10x4, asymmetric pads.
CASES = [
    (3, 16, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),
    (5, 16, 32, 32, 32, 3, 3, 2, (1, 1, 1, 1)),
    (5, 16, 32, 32, 32, 1, 1, 2, (0, 0, 0, 0)),
    (9, 32, 32, 16, 16, 3, 3, 1, (1, 1, 1, 1)),
    (7, 32, 32, 8, 8, 3, 3, 1, (1, 1, 1, 1)),
    (37, 24, 20, 4, 4, 3, 3, 1, (1, 1, 1, 1)),
    (2, 8, 8, 25, 5, 3, 3, 1, (1, 1, 1, 1)),
    (2, 10, 13, 19, 23, 3, 3, 1, (1, 1, 1, 1)),
    (2, 17, 30, 19, 23, 3, 3, 2, (1, 0, 0, 1)),
    (1, 32, 32, 40, 100, 3, 3, 1, (1, 1, 1, 1)),
    (2, 16, 8, 70, 66, 1, 1, 1, (0, 0, 0, 0)),
    (3, 5, 32, 14, 14, 5, 5, 1, (2, 2, 2, 2)),
    (2, 16, 16, 9, 30, 1, 3, 1, (0, 0, 1, 1)),
    (3, 7, 12, 49, 10, 10, 4, 2, (4, 5, 1, 1)),
    (300, 16, 16, 3, 3, 3, 3, 1, (1, 1, 1, 1)),
    (2, 32, 16, 33, 31, 3, 3, 2, (0, 1, 1, 0)),
    (6, 32, 64, 16, 16, 3, 3, 2, (1, 1, 1, 1)),
    (6, 32, 64, 16, 16, 1, 1, 2, (0, 0, 0, 0)),
    (3, 20, 72, 11, 13, 3, 3, 1, (1, 1, 1, 1)),
    (2, 16, 130, 9, 9, 1, 1, 1, (0, 0, 0, 0)),
    (4, 3, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),
    (2, 21, 16, 12, 12, 3, 3, 1, (1, 1, 1, 1)),
]


@pytest.mark.parametrize("math", ["tf32", "3xtf32"])
@pytest.mark.parametrize("case", CASES)
def test_conv_warp_mma(case, math):
    N, C, K, H, W, FH, FW, S, pad = case
    x, w, b = rnd((N, C, H, W), 1), rnd((K, C, FH, FW), 2), rnd((K,), 3)
    m = B.MATH[math]
    wb = torch.empty(B.small_conv_weight_elems(C, K, FH, FW, m), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, FH, FW, m)
    bx = to_blk(x)
    ref = oracle.conv2d(x, w, b, S, pad, relu=True)
    OH, OW = ref.shape[2:]
    with conv_path("warp_mma"):
        assert B.small_conv2d_path(ctx(), N, C, K, H, W, FH, FW, S, pad, m) == WARP_MMA
        out = new_blk(N, K, OH, OW)
        B.small_conv2d(ctx(), bx, wb, dev(b), out, N, C, K, H, W, FH, FW, S, pad, B.RELU | m)
        assert B.small_device_status(ctx()) == 0
        err = rel_err(from_blk(out, N, K, OH, OW), ref)
        assert err <= TOL[math], err
        assert pad_lanes_are_zero(out, N, K, OH, OW)
        # the residual join: no bias, no ReLU, added to the tensor already in `out`
        prev = rnd((N, K, OH, OW), 4)
        acc = to_blk(prev)
        B.small_conv2d(ctx(), bx, wb, None, acc, N, C, K, H, W, FH, FW, S, pad, B.ACCUMULATE | m)
        assert B.small_device_status(ctx()) == 0
        err = rel_err(from_blk(acc, N, K, OH, OW), oracle.conv2d(x, w, None, S, pad, accumulate_into=prev))
        assert err <= TOL[math], err
        assert pad_lanes_are_zero(acc, N, K, OH, OW)


def test_warp_mma_is_not_the_fp32_kernel():
    """The 3xTF32 result differs in its last bits from the FP32 CUDA-core kernel's (another order of summation)."""
    N, C, K, H, W = 2, 16, 16, 32, 32
    x, w = rnd((N, C, H, W), 5), rnd((K, C, 3, 3), 6)
    wb = torch.empty(B.small_conv_weight_elems(C, K, 3, 3, B.MATH_3XTF32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, 3, 3, B.MATH_3XTF32)
    bx = to_blk(x)
    a, b = new_blk(N, K, H, W), new_blk(N, K, H, W)
    with conv_path("warp_mma"):
        B.small_conv2d(ctx(), bx, wb, None, a, N, C, K, H, W, 3, 3, 1, (1, 1, 1, 1), B.MATH_3XTF32)
    B.small_conv2d(ctx(), bx, wb, None, b, N, C, K, H, W, 3, 3, 1, (1, 1, 1, 1), B.MATH_FP32)
    torch.cuda.synchronize()
    assert not torch.equal(a.view(torch.int32), b.view(torch.int32))
    assert rel_err(from_blk(a, N, K, H, W), from_blk(b, N, K, H, W)) <= 1e-5
