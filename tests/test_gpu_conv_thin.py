"""GPU parity of the convolution kernel for layers with at most four input channels (network stems): filters in
registers, FP32 FMAs in every math mode, against the oracle's plain definition."""
import numpy as np
import pytest
import torch

import oracle
import synth
from paper_2303_04769_b200 import binding as B
from gpu_util import ctx, dev, to_blk, from_blk, new_blk, rel_err, pad_lanes_are_zero

pytestmark = pytest.mark.gpu


def rnd(shape, tid, lo=-1.0, hi=1.0):
    return synth.uniform(shape, lo, hi, tid)


CASES = [  # N, C, K, H, W, FH, FW, stride, pad
    (4, 3, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),        # residual network stem
    (3, 3, 8, 96, 96, 3, 3, 2, (1, 1, 1, 1)),         # depthwise-separable stem: bands of rows, six column groups
    (7, 1, 64, 49, 10, 10, 4, 2, (4, 5, 1, 1)),       # keyword-spotting stem: several images per tile, two filters per lane
    (5, 1, 12, 49, 10, 10, 4, 2, (4, 5, 1, 1)),       # the same window with one filter block
    (2, 1, 40, 13, 50, 10, 4, 2, (0, 0, 0, 0)),       # the same window on a wide plane, no padding (eight pixels per warp)
    (2, 2, 70, 9, 11, 3, 3, 1, (0, 1, 1, 0)),         # three filter blocks (two filter groups, the last half empty), ragged plane
    (3, 4, 33, 17, 19, 3, 3, 2, (1, 0, 0, 1)),        # four channels, odd sizes, pads on one side only
    (1, 4, 5, 3, 3, 3, 3, 1, (1, 1, 1, 1)),           # plane no larger than the window
    (2, 3, 32, 70, 9, 3, 3, 1, (2, 2, 2, 2)),         # pads of two, tall narrow plane
    (600, 1, 8, 5, 6, 3, 3, 1, (1, 1, 1, 1)),         # many tiny images: more tiles than resident thread blocks
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("math", [B.MATH_FP32, B.MATH_TF32, B.MATH_3XTF32])
def test_thin_conv_matches_oracle(case, math):
    N, C, K, H, W, FH, FW, S, pad = case
    x, w, b = rnd((N, C, H, W), 61), rnd((K, C, FH, FW), 62), rnd((K,), 63)
    wb = torch.empty(B.small_conv_weight_elems(C, K, FH, FW, math), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, FH, FW, math)
    assert not B.small_conv2d_uses_tensor_cores(N, C, K, H, W, FH, FW, S, pad)
    bx = to_blk(x)
    ref = oracle.conv2d(x, w, b, S, pad, relu=True)
    OH, OW = ref.shape[2:]
    out = new_blk(N, K, OH, OW)
    B.small_conv2d(ctx(), bx, wb, dev(b), out, N, C, K, H, W, FH, FW, S, pad, B.RELU | math)
    assert rel_err(from_blk(out, N, K, OH, OW), ref) <= 1e-5      # FP32 arithmetic whatever the mode allows
    assert pad_lanes_are_zero(out, N, K, OH, OW)
    # no bias, no ReLU
    B.small_conv2d(ctx(), bx, wb, None, out, N, C, K, H, W, FH, FW, S, pad, math)
    assert rel_err(from_blk(out, N, K, OH, OW), oracle.conv2d(x, w, None, S, pad)) <= 1e-5
    # accumulate onto an existing tensor, then ReLU
    prev = rnd((N, K, OH, OW), 64)
    acc = to_blk(prev)
    B.small_conv2d(ctx(), bx, wb, dev(b), acc, N, C, K, H, W, FH, FW, S, pad, B.RELU | B.ACCUMULATE | math)
    assert rel_err(from_blk(acc, N, K, OH, OW), oracle.conv2d(x, w, b, S, pad, relu=True, accumulate_into=prev)) <= 1e-5
    assert pad_lanes_are_zero(acc, N, K, OH, OW)
    assert B.small_device_status(ctx()) == 0


def test_thin_conv_is_exact_on_small_integers():
    """Integer-valued inputs and filters: every product and partial sum is an integer below 2^24, so FP32 FMAs in any
    order give the oracle's result bit for bit."""
    N, C, K, H, W = 3, 3, 16, 12, 20
    rng = np.random.default_rng(5)
    x = rng.integers(-8, 9, size=(N, C, H, W)).astype(np.float32)
    w = rng.integers(-8, 9, size=(K, C, 3, 3)).astype(np.float32)
    b = rng.integers(-8, 9, size=(K,)).astype(np.float32)
    wb = torch.empty(B.small_conv_weight_elems(C, K, 3, 3, B.MATH_3XTF32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, 3, 3, B.MATH_3XTF32)
    ref = oracle.conv2d(x, w, b, 2, (1, 1, 1, 1))
    OH, OW = ref.shape[2:]
    out = new_blk(N, K, OH, OW)
    B.small_conv2d(ctx(), to_blk(x), wb, dev(b), out, N, C, K, H, W, 3, 3, 2, (1, 1, 1, 1), B.MATH_3XTF32)
    np.testing.assert_array_equal(from_blk(out, N, K, OH, OW), ref.astype(np.float32))
