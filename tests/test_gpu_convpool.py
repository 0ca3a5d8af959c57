"""The fused convolution -> 2x2 stride-2 max pool layer (small_conv_maxpool2d) against the oracle's two layers, and bit for
bit against the library's own two launches: the pooled values must be exactly the maxima of the values the unfused
convolution kernel writes."""
import numpy as np
import pytest
import torch

import oracle
import synth
from paper_2303_04769_b200 import binding as B
from gpu_util import ctx, dev, to_blk, from_blk, new_blk, rel_err, pad_lanes_are_zero, conv_path

pytestmark = pytest.mark.gpu

CASES = [  # N, C, K, H, W, FH, FW, S, pad
    (1, 16, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),       # the single-convolution workload
    (5, 16, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),
    (3, 3, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),
    (4, 32, 40, 16, 16, 3, 3, 1, (1, 1, 1, 1)),       # ragged filters
    (6, 64, 64, 8, 8, 3, 3, 1, (1, 1, 1, 1)),         # several images per row warp
    (2, 70, 45, 18, 22, 3, 3, 1, (1, 1, 1, 1)),       # ragged channels, a partial column tile
    (2, 16, 32, 33, 35, 3, 3, 1, (1, 1, 1, 1)),       # odd convolution output: last row and column dropped by the pool
    (3, 16, 32, 32, 32, 3, 3, 2, (1, 1, 1, 1)),       # stride-2 convolution, then the pool
    (2, 64, 64, 56, 56, 1, 1, 1, (0, 0, 0, 0)),
    (2, 8, 8, 12, 20, 5, 3, 1, (2, 2, 1, 1)),
]


@pytest.mark.parametrize("case", CASES)
def test_convpool_matches_the_two_layers(case):
    N, C, K, H, W, FH, FW, S, pad = case
    x = synth.uniform((N, C, H, W), -1.0, 1.0, 71, seed=5)
    w = synth.uniform((K, C, FH, FW), -1.0, 1.0, 72, seed=5)
    b = synth.uniform((K,), -1.0, 1.0, 73, seed=5)
    wb = torch.empty(B.small_conv_weight_elems(C, K, FH, FW, B.MATH_FP32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, FH, FW, B.MATH_FP32)
    bx = to_blk(x)
    assert B.small_conv_maxpool_fused(N, C, K, H, W, FH, FW, S, pad)
    for relu in (True, False):
        mid_ref = oracle.conv2d(x, w, b, S, pad, relu=relu)
        ref = oracle.pool2d(mid_ref, 2, 2, 2)
        OH, OW = mid_ref.shape[2:]
        out = new_blk(N, K, OH // 2, OW // 2)
        B.small_conv_maxpool2d(ctx(), bx, wb, dev(b), out, None, N, C, K, H, W, FH, FW, S, pad, B.RELU if relu else 0)
        got = from_blk(out, N, K, OH // 2, OW // 2)
        assert got.shape == ref.shape
        assert rel_err(got, ref) <= 1e-5
        assert pad_lanes_are_zero(out, N, K, OH // 2, OW // 2)
        # the library's own two launches with the same convolution kernel: the same bits
        mid = new_blk(N, K, OH, OW)
        two = new_blk(N, K, OH // 2, OW // 2)
        with conv_path("cuda_cores"):
            same_kernel = B.small_conv2d_path(ctx(), N, C, K, H, W, FH, FW, S, pad, B.MATH_FP32) == 1   # (stems take another kernel)
            B.small_conv2d(ctx(), bx, wb, dev(b), mid, N, C, K, H, W, FH, FW, S, pad, B.RELU if relu else 0)
        B.small_pool2d(ctx(), mid, two, None, N, K, OH, OW, 2, 2, 2, (0, 0, 0, 0), B.POOL_MAX)
        if same_kernel:
            assert torch.equal(out.view(torch.int32), two.view(torch.int32))
        else:
            assert rel_err(got, from_blk(two, N, K, OH // 2, OW // 2)) <= 1e-5
    assert B.small_device_status(ctx()) == 0


def test_convpool_unfused_shapes_need_scratch():
    N, C, K, H, W = 2, 16, 16, 9, 9       # 9 convolution rows per image and several images per row warp: pairs would straddle images
    assert not B.small_conv_maxpool_fused(N, C, K, H, W, 3, 3, 1, (1, 1, 1, 1))
    x = synth.uniform((N, C, H, W), -1.0, 1.0, 74, seed=5)
    w = synth.uniform((K, C, 3, 3), -1.0, 1.0, 75, seed=5)
    wb = torch.empty(B.small_conv_weight_elems(C, K, 3, 3, B.MATH_FP32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, 3, 3, B.MATH_FP32)
    bx = to_blk(x)
    out = new_blk(N, K, 4, 4)
    with pytest.raises(B.SmallError) as e:
        B.small_conv_maxpool2d(ctx(), bx, wb, None, out, None, N, C, K, H, W, 3, 3, 1, (1, 1, 1, 1), B.RELU)
    assert e.value.status == 5
    scratch = new_blk(N, K, H, W)
    B.small_conv_maxpool2d(ctx(), bx, wb, None, out, scratch, N, C, K, H, W, 3, 3, 1, (1, 1, 1, 1), B.RELU)
    ref = oracle.pool2d(oracle.conv2d(x, w, None, 1, (1, 1, 1, 1), relu=True), 2, 2, 2)
    assert rel_err(from_blk(out, N, K, 4, 4), ref) <= 1e-5
