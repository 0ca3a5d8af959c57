"""Fused depthwise 3x3 -> 1x1 convolution against the oracle's two layers applied one after the other."""
import numpy as np
import pytest
import torch

import oracle
import synth
from paper_2303_04769_b200 import binding as B
from gpu_util import ctx, dev, to_blk, from_blk, new_blk, rel_err, pad_lanes_are_zero

pytestmark = pytest.mark.gpu


def rnd(shape, tid, lo=-1.0, hi=1.0):
    return synth.uniform(shape, lo, hi, tid, seed=777)


CASES = [  # N, C, K, H, W, stride, pad
    (2, 64, 64, 25, 5, 1, (1, 1, 1, 1)),        # keyword-spotting blocks
    (3, 64, 128, 24, 24, 1, (1, 1, 1, 1)),      # depthwise-separable blocks: several row tiles per image
    (2, 32, 64, 48, 48, 2, (1, 1, 1, 1)),       # stride-2 depthwise
    (5, 128, 128, 12, 12, 1, (1, 1, 1, 1)),     # whole images per tile
    (4, 256, 256, 6, 6, 2, (1, 1, 1, 1)),       # 3x3 output planes, eight channel blocks
    (2, 8, 16, 48, 48, 1, (1, 1, 1, 1)),        # fewer channels than a block
    (2, 70, 45, 9, 11, 1, (1, 0, 0, 1)),        # ragged channels, one-sided pads
    (1, 128, 300, 7, 7, 1, (1, 1, 1, 1)),       # two filter tiles
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("math", ["tf32", "3xtf32", "fp32"])
def test_dwpw_matches_the_two_layers(case, math):
    N, C, K, H, W, S, pad = case
    x = rnd((N, C, H, W), 71)
    wd, bd = rnd((C, 3, 3), 72), rnd((C,), 73)
    wp, bp = rnd((K, C, 1, 1), 74), rnd((K,), 75)
    mid = oracle.dwconv2d(x, wd, bd, S, pad, relu=True)
    ref = oracle.conv2d(mid, wp, bp, 1, (0, 0, 0, 0), relu=True)
    OH, OW = ref.shape[2:]
    wdb = torch.empty(B.small_dw_weight_elems(C, 3, 3), device="cuda")
    B.small_pack_dw_weights(ctx(), dev(wd), wdb, C, 3, 3)
    wpb = torch.empty(B.small_conv_weight_elems(C, K, 1, 1, B.MATH_3XTF32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(wp), wpb, C, K, 1, 1, B.MATH_3XTF32)
    out = new_blk(N, K, OH, OW)
    scratch = new_blk(N, C, OH, OW)
    fused = math != "fp32" and B.small_dwpw_fused(N, C, K, H, W, S, pad, B.MATH[math])
    B.small_dwpw_conv2d(ctx(), to_blk(x), wdb, dev(bd), wpb, dev(bp), out, None if fused else scratch,
                        N, C, K, H, W, S, pad, B.RELU | B.RELU_MID | B.MATH[math])
    assert B.small_device_status(ctx()) == 0
    err = rel_err(from_blk(out, N, K, OH, OW), ref)
    assert err <= {"tf32": 2e-3, "3xtf32": 1e-5, "fp32": 1e-5}[math], err
    assert pad_lanes_are_zero(out, N, K, OH, OW)
    if math != "fp32":
        assert fused, "the tensor-core modes take every shape of this list as one kernel"


def test_dwpw_needs_scratch_only_when_not_fused():
    N, C, K, H, W = 1, 32, 32, 8, 8
    x = to_blk(rnd((N, C, H, W), 76))
    wdb = torch.zeros(B.small_dw_weight_elems(C, 3, 3), device="cuda")
    wpb = torch.zeros(B.small_conv_weight_elems(C, K, 1, 1, B.MATH_TF32), device="cuda")
    out = new_blk(N, K, H, W)
    with pytest.raises(B.SmallError):
        B.small_dwpw_conv2d(ctx(), x, wdb, None, wpb, None, out, None, N, C, K, H, W, 1, (1, 1, 1, 1), B.MATH_FP32)
    B.small_dwpw_conv2d(ctx(), x, wdb, None, wpb, None, out, None, N, C, K, H, W, 1, (1, 1, 1, 1), B.MATH_TF32)
    assert float(from_blk(out, N, K, H, W).max()) == 0.0
