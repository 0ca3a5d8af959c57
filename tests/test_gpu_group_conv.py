"""Group convolution (partial channel reduction, Section 3.1.2 / Figure 1) on the GPU against the oracle's statement of
Algorithm 1, which slides the window over the channels too.  The abstract layer has no padding and takes one image, so
padded cases pad the input on the host first and images go through it one by one."""
import numpy as np
import pytest
import torch

import oracle
from paper_2303_04769_b200 import binding as B
from gpu_util import ctx, dev, to_blk, from_blk, new_blk, rel_err, pad_lanes_are_zero
import synth

pytestmark = pytest.mark.gpu


def rnd(shape, tid, lo=-1.0, hi=1.0):
    return synth.uniform(shape, lo, hi, tid, seed=4242)

CASES = [  # N, C, F_C, S_C, K, H, W, FH, FW, stride, pad
    (2, 64, 16, 16, 16, 14, 14, 3, 3, 1, (1, 1, 1, 1)),     # 4 groups of 16 channels, 16 filters each
    (2, 128, 32, 32, 32, 9, 11, 3, 3, 1, (1, 1, 1, 1)),     # groups = whole channel blocks
    (3, 40, 1, 1, 1, 9, 9, 3, 3, 1, (1, 1, 1, 1)),          # one channel, one filter per group: a depthwise convolution
    (2, 24, 1, 1, 3, 8, 8, 3, 3, 2, (1, 1, 1, 1)),          # channel multiplier 3, stride 2
    (1, 8, 4, 2, 3, 6, 7, 3, 3, 1, (0, 0, 0, 0)),           # Figure 1's shape: overlapping groups (F_C = 4, S_C = 2)
    (2, 96, 48, 48, 20, 7, 7, 1, 1, 1, (0, 0, 0, 0)),       # groups across block boundaries, ragged filter count
    (2, 70, 10, 10, 5, 6, 6, 5, 3, (1), (2, 2, 1, 1)),      # 7 groups, nothing a multiple of 32
    (2, 64, 64, 1, 8, 6, 6, 3, 3, 1, (1, 1, 1, 1)),         # a single group: the full reduction
    (1, 36, 8, 4, 40, 5, 5, 2, 2, 1, (0, 1, 1, 0)),         # more filters per group than a block, overlapping groups
]


def oracle_group_conv(x, w, bias, F_C, S_C, K, stride, pad, relu):
    pt, pb, pl, pr = pad
    xp = np.pad(x, ((0, 0), (0, 0), (pt, pb), (pl, pr)))
    G = w.shape[0]
    outs = [oracle.abstract_layer(xp[n], w, w.shape[3], w.shape[4], F_C, stride, stride, S_C, K)
            for n in range(x.shape[0])]
    out = np.stack(outs).astype(np.float64) + bias.astype(np.float64)[None, :, None, None]
    out = out.astype(np.float32)
    return np.maximum(out, 0.0) if relu else out


@pytest.mark.parametrize("case", CASES)
def test_group_conv_matches_algorithm_1(case):
    N, C, F_C, S_C, K, H, W, FH, FW, S, pad = case
    G = B.small_group_count(C, F_C, S_C)
    assert G == oracle.groups(C, F_C, S_C) and G >= 1
    OC = K * G
    x, w, b = rnd((N, C, H, W), 46), rnd((G, K, F_C, FH, FW), 47), rnd((OC,), 48)
    wb = torch.full((B.small_group_conv_weight_elems(C, F_C, S_C, K, FH, FW),), float("nan"), device="cuda")
    B.small_pack_group_conv_weights(ctx(), dev(w), wb, C, F_C, S_C, K, FH, FW)
    ref = oracle_group_conv(x, w, b, F_C, S_C, K, S, pad, relu=True)
    OH, OW = ref.shape[2:]
    out = new_blk(N, OC, OH, OW)
    B.small_group_conv2d(ctx(), to_blk(x), wb, dev(b), out, N, C, F_C, S_C, K, H, W, FH, FW, S, pad, B.RELU)
    got = from_blk(out, N, OC, OH, OW)
    # the abstract layer rounds its sum before the bias is added here, the kernel adds the bias first: one more rounding
    assert rel_err(got, ref) <= 1e-5
    assert pad_lanes_are_zero(out, N, OC, OH, OW)
    # accumulate epilogue
    prev = rnd((N, OC, OH, OW), 49)
    acc = to_blk(prev)
    B.small_group_conv2d(ctx(), to_blk(x), wb, None, acc, N, C, F_C, S_C, K, H, W, FH, FW, S, pad, B.ACCUMULATE)
    ref_acc = oracle_group_conv(x, w, np.zeros(OC, np.float32), F_C, S_C, K, S, pad, relu=False).astype(np.float64) + prev
    assert rel_err(from_blk(acc, N, OC, OH, OW), ref_acc.astype(np.float32)) <= 1e-5


def test_group_conv_special_cases_equal_the_other_layers():
    # one group = small_conv2d's result; one channel and one filter per group = small_dwconv2d's result
    N, C, K, H, W = 2, 48, 20, 9, 9
    x, w, b = rnd((N, C, H, W), 50), rnd((K, C, 3, 3), 51), rnd((K,), 52)
    wb = torch.empty(B.small_group_conv_weight_elems(C, C, 1, K, 3, 3), device="cuda")
    B.small_pack_group_conv_weights(ctx(), dev(w), wb, C, C, 1, K, 3, 3)
    out = new_blk(N, K, H, W)
    B.small_group_conv2d(ctx(), to_blk(x), wb, dev(b), out, N, C, C, 1, K, H, W, 3, 3, 1, (1, 1, 1, 1), B.RELU)
    assert rel_err(from_blk(out, N, K, H, W), oracle.conv2d(x, w, b, 1, (1, 1, 1, 1), relu=True)) <= 1e-5
    wd = rnd((C, 3, 3), 53)
    wb = torch.empty(B.small_group_conv_weight_elems(C, 1, 1, 1, 3, 3), device="cuda")
    B.small_pack_group_conv_weights(ctx(), dev(wd), wb, C, 1, 1, 1, 3, 3)
    bc = rnd((C,), 54)
    out = new_blk(N, C, H, W)
    B.small_group_conv2d(ctx(), to_blk(x), wb, dev(bc), out, N, C, 1, 1, 1, H, W, 3, 3, 1, (1, 1, 1, 1), 0)
    assert rel_err(from_blk(out, N, C, H, W), oracle.dwconv2d(x, wd, bc, 1, (1, 1, 1, 1))) <= 1e-5


def test_group_conv_rejects_bad_channel_windows():
    assert B.small_group_count(10, 4, 4) == 0 and B.small_group_conv_weight_elems(10, 4, 4, 2, 3, 3) == 0
    x = new_blk(1, 10, 4, 4, 0.0)
    out = new_blk(1, 4, 4, 4, 0.0)
    w = torch.zeros(1024, device="cuda")
    with pytest.raises(B.SmallError) as e:
        B.small_group_conv2d(ctx(), x, w, None, out, 1, 10, 4, 4, 2, 4, 4, 1, 1, 1, (0, 0, 0, 0), 0)
    assert "shape" in str(e.value).lower() or e.value.status != 0


TC_CASES = [  # groups of whole channel blocks: N, C, F_C, K, H, W, FH, FW, stride, pad
    (2, 128, 32, 32, 9, 11, 3, 3, 1, (1, 1, 1, 1)),
    (3, 256, 64, 64, 14, 14, 3, 3, 1, (1, 1, 1, 1)),       # two channel blocks per group
    (2, 128, 32, 32, 16, 16, 3, 3, 2, (1, 1, 1, 1)),       # stride 2: phase planes per group
    (2, 64, 32, 128, 9, 9, 1, 1, 1, (0, 0, 0, 0)),         # more filters than channels per group
    (5, 512, 32, 32, 7, 7, 3, 3, 1, (1, 1, 1, 1)),         # 16 groups, several images per strip
    (2, 96, 32, 96, 12, 10, 3, 1, 1, (1, 1, 0, 0)),        # three groups, rectangular window
]


@pytest.mark.parametrize("case", TC_CASES)
def test_group_conv_on_tensor_cores(case):
    N, C, F_C, K, H, W, FH, FW, S, pad = case
    G = C // F_C
    OC = K * G
    x, w, b = rnd((N, C, H, W), 56), rnd((G, K, F_C, FH, FW), 57), rnd((OC,), 58)
    wb = torch.full((B.small_group_conv_weight_elems(C, F_C, F_C, K, FH, FW),), float("nan"), device="cuda")
    B.small_pack_group_conv_weights(ctx(), dev(w), wb, C, F_C, F_C, K, FH, FW)
    ref = oracle_group_conv(x, w, b, F_C, F_C, K, S, pad, relu=True)
    OH, OW = ref.shape[2:]
    bx = to_blk(x)
    outs = {}
    for math, tol in (("fp32", 1e-5), ("tf32", 2e-3), ("3xtf32", 1e-5)):
        out = new_blk(N, OC, OH, OW)
        B.small_group_conv2d(ctx(), bx, wb, dev(b), out, N, C, F_C, F_C, K, H, W, FH, FW, S, pad, B.RELU | B.MATH[math])
        assert B.small_device_status(ctx()) == 0
        got = from_blk(out, N, OC, OH, OW)
        err = rel_err(got, ref)
        assert err <= tol, (math, err)
        assert pad_lanes_are_zero(out, N, OC, OH, OW)
        outs[math] = (out, err)
    assert outs["tf32"][1] > 1e-6                                    # TF32 products: the tensor-core kernel ran
    assert not torch.equal(outs["3xtf32"][0].view(torch.int32), outs["fp32"][0].view(torch.int32))
    prev = rnd((N, OC, OH, OW), 59)
    acc = to_blk(prev)
    B.small_group_conv2d(ctx(), bx, wb, None, acc, N, C, F_C, F_C, K, H, W, FH, FW, S, pad, B.ACCUMULATE | B.MATH_3XTF32)
    ref_acc = oracle_group_conv(x, w, np.zeros(OC, np.float32), F_C, F_C, K, S, pad, relu=False).astype(np.float64) + prev
    assert rel_err(from_blk(acc, N, OC, OH, OW), ref_acc.astype(np.float32)) <= 1e-5
