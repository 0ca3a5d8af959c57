"""GPU parity of the fused classifier head (global average pool, then the full reduction) against the oracle's two
layers one after the other, through small_gap_fc and as small_run_net forms the pair from plain descriptors."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import nets
from synth import configs
from paper_2303_04769_b200 import binding as B
from paper_2303_04769_b200.net import Net
from gpu_util import ctx, dev, to_blk, from_blk, new_blk, rel_err, pad_lanes_are_zero, net_tol

pytestmark = pytest.mark.gpu


def rnd(shape, tid, lo=-1.0, hi=1.0):
    return synth.uniform(shape, lo, hi, tid, seed=909)


def reference(x, w, b, relu):
    N, C, H, W = x.shape
    pooled = oracle.pool2d(x, H, W, 1, (0, 0, 0, 0), mode="avg")           # [N][C][1][1], rounded to float
    return oracle.fc(pooled, w, b, relu=relu)


# (N, C, H, W, K): the three networks' heads, ragged channel and filter counts, planes of one pixel and of more pixels
# than a thread block has warps several times over, more images than resident thread blocks
CASES = [(6, 64, 8, 8, 10), (5, 256, 3, 3, 2), (9, 64, 25, 5, 12), (3, 70, 7, 5, 45), (2, 1, 1, 1, 1), (4, 33, 1, 9, 33),
         (2, 300, 4, 4, 100), (2000, 16, 2, 2, 5)]


@pytest.mark.parametrize("case", CASES)
def test_gap_fc_matches_oracle(case):
    N, C, H, W, K = case
    x, w, b = rnd((N, C, H, W), 1), rnd((K, C), 2), rnd((K,), 3)
    wb = torch.empty(B.small_fc_weight_elems(C, K), device="cuda")
    B.small_pack_fc_weights(ctx(), dev(w), wb, C, K)
    bx = to_blk(x)
    assert B.small_gap_fc_fused(N, C, K, B.MATH_FP32)
    for relu in (False, True):
        out = new_blk(N, K, 1, 1)
        B.small_gap_fc(ctx(), bx, wb, dev(b), out, None, N, C, H, W, K, B.RELU if relu else 0)
        assert rel_err(from_blk(out, N, K, 1, 1).reshape(N, K), reference(x, w, b, relu)) <= 1e-5
        assert pad_lanes_are_zero(out, N, K, 1, 1)
    out = new_blk(N, K, 1, 1)
    B.small_gap_fc(ctx(), bx, wb, None, out, None, N, C, H, W, K, 0)
    assert rel_err(from_blk(out, N, K, 1, 1).reshape(N, K), reference(x, w, None, False)) <= 1e-5
    # the library's own two launches give the same result within rounding of the sums
    mid, two = new_blk(N, C, 1, 1), new_blk(N, K, 1, 1)
    B.small_pool2d(ctx(), bx, mid, None, N, C, H, W, H, W, 1, (0, 0, 0, 0), B.POOL_AVG)
    B.small_fc(ctx(), mid, wb, None, two, N, C, K, 0)
    assert rel_err(from_blk(out, N, K, 1, 1), from_blk(two, N, K, 1, 1)) <= 1e-5
    assert B.small_device_status(ctx()) == 0


def test_large_full_reduction_runs_unfused_through_scratch():
    """A full reduction large enough for the tensor-core route keeps it: the pair runs as two layers through the
    caller's scratch tensor, and without one the call is refused."""
    N, C, H, W, K = 4096, 128, 2, 2, 128
    assert not B.small_gap_fc_fused(N, C, K, B.MATH_TF32) and B.small_gap_fc_fused(N, C, K, B.MATH_FP32)
    x, w, b = rnd((N, C, H, W), 4), rnd((K, C), 5), rnd((K,), 6)
    wb = torch.empty(B.small_fc_weight_elems(C, K, B.MATH_TF32), device="cuda")
    B.small_pack_fc_weights(ctx(), dev(w), wb, C, K, B.MATH_TF32)
    bx, out, scratch = to_blk(x), new_blk(N, K, 1, 1), new_blk(N, C, 1, 1)
    B.small_gap_fc(ctx(), bx, wb, dev(b), out, scratch, N, C, H, W, K, B.MATH_TF32)
    assert rel_err(from_blk(out, N, K, 1, 1).reshape(N, K), reference(x, w, b, False)) <= 2e-3
    with pytest.raises(B.SmallError):
        B.small_gap_fc(ctx(), bx, wb, dev(b), out, None, N, C, H, W, K, B.MATH_TF32)


@pytest.mark.parametrize("math", ["fp32", "3xtf32"])
def test_runner_forms_the_pair(math):
    """small_run_net runs the residual network's average pool and classifier as one launch (one launch fewer than with
    that fusion off) and gives the result of the unfused run within the network tolerance."""
    batch = 8
    net = configs.residual_cnn(batch=batch)
    params = configs.make_params(net)
    x = configs.make_input(net, batch)
    fused, plain = Net(ctx(), net, params, batch=batch, math=math), Net(ctx(), net, params, batch=batch, math=math, fuse_poolfc=False)
    assert fused.launches() == plain.launches() - 1
    in_blk = to_blk(x)
    oc, oh, ow = fused.out_shape
    got = from_blk(fused.run(in_blk), batch, oc, oh, ow)
    want = from_blk(plain.run(in_blk), batch, oc, oh, ow)
    ref = nets.run_net(net, params, x)["out"]
    assert rel_err(got, ref) <= net_tol("residual_cnn", math)
    assert rel_err(got, want) <= 1e-5
    assert B.small_device_status(ctx()) == 0
