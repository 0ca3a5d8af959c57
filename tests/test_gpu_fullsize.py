"""Parity at the full workload sizes, in the launch configuration bench.py times.  The whole batch runs on the GPU;
images are independent (batch is only an outer dimension of every layer), so the oracle computes a sample of images
one by one and those rows of the GPU result are compared with them, in relative L2 norm and element by element
(gpu_util.rel_err)."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import nets
from synth import configs
from paper_2303_04769_b200 import binding as B
from paper_2303_04769_b200.net import Net
from gpu_util import ctx, dev, to_blk, from_blk, new_blk, rel_err, pad_lanes_are_zero, TOL, net_tol

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("math", ["3xtf32", "tf32", "fp32"])
def test_residual_cnn_batch_256_sampled_images(math):
    net = configs.residual_cnn()                      # batch 256: the benchmark's step
    N = net["batch"]
    params = configs.make_params(net)
    x = configs.make_input(net, N)
    gnet = Net(ctx(), net, params, math=math)
    out = gnet.run(to_blk(x))
    oc, oh, ow = gnet.out_shape
    got = from_blk(out, N, oc, oh, ow)
    assert B.small_device_status(ctx()) == 0
    sample = [0, 1, 97, 128, 255]
    ref = nets.run_net(net, params, x[sample])["out"]
    assert rel_err(got[sample], ref) <= net_tol("residual_cnn", math)
    for j, n in enumerate(sample):                    # each sampled image on its own, not only in the mean
        assert rel_err(got[n], ref[j]) <= net_tol("residual_cnn", math), n


@pytest.mark.parametrize("name,sample", [("kws_cnn", [0, 6, 7, 511, 1021, 1023]), ("dwsep_cnn", [0, 31, 63]),
                                         ("autoencoder_fc", [0, 255, 256, 4095])])
@pytest.mark.parametrize("math", ["3xtf32", "tf32", "fp32"])
def test_other_networks_full_batch_sampled_images(name, sample, math):
    """The other network workloads the benchmark reports, at their full batch and with the benchmark's layer
    fusion: images from the first, a middle and the ragged last tile against the oracle."""
    net = configs.NETWORKS[name]()
    N = net["batch"]
    params = configs.make_params(net)
    x = configs.make_input(net, N)
    gnet = Net(ctx(), net, params, math=math)
    out = gnet.run(to_blk(x))
    oc, oh, ow = gnet.out_shape
    got = from_blk(out, N, oc, oh, ow)
    assert B.small_device_status(ctx()) == 0
    ref = nets.run_net(net, params, x[sample])["out"]
    assert rel_err(got[sample], ref) <= net_tol(name, math)
    for j, n in enumerate(sample):
        assert rel_err(got[n], ref[j]) <= net_tol(name, math), n


SWEEP = [(C, HW) for C, HW in configs.SWEEP_SIZES]


@pytest.mark.parametrize("C,HW", SWEEP)
def test_sweep_layers_batch_128_sampled_images(C, HW):
    N = configs.SWEEP_BATCH
    x = synth.uniform((N, C, HW, HW), -1.0, 1.0, 500 + C)
    bias = synth.uniform((C,), -1.0, 1.0, 600 + C)
    bx = to_blk(x)
    sample = [0, 63, N - 1]
    xs = x[sample]
    for F, pad in ((3, (1, 1, 1, 1)), (1, (0, 0, 0, 0))):
        w = synth.uniform((C, C, F, F), -1.0, 1.0, 700 + C + F)
        wb = torch.empty(B.small_conv_weight_elems(C, C, F, F, B.MATH_3XTF32), device="cuda")
        B.small_pack_conv_weights(ctx(), dev(w), wb, C, C, F, F, B.MATH_3XTF32)
        ref = oracle.conv2d(xs, w, bias, 1, pad, relu=True)
        for math in ("tf32", "3xtf32"):
            out = new_blk(N, C, HW, HW)
            B.small_conv2d(ctx(), bx, wb, dev(bias), out, N, C, C, HW, HW, F, F, 1, pad, B.RELU | B.MATH[math])
            got = from_blk(out, N, C, HW, HW)
            assert B.small_device_status(ctx()) == 0
            assert rel_err(got[sample], ref) <= TOL[math], (F, math)
            assert pad_lanes_are_zero(out, N, C, HW, HW)
    wd = synth.uniform((C, 3, 3), -1.0, 1.0, 800 + C)
    wdb = torch.empty(B.small_dw_weight_elems(C, 3, 3), device="cuda")
    B.small_pack_dw_weights(ctx(), dev(wd), wdb, C, 3, 3)
    out = new_blk(N, C, HW, HW)
    B.small_dwconv2d(ctx(), bx, wdb, dev(bias), out, N, C, HW, HW, 3, 3, 1, (1, 1, 1, 1), B.RELU)
    assert rel_err(from_blk(out, N, C, HW, HW)[sample], oracle.dwconv2d(xs, wd, bias, 1, (1, 1, 1, 1), relu=True)) <= 1e-5
    OHW = (HW - 2) // 2 + 1
    out = new_blk(N, C, OHW, OHW)
    idx = torch.full((B.small_packed_elems(N, C, OHW, OHW),), -1, dtype=torch.int32, device="cuda")
    B.small_pool2d(ctx(), bx, out, idx, N, C, HW, HW, 2, 2, 2, (0, 0, 0, 0), B.POOL_MAX)
    ref_v, ref_i = oracle.pool2d(xs, 2, 2, 2, mode="max", with_indices=True)
    got_v = from_blk(out, N, C, OHW, OHW)[sample]
    assert np.array_equal(got_v.view(np.int32), ref_v.view(np.int32))          # values bit-exact
    got_i = from_blk(idx.view(torch.float32), N, C, OHW, OHW)[sample].view(np.int32)
    assert np.array_equal(got_i, ref_i)                                          # indices bit-exact
    out = new_blk(N, C, HW, HW)
    B.small_relu(ctx(), bx, out, N, C, HW, HW)
    assert np.array_equal(from_blk(out, N, C, HW, HW)[sample].view(np.int32), oracle.relu(xs).view(np.int32))
