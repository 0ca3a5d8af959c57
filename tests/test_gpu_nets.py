"""GPU parity of the network workloads (reduced batch) against the oracle: every layer on the tensor the GPU fed it
and the final result, through small_run_net, and end to end from host buffers through small_run_net_host.  Float
results are bounded in relative L2 norm and element by element (gpu_util.rel_err)."""
import numpy as np
import pytest
import torch

from oracle import nets
from synth import configs
from paper_2303_04769_b200 import binding as B
from paper_2303_04769_b200.net import Net
from gpu_util import ctx, to_blk, from_blk, rel_err, TOL, net_tol

pytestmark = pytest.mark.gpu

CASES = [("single_conv_pool", 1), ("residual_cnn", 4), ("dwsep_cnn", 2), ("kws_cnn", 8),
         ("autoencoder_fc", 64), ("autoencoder_fc", 300)]      # 300 images: a full strip of 256 and a ragged one


@pytest.mark.parametrize("name,batch", CASES)
@pytest.mark.parametrize("math", ["fp32", "tf32", "3xtf32"])
def test_network_matches_oracle_layer_by_layer(name, batch, math):
    """Every layer at the mode's tolerance against the oracle applied to the tensor the GPU fed that layer (so a
    layer's own error is not mixed with what came before it), and the network's result at the network tolerance
    against the oracle run from the input."""
    net = configs.NETWORKS[name]() if name == "single_conv_pool" else configs.NETWORKS[name](batch=batch)
    params = configs.make_params(net)
    x = configs.make_input(net, batch)
    gnet = Net(ctx(), net, params, batch=batch, math=math, fuse_dwpw="all")     # every pair the fused kernel takes
    in_blk = to_blk(x)
    tol = TOL[math]
    oc, oh, ow = gnet.out_shape

    def gpu_tensor(tname):
        if tname == "in":
            return x
        if tname == "out":
            return from_blk(gnet.out_blk, batch, oc, oh, ow)
        c, h, w = gnet.dims[tname]
        return from_blk(gnet.slot_tensor(tname), batch, c, h, w)

    worst = 0.0
    for i, row in enumerate(gnet.layer_rows):
        first, upto = row["first"], row["upto"]     # configuration layers this descriptor covers (two for a fused pair)
        sub_layers = [dict(L) for L in net["layers"][first:upto]]
        # what the GPU hands this layer: its source, and for an accumulating layer the tensor already in its target
        if i > 0:
            gnet.run(in_blk, n_layers=i)
        src = gpu_tensor(sub_layers[0]["src"])
        init = {}
        if sub_layers[-1].get("accumulate"):
            init[sub_layers[-1]["dst"]] = gpu_tensor(sub_layers[-1]["dst"])
        gnet.run(in_blk, n_layers=i + 1)
        got = gpu_tensor(row["dst"])
        sub_layers[0]["src"] = "in"
        ref_i = nets.run_net(dict(net, layers=sub_layers), params[first:upto], src, init=init)[row["dst"]]
        err = rel_err(got, ref_i)
        worst = max(worst, err)
        assert err <= tol, (row["name"], err)
    out = gnet.run(in_blk)
    got = from_blk(out, batch, oc, oh, ow)
    ref = nets.run_net(net, params, x)["out"]
    assert got.shape == ref.shape
    err = rel_err(got, ref)
    print(f"network error {name} batch {batch} {math}: result {err:.3e} (tolerance {net_tol(name, math):.1e}), worst single layer {worst:.3e} (tolerance {tol:.1e})")
    assert err <= net_tol(name, math), err
    assert B.small_device_status(ctx()) == 0


@pytest.mark.parametrize("name,batch", [("residual_cnn", 96), ("dwsep_cnn", 24), ("kws_cnn", 200), ("autoencoder_fc", 1500)])
@pytest.mark.parametrize("math", ["fp32", "tf32", "3xtf32"])
def test_layer_overlap_changes_no_bit(name, batch, math):
    """Layers launched as dependent launches (the default) give exactly the tensor that fully serialised launches
    give, run after run, eagerly and replayed from a CUDA graph: a layer that read or wrote a tensor before the layer
    in front of it had finished would show up here.  The batch is large enough for several tiles per SM."""
    net = configs.NETWORKS[name](batch=batch)
    params = configs.make_params(net)
    in_blk = to_blk(configs.make_input(net, batch))
    try:
        B.small_set_layer_overlap(ctx(), 0)
        want = Net(ctx(), net, params, batch=batch, math=math).run(in_blk).clone()
        B.small_set_layer_overlap(ctx(), 1)
        gnet = Net(ctx(), net, params, batch=batch, math=math)
        for _ in range(3):
            assert torch.equal(gnet.run(in_blk), want)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            out = gnet.run(in_blk)
        for _ in range(5):
            out.fill_(float("nan"))
            g.replay()
            assert torch.equal(out, want)
    finally:
        B.small_set_layer_overlap(ctx(), 1)
    assert B.small_device_status(ctx()) == 0


@pytest.mark.parametrize("math", ["fp32", "tf32", "3xtf32"])
def test_branch_overlap_changes_no_bit(math):
    """A residual stage's shortcut convolution runs on the context's side stream next to the stage's first convolution:
    the result must be the one that strictly consecutive launches give, eagerly and replayed from a CUDA graph."""
    batch = 96
    net = configs.residual_cnn(batch=batch)
    params = configs.make_params(net)
    in_blk = to_blk(configs.make_input(net, batch))
    gnet = Net(ctx(), net, params, batch=batch, math=math)
    try:
        B.small_set_branch_overlap(ctx(), 0)
        want = gnet.run(in_blk).clone()
        B.small_set_branch_overlap(ctx(), 1)
        for _ in range(3):
            assert torch.equal(gnet.run(in_blk), want)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            out = gnet.run(in_blk)
        for _ in range(5):
            out.fill_(float("nan"))
            g.replay()
            assert torch.equal(out, want)
    finally:
        B.small_set_branch_overlap(ctx(), 1)
    assert B.small_device_status(ctx()) == 0


def test_the_runner_fuses_plain_descriptors_itself():
    """Plain layer descriptors through the C ABI: small_run_net decides which neighbours run as one fused layer.  The launch
    counts it reports follow the fusion setting, and the results stay the same within the mode's tolerance."""
    c = ctx()
    net = configs.dwsep_cnn(batch=2)
    params = configs.make_params(net)
    x = configs.make_input(net, 2)
    ref = nets.run_net(net, params, x)["out"]
    gnet = Net(c, net, params, batch=2, math="tf32")
    n_layers = len(gnet.layers)
    assert n_layers == len(net["layers"]) == 29          # every descriptor is a plain layer
    in_blk = to_blk(x)
    counts = {}
    for mask in (0, B.FUSE_DWPW, B.FUSE_DWPW | B.FUSE_DWPW_ALWAYS, B.FUSE_DEFAULT):
        B.small_set_net_fusion(c, mask)
        try:
            counts[mask] = B.small_net_launches(c, gnet.layers, 2)
            out = torch.full_like(gnet.out_blk, float("nan"))
            B.small_run_net(c, gnet.layers, 2, in_blk, out, gnet.workspace, gnet.ws_bytes)
        finally:
            B.small_set_net_fusion(c, B.FUSE_DEFAULT)
        assert rel_err(from_blk(out, 2, 2, 1, 1), ref) <= net_tol("dwsep_cnn", "tf32")
    assert counts[0] == 29
    assert counts[B.FUSE_DWPW] == 29 - 13        # all thirteen depthwise / 1x1 pairs at this batch
    assert counts[B.FUSE_DEFAULT] == 29 - 13 - 1     # and the average pool with the classifier behind it
    assert counts[B.FUSE_DWPW | B.FUSE_DWPW_ALWAYS] == 16
    # in FP32 mode only the classifier head of this network fuses; the single-convolution workload is one launch in every mode
    assert Net(c, net, params, batch=2, math="fp32").launches() == 28
    one = configs.single_conv_pool()
    assert Net(c, one, configs.make_params(one), math="3xtf32").launches() == 1
    assert Net(c, one, configs.make_params(one), math="3xtf32", fuse_convpool=False).launches() == 2
    # a full reduction under a tensor-core mode is routed by the library, not by the caller
    assert B.small_fc_uses_tensor_cores(4096, 128, 128, B.MATH_TF32) and not B.small_fc_uses_tensor_cores(256, 64, 10, B.MATH_TF32)
    with pytest.raises(B.SmallError):
        B.small_set_net_fusion(c, 32)
    assert B.small_device_status(c) == 0


def test_run_net_host_end_to_end():
    net = configs.residual_cnn(batch=8)
    params = configs.make_params(net)
    x = configs.make_input(net)
    ref = nets.run_net(net, params, x)["out"]
    gnet = Net(ctx(), net, params)
    in_host = torch.from_numpy(x).pin_memory()
    out_host = torch.empty((8, 10, 1, 1)).pin_memory()
    gnet.run_host(in_host, out_host)
    torch.cuda.synchronize()
    assert rel_err(out_host.numpy(), ref) <= 1e-5
    # same result as the device-resident call
    got = from_blk(gnet.run(to_blk(x)), 8, 10, 1, 1)
    np.testing.assert_array_equal(got, out_host.numpy())
    # back-to-back calls: the input copy of a call runs while the call before it computes, through two staging areas;
    # every call must still see its own input (five calls: each staging area is reused)
    xs = [configs.make_input(net, 8, seed=100 + i) for i in range(5)]
    ins = [torch.from_numpy(a).pin_memory() for a in xs]
    outs = [torch.full((8, 10, 1, 1), float("nan")).pin_memory() for _ in xs]
    for a, o in zip(ins, outs):
        gnet.run_host(a, o)
    torch.cuda.synchronize()
    for a, o in zip(xs, outs):
        np.testing.assert_array_equal(o.numpy(), from_blk(gnet.run(to_blk(a)), 8, 10, 1, 1))


def test_run_net_rejects_bad_workspace_and_descriptors():
    net = configs.kws_cnn(batch=2)
    gnet = Net(ctx(), net, configs.make_params(net))
    x = to_blk(configs.make_input(net))
    L = B.lib()
    st = torch.cuda.current_stream().cuda_stream
    args = (ctx(), gnet.layers, len(gnet.layers), 2, x.data_ptr(), gnet.out_blk.data_ptr(), gnet.workspace.data_ptr())
    assert L.small_run_net(*args, gnet.ws_bytes, st) == 0
    assert L.small_run_net(*args, gnet.ws_bytes - 256, st) == 5          # workspace too small
    assert L.small_run_net(ctx(), gnet.layers, len(gnet.layers), 2, x.data_ptr(), gnet.out_blk.data_ptr(),
                           gnet.workspace.data_ptr() + 16, gnet.ws_bytes, st) == 3   # workspace misaligned
    bad = (B.small_layer * len(gnet.layers))(*gnet.layers)
    bad[3].w_blk = None
    assert L.small_run_net(ctx(), bad, len(bad), 2, x.data_ptr(), gnet.out_blk.data_ptr(), gnet.workspace.data_ptr(),
                           gnet.ws_bytes, st) == 1
    torch.cuda.synchronize()
