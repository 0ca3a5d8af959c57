"""GPU parity of the four network workloads (reduced batch) against the oracle: every intermediate the network
produces and the final result, through small_run_net, and end to end from host buffers through small_run_net_host."""
import numpy as np
import pytest
import torch

from oracle import nets
from synth import configs
from paper_2303_04769_b200 import binding as B
from paper_2303_04769_b200.net import Net
from gpu_util import ctx, to_blk, from_blk, rel_l2

pytestmark = pytest.mark.gpu
TOL = {"fp32": 1e-5, "3xtf32": 1e-5, "tf32": 2e-3}

CASES = [("single_conv_pool", 1), ("residual_cnn", 4), ("dwsep_cnn", 2), ("kws_cnn", 8),
         ("autoencoder_fc", 64), ("autoencoder_fc", 300)]      # 300 images: a full strip of 256 and a ragged one


@pytest.mark.parametrize("name,batch", CASES)
@pytest.mark.parametrize("math", ["fp32", "tf32", "3xtf32"])
def test_network_matches_oracle_layer_by_layer(name, batch, math):
    net = configs.NETWORKS[name]() if name == "single_conv_pool" else configs.NETWORKS[name](batch=batch)
    params = configs.make_params(net)
    x = configs.make_input(net, batch)
    ref = nets.run_net(net, params, x)
    gnet = Net(ctx(), net, params, batch=batch, math=math, fuse_dwpw="all")     # every pair the fused kernel takes
    in_blk = to_blk(x)
    tol = TOL[math]
    # prefixes of the layer list: the tensor each layer has just written is checked before a later layer reuses its slot
    for i, row in enumerate(gnet.layer_rows):
        if row["dst"] == "out":
            continue
        # a prefix cannot end on an accumulate target that the oracle dict has since overwritten: recompute the oracle prefix
        upto = row["upto"]          # configuration layers this descriptor completes (two for a fused depthwise + 1x1 pair)
        sub = dict(net, layers=net["layers"][:upto])
        ref_i = nets.run_net(sub, params[:upto], x)[row["dst"]]
        gnet.run(in_blk, n_layers=i + 1)
        got = from_blk(gnet.slot_tensor(row["dst"]), batch, row["K"], row["OH"], row["OW"])
        assert rel_l2(got, ref_i) <= tol * (1 + i), (row["name"], rel_l2(got, ref_i))
    out = gnet.run(in_blk)
    oc, oh, ow = gnet.out_shape
    got = from_blk(out, batch, oc, oh, ow)
    assert got.shape == ref["out"].shape
    err = rel_l2(got, ref["out"])
    assert err <= tol * 4, err   # error compounds over up to 28 layers; each layer alone meets `tol` (test_gpu_layers)
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
    assert rel_l2(out_host.numpy(), ref) <= 4e-5
    # same result as the device-resident call
    got = from_blk(gnet.run(to_blk(x)), 8, 10, 1, 1)
    np.testing.assert_array_equal(got, out_host.numpy())


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
