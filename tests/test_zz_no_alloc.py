"""small_run_net_static - the network runner for callers that cannot allocate device memory (their memory belongs
to another allocator, or an allocation's device-wide stall is not acceptable where they call from) - must give
exactly what small_run_net gives with a caller workspace, and must itself take no device memory.  Collected last on
purpose (file name), so a run that stops at the first failure has already run every other test.  Passes alone in a
fresh process and after the others."""
import pytest
import torch

from synth import configs
from paper_2303_04769_b200 import binding as B
from paper_2303_04769_b200.net import Net
from gpu_util import ctx, to_blk

pytestmark = pytest.mark.gpu


def test_static_workspace_matches_caller_workspace_twice_in_a_row():
    batch = 8
    # another network through the same array first: what it leaves there has a different layout than anything the
    # network under test writes, so a layer that read a stale byte would not find a plausible value
    other = configs.autoencoder_fc(batch=64)
    onet = Net(ctx(), other, configs.make_params(other), batch=64)
    oin = to_blk(configs.make_input(other, 64))
    want_o = onet.run(oin).clone()
    got_o = torch.full_like(want_o, float("nan"))
    B.small_run_net_static(ctx(), onet.layers, 64, oin, got_o)
    assert torch.equal(got_o, want_o)
    net = configs.kws_cnn(batch=batch)
    gnet = Net(ctx(), net, configs.make_params(net))
    assert 0 < gnet.ws_bytes <= B.small_static_workspace_bytes() == 32 << 20
    for call, seed in enumerate((11, 12)):          # two calls in a row, different inputs: the second one finds
        x = configs.make_input(net, batch, seed=seed)   # the first one's leftovers in the shared array
        in_blk = to_blk(x)
        want = gnet.run(in_blk).clone()                                  # existing entry point, caller's workspace (also warms the kernels)
        got = torch.full_like(want, float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.small_run_net_static(ctx(), gnet.layers, batch, in_blk, got)   # new entry point, built-in workspace
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, call         # the call took no device memory
        assert torch.equal(got, want), call                              # same kernels, same inputs: the same bits
    assert B.small_device_status(ctx()) == 0


def test_static_workspace_rejects_what_does_not_fit():
    net = configs.residual_cnn(batch=256)               # three 32 MiB activation slots: too large for the array
    gnet = Net(ctx(), net, configs.make_params(net))
    assert gnet.ws_bytes > B.small_static_workspace_bytes()
    x = torch.zeros(B.small_packed_elems(256, 3, 32, 32), device="cuda")
    out = torch.full((B.small_packed_elems(256, 10, 1, 1),), 7.0, device="cuda")
    with pytest.raises(B.SmallError) as e:
        B.small_run_net_static(ctx(), gnet.layers, 256, x, out)
    assert e.value.status == 5                          # SMALL_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())                     # nothing was launched
