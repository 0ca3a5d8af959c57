"""The fused chain of full reductions (small_fc_chain: one kernel, activations resident in shared memory between layers)
against the oracle's layers applied one after the other, in both tensor-core modes, on full, ragged and tiny tiles."""
import numpy as np
import pytest
import torch

import oracle
import synth
from paper_2303_04769_b200 import binding as B
from gpu_util import ctx, dev, to_blk, from_blk, new_blk, rel_err, pad_lanes_are_zero, TOL

pytestmark = pytest.mark.gpu

CASES = [  # widths, N
    ([128, 128, 128], 256),
    ([128, 128, 128, 128, 8, 128, 128, 128, 128], 1000),     # the autoencoder's eight inner layers, ragged last tile
    ([70, 45, 100, 8, 33], 300),                             # ragged widths: partial channel blocks and filter blocks
    ([32, 16, 64], 5),                                       # less than one tile
    ([96, 128, 40, 128, 128, 10], 4096),
    ([640, 128, 128], 300),                                  # wide first layer: its input streams through the operand slots
    ([128, 128, 640], 300),                                  # wide last layer: chunks of 128 filters
    ([300, 64, 200], 260),                                   # both, ragged
    ([640, 128, 128, 128, 128, 8, 128, 128, 128, 128, 640], 1000),    # the whole autoencoder
]


def chain_params(widths, seed):
    ws, bs = [], []
    for i in range(len(widths) - 1):
        ws.append(synth.he_normal((widths[i + 1], widths[i]), widths[i], 300 + 2 * i, seed))
        bs.append(synth.uniform((widths[i + 1],), -0.1, 0.1, 301 + 2 * i, seed))
    return ws, bs


@pytest.mark.parametrize("widths,N", CASES)
@pytest.mark.parametrize("math", ["tf32", "3xtf32"])
def test_fc_chain_matches_the_layers_one_by_one(widths, N, math):
    L = len(widths) - 1
    ws, bs = chain_params(widths, 77)
    relu = [i != L - 1 for i in range(L)]
    x = synth.normal((N, widths[0], 1, 1), 0.0, 1.0, 299, 77)
    ref = x.reshape(N, widths[0])
    for w, b, r in zip(ws, bs, relu):
        ref = oracle.fc(ref, w, b, relu=r)
    assert B.small_fc_chain_fused(widths, B.MATH[math])
    wbs = []
    for i, w in enumerate(ws):
        wb = torch.empty(B.small_fc_weight_elems(widths[i], widths[i + 1], B.MATH[math]), device="cuda")
        B.small_pack_fc_weights(ctx(), dev(w), wb, widths[i], widths[i + 1], B.MATH[math])
        wbs.append(wb)
    dbs = [dev(b) for b in bs]
    bx = to_blk(x)
    out = new_blk(N, widths[-1], 1, 1)
    B.small_fc_chain(ctx(), bx, wbs, dbs, widths, relu, out, None, N, B.MATH[math])
    got = from_blk(out, N, widths[-1], 1, 1).reshape(N, widths[-1])
    assert B.small_device_status(ctx()) == 0
    # a chain compounds each layer's rounding: the bound grows with its length (every single layer meets 1x, test_fc)
    factor = 1.0 if L <= 2 else 2.5
    err = rel_err(got, ref)
    assert err <= factor * TOL[math], err
    if math == "tf32":
        assert err > 1e-7                 # TF32 products: the tensor cores ran
    assert pad_lanes_are_zero(out, N, widths[-1], 1, 1)
    # the same chain layer by layer through scratch (fused kernel switched off by the general-path setting)
    scratch = torch.empty(2 * B.small_packed_elems(N, max(widths[1:-1]), 1, 1), device="cuda")
    two = new_blk(N, widths[-1], 1, 1)
    B.small_set_conv_path(ctx(), "cuda_cores")
    try:
        B.small_fc_chain(ctx(), bx, wbs, dbs, widths, relu, two, scratch, N, B.MATH[math])
    finally:
        B.small_set_conv_path(ctx(), "auto")
    assert rel_err(from_blk(two, N, widths[-1], 1, 1).reshape(N, widths[-1]), ref) <= 1e-5      # FP32 FMAs layer by layer
    # deterministic
    out2 = new_blk(N, widths[-1], 1, 1)
    B.small_fc_chain(ctx(), bx, wbs, dbs, widths, relu, out2, None, N, B.MATH[math])
    assert torch.equal(out.view(torch.int32), out2.view(torch.int32))


def test_fc_chain_falls_back_and_rejects():
    widths = [640, 256, 128]                     # a width between two layers above 128: not one kernel
    assert not B.small_fc_chain_fused(widths, B.MATH_TF32)
    assert not B.small_fc_chain_fused([128] * 14, B.MATH_TF32)       # too long
    assert not B.small_fc_chain_fused([128, 128, 128], B.MATH_FP32)
    N = 64
    ws, bs = chain_params(widths, 78)
    x = synth.normal((N, 640, 1, 1), 0.0, 1.0, 298, 78)
    ref = oracle.fc(oracle.fc(x.reshape(N, 640), ws[0], bs[0], relu=True), ws[1], bs[1])
    assert ref.shape == (N, 128)
    wbs = []
    for i, w in enumerate(ws):
        wb = torch.empty(B.small_fc_weight_elems(widths[i], widths[i + 1], B.MATH_3XTF32), device="cuda")
        B.small_pack_fc_weights(ctx(), dev(w), wb, widths[i], widths[i + 1], B.MATH_3XTF32)
        wbs.append(wb)
    out = new_blk(N, 128, 1, 1)
    with pytest.raises(B.SmallError) as e:
        B.small_fc_chain(ctx(), to_blk(x), wbs, [dev(b) for b in bs], widths, [True, False], out, None, N, B.MATH_3XTF32)
    assert e.value.status == 5                   # scratch needed
    scratch = torch.empty(2 * B.small_packed_elems(N, 256, 1, 1), device="cuda")
    B.small_fc_chain(ctx(), to_blk(x), wbs, [dev(b) for b in bs], widths, [True, False], out, scratch, N, B.MATH_3XTF32)
    assert rel_err(from_blk(out, N, 128, 1, 1).reshape(N, 128), ref) <= 1e-5


@pytest.mark.parametrize("math", ["tf32", "3xtf32"])
def test_fc_chain_tile_sizes_agree(math):
    """Every tile size gives the same bits, on a batch that gives the thread blocks of the smallest tile several tiles
    each (the slots and accumulators are then reused across tiles) and ends in a ragged tile."""
    widths, N = [200, 128, 16, 300], 32 * 148 * 2 + 37
    L = len(widths) - 1
    ws, bs = chain_params(widths, 79)
    relu = [True, True, False]
    x = synth.normal((N, widths[0], 1, 1), 0.0, 1.0, 297, 79)
    ref = x.reshape(N, widths[0])
    for w, b, r in zip(ws, bs, relu):
        ref = oracle.fc(ref, w, b, relu=r)
    wbs = []
    for i, w in enumerate(ws):
        wb = torch.empty(B.small_fc_weight_elems(widths[i], widths[i + 1], B.MATH[math]), device="cuda")
        B.small_pack_fc_weights(ctx(), dev(w), wb, widths[i], widths[i + 1], B.MATH[math])
        wbs.append(wb)
    dbs = [dev(b) for b in bs]
    bx = to_blk(x)
    outs = []
    try:
        for tile in (32, 64, 128, 0):
            B.small_set_fc_chain_tile(ctx(), tile)
            out = new_blk(N, widths[-1], 1, 1)
            B.small_fc_chain(ctx(), bx, wbs, dbs, widths, relu, out, None, N, B.MATH[math])
            assert B.small_device_status(ctx()) == 0
            outs.append(out)
    finally:
        B.small_set_fc_chain_tile(ctx(), 0)
    assert rel_err(from_blk(outs[0], N, widths[-1], 1, 1).reshape(N, widths[-1]), ref) <= 2.5 * TOL[math]
    assert pad_lanes_are_zero(outs[0], N, widths[-1], 1, 1)
    for o in outs[1:]:
        assert torch.equal(o.view(torch.int32), outs[0].view(torch.int32))
    with pytest.raises(B.SmallError):
        B.small_set_fc_chain_tile(ctx(), 48)
