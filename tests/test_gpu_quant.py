"""GPU parity of the quantised layers (uint8 tensors, int32 accumulation) against the oracle's integer definitions:
bit-exact, through the C ABI, on shapes that span several tiles, ragged channel counts, borders on every side, both
strides, small planes with several images per tile, and the degenerate 1 x 1 plane (a fully-connected layer)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2303_04769_b200 import binding as B
from gpu_util import ctx

pytestmark = pytest.mark.gpu


def u8(shape, seed, lo=0, hi=256):
    return np.random.RandomState(seed).randint(lo, hi, size=shape).astype(np.uint8)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def q_blk(x):
    N, C, H, W = x.shape
    blk = torch.full((B.small_q_packed_bytes(N, C, H, W),), 0xAB, dtype=torch.uint8, device="cuda")
    B.small_q_pack(ctx(), dev(x), blk, N, C, H, W)
    return blk


def q_nchw(blk, N, C, H, W):
    out = torch.full((N, C, H, W), 0xCD, dtype=torch.uint8, device="cuda")
    B.small_q_unpack(ctx(), blk, out, N, C, H, W)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def pad_lanes_zero(blk, N, C, H, W):
    cb = (C + 31) // 32
    v = blk.view(N, cb, H, W, 32)[:, -1, :, :, C - (cb - 1) * 32:]
    return v.numel() == 0 or bool((v == 0).all().item())


@pytest.mark.parametrize("shape", [(1, 16, 32, 32), (2, 3, 5, 7), (3, 33, 4, 4), (2, 70, 9, 11), (1, 1, 1, 1)])
def test_q_pack_unpack_are_byte_moves(shape):
    x = u8(shape, 1)
    blk = q_blk(x)
    assert pad_lanes_zero(blk, *shape)
    np.testing.assert_array_equal(q_nchw(blk, *shape), x)
    # the blocked form itself: [N][CB][H][W][32]
    N, C, H, W = shape
    cb = (C + 31) // 32
    ref = np.zeros((N, cb * 32, H, W), dtype=np.uint8)
    ref[:, :C] = x
    ref = ref.reshape(N, cb, 32, H, W).transpose(0, 1, 3, 4, 2)
    np.testing.assert_array_equal(blk.cpu().numpy().reshape(N, cb, H, W, 32), ref)


Q_CONV_CASES = [  # N, C, K, H, W, FH, FW, S, pad
    (1, 16, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),       # the single-convolution workload's shape
    (5, 16, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),       # several row bands and images
    (3, 16, 32, 32, 32, 3, 3, 2, (1, 1, 1, 1)),       # stride 2
    (3, 16, 32, 32, 32, 1, 1, 2, (0, 0, 0, 0)),       # 1x1 stride 2: the copy skips every other pixel
    (4, 32, 32, 16, 16, 3, 3, 1, (1, 1, 1, 1)),
    (9, 64, 64, 8, 8, 3, 3, 1, (1, 1, 1, 1)),         # several images per row warp, two filter tiles of 32
    (7, 64, 64, 25, 5, 1, 1, 1, (0, 0, 0, 0)),        # keyword-spotting 1x1
    (2, 3, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),        # three channels
    (2, 70, 45, 9, 11, 3, 3, 1, (1, 1, 1, 1)),        # ragged channel counts, three channel blocks
    (2, 33, 100, 17, 19, 5, 3, 1, (2, 1, 0, 2)),      # tall window, asymmetric pads
    (2, 5, 10, 40, 70, 3, 3, 2, (0, 1, 1, 0)),        # wide plane: several column tiles
    (3, 40, 8, 7, 7, 3, 1, 1, (1, 1, 0, 0)),          # 3 x 1 window, one filter group
    (37, 128, 10, 1, 1, 1, 1, 1, (0, 0, 0, 0)),       # a fully-connected layer: 1 x 1 plane
    (2, 64, 64, 56, 56, 3, 3, 1, (1, 1, 1, 1)),       # a sweep shape at small batch
]
ZP = [(0, 0, 0), (128, 131, 7), (140, 119, 200)]       # zero points of input, weights, output


def multiplier(n_terms, zx, zw, shift=40):
    """A requantisation multiplier that spreads this reduction's results over the byte range instead of saturating:
    with both zero points 0 the sums sit near n * 127.5^2, otherwise they scatter around 0 with deviation sqrt(n) * 74^2."""
    scale = 128.0 / (n_terms * 16256.0) if (zx == 0 and zw == 0) else 40.0 / (n_terms ** 0.5 * 5476.0)
    return min((1 << 31) - 1, max(1, int(scale * 2.0 ** shift))), shift


@pytest.mark.parametrize("case", Q_CONV_CASES)
def test_q_conv_bit_exact(case):
    N, C, K, H, W, FH, FW, S, pad = case
    x, w = u8((N, C, H, W), 3), u8((K, C, FH, FW), 4)
    b = np.random.RandomState(5).randint(-20000, 20000, size=K).astype(np.int32)
    wb = torch.full((B.small_q_conv_weight_bytes(C, K, FH, FW),), 0x5A, dtype=torch.uint8, device="cuda")
    B.small_q_pack_conv_weights(ctx(), dev(w), wb, C, K, FH, FW)
    bx = q_blk(x)
    for i, (zx, zw, zo) in enumerate(ZP):
        relu, bias = bool(i & 1), (b if i != 2 else None)
        mult_i, shift = multiplier(C * FH * FW, zx, zw)
        ref = oracle.q_conv2d(x, w, bias, S, pad, zx, zw, zo, mult_i, shift, relu)
        OH, OW = ref.shape[2:]
        out = torch.full((B.small_q_packed_bytes(N, K, OH, OW),), 0xEE, dtype=torch.uint8, device="cuda")
        B.small_q_conv2d(ctx(), bx, wb, None if bias is None else dev(bias), out, N, C, K, H, W, FH, FW, S, pad,
                         (zx, zw, zo, mult_i, shift), B.RELU if relu else 0)
        got = q_nchw(out, N, K, OH, OW)
        assert B.small_device_status(ctx()) == 0
        assert len(np.unique(ref)) > 3                      # not a saturated tensor
        np.testing.assert_array_equal(got, ref, err_msg=str((case, i)))
        assert pad_lanes_zero(out, N, K, OH, OW)


@pytest.mark.parametrize("case", [(2, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)), (3, 64, 25, 5, 3, 3, 1, (1, 1, 1, 1)), (2, 70, 9, 11, 3, 3, 2, (1, 1, 1, 1)),
                                  (2, 5, 12, 10, 5, 2, 3, (2, 1, 0, 1)), (4, 8, 48, 48, 3, 3, 2, (1, 1, 1, 1))])
def test_q_depthwise_bit_exact(case):
    N, C, H, W, FH, FW, S, pad = case
    x, w = u8((N, C, H, W), 6), u8((C, FH, FW), 7)
    b = np.random.RandomState(8).randint(-3000, 3000, size=C).astype(np.int32)
    wb = torch.empty(B.small_q_dw_weight_bytes(C, FH, FW), dtype=torch.uint8, device="cuda")
    B.small_q_pack_dw_weights(ctx(), dev(w), wb, C, FH, FW)
    bx = q_blk(x)
    for zx, zw, zo, mult, shift, relu in [(0, 0, 0, 1 << 19, 30, False), (120, 131, 90, 1518500250, 43, True)]:
        ref = oracle.q_dwconv2d(x, w, b, S, pad, zx, zw, zo, mult, shift, relu)
        OH, OW = ref.shape[2:]
        out = torch.full((B.small_q_packed_bytes(N, C, OH, OW),), 0xEE, dtype=torch.uint8, device="cuda")
        B.small_q_dwconv2d(ctx(), bx, wb, dev(b), out, N, C, H, W, FH, FW, S, pad, (zx, zw, zo, mult, shift), B.RELU if relu else 0)
        np.testing.assert_array_equal(q_nchw(out, N, C, OH, OW), ref)
        assert pad_lanes_zero(out, N, C, OH, OW)


@pytest.mark.parametrize("case", [(2, 16, 32, 32, 2, 2, 2, (0, 0, 0, 0)), (3, 70, 7, 7, 2, 2, 2, (0, 0, 0, 0)), (2, 33, 9, 8, 3, 3, 2, (1, 1, 1, 1)),
                                  (1, 5, 6, 6, 3, 2, 1, (2, 0, 0, 1))])
def test_q_maxpool_and_relu_bit_exact(case):
    N, C, H, W, FH, FW, S, pad = case
    x = u8((N, C, H, W), 9)
    bx = q_blk(x)
    z = 77
    ref = oracle.q_maxpool2d(x, FH, FW, S, pad, z)
    OH, OW = ref.shape[2:]
    out = torch.full((B.small_q_packed_bytes(N, C, OH, OW),), 0xEE, dtype=torch.uint8, device="cuda")
    B.small_q_maxpool2d(ctx(), bx, out, N, C, H, W, FH, FW, S, pad, z)
    np.testing.assert_array_equal(q_nchw(out, N, C, OH, OW), ref)
    assert pad_lanes_zero(out, N, C, OH, OW)
    r = torch.full_like(bx, 0xEE)
    B.small_q_relu(ctx(), bx, r, N, C, H, W, z)
    np.testing.assert_array_equal(q_nchw(r, N, C, H, W), oracle.q_relu(x, z))
    assert pad_lanes_zero(r, N, C, H, W)
    B.small_q_relu(ctx(), bx, bx, N, C, H, W, z)            # in place
    assert torch.equal(bx, r)


def test_quantised_single_conv_workload_and_errors():
    """The single-convolution workload's shape in uint8: 3x3 convolution + ReLU, then 2x2 stride-2 max pool."""
    N, C, K, H, W = 1, 16, 16, 32, 32
    x, w = u8((N, C, H, W), 10), u8((K, C, 3, 3), 11)
    b = np.random.RandomState(12).randint(-9000, 9000, size=K).astype(np.int32)
    qp = (128, 128, 30, 1518500250, 48)
    wb = torch.empty(B.small_q_conv_weight_bytes(C, K, 3, 3), dtype=torch.uint8, device="cuda")
    B.small_q_pack_conv_weights(ctx(), dev(w), wb, C, K, 3, 3)
    bx = q_blk(x)
    mid = torch.empty(B.small_q_packed_bytes(N, K, H, W), dtype=torch.uint8, device="cuda")
    out = torch.empty(B.small_q_packed_bytes(N, K, 16, 16), dtype=torch.uint8, device="cuda")
    B.small_q_conv2d(ctx(), bx, wb, dev(b), mid, N, C, K, H, W, 3, 3, 1, (1, 1, 1, 1), qp, B.RELU)
    B.small_q_maxpool2d(ctx(), mid, out, N, K, H, W, 2, 2, 2, (0, 0, 0, 0), qp[2])
    ref = oracle.q_maxpool2d(oracle.q_conv2d(x, w, b, 1, (1, 1, 1, 1), *qp, relu=True), 2, 2, 2, (0, 0, 0, 0), qp[2])
    np.testing.assert_array_equal(q_nchw(out, N, K, 16, 16), ref)
    L, c, st = B.lib(), ctx(), torch.cuda.current_stream().cuda_stream
    args = (N, C, K, H, W, 3, 3, 1, 1, 1, 1, 1)
    assert L.small_q_conv2d(c, bx.data_ptr(), wb.data_ptr(), None, mid.data_ptr(), *args, 128, 128, 30, 1, 0, 0, st) == 1     # shift 0
    assert L.small_q_conv2d(c, bx.data_ptr(), wb.data_ptr(), None, mid.data_ptr(), *args, 256, 128, 30, 1, 30, 0, st) == 1   # zero point out of range
    assert L.small_q_conv2d(c, bx.data_ptr(), wb.data_ptr(), None, mid.data_ptr(), *args, 1, 1, 1, 1, 30, 2, st) == 1        # accumulate is not a quantised flag
    assert L.small_q_conv2d(c, bx.data_ptr(), wb.data_ptr(), None, bx.data_ptr(), *args, 1, 1, 1, 1, 30, 0, st) == 4         # in place
    assert L.small_q_conv2d(c, bx.data_ptr(), wb.data_ptr(), None, mid.data_ptr(), N, C, K, H, W, 5, 5, 1, 2, 2, 2, 2, 1, 1, 1, 1, 30, 0, st) == 6   # 5-wide window
    assert L.small_q_conv2d(c, bx.data_ptr(), wb.data_ptr(), None, mid.data_ptr(), N, 4000, K, 4, 4, 3, 3, 1, 1, 1, 1, 1, 1, 1, 1, 1, 30, 0, st) == 2   # sums could leave 32 bits
    torch.cuda.synchronize()
    assert B.small_device_status(ctx()) == 0
