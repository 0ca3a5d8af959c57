"""GPU parity: every layer of the C ABI against the CPU oracle, element by element, on seeded inputs.
Tolerances (relative L2 over the whole output): FP32 CUDA-core path 1e-5; moves, ReLU, max-pool values and
indices bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import synth
from paper_2303_04769_b200 import binding as B
from gpu_util import ctx, dev, to_blk, from_blk, new_blk, rel_err, pad_lanes_are_zero, conv_path, runs_on_tensor_cores

pytestmark = pytest.mark.gpu
TOL_FP32 = 1e-5


def rnd(shape, tid, lo=-1.0, hi=1.0):
    return synth.uniform(shape, lo, hi, tid, seed=4242)


@pytest.mark.parametrize("shape", [(1, 16, 32, 32), (2, 3, 5, 7), (3, 33, 4, 4), (2, 70, 9, 11), (5, 1, 49, 10),
                                   (4, 64, 1, 1), (2, 32, 33, 31), (1, 129, 1, 3)])
def test_pack_unpack_bit_exact(shape):
    N, C, H, W = shape
    x = rnd(shape, 1)
    blk = to_blk(x)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(blk.cpu().numpy().view(np.int32), oracle.pack(x, 32).view(np.int32))
    np.testing.assert_array_equal(from_blk(blk, N, C, H, W).view(np.int32), x.view(np.int32))
    assert pad_lanes_are_zero(blk, N, C, H, W)


@pytest.mark.parametrize("shape", [(2, 16, 9, 7), (3, 40, 5, 5), (1, 64, 56, 56)])
def test_relu_and_add_bit_exact(shape):
    N, C, H, W = shape
    x, y = rnd(shape, 2), rnd(shape, 3)
    x.ravel()[:4] = [0.0, -0.0, 1e-40, -1e-40]
    bx, by = to_blk(x), to_blk(y)
    out = new_blk(N, C, H, W)
    B.small_relu(ctx(), bx, out, N, C, H, W)
    got = from_blk(out, N, C, H, W)
    np.testing.assert_array_equal(got.view(np.int32), oracle.relu(x).view(np.int32))
    assert pad_lanes_are_zero(out, N, C, H, W)
    B.small_add(ctx(), bx, by, out, N, C, H, W, B.RELU)
    np.testing.assert_array_equal(from_blk(out, N, C, H, W), oracle.add(x, y, relu=True))
    B.small_add(ctx(), bx, by, out, N, C, H, W, 0)
    np.testing.assert_array_equal(from_blk(out, N, C, H, W), oracle.add(x, y))
    B.small_relu(ctx(), bx, bx, N, C, H, W)   # in place
    np.testing.assert_array_equal(from_blk(bx, N, C, H, W), oracle.relu(x))


POOL_CASES = [  # N, C, H, W, FH, FW, S, pad
    (1, 16, 32, 32, 2, 2, 2, (0, 0, 0, 0)),
    (2, 40, 7, 7, 2, 2, 2, (0, 0, 0, 0)),      # 7 -> 3: last row and column dropped
    (2, 3, 9, 8, 3, 3, 2, (1, 1, 1, 1)),
    (1, 33, 6, 11, 3, 2, 1, (2, 0, 1, 1)),
    (3, 64, 8, 8, 8, 8, 1, (0, 0, 0, 0)),      # whole plane
    (2, 64, 25, 5, 25, 5, 1, (0, 0, 0, 0)),
    (2, 5, 5, 5, 1, 1, 1, (0, 0, 0, 0)),
]


@pytest.mark.parametrize("case", POOL_CASES)
def test_max_pool_values_and_indices_bit_exact(case):
    N, C, H, W, FH, FW, S, pad = case
    x = rnd((N, C, H, W), 4)
    x[0, 0, :2, :2] = 0.5   # ties: the first maximum of the row-major scan must win
    ref, ridx = oracle.pool2d(x, FH, FW, S, pad, "max", with_indices=True)
    OH, OW = ref.shape[2:]
    out = new_blk(N, C, OH, OW)
    idx = torch.full((B.small_packed_elems(N, C, OH, OW),), -7, dtype=torch.int32, device="cuda")
    B.small_pool2d(ctx(), to_blk(x), out, idx, N, C, H, W, FH, FW, S, pad, B.POOL_MAX)
    np.testing.assert_array_equal(from_blk(out, N, C, OH, OW).view(np.int32), ref.view(np.int32))
    got_idx = from_blk(idx.view(torch.float32), N, C, OH, OW).view(np.int32)
    np.testing.assert_array_equal(got_idx, ridx)
    assert pad_lanes_are_zero(out, N, C, OH, OW) and pad_lanes_are_zero(idx.view(torch.float32), N, C, OH, OW)
    out2 = new_blk(N, C, OH, OW)
    B.small_pool2d(ctx(), to_blk(x), out2, None, N, C, H, W, FH, FW, S, pad, B.POOL_MAX)
    assert torch.equal(out.view(torch.int32), out2.view(torch.int32))


@pytest.mark.parametrize("case", POOL_CASES)
def test_avg_pool(case):
    N, C, H, W, FH, FW, S, pad = case
    x = rnd((N, C, H, W), 5)
    ref = oracle.pool2d(x, FH, FW, S, pad, "avg")
    OH, OW = ref.shape[2:]
    out = new_blk(N, C, OH, OW)
    B.small_pool2d(ctx(), to_blk(x), out, None, N, C, H, W, FH, FW, S, pad, B.POOL_AVG)
    assert rel_err(from_blk(out, N, C, OH, OW), ref) <= 2e-6
    assert pad_lanes_are_zero(out, N, C, OH, OW)


DW_CASES = [  # N, C, H, W, FH, FW, S, pad
    (2, 64, 25, 5, 3, 3, 1, (1, 1, 1, 1)),
    (2, 8, 48, 48, 3, 3, 1, (1, 1, 1, 1)),
    (2, 16, 48, 48, 3, 3, 2, (1, 1, 1, 1)),
    (1, 128, 6, 6, 3, 3, 1, (1, 1, 1, 1)),
    (3, 256, 3, 3, 3, 3, 1, (1, 1, 1, 1)),
    (2, 70, 9, 11, 3, 3, 2, (1, 1, 1, 1)),
    (1, 33, 17, 13, 5, 3, 1, (2, 1, 0, 2)),
    (2, 64, 56, 56, 3, 3, 1, (1, 1, 1, 1)),
    (1, 40, 7, 9, 2, 4, 3, (0, 1, 3, 0)),
    (1, 32, 1, 1, 3, 3, 1, (1, 1, 1, 1)),
    (2, 96, 14, 14, 3, 3, 1, (0, 0, 0, 0)),
]


@pytest.mark.parametrize("case", DW_CASES)
@pytest.mark.parametrize("relu", [False, True])
def test_depthwise(case, relu):
    N, C, H, W, FH, FW, S, pad = case
    x, w, b = rnd((N, C, H, W), 6), rnd((C, FH, FW), 7), rnd((C,), 8)
    ref = oracle.dwconv2d(x, w, b, S, pad, relu)
    OH, OW = ref.shape[2:]
    wb = torch.empty(B.small_dw_weight_elems(C, FH, FW), device="cuda")
    B.small_pack_dw_weights(ctx(), dev(w), wb, C, FH, FW)
    out = new_blk(N, C, OH, OW)
    B.small_dwconv2d(ctx(), to_blk(x), wb, dev(b), out, N, C, H, W, FH, FW, S, pad, B.RELU if relu else 0)
    assert rel_err(from_blk(out, N, C, OH, OW), ref) <= TOL_FP32
    assert pad_lanes_are_zero(out, N, C, OH, OW)
    if not relu:
        B.small_dwconv2d(ctx(), to_blk(x), wb, None, out, N, C, H, W, FH, FW, S, pad, 0)
        assert rel_err(from_blk(out, N, C, OH, OW), oracle.dwconv2d(x, w, None, S, pad)) <= TOL_FP32


CONV_CASES = [  # N, C, K, H, W, FH, FW, S, pad
    (1, 16, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),      # the single-conv workload
    (2, 3, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),       # 3-channel stem
    (2, 16, 32, 32, 32, 3, 3, 2, (1, 1, 1, 1)),      # stride 2
    (2, 16, 32, 32, 32, 1, 1, 2, (0, 0, 0, 0)),      # 1x1 stride-2 shortcut
    (2, 64, 64, 8, 8, 3, 3, 1, (1, 1, 1, 1)),
    (3, 1, 64, 49, 10, 10, 4, 2, (4, 5, 1, 1)),      # keyword-spotting stem, 'same' padding
    (2, 3, 8, 96, 96, 3, 3, 2, (1, 1, 1, 1)),
    (2, 64, 64, 25, 5, 1, 1, 1, (0, 0, 0, 0)),
    (1, 128, 256, 3, 3, 1, 1, 1, (0, 0, 0, 0)),
    (2, 70, 45, 9, 11, 3, 3, 1, (1, 1, 1, 1)),       # ragged channel counts
    (1, 33, 10, 17, 19, 5, 3, 3, (2, 1, 0, 2)),      # asymmetric pads, rectangular window, stride 3
    (1, 40, 40, 17, 17, 2, 2, 1, (0, 1, 1, 0)),
    (2, 64, 64, 14, 14, 3, 3, 1, (1, 1, 1, 1)),
    (1, 96, 32, 6, 6, 6, 6, 1, (0, 0, 0, 0)),        # full reduction as a full-window convolution
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_fp32(case):
    N, C, K, H, W, FH, FW, S, pad = case
    x, w, b = rnd((N, C, H, W), 9), rnd((K, C, FH, FW), 10), rnd((K,), 11)
    wb = torch.empty(B.small_conv_weight_elems(C, K, FH, FW, B.MATH_FP32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, FH, FW, B.MATH_FP32)
    bx = to_blk(x)
    ref = oracle.conv2d(x, w, b, S, pad, relu=True)
    OH, OW = ref.shape[2:]
    out = new_blk(N, K, OH, OW)
    B.small_conv2d(ctx(), bx, wb, dev(b), out, N, C, K, H, W, FH, FW, S, pad, B.RELU | B.MATH_FP32)
    assert rel_err(from_blk(out, N, K, OH, OW), ref) <= TOL_FP32
    assert pad_lanes_are_zero(out, N, K, OH, OW)
    # no bias, no ReLU
    B.small_conv2d(ctx(), bx, wb, None, out, N, C, K, H, W, FH, FW, S, pad, 0)
    assert rel_err(from_blk(out, N, K, OH, OW), oracle.conv2d(x, w, None, S, pad)) <= TOL_FP32
    # accumulate onto an existing tensor (the residual join), then ReLU
    prev = rnd((N, K, OH, OW), 12)
    acc = to_blk(prev)
    B.small_conv2d(ctx(), bx, wb, dev(b), acc, N, C, K, H, W, FH, FW, S, pad, B.RELU | B.ACCUMULATE)
    assert rel_err(from_blk(acc, N, K, OH, OW), oracle.conv2d(x, w, b, S, pad, relu=True, accumulate_into=prev)) <= TOL_FP32
    assert pad_lanes_are_zero(acc, N, K, OH, OW)


@pytest.mark.parametrize("N,J,K", [(4, 64, 10), (3, 256, 2), (5, 64, 12), (2, 70, 45), (1, 1, 1), (7, 128, 128)])
def test_fc(N, J, K):
    x, w, b = rnd((N, J, 1, 1), 13), rnd((K, J), 14), rnd((K,), 15)
    wb = torch.empty(B.small_fc_weight_elems(J, K), device="cuda")
    B.small_pack_fc_weights(ctx(), dev(w), wb, J, K)
    out = new_blk(N, K, 1, 1)
    B.small_fc(ctx(), to_blk(x), wb, dev(b), out, N, J, K, 0)
    assert rel_err(from_blk(out, N, K, 1, 1).reshape(N, K), oracle.fc(x, w, b)) <= TOL_FP32
    assert pad_lanes_are_zero(out, N, K, 1, 1)
    B.small_fc(ctx(), to_blk(x), wb, None, out, N, J, K, B.RELU)
    assert rel_err(from_blk(out, N, K, 1, 1).reshape(N, K), oracle.fc(x, w, None, relu=True)) <= TOL_FP32


def test_argument_errors_launch_nothing():
    c = ctx()
    L = B.lib()
    x = new_blk(1, 32, 4, 4, 0.0)
    y = new_blk(1, 32, 4, 4, 0.0)
    w = torch.zeros(B.small_conv_weight_elems(32, 32, 3, 3, B.MATH_FP32), device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    def conv(inp, wt, out, N=1, C=32, K=32, H=4, W=4, FH=3, FW=3, S=1, pads=(1, 1, 1, 1), flags=0):
        return L.small_conv2d(c, inp, wt, None, out, N, C, K, H, W, FH, FW, S, *pads, flags, st)
    assert conv(x.data_ptr(), w.data_ptr(), y.data_ptr()) == 0
    assert conv(None, w.data_ptr(), y.data_ptr()) == 1                      # null
    assert conv(x.data_ptr() + 4, w.data_ptr(), y.data_ptr()) == 3          # misaligned
    assert conv(x.data_ptr(), w.data_ptr(), x.data_ptr()) == 4              # overlap
    assert conv(x.data_ptr(), w.data_ptr(), y.data_ptr(), N=0) == 2         # shape
    assert conv(x.data_ptr(), w.data_ptr(), y.data_ptr(), pads=(3, 1, 1, 1)) == 2   # pad >= window
    assert conv(x.data_ptr(), w.data_ptr(), y.data_ptr(), FH=7, FW=7, pads=(0, 0, 0, 0)) == 2   # empty output
    assert conv(x.data_ptr(), w.data_ptr(), y.data_ptr(), flags=3 << 4) == 1   # unknown math mode
    assert conv(x.data_ptr(), w.data_ptr(), y.data_ptr(), flags=1 << 8) == 1   # unknown flag
    assert L.small_pool2d(c, x.data_ptr(), y.data_ptr(), None, 1, 32, 4, 4, 2, 2, 2, 0, 0, 0, 0, 5, st) == 1
    assert L.small_relu(c, x.data_ptr(), x.data_ptr() + 64, 1, 32, 4, 4, st) == 4   # partial overlap
    torch.cuda.synchronize()
    assert B.small_device_status(c) == 0


CONV_TC_CASES = [  # N, C, K, H, W, FH, FW, pad  (stride 1: the shapes the tensor-core kernel takes)
    (1, 16, 16, 32, 32, 3, 3, (1, 1, 1, 1)),       # the single-conv workload
    (2, 64, 64, 56, 56, 3, 3, (1, 1, 1, 1)),       # sweep shapes at small batch: row tiles of one image
    (3, 128, 128, 28, 28, 3, 3, (1, 1, 1, 1)),
    (5, 256, 256, 14, 14, 3, 3, (1, 1, 1, 1)),     # several images per strip, two filter tiles
    (19, 512, 512, 7, 7, 3, 3, (1, 1, 1, 1)),      # ragged last strip (19 = 2 x 8 + 3 images)
    (2, 64, 64, 56, 56, 1, 1, (0, 0, 0, 0)),
    (23, 512, 512, 7, 7, 1, 1, (0, 0, 0, 0)),
    (3, 64, 64, 25, 5, 1, 1, (0, 0, 0, 0)),
    (2, 5, 16, 32, 32, 3, 3, (1, 1, 1, 1)),        # few input channels: the rest of the block is zero
    (2, 3, 16, 32, 32, 3, 3, (1, 1, 1, 1)),        # at most four: the register-filter CUDA-core kernel in every mode
    (2, 70, 45, 9, 11, 3, 3, (1, 1, 1, 1)),        # ragged channel counts
    (2, 33, 200, 17, 19, 5, 3, (2, 1, 0, 2)),      # asymmetric pads, rectangular window, ragged filter tile
    (1, 40, 40, 17, 17, 2, 2, (0, 1, 1, 0)),
    (3, 32, 32, 40, 120, 3, 3, (1, 1, 1, 1)),      # wide rows
    (3, 32, 32, 40, 200, 3, 3, (1, 1, 1, 1)),      # rows so wide that two strips exceed shared memory: FP32 kernel
    (4, 32, 64, 6, 6, 3, 3, (2, 0, 0, 2)),
    (1, 96, 32, 6, 6, 6, 6, (0, 0, 0, 0)),         # full reduction as a full-window convolution
    (2, 32, 32, 3, 300, 1, 1, (0, 0, 0, 0)),       # row wider than the kernel's tile: runs the FP32 kernel instead
]


@pytest.fixture
def tensor_path():
    """The tests below are about the tensor-core kernel: they force it wherever it takes the shape (the automatic
    choice hands layers with few channels to the CUDA-core kernel)."""
    with conv_path("tensor"):
        yield


@pytest.mark.usefixtures("tensor_path")
@pytest.mark.parametrize("case", CONV_TC_CASES)
def test_conv_tf32_tensor_cores(case):
    N, C, K, H, W, FH, FW, pad = case
    x, w, b = rnd((N, C, H, W), 16), rnd((K, C, FH, FW), 17), rnd((K,), 18)
    wb = torch.empty(B.small_conv_weight_elems(C, K, FH, FW, B.MATH_TF32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, FH, FW, B.MATH_TF32)
    bx = to_blk(x)
    ref = oracle.conv2d(x, w, b, 1, pad, relu=True)
    OH, OW = ref.shape[2:]
    uses = runs_on_tensor_cores(N, C, K, H, W, FH, FW, 1, pad)
    if W > 255:
        assert not uses      # the padded row must fit a 256-pixel TMA box (very wide rows may also exceed shared memory)
    out = new_blk(N, K, OH, OW)
    B.small_conv2d(ctx(), bx, wb, dev(b), out, N, C, K, H, W, FH, FW, 1, pad, B.RELU | B.MATH_TF32)
    err = rel_err(from_blk(out, N, K, OH, OW), ref)
    assert B.small_device_status(ctx()) == 0
    assert err <= 2e-3, err
    if uses:
        assert err > 1e-7     # TF32 products: not the FP32 kernel in disguise
    assert pad_lanes_are_zero(out, N, K, OH, OW)
    prev = rnd((N, K, OH, OW), 19)
    acc = to_blk(prev)
    B.small_conv2d(ctx(), bx, wb, None, acc, N, C, K, H, W, FH, FW, 1, pad, B.ACCUMULATE | B.MATH_TF32)
    assert rel_err(from_blk(acc, N, K, OH, OW), oracle.conv2d(x, w, None, 1, pad, accumulate_into=prev)) <= 2e-3
    # deterministic: the same launch twice gives the same bits
    out2 = new_blk(N, K, OH, OW)
    B.small_conv2d(ctx(), bx, wb, dev(b), out2, N, C, K, H, W, FH, FW, 1, pad, B.RELU | B.MATH_TF32)
    assert torch.equal(out.view(torch.int32), out2.view(torch.int32))


CONV_TC_STRIDE2_CASES = [  # N, C, K, H, W, FH, FW, pad  (stride 2: read as a stride-1 window over the input's four phase planes)
    (3, 16, 32, 32, 32, 3, 3, (1, 1, 1, 1)),       # the residual network's downsampling convolutions
    (3, 16, 32, 32, 32, 1, 1, (0, 0, 0, 0)),       # and its 1x1 shortcut: a single phase plane
    (2, 32, 64, 16, 16, 3, 3, (1, 1, 1, 1)),
    (2, 5, 8, 96, 96, 3, 3, (1, 1, 1, 1)),         # the depthwise-separable stem's shape with five channels
    (5, 5, 64, 49, 10, 10, 4, (4, 5, 1, 1)),       # the keyword-spotting stem's: tall window, odd height, asymmetric pads
    (2, 70, 45, 17, 19, 3, 3, (0, 1, 1, 0)),       # odd planes, ragged channels, pads on one side only
    (2, 40, 40, 15, 15, 2, 2, (0, 0, 0, 0)),       # window = stride: every phase plane has one tap
    (3, 64, 64, 9, 9, 5, 5, (2, 2, 2, 2)),
    (2, 32, 32, 31, 33, 1, 1, (0, 0, 0, 0)),
    (2, 32, 300, 12, 12, 3, 3, (1, 0, 0, 1)),      # two filter tiles
]


@pytest.mark.usefixtures("tensor_path")
@pytest.mark.parametrize("case", CONV_TC_STRIDE2_CASES)
def test_conv_tf32_tensor_cores_stride2(case):
    N, C, K, H, W, FH, FW, pad = case
    x, w, b = rnd((N, C, H, W), 26), rnd((K, C, FH, FW), 27), rnd((K,), 28)
    wb = torch.empty(B.small_conv_weight_elems(C, K, FH, FW, B.MATH_TF32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, FH, FW, B.MATH_TF32)
    bx = to_blk(x)
    ref = oracle.conv2d(x, w, b, 2, pad, relu=True)
    OH, OW = ref.shape[2:]
    assert runs_on_tensor_cores(N, C, K, H, W, FH, FW, 2, pad)
    out = new_blk(N, K, OH, OW)
    B.small_conv2d(ctx(), bx, wb, dev(b), out, N, C, K, H, W, FH, FW, 2, pad, B.RELU | B.MATH_TF32)
    err = rel_err(from_blk(out, N, K, OH, OW), ref)
    assert B.small_device_status(ctx()) == 0
    assert 1e-7 < err <= 2e-3, err
    assert pad_lanes_are_zero(out, N, K, OH, OW)
    prev = rnd((N, K, OH, OW), 29)
    acc = to_blk(prev)
    B.small_conv2d(ctx(), bx, wb, None, acc, N, C, K, H, W, FH, FW, 2, pad, B.ACCUMULATE | B.MATH_TF32)
    assert rel_err(from_blk(acc, N, K, OH, OW), oracle.conv2d(x, w, None, 2, pad, accumulate_into=prev)) <= 2e-3
    # the FP32 mode of the same layer stays within its own bound
    out32 = new_blk(N, K, OH, OW)
    B.small_conv2d(ctx(), bx, wb, dev(b), out32, N, C, K, H, W, FH, FW, 2, pad, B.RELU | B.MATH_FP32)
    assert rel_err(from_blk(out32, N, K, OH, OW), ref) <= 1e-5


CONV_3XTF32_CASES = [  # N, C, K, H, W, FH, FW, stride, pad
    (1, 16, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),
    (2, 64, 64, 56, 56, 3, 3, 1, (1, 1, 1, 1)),
    (3, 128, 128, 28, 28, 3, 3, 1, (1, 1, 1, 1)),
    (5, 256, 256, 14, 14, 3, 3, 1, (1, 1, 1, 1)),     # long reductions: channel blocks rotate over 2 ...
    (19, 512, 512, 7, 7, 3, 3, 1, (1, 1, 1, 1)),      # ... or 4 accumulators
    (19, 512, 512, 7, 7, 1, 1, 1, (0, 0, 0, 0)),
    (2, 64, 64, 56, 56, 1, 1, 1, (0, 0, 0, 0)),
    (2, 5, 16, 32, 32, 3, 3, 1, (1, 1, 1, 1)),
    (2, 70, 45, 9, 11, 3, 3, 1, (1, 1, 1, 1)),
    (2, 33, 200, 17, 19, 5, 3, 1, (2, 1, 0, 2)),
    (3, 16, 32, 32, 32, 3, 3, 2, (1, 1, 1, 1)),
    (3, 16, 32, 32, 32, 1, 1, 2, (0, 0, 0, 0)),
    (5, 5, 64, 49, 10, 10, 4, 2, (4, 5, 1, 1)),
]


@pytest.mark.usefixtures("tensor_path")
@pytest.mark.parametrize("case", CONV_3XTF32_CASES)
def test_conv_3xtf32_tensor_cores(case):
    """3xTF32: TF32 part and residual of both operands, three MMAs per K step, FP32-level accuracy."""
    N, C, K, H, W, FH, FW, S, pad = case
    x, w, b = rnd((N, C, H, W), 36), rnd((K, C, FH, FW), 37), rnd((K,), 38)
    wb = torch.empty(B.small_conv_weight_elems(C, K, FH, FW, B.MATH_3XTF32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, FH, FW, B.MATH_3XTF32)
    bx = to_blk(x)
    ref = oracle.conv2d(x, w, b, S, pad, relu=True)
    OH, OW = ref.shape[2:]
    out = new_blk(N, K, OH, OW)
    B.small_conv2d(ctx(), bx, wb, dev(b), out, N, C, K, H, W, FH, FW, S, pad, B.RELU | B.MATH_3XTF32)
    assert B.small_device_status(ctx()) == 0
    err = rel_err(from_blk(out, N, K, OH, OW), ref)
    assert err <= 1e-5, err
    assert pad_lanes_are_zero(out, N, K, OH, OW)
    # not the CUDA-core kernel under another name: the same layer in FP32 mode sums in another order
    out32 = new_blk(N, K, OH, OW)
    B.small_conv2d(ctx(), bx, wb, dev(b), out32, N, C, K, H, W, FH, FW, S, pad, B.RELU | B.MATH_FP32)
    assert not torch.equal(out.view(torch.int32), out32.view(torch.int32))
    prev = rnd((N, K, OH, OW), 39)
    acc = to_blk(prev)
    B.small_conv2d(ctx(), bx, wb, None, acc, N, C, K, H, W, FH, FW, S, pad, B.ACCUMULATE | B.MATH_3XTF32)
    assert rel_err(from_blk(acc, N, K, OH, OW), oracle.conv2d(x, w, None, S, pad, accumulate_into=prev)) <= 1e-5


def test_tf32_issue_probe():
    """The probe's straight-line MMA chains run at the pipe's rate: N / 2 cycles per 128 x N x 8 MMA for N >= 128."""
    tf256, c256 = B.small_measure_tf32_peak(ctx(), 256, 2048)
    tf128, c128 = B.small_measure_tf32_peak(ctx(), 128, 2048)
    tf32, c32 = B.small_measure_tf32_peak(ctx(), 32, 2048)
    assert B.small_device_status(ctx()) == 0
    assert 120.0 <= c256 <= 140.0 and 60.0 <= c128 <= 75.0 and 20.0 <= c32 <= 75.0, (c256, c128, c32)
    assert tf256 > 600.0 and abs(tf128 / tf256 - 1.0) < 0.15
    with pytest.raises(B.SmallError):
        B.small_measure_tf32_peak(ctx(), 48, 2048)


@pytest.mark.parametrize("shape", [(2, 16, 9, 7), (3, 40, 5, 5), (1, 64, 56, 56), (2, 3, 4, 4), (1, 70, 3, 11)])
def test_scale_shift(shape):
    """Batch normalisation as a per-channel FMA: one fused multiply-add per element, so within one rounding of the oracle."""
    N, C, H, W = shape
    x, s, t = rnd(shape, 81), rnd((C,), 82), rnd((C,), 83)
    for relu in (False, True):
        ref = oracle.scale_shift(x, s, t, relu)
        out = new_blk(N, C, H, W)
        B.small_scale_shift(ctx(), to_blk(x), dev(s), dev(t), out, N, C, H, W, B.RELU if relu else 0)
        got = from_blk(out, N, C, H, W)
        assert np.array_equal(got.view(np.int32), ref.view(np.int32))      # a single FMA rounds once, like the oracle
        assert pad_lanes_are_zero(out, N, C, H, W)
    buf = to_blk(x)                                                          # in place
    B.small_scale_shift(ctx(), buf, dev(s), dev(t), buf, N, C, H, W, 0)
    assert np.array_equal(from_blk(buf, N, C, H, W).view(np.int32), oracle.scale_shift(x, s, t).view(np.int32))


@pytest.mark.parametrize("shape,f", [((2, 16, 9, 7), 2), ((1, 40, 5, 5), 3), ((2, 3, 4, 4), 1), ((1, 64, 14, 14), 2), ((3, 33, 1, 6), 4)])
def test_upsample_nearest_bit_exact(shape, f):
    N, C, H, W = shape
    x = rnd(shape, 84)
    out = new_blk(N, C, H * f, W * f)
    B.small_upsample_nearest(ctx(), to_blk(x), out, N, C, H, W, f)
    got = from_blk(out, N, C, H * f, W * f)
    assert np.array_equal(got.view(np.int32), oracle.upsample_nearest(x, f).view(np.int32))
    assert pad_lanes_are_zero(out, N, C, H * f, W * f)
    with pytest.raises(B.SmallError):
        B.small_upsample_nearest(ctx(), to_blk(x), out, N, C, H, W, 0)


def test_bounded_wait_runs_out_records_timeout_and_the_context_stays_usable():
    """The give-up-and-return path of the device-side waits: with the limit lowered to a few hundred polls, a kernel that
    waits on a barrier nothing arms returns by itself, the status word reads SMALL_ERR_TIMEOUT once, and ordinary calls
    (tensor-core, TMA-fed CUDA-core and depthwise kernels, which use the same wait routine and limit) work as before."""
    c = ctx()
    assert B.small_device_status(c) == 0
    try:
        B.small_set_wait_limit(c, 300)
        B.small_selftest_wait_timeout(c)
        torch.cuda.synchronize()                       # the kernel returned: nothing hangs, nothing traps
        assert B.small_device_status(c) == 8           # SMALL_ERR_TIMEOUT
        assert B.small_device_status(c) == 0           # read once, then clear
    finally:
        B.small_set_wait_limit(c, 1 << 22)
    with pytest.raises(B.SmallError):
        B.small_set_wait_limit(c, 3)
    N, C, K, H, W = 2, 64, 64, 14, 14
    x, w, b = rnd((N, C, H, W), 81), rnd((K, C, 3, 3), 82), rnd((K,), 83)
    wb = torch.empty(B.small_conv_weight_elems(C, K, 3, 3, B.MATH_3XTF32), device="cuda")
    B.small_pack_conv_weights(c, dev(w), wb, C, K, 3, 3, B.MATH_3XTF32)
    ref = oracle.conv2d(x, w, b, 1, (1, 1, 1, 1), relu=True)
    for math, tol in (("fp32", 1e-5), ("tf32", 2e-3), ("3xtf32", 1e-5)):
        out = new_blk(N, K, H, W)
        B.small_conv2d(c, to_blk(x), wb, dev(b), out, N, C, K, H, W, 3, 3, 1, (1, 1, 1, 1), B.RELU | B.MATH[math])
        assert rel_err(from_blk(out, N, K, H, W), ref) <= tol
    assert B.small_device_status(c) == 0
