"""Pins for the CPU oracle: each test fixes it to something other than itself - brute force written
independently here, library routines (numpy matmul, scipy correlate, torch conv in float64),
closed forms, invariants, and the values the paper prints.  No GPU, no CUDA library."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from oracle import nets
import synth
from synth import configs
from conftest import read_golden

GOLD = read_golden("paper_values.txt")


def rnd(shape, tid, lo=-1.0, hi=1.0):
    return synth.uniform(shape, lo, hi, tid, seed=77)


# ---------------------------------------------------------------- brute force, written separately
def brute_conv(x, w, b, S, pad, relu=False, prev=None):
    """One output at a time, seven loops, extended precision."""
    N, C, H, W = x.shape
    K, _, FH, FW = w.shape
    pt, pb, pl, pr = pad
    OH = (H + pt + pb - FH) // S + 1
    OW = (W + pl + pr - FW) // S + 1
    out = np.zeros((N, K, OH, OW), dtype=np.float32)
    for n, k, oh, ow in itertools.product(range(N), range(K), range(OH), range(OW)):
        acc = np.longdouble(b[k]) if b is not None else np.longdouble(0)
        for c, fx, fy in itertools.product(range(C), range(FH), range(FW)):
            ih, iw = oh * S + fx - pt, ow * S + fy - pl
            if 0 <= ih < H and 0 <= iw < W:
                acc += np.longdouble(x[n, c, ih, iw]) * np.longdouble(w[k, c, fx, fy])
        if prev is not None:
            acc += np.longdouble(prev[n, k, oh, ow])
        v = np.float32(acc)
        out[n, k, oh, ow] = max(v, np.float32(0)) if relu else v
    return out


@pytest.mark.parametrize("S,pad,F", [(1, (0, 0, 0, 0), (3, 2)), (2, (1, 0, 2, 1), (3, 2)), (1, (1, 1, 1, 1), (3, 3)),
                                      (2, (0, 1, 0, 1), (1, 1)), (3, (2, 2, 1, 0), (4, 3))])
def test_conv_matches_brute_force(S, pad, F):
    x = rnd((2, 3, 5, 6), 1)
    w = rnd((4, 3) + F, 2)
    b = rnd((4,), 3)
    got = oracle.conv2d(x, w, b, S, pad, relu=True)
    ref = brute_conv(x, w, b, S, pad, relu=True)
    assert got.shape == ref.shape
    np.testing.assert_array_max_ulp(got, ref, maxulp=1)


def test_conv_accumulate_matches_brute_force():
    x = rnd((2, 3, 5, 6), 4)
    w = rnd((4, 3, 3, 3), 5)
    b = rnd((4,), 6)
    prev = rnd((2, 4, 5, 6), 7)
    got = oracle.conv2d(x, w, b, 1, (1, 1, 1, 1), relu=True, accumulate_into=prev)
    ref = brute_conv(x, w, b, 1, (1, 1, 1, 1), relu=True, prev=prev)
    np.testing.assert_array_max_ulp(got, ref, maxulp=1)
    # and it equals conv followed by the single-element addition layer
    plain = oracle.conv2d(x, w, b, 1, (1, 1, 1, 1))
    np.testing.assert_allclose(got, oracle.add(plain, prev, relu=True), rtol=0, atol=1e-6)


def test_dwconv_matches_brute_force_and_block_diagonal_conv():
    # Section 5.2.2: a depthwise convolution cast as a full convolution gives the same result
    # (with more work); Table 1: depthwise is F_C = 1, K = 1, G = I_C.
    x = rnd((2, 5, 7, 6), 8)
    w = rnd((5, 3, 3), 9)
    b = rnd((5,), 10)
    for S, pad in [(1, (1, 1, 1, 1)), (2, (1, 1, 1, 1)), (2, (0, 1, 0, 2))]:
        got = oracle.dwconv2d(x, w, b, S, pad, relu=True)
        full = np.zeros((5, 5, 3, 3), dtype=np.float32)
        for c in range(5):
            full[c, c] = w[c]
        np.testing.assert_array_max_ulp(got, brute_conv(x, full, b, S, pad, relu=True), maxulp=1)
        np.testing.assert_array_max_ulp(got, oracle.conv2d(x, full, b, S, pad, relu=True), maxulp=1)


# ---------------------------------------------------------------- library routines
@pytest.mark.parametrize("S,p,F,C,K", [(1, 1, 3, 4, 6), (2, 1, 3, 5, 3), (1, 0, 1, 7, 5), (2, 0, 1, 6, 4), (1, 2, 5, 3, 2)])
def test_conv_matches_torch_float64(S, p, F, C, K):
    x = rnd((3, C, 9, 11), 11)
    w = rnd((K, C, F, F), 12)
    b = rnd((K,), 13)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(),
                                     torch.from_numpy(b).double(), stride=S, padding=p).float().numpy()
    got = oracle.conv2d(x, w, b, S, (p, p, p, p))
    np.testing.assert_array_max_ulp(got, ref, maxulp=1)


def test_asymmetric_pad_equals_explicit_zero_border():
    x = rnd((2, 3, 6, 5), 14)
    w = rnd((4, 3, 3, 2), 15)
    pad = (2, 0, 1, 3)
    xp = np.pad(x, ((0, 0), (0, 0), (pad[0], pad[1]), (pad[2], pad[3])))
    for S in (1, 2):
        np.testing.assert_array_equal(oracle.conv2d(x, w, None, S, pad), oracle.conv2d(xp, w, None, S, (0, 0, 0, 0)))


def test_single_channel_conv_matches_scipy_correlate():
    from scipy.signal import correlate2d
    x = rnd((1, 1, 8, 9), 16)
    w = rnd((1, 1, 3, 4), 17)
    ref = correlate2d(x[0, 0].astype(np.float64), w[0, 0].astype(np.float64), mode="valid")
    np.testing.assert_array_max_ulp(oracle.conv2d(x, w)[0, 0], ref.astype(np.float32), maxulp=1)


def test_pointwise_conv_is_a_matrix_product():
    # Section 3.2 item 4: a 1x1 convolution reduces the channels of one pixel; pixels are independent.
    x = rnd((2, 6, 4, 5), 18)
    w = rnd((7, 6, 1, 1), 19)
    A = x.transpose(0, 2, 3, 1).reshape(-1, 6).astype(np.float64)
    ref = (A @ w.reshape(7, 6).astype(np.float64).T).reshape(2, 4, 5, 7).transpose(0, 3, 1, 2)
    np.testing.assert_array_max_ulp(oracle.conv2d(x, w), ref.astype(np.float32), maxulp=1)


def test_fc_is_matrix_product_full_window_conv_and_1x1_conv():
    # Section 3.2 item 5 / Table 1 row 5: F_H = I_H, F_W = I_W, F_C = I_C; Section 5.4: looks like a 1x1 conv.
    x = rnd((3, 4, 3, 2), 20)
    w = rnd((5, 24), 21)
    b = rnd((5,), 22)
    got = oracle.fc(x, w, b)
    ref = x.reshape(3, 24).astype(np.float64) @ w.astype(np.float64).T + b.astype(np.float64)
    np.testing.assert_array_max_ulp(got, ref.astype(np.float32), maxulp=1)
    as_conv = oracle.conv2d(x, w.reshape(5, 4, 3, 2), b)
    np.testing.assert_array_max_ulp(got, as_conv.reshape(3, 5), maxulp=1)
    flat = x.reshape(3, 24, 1, 1)
    np.testing.assert_array_max_ulp(got, oracle.conv2d(flat, w.reshape(5, 24, 1, 1), b).reshape(3, 5), maxulp=1)


def test_maxpool_matches_torch_values_and_indices():
    x = rnd((2, 3, 9, 8), 23)
    for F, S, p in [(2, 2, 0), (3, 2, 1), (3, 1, 1), (2, 1, 0)]:
        ref, ridx = torch.nn.functional.max_pool2d(torch.from_numpy(x), F, S, p, return_indices=True)
        got, idx = oracle.pool2d(x, F, F, S, (p, p, p, p), "max", with_indices=True)
        np.testing.assert_array_equal(got, ref.numpy())
        np.testing.assert_array_equal(idx, ridx.numpy().astype(np.int32))


def test_avgpool_matches_torch_excluding_pad():
    x = rnd((2, 3, 9, 8), 24)
    for F, S, p in [(2, 2, 0), (3, 2, 1), (3, 1, 1)]:
        ref = torch.nn.functional.avg_pool2d(torch.from_numpy(x).double(), F, S, p, count_include_pad=False)
        got = oracle.pool2d(x, F, F, S, (p, p, p, p), "avg")
        np.testing.assert_array_max_ulp(got, ref.float().numpy(), maxulp=1)


# ---------------------------------------------------------------- closed forms and invariants
def test_all_ones_input_gives_weight_sums():
    K, C = 5, 4
    w = rnd((K, C, 3, 3), 25)
    b = rnd((K,), 26)
    x = np.ones((1, C, 6, 7), dtype=np.float32)
    full = (b.astype(np.float64) + w.astype(np.float64).sum(axis=(1, 2, 3))).astype(np.float32)
    out = oracle.conv2d(x, w, b)                     # no padding: every output is the filter sum
    for k in range(K):
        np.testing.assert_array_max_ulp(out[0, k], np.full((4, 5), full[k], np.float32), maxulp=1)
    outp = oracle.conv2d(x, w, b, 1, (1, 1, 1, 1))   # padding: interior = full sum, corner = partial sum
    for k in range(K):
        np.testing.assert_array_max_ulp(outp[0, k, 1:-1, 1:-1], np.full((4, 5), full[k], np.float32), maxulp=1)
        corner = np.float32(b[k].astype(np.float64) + w[k, :, 1:, 1:].astype(np.float64).sum())
        np.testing.assert_array_max_ulp(outp[0, k, 0, 0], corner, maxulp=1)
        edge = np.float32(b[k].astype(np.float64) + w[k, :, :2, :].astype(np.float64).sum())
        np.testing.assert_array_max_ulp(outp[0, k, -1, 2], edge, maxulp=1)


def test_delta_input_reads_back_the_filter():
    # a unit impulse at (c0, h0, w0): out[k, h0 - x + pt, w0 - y + pl] = w[k, c0, x, y] (cross-correlation,
    # no flip); catches a transposed or flipped filter index and a wrong pad sign
    w = rnd((3, 2, 3, 2), 27)
    x = np.zeros((1, 2, 7, 7), dtype=np.float32)
    x[0, 1, 3, 4] = 1.0
    out = oracle.conv2d(x, w, None, 1, (1, 0, 0, 1))
    for k, fx, fy in itertools.product(range(3), range(3), range(2)):
        assert out[0, k, 3 - fx + 1, 4 - fy + 0] == w[k, 1, fx, fy]
    assert np.count_nonzero(out) == 3 * 3 * 2


def test_linearity_and_shift_equivariance():
    a, b2 = rnd((1, 3, 8, 8), 28), rnd((1, 3, 8, 8), 29)
    w = rnd((4, 3, 3, 3), 30)
    lhs = oracle.conv2d((2.0 * a + 0.5 * b2).astype(np.float32), w)
    rhs = 2.0 * oracle.conv2d(a, w) + 0.5 * oracle.conv2d(b2, w)
    np.testing.assert_allclose(lhs, rhs, rtol=0, atol=2e-5)
    shifted = np.zeros_like(a)
    shifted[:, :, 1:, 2:] = a[:, :, :-1, :-2]
    np.testing.assert_array_equal(oracle.conv2d(shifted, w)[:, :, 1:, 2:], oracle.conv2d(a, w)[:, :, :-1, :-2])


def test_output_size_rule():
    # Section 3.1.2 with pads 0; floor division; the cases the workloads need
    assert oracle.out_size(32, 3, 1, 1, 1) == 32
    assert oracle.out_size(32, 3, 2, 1, 1) == 16
    assert oracle.out_size(7, 2, 2) == 3
    assert oracle.out_size(96, 3, 2, 1, 1) == 48
    assert oracle.out_size(5, 6, 1) == 0
    for I, F, S in itertools.product(range(1, 12), range(1, 5), range(1, 4)):
        if F <= I:
            assert oracle.out_size(I, F, S) == len(range(0, I - F + 1, S))
    # 'same' padding of the keyword-spotting stem: 49x10, 10x4 window, stride 2 -> 25x5 (model table)
    assert oracle.same_pad(49, 10, 2) == (GOLD["dscnn_stem_out_h"], 4, 5)
    assert oracle.same_pad(10, 4, 2) == (GOLD["dscnn_stem_out_w"], 1, 1)
    stem = configs.kws_cnn()["layers"][0]
    assert stem["pad"] == (4, 5, 1, 1)


def test_figure1_group_arithmetic():
    # Figure 1: G = 2, K = 3 -> O_C = 6, with F_C = 4 and overlapping groups (S_C < F_C)
    assert oracle.out_channels(GOLD["fig1_K"], GOLD["fig1_G"]) == GOLD["fig1_OC"]
    I_C, S_C = 6, 2   # (6 - 4)/2 + 1 = 2 groups, overlapping
    assert oracle.groups(I_C, GOLD["fig1_FC"], S_C) == GOLD["fig1_G"]
    # Table 1 rows: depthwise G = I_C; convolution G = 1
    assert oracle.groups(16, 1, 1) == 16
    assert oracle.groups(16, 16, 1) == 1
    assert 64 // GOLD["rpi_channel_block"] == GOLD["rpi_blocks_of_64"]


def test_maxpool_invariants():
    x = rnd((2, 3, 8, 10), 31)
    out, idx = oracle.pool2d(x, 2, 2, 2, mode="max", with_indices=True)
    for n, c, oh, ow in itertools.product(range(2), range(3), range(4), range(5)):
        win = x[n, c, 2 * oh:2 * oh + 2, 2 * ow:2 * ow + 2]
        assert out[n, c, oh, ow] == win.max()
        assert x[n, c].ravel()[idx[n, c, oh, ow]] == out[n, c, oh, ow]
    const = np.full((1, 2, 6, 6), 3.25, dtype=np.float32)
    o, i = oracle.pool2d(const, 3, 3, 1, (1, 1, 1, 1), "max", with_indices=True)
    assert np.all(o == 3.25)
    assert i[0, 0, 0, 0] == 0 and i[0, 0, 2, 2] == 1 * 6 + 1   # ties: first element in row-major scan
    np.testing.assert_array_equal(oracle.pool2d(x, 1, 1, 1, mode="max"), x)
    ramp = np.arange(36, dtype=np.float32).reshape(1, 1, 6, 6)
    o, i = oracle.pool2d(ramp, 2, 2, 2, mode="max", with_indices=True)
    np.testing.assert_array_equal(o[0, 0], ramp[0, 0, 1::2, 1::2])
    np.testing.assert_array_equal(i[0, 0], ramp[0, 0, 1::2, 1::2].astype(np.int32))
    # 7x7 -> 3x3: the last row and column are dropped (floor)
    assert oracle.pool2d(rnd((1, 1, 7, 7), 32), 2, 2, 2).shape == (1, 1, 3, 3)
    # negative-only input with padding: pad positions never win
    neg = -np.ones((1, 1, 4, 4), dtype=np.float32)
    assert np.all(oracle.pool2d(neg, 3, 3, 1, (1, 1, 1, 1), "max") == -1.0)


def test_avgpool_invariants():
    const = np.full((2, 3, 5, 4), -1.5, dtype=np.float32)
    assert np.all(oracle.pool2d(const, 5, 4, 1, mode="avg") == -1.5)
    assert np.all(oracle.pool2d(const, 3, 3, 2, (1, 1, 1, 1), "avg") == -1.5)
    x = rnd((2, 3, 6, 8), 33)
    out = oracle.pool2d(x, 2, 2, 2, mode="avg")
    np.testing.assert_allclose(out.astype(np.float64).sum() * 4, x.astype(np.float64).sum(), rtol=1e-6)
    g = oracle.pool2d(x, 6, 8, 1, mode="avg")
    np.testing.assert_array_max_ulp(g[:, :, 0, 0], x.astype(np.float64).mean(axis=(2, 3)).astype(np.float32), maxulp=1)


def test_relu_invariants():
    x = rnd((4, 5, 3, 3), 34)
    x.ravel()[:3] = [0.0, -0.0, -1e-30]
    r = oracle.relu(x)
    assert np.all(r >= 0) and not np.any(np.signbit(r))          # -0 becomes +0
    np.testing.assert_array_equal(oracle.relu(r), r)
    np.testing.assert_array_equal(r - oracle.relu(-x), np.where(x == 0, 0, x).astype(np.float32))
    np.testing.assert_array_equal(r, np.maximum(x, 0) + 0.0)


def test_float_accumulator_variant_is_exact_on_integers_and_within_the_rounding_bound():
    """so_conv2d_f32acc (timed as a second CPU baseline, never used for parity): on small integers every partial sum is
    an integer below 2^24, so float accumulation is exact and must equal the double version bit for bit - including
    padding, stride, bias, accumulate and ReLU; on general data it may differ from the double version by at most the
    forward error bound of a recursive float sum, n * 2^-24 * sum |terms| (Higham, Accuracy and Stability, Section 4.2)."""
    rng = np.random.RandomState(7)
    xi = rng.randint(-8, 9, size=(2, 5, 9, 8)).astype(np.float32)
    wi = rng.randint(-4, 5, size=(6, 5, 3, 2)).astype(np.float32)
    bi = rng.randint(-9, 10, size=(6,)).astype(np.float32)
    for S, pad in [(1, (0, 0, 0, 0)), (2, (1, 2, 0, 1)), (1, (2, 1, 1, 0))]:
        a = oracle.conv2d(xi, wi, bi, S, pad, relu=True)
        b = oracle.conv2d(xi, wi, bi, S, pad, relu=True, f32acc=True)
        np.testing.assert_array_equal(a.view(np.int32), b.view(np.int32))
        prev = rng.randint(-20, 21, size=a.shape).astype(np.float32)
        np.testing.assert_array_equal(oracle.conv2d(xi, wi, bi, S, pad, accumulate_into=prev),
                                      oracle.conv2d(xi, wi, bi, S, pad, accumulate_into=prev, f32acc=True))
    x, w, b = rnd((2, 7, 10, 9), 71), rnd((4, 7, 3, 3), 72), rnd((4,), 73)
    d = oracle.conv2d(x, w, b, 1, (1, 1, 1, 1)).astype(np.float64)
    f = oracle.conv2d(x, w, b, 1, (1, 1, 1, 1), f32acc=True).astype(np.float64)
    n_terms = 7 * 9 + 1
    mag = oracle.conv2d(np.abs(x), np.abs(w), np.abs(b), 1, (1, 1, 1, 1)).astype(np.float64)   # sum of |terms|
    assert np.all(np.abs(f - d) <= (n_terms + 1) * 2.0 ** -24 * mag)
    assert np.any(f != d)          # and it really is another accumulator, not the double routine again


# ---------------------------------------------------------------- the abstract layer vs the layer classes
def test_abstract_layer_as_convolution():
    # Table 1 row 4: F_C = I_C, K = O_C, G = 1
    x = rnd((1, 5, 8, 9), 35)
    w = rnd((6, 5, 3, 2), 36)
    for S in (1, 2):
        got = oracle.abstract_layer(x[0], w.reshape(1, 6, 5, 3, 2), 3, 2, 5, S, S, 1, 6)
        np.testing.assert_array_max_ulp(got, oracle.conv2d(x, w, None, S)[0], maxulp=1)


def test_abstract_layer_as_depthwise_and_pool_and_relu():
    # Table 1 row 2: F_C = 1, K = 1, G = I_C.  Table 2: depthwise = FMA, max pool = Max, ReLU = Max.
    x = rnd((1, 7, 8, 9), 37)
    w = rnd((7, 3, 3), 38)
    got = oracle.abstract_layer(x[0], w.reshape(7, 1, 1, 3, 3), 3, 3, 1, 2, 2, 1, 1)
    np.testing.assert_array_max_ulp(got, oracle.dwconv2d(x, w, None, 2)[0], maxulp=1)
    got = oracle.abstract_layer(x[0], None, 2, 2, 1, 2, 2, 1, 1, op="max", init=-np.inf)
    np.testing.assert_array_equal(got, oracle.pool2d(x, 2, 2, 2)[0])
    # Table 1 row 1 (single element): ReLU is the Max reduction over a 1x1x1 window started at zero
    got = oracle.abstract_layer(x[0], None, 1, 1, 1, 1, 1, 1, 1, op="max", init=0.0)
    np.testing.assert_array_equal(got, oracle.relu(x)[0])


def test_abstract_layer_figure1_group_convolution():
    # Figure 1's shape: two overlapping groups of three filters over four channels each
    x = rnd((1, 6, 6, 7), 39)
    w = rnd((2, 3, 4, 3, 3), 40)
    got = oracle.abstract_layer(x[0], w, 3, 3, 4, 1, 1, 2, 3)
    assert got.shape[0] == GOLD["fig1_OC"]
    for g in range(2):
        ref = oracle.conv2d(x[:, 2 * g:2 * g + 4], w[g])[0]
        np.testing.assert_array_max_ulp(got[3 * g:3 * g + 3], ref, maxulp=1)
    # brute force, written a second time with the indices in another order: output channel oc = g*K + k
    xd, wd = x[0].astype(np.float64), w.astype(np.float64)
    for oc, oh, ow in [(0, 0, 0), (2, 3, 4), (3, 0, 1), (5, 3, 4)]:
        g, k = divmod(oc, 3)
        want = sum(xd[g * 2 + c, oh + a, ow + b] * wd[g, k, c, a, b] for c in range(4) for a in range(3) for b in range(3))
        assert abs(float(got[oc, oh, ow]) - want) <= 4e-7 * max(1.0, abs(want))


def test_abstract_layer_full_reduction_is_fc():
    x = rnd((1, 4, 3, 5), 41)
    w = rnd((6, 60), 42)
    got = oracle.abstract_layer(x[0], w.reshape(1, 6, 4, 3, 5), 3, 5, 4, 1, 1, 1, 6)
    np.testing.assert_array_max_ulp(got.reshape(6), oracle.fc(x, w)[0], maxulp=1)


def test_abstract_layer_rejects_windows_that_do_not_tile_the_channels():
    x = rnd((1, 6, 4, 4), 44)
    with pytest.raises(ValueError):
        oracle.abstract_layer(x[0], None, 1, 1, 4, 1, 1, 3, 1, op="max")       # (6 - 4) % 3 != 0


# ---------------------------------------------------------------- layout
def test_pack_unpack_and_index():
    for C, Cb in [(5, 4), (16, 16), (3, 32), (70, 32), (33, 16)]:
        N, H, W = 2, 3, 5
        x = rnd((N, C, H, W), 43)
        blk = oracle.pack(x, Cb)
        nb = -(-C // Cb)
        assert blk.size == N * nb * Cb * H * W == oracle.blk_elems(N, C, H, W, Cb)
        np.testing.assert_array_equal(oracle.unpack(blk, N, C, H, W, Cb), x)
        # independent statement of Figure 2: [N][C/Cb][H][W][Cb]
        ref = np.zeros((N, nb * Cb, H, W), dtype=np.float32)
        ref[:, :C] = x
        ref = ref.reshape(N, nb, Cb, H, W).transpose(0, 1, 3, 4, 2).ravel()
        np.testing.assert_array_equal(blk, ref)
        pads = blk.reshape(N, nb, H, W, Cb)[:, -1, :, :, C - (nb - 1) * Cb:]
        assert np.all(pads == 0) and not np.any(np.signbit(pads))
        assert oracle.blk_index(1, C - 1, 2, 4, C, H, W, Cb) == blk.size - Cb + (C - 1) % Cb
    # neighbouring channels of one pixel are adjacent; the next pixel is Cb away (channels fastest, then width)
    assert oracle.blk_index(0, 1, 0, 0, 64, 4, 4, 16) - oracle.blk_index(0, 0, 0, 0, 64, 4, 4, 16) == 1
    assert oracle.blk_index(0, 0, 0, 1, 64, 4, 4, 16) == 16
    assert oracle.blk_index(0, 0, 1, 0, 64, 4, 4, 16) == 16 * 4
    assert oracle.blk_index(0, 16, 0, 0, 64, 4, 4, 16) == 16 * 4 * 4


# ---------------------------------------------------------------- memory model and the workload definitions
def test_memory_model_reproduces_table5():
    # Section 5.3: bytes = 4 x (parameters + largest in/out buffer pair [+ the model input]); Table 5 prints MB = 2^20 B
    plan = nets.buffer_plan(configs.residual_cnn())
    assert plan["largest_pair"] == 2 * 16 * 32 * 32 and plan["model_input"] == 3 * 32 * 32
    got = oracle.model_memory_mib(GOLD["params_resnet"], plan["largest_pair"], plan["model_input"])
    assert round(got, 3) == GOLD["mem_resnet"]
    # MobileNet at full width: stem 3->32 stride 2 on 96x96, then depthwise 32 and pointwise 64 at 48x48
    pair = 48 * 48 * 32 + 48 * 48 * 64
    assert round(oracle.model_memory_mib(GOLD["params_mobilenet"], pair, 96 * 96 * 3), 3) == GOLD["mem_mobilenet"]
    assert round(oracle.model_memory_mib(GOLD["params_autoencoder"], 128 + 128, 128), 3) == GOLD["mem_autoencoder"]


def test_workload_shapes():
    res = nets.shapes(configs.residual_cnn())
    assert [r["out"] for r in res] == [(16, 32, 32), (16, 32, 32), (16, 32, 32), (32, 16, 16), (32, 16, 16), (32, 16, 16),
                                       (64, 8, 8), (64, 8, 8), (64, 8, 8), (64, 1, 1), (10, 1, 1)]
    plan = nets.buffer_plan(configs.residual_cnn())
    assert plan["weights"] == 77360 and plan["biases"] == 346     # the paper's ResNet has 77744 parameters
    assert abs(plan["weights"] + plan["biases"] - GOLD["params_resnet"]) < 100
    mob = nets.shapes(configs.dwsep_cnn())
    assert mob[0]["out"] == (8, 48, 48)
    assert [r["out"][1] for r in mob[2:27:2]] == [48, 24, 24, 12, 12, 6, 6, 6, 6, 6, 6, 3, 3]
    assert mob[-1]["out"] == (2, 1, 1) and mob[-2]["inp"] == (256, 3, 3)
    kws = nets.shapes(configs.kws_cnn())
    assert kws[0]["out"] == (64, 25, 5) and kws[-1]["out"] == (12, 1, 1)
    one = nets.shapes(configs.single_conv_pool())
    assert one[0]["out"] == (16, 32, 32) and one[1]["out"] == (16, 16, 16)


def test_network_runner_matches_torch_float64():
    # whole-network cross-check against torch CPU ops in float64 (a library statement of the same layers)
    net = configs.residual_cnn(batch=2)
    params = configs.make_params(net)
    x = configs.make_input(net)
    t = nets.run_net(net, params, x)
    F = torch.nn.functional
    tp = [(None if w is None else torch.from_numpy(w).double(), None if b is None else torch.from_numpy(b).double())
          for w, b in params]
    X = torch.from_numpy(x).double()
    x1 = F.relu(F.conv2d(X, *tp[0], padding=1))
    a1 = F.relu(F.conv2d(x1, *tp[1], padding=1))
    x1 = F.relu(x1 + F.conv2d(a1, *tp[2], padding=1))
    a2 = F.relu(F.conv2d(x1, *tp[3], stride=2, padding=1))
    x2 = F.conv2d(x1, *tp[4], stride=2)
    x2 = F.relu(x2 + F.conv2d(a2, *tp[5], padding=1))
    a3 = F.relu(F.conv2d(x2, *tp[6], stride=2, padding=1))
    x3 = F.conv2d(x2, *tp[7], stride=2)
    x3 = F.relu(x3 + F.conv2d(a3, *tp[8], padding=1))
    g = x3.mean(dim=(2, 3))
    out = g @ tp[10][0].T + tp[10][1]
    np.testing.assert_allclose(t["out"].reshape(2, 10), out.numpy(), rtol=2e-6, atol=2e-6)
    np.testing.assert_allclose(t["x2"], x2.numpy(), rtol=2e-6, atol=2e-6)


def test_dwsep_and_kws_runner_match_torch_float64():
    F = torch.nn.functional
    for net in (configs.dwsep_cnn(batch=1), configs.kws_cnn(batch=2)):
        params = configs.make_params(net)
        x = configs.make_input(net)
        t = nets.run_net(net, params, x)
        cur = torch.from_numpy(x).double()
        for layer, (w, b) in zip(net["layers"], params):
            W = None if w is None else torch.from_numpy(w).double()
            B = None if b is None else torch.from_numpy(b).double()
            pt, pb, pl, pr = layer["pad"]
            if layer["op"] == "conv":
                cur = F.conv2d(F.pad(cur, (pl, pr, pt, pb)), W, B, stride=layer["stride"])
            elif layer["op"] == "dwconv":
                cur = F.conv2d(F.pad(cur, (pl, pr, pt, pb)), W.unsqueeze(1), B, stride=layer["stride"], groups=layer["C"])
            elif layer["op"] == "pool":
                cur = cur.mean(dim=(2, 3), keepdim=True)
            else:
                cur = (cur.flatten(1) @ W.T + B).reshape(cur.shape[0], -1, 1, 1)
            if layer["relu"]:
                cur = F.relu(cur)
        np.testing.assert_allclose(t["out"], cur.numpy(), rtol=1e-5, atol=1e-6)


# ---------------------------------------------------------------- the generator itself
def test_generator_is_counter_based_and_in_range():
    a = synth.uniform((1000,), -1, 1, 5)
    b = synth.uniform((1000,), -1, 1, 5)
    np.testing.assert_array_equal(a, b)
    assert a.min() >= -1 and a.max() < 1 and abs(a.mean()) < 0.1
    np.testing.assert_array_equal(synth.unit_uniform(1, 2, 10, start=5), synth.unit_uniform(1, 2, 15)[5:])
    assert not np.array_equal(a, synth.uniform((1000,), -1, 1, 6))
    z = synth.normal((20000,), 0, 1, 7)
    assert abs(z.mean()) < 0.03 and abs(z.std() - 1) < 0.03
    w = synth.he_normal((64, 64, 3, 3), 576, 8)
    assert abs(w.std() - np.sqrt(2 / 576)) < 2e-3


# ---- the other single-element layers of Table 2: batch normalisation (FMA) and upsampling (nearest neighbour)
def test_scale_shift_pins():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 5, 3, 4)).astype(np.float32)
    s = rng.standard_normal(5).astype(np.float32)
    t = rng.standard_normal(5).astype(np.float32)
    got = oracle.scale_shift(x, s, t)
    # brute force, one element at a time, exact rational arithmetic rounded once
    from fractions import Fraction
    for n, c, h, w in [(0, 0, 0, 0), (1, 4, 2, 3), (0, 2, 1, 1), (1, 1, 0, 2)]:
        exact = Fraction(float(s[c])) * Fraction(float(x[n, c, h, w])) + Fraction(float(t[c]))
        assert got[n, c, h, w] == np.float32(float(exact))
    # special cases: identity, pure shift, a 1x1 depthwise convolution with bias is the same layer
    assert np.array_equal(oracle.scale_shift(x, np.ones(5, np.float32), np.zeros(5, np.float32)), x)
    assert np.array_equal(oracle.scale_shift(np.zeros_like(x), s, t), np.broadcast_to(t[None, :, None, None], x.shape))
    assert np.array_equal(got, oracle.dwconv2d(x, s.reshape(5, 1, 1), t, 1, (0, 0, 0, 0)))
    assert np.array_equal(oracle.scale_shift(x, s, t, relu=True), np.maximum(got, 0))


def test_upsample_nearest_pins():
    rng = np.random.default_rng(6)
    x = rng.standard_normal((2, 3, 4, 5)).astype(np.float32)
    for f in (1, 2, 3):
        up = oracle.upsample_nearest(x, f)
        assert up.shape == (2, 3, 4 * f, 5 * f)
        assert np.array_equal(up, np.repeat(np.repeat(x, f, axis=2), f, axis=3))       # library statement of the same thing
        assert np.array_equal(up[:, :, ::f, ::f], x)                                    # subsampling undoes it
        assert np.array_equal(oracle.pool2d(up, f, f, f, mode="max"), x)                # so does pooling each f x f block
    up = oracle.upsample_nearest(x, 2)
    assert up[1, 2, 7, 9] == x[1, 2, 3, 4] and up[0, 1, 2, 1] == x[0, 1, 1, 0]
