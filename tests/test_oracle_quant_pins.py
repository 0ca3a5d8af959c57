"""Pins of the oracle's quantised routines (uint8 data, int32 accumulation, one integer requantisation per output)
against things other than themselves: exact rational arithmetic, brute force in Python integers, the float oracle and a
library convolution on the same integers, the layer-class equivalences of Table 1, and the one row of Table 5's
quantised column that the printed memory formula reproduces."""
from fractions import Fraction
import math

import numpy as np
import pytest

import oracle
from conftest import read_golden

GOLD = read_golden("paper_values.txt")


def u8(shape, seed, lo=0, hi=256):
    return np.random.RandomState(seed).randint(lo, hi, size=shape).astype(np.uint8)


def test_requantize_is_one_round_half_up_of_the_exact_product():
    rng = np.random.RandomState(3)
    cases = [(0, 1 << 30, 30, 0, 0), (5, 1 << 29, 30, 0, 0), (-5, 1 << 29, 30, 10, 0), (3, 1 << 29, 30, 0, 0), (-3, 1 << 29, 30, 7, 0),
             (1 << 30, (1 << 31) - 1, 31, 0, 0), (-(1 << 30), (1 << 31) - 1, 40, 128, 0), (1000, 12345, 20, 3, 3), (-1000, 12345, 12, 200, 200)]
    for _ in range(300):
        cases.append((int(rng.randint(-(1 << 24), 1 << 24)), int(rng.randint(0, (1 << 31) - 1)), int(rng.randint(1, 50)),
                      int(rng.randint(0, 256)), int(rng.choice([0, 17, 128]))))
    for acc, mult, shift, z, lo in cases:
        exact = Fraction(acc * mult, 1 << shift)
        r = math.floor(exact + Fraction(1, 2))            # half up: ties go towards +infinity
        want = min(255, max(lo, z + r))
        assert oracle.requantize(acc, mult, shift, z, lo) == want, (acc, mult, shift, z, lo)
    # ties: 2.5 -> 3, -2.5 -> -2 (z = 100 keeps the result in range)
    assert oracle.requantize(5, 1 << 29, 30, 100) == 103
    assert oracle.requantize(-5, 1 << 29, 30, 100) == 98


def brute_q_conv(x, w, b, S, pad, zx, zw, zo, mult, shift, relu):
    N, C, H, W = x.shape
    K, _, FH, FW = w.shape
    pt, pb, pl, pr = pad
    OH, OW = (H + pt + pb - FH) // S + 1, (W + pl + pr - FW) // S + 1
    out = np.zeros((N, K, OH, OW), dtype=np.uint8)
    for n in range(N):
        for k in range(K):
            for oh in range(OH):
                for ow in range(OW):
                    acc = int(b[k]) if b is not None else 0
                    for fy in range(FW):            # loops in another order than the routine under test
                        for fx in range(FH):
                            ih, iw = oh * S + fx - pt, ow * S + fy - pl
                            if 0 <= ih < H and 0 <= iw < W:
                                for c in range(C):
                                    acc += (int(x[n, c, ih, iw]) - zx) * (int(w[k, c, fx, fy]) - zw)
                    r = math.floor(Fraction(acc * mult, 1 << shift) + Fraction(1, 2))
                    out[n, k, oh, ow] = min(255, max(zo if relu else 0, zo + r))
    return out


@pytest.mark.parametrize("S,pad,F", [(1, (0, 0, 0, 0), (3, 3)), (1, (1, 1, 1, 1), (3, 3)), (2, (1, 0, 2, 1), (3, 4)), (2, (0, 0, 0, 0), (1, 1)), (3, (2, 1, 0, 2), (5, 3))])
def test_q_conv_matches_brute_force_in_python_integers(S, pad, F):
    x, w = u8((2, 3, 7, 8), 11), u8((4, 3) + F, 12)
    b = np.random.RandomState(13).randint(-5000, 5000, size=4).astype(np.int32)
    for zx, zw, zo, mult, shift, relu in [(0, 0, 0, 1 << 20, 30, False), (128, 131, 7, 1518500250, 44, True), (3, 250, 200, 987654321, 43, False)]:
        got = oracle.q_conv2d(x, w, b, S, pad, zx, zw, zo, mult, shift, relu)
        np.testing.assert_array_equal(got, brute_q_conv(x, w, b, S, pad, zx, zw, zo, mult, shift, relu))


def test_q_conv_padding_is_the_input_zero_point():
    # padded positions are real zeros, i.e. bytes equal to z_in: padding the tensor explicitly with z_in gives the same result
    x, w = u8((1, 2, 5, 6), 21), u8((3, 2, 3, 3), 22)
    zx = 77
    xp = np.full((1, 2, 5 + 1 + 2, 6 + 2 + 1), zx, dtype=np.uint8)
    xp[:, :, 1:6, 2:8] = x
    a = oracle.q_conv2d(x, w, None, 1, (1, 2, 2, 1), zx, 9, 100, 1 << 18, 30)
    b = oracle.q_conv2d(xp, w, None, 1, (0, 0, 0, 0), zx, 9, 100, 1 << 18, 30)
    np.testing.assert_array_equal(a, b)


def test_q_conv_with_identity_requantisation_is_the_float_convolution_of_the_same_integers():
    torch = pytest.importorskip("torch")
    x, w = u8((2, 4, 6, 7), 31, 0, 6), u8((5, 4, 3, 3), 32, 0, 4)         # small values: results stay below 256
    got = oracle.q_conv2d(x, w, None, 1, (1, 1, 1, 1), 0, 0, 0, 1 << 30, 30)
    ref = oracle.conv2d(x.astype(np.float32), w.astype(np.float32), None, 1, (1, 1, 1, 1))
    assert ref.max() > 100
    np.testing.assert_array_equal(got, np.clip(ref, 0, 255).astype(np.uint8))
    lib = torch.nn.functional.conv2d(torch.from_numpy(x.astype(np.float64)), torch.from_numpy(w.astype(np.float64)), padding=1).numpy()
    np.testing.assert_array_equal(got, np.clip(lib, 0, 255).astype(np.uint8))
    # with zero points: the same library routine on the offset integers, then the exact requantisation
    zx, zw, zo, mult, shift = 2, 1, 30, 1 << 27, 30
    lib = torch.nn.functional.conv2d(torch.from_numpy(x.astype(np.float64) - zx), torch.from_numpy(w.astype(np.float64) - zw), padding=0).numpy()
    want = np.clip(zo + np.floor(lib * mult / 2.0 ** shift + 0.5), 0, 255).astype(np.uint8)      # values are small: exact in float64
    np.testing.assert_array_equal(oracle.q_conv2d(x, w, None, 1, (0, 0, 0, 0), zx, zw, zo, mult, shift), want)


def test_q_depthwise_is_a_convolution_whose_other_filter_taps_equal_the_weight_zero_point():
    x, wd = u8((2, 5, 6, 6), 41), u8((5, 3, 3), 42)
    b = np.random.RandomState(43).randint(-300, 300, size=5).astype(np.int32)
    zw = 120
    wfull = np.full((5, 5, 3, 3), zw, dtype=np.uint8)          # (w - z_w) = 0 off the diagonal
    for c in range(5):
        wfull[c, c] = wd[c]
    for S in (1, 2):
        a = oracle.q_dwconv2d(x, wd, b, S, (1, 1, 1, 1), 10, zw, 128, 1 << 22, 30, relu=True)
        np.testing.assert_array_equal(a, oracle.q_conv2d(x, wfull, b, S, (1, 1, 1, 1), 10, zw, 128, 1 << 22, 30, relu=True))


def test_q_maxpool_and_relu_commute_with_dequantisation():
    x = u8((2, 3, 7, 7), 51)
    scale, z = 0.037, 93
    real = (scale * (x.astype(np.float64) - z)).astype(np.float32)
    pooled = oracle.q_maxpool2d(x, 2, 2, 2, (0, 0, 0, 0), z)
    np.testing.assert_array_equal((scale * (pooled.astype(np.float64) - z)).astype(np.float32), oracle.pool2d(real, 2, 2, 2))
    np.testing.assert_array_equal(pooled, oracle.pool2d(x.astype(np.float32), 2, 2, 2).astype(np.uint8))
    padded = oracle.q_maxpool2d(x, 3, 3, 2, (1, 1, 1, 1), z)
    np.testing.assert_array_equal(padded, oracle.pool2d(x.astype(np.float32), 3, 3, 2, (1, 1, 1, 1)).astype(np.uint8))
    r = oracle.q_relu(x, z)
    np.testing.assert_array_equal(r, np.maximum(x, z))
    np.testing.assert_array_equal((scale * (r.astype(np.float64) - z)).astype(np.float32), oracle.relu(real))


def test_quantised_memory_model_reproduces_the_autoencoder_row_of_table5():
    # Section 5.3: parameters + intermediates + 4 x the largest plane; for the fully-connected autoencoder the
    # intermediates are the largest input/output pair (640 + 128) and the model input (640), every plane is 1 x 1
    got = oracle.model_memory_q_mib(int(GOLD["params_autoencoder"]), 640 + 128 + 640, 1)
    assert round(got, 3) == GOLD["mem_q_autoencoder"]
