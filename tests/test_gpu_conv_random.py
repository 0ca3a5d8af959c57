"""Seeded random geometries through small_conv2d in both tensor-core modes against the oracle: the planner picks tiles,
orientation, residency, chunk counts and the stride-2 view from the shape, so odd shapes are where its branches meet."""
import numpy as np
import pytest
import torch

import oracle
import synth
from paper_2303_04769_b200 import binding as B
from gpu_util import ctx, dev, to_blk, from_blk, new_blk, rel_err, pad_lanes_are_zero, conv_path

pytestmark = pytest.mark.gpu


def _cases(count, seed):
    rng = np.random.RandomState(seed)      # shapes only; tensor values come from the counter-based generator
    out = []
    while len(out) < count:
        S = int(rng.choice([1, 1, 2]))
        FH, FW = int(rng.randint(1, 6)), int(rng.randint(1, 6))
        H, W = int(rng.randint(FH, 41)), int(rng.randint(FW, 41))
        pad = tuple(int(rng.randint(0, min(3, f))) for f in (FH, FH, FW, FW))
        C = int(rng.choice([1, 3, 8, 16, 17, 32, 33, 48, 64, 96, 130]))
        K = int(rng.choice([1, 5, 16, 32, 40, 64, 100, 128, 160, 260]))
        N = int(rng.randint(1, 7))
        if (H + pad[0] + pad[1] - FH) // S + 1 < 1 or (W + pad[2] + pad[3] - FW) // S + 1 < 1:
            continue
        if 2.0 * N * H * W * C * K * FH * FW > 3e9:      # keep the oracle quick
            continue
        out.append((N, C, K, H, W, FH, FW, S, pad))
    return out


@pytest.mark.parametrize("path", ["tensor", "cuda_cores"])
@pytest.mark.parametrize("case", _cases(48, 20230304))
def test_random_geometry_tf32_and_3xtf32(case, path):
    """Each geometry with the tensor-core kernel forced wherever it takes the shape, and with the register-tiled
    CUDA-core kernel forced wherever that one does (the automatic choice between them is by channel counts)."""
    N, C, K, H, W, FH, FW, S, pad = case
    x = synth.uniform((N, C, H, W), -1.0, 1.0, 61, seed=99)
    w = synth.uniform((K, C, FH, FW), -1.0, 1.0, 62, seed=99)
    b = synth.uniform((K,), -1.0, 1.0, 63, seed=99)
    wb = torch.empty(B.small_conv_weight_elems(C, K, FH, FW, B.MATH_3XTF32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, FH, FW, B.MATH_3XTF32)
    ref = oracle.conv2d(x, w, b, S, pad, relu=True)
    OH, OW = ref.shape[2:]
    bx = to_blk(x)
    for math, tol in (("tf32", 2e-3), ("3xtf32", 1e-5)):
        out = new_blk(N, K, OH, OW)
        with conv_path(path):
            B.small_conv2d(ctx(), bx, wb, dev(b), out, N, C, K, H, W, FH, FW, S, pad, B.RELU | B.MATH[math])
        assert B.small_device_status(ctx()) == 0
        err = rel_err(from_blk(out, N, K, OH, OW), ref)
        assert err <= tol, (math, err)
        assert pad_lanes_are_zero(out, N, K, OH, OW)


def _cases_few_channels(count, seed):
    """Shapes the warp-level tensor-core kernel takes: one channel block, filters in tiles of 32."""
    rng = np.random.RandomState(seed)
    out = []
    while len(out) < count:
        S = int(rng.choice([1, 1, 2]))
        FH, FW = (int(v) for v in rng.choice([1, 2, 3, 3, 3, 5], size=2))
        H, W = int(rng.randint(FH, 45)), int(rng.randint(FW, 80))
        pad = tuple(int(rng.randint(0, min(3, f))) for f in (FH, FH, FW, FW))
        C = int(rng.choice([1, 3, 5, 8, 9, 16, 17, 24, 31, 32]))
        K = int(rng.choice([1, 5, 8, 12, 16, 20, 32, 33, 64, 70, 200]))
        N = int(rng.choice([1, 2, 3, 5, 9, 40]))
        if (H + pad[0] + pad[1] - FH) // S + 1 < 1 or (W + pad[2] + pad[3] - FW) // S + 1 < 1:
            continue
        if 2.0 * N * H * W * C * K * FH * FW > 6e8:       # keep the oracle quick
            continue
        out.append((N, C, K, H, W, FH, FW, S, pad))
    return out


@pytest.mark.parametrize("case", _cases_few_channels(40, 20230305))
def test_random_geometry_warp_level_kernel(case):
    """The same comparison with the warp-level kernel forced: its planner picks fragment shapes, bands, column tiles,
    images per tile, filter tiles and the row-sharing form from the shape; plain and accumulating form."""
    N, C, K, H, W, FH, FW, S, pad = case
    x = synth.uniform((N, C, H, W), -1.0, 1.0, 71, seed=98)
    w = synth.uniform((K, C, FH, FW), -1.0, 1.0, 72, seed=98)
    b = synth.uniform((K,), -1.0, 1.0, 73, seed=98)
    wb = torch.empty(B.small_conv_weight_elems(C, K, FH, FW, B.MATH_3XTF32), device="cuda")
    B.small_pack_conv_weights(ctx(), dev(w), wb, C, K, FH, FW, B.MATH_3XTF32)
    ref = oracle.conv2d(x, w, b, S, pad, relu=True)
    OH, OW = ref.shape[2:]
    prev = synth.uniform((N, K, OH, OW), -1.0, 1.0, 74, seed=98)
    ref_acc = oracle.conv2d(x, w, None, S, pad, accumulate_into=prev)
    bx = to_blk(x)
    with conv_path("warp_mma"):
        for math, tol in (("tf32", 2e-3), ("3xtf32", 1e-5)):
            assert B.small_conv2d_path(ctx(), N, C, K, H, W, FH, FW, S, pad, B.MATH[math]) == 4
            out = new_blk(N, K, OH, OW)
            B.small_conv2d(ctx(), bx, wb, dev(b), out, N, C, K, H, W, FH, FW, S, pad, B.RELU | B.MATH[math])
            assert B.small_device_status(ctx()) == 0
            err = rel_err(from_blk(out, N, K, OH, OW), ref)
            assert err <= tol, (math, err)
            assert pad_lanes_are_zero(out, N, K, OH, OW)
            acc = to_blk(prev)
            B.small_conv2d(ctx(), bx, wb, None, acc, N, C, K, H, W, FH, FW, S, pad, B.ACCUMULATE | B.MATH[math])
            err = rel_err(from_blk(acc, N, K, OH, OW), ref_acc)
            assert err <= tol, (math, "accumulate", err)
