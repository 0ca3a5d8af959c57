"""Host-only checks of the C-ABI library: it loads, exports every function include/small.h declares, and its
host-side helpers agree with the oracle's independent size rules.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

import oracle
from conftest import ROOT

B = pytest.importorskip("paper_2303_04769_b200.binding")


@pytest.fixture(scope="module")
def lib():
    from paper_2303_04769_b200 import build
    build.build()
    return B.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "small.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(small_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 25
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in small.h but not exported"
    assert sorted(B.EXPORTS) == names


def test_host_helpers_match_oracle(lib):
    cb = B.small_channel_block()
    assert cb == 32
    for N, C, H, W in [(1, 16, 32, 32), (2, 3, 5, 7), (3, 33, 4, 4), (256, 64, 8, 8), (1, 1, 1, 1)]:
        assert B.small_packed_elems(N, C, H, W) == oracle.blk_elems(N, C, H, W, cb)
    assert B.small_packed_elems(0, 3, 4, 4) == 0
    for I in range(1, 14):
        for F in range(1, 6):
            for S in range(1, 4):
                for pa, pb in [(0, 0), (1, 1), (0, 2), (2, 1)]:
                    assert B.small_out_size(I, F, S, pa, pb) == oracle.out_size(I, F, S, pa, pb)
    assert B.small_out_size(5, 3, 1, -1, 0) == 0


def test_weight_sizes(lib):
    assert B.small_conv_weight_elems(64, 64, 3, 3, B.MATH_FP32) == 2 * 2 * 9 * 32 * 32
    assert B.small_conv_weight_elems(64, 64, 3, 3, B.MATH_TF32) == 2 * (2 * 2 * 9 * 32 * 32)
    assert B.small_conv_weight_elems(64, 64, 3, 3, B.MATH_3XTF32) == 3 * (2 * 2 * 9 * 32 * 32)
    assert B.small_conv_weight_elems(3, 16, 3, 3, B.MATH_FP32) == 9 * 32 * 32
    assert B.small_conv_weight_elems(3, 16, 3, 3, 3 << 4) == 0
    assert B.small_dw_weight_elems(70, 3, 3) == 3 * 9 * 32
    assert B.small_fc_weight_elems(64, 10) == 2 * 32 * 32
    assert B.small_fc_weight_elems(64, 10, B.MATH_3XTF32) == 3 * 2 * 32 * 32
    assert B.small_fc_weight_elems(0, 10) == 0


def test_group_convolution_sizes(lib):
    # the group count is Section 3.1.2's sliding-window formula applied to the channels
    for C, F_C, S_C in [(8, 4, 2), (64, 16, 16), (40, 1, 1), (96, 48, 48), (64, 64, 1), (36, 8, 4)]:
        assert B.small_group_count(C, F_C, S_C) == oracle.groups(C, F_C, S_C)
    assert B.small_group_count(10, 4, 4) == 0 and B.small_group_count(8, 9, 1) == 0 and B.small_group_count(8, 4, 0) == 0
    # packed size = filter blocks x channel blocks one filter block can touch x window x 32 x 32
    assert B.small_group_conv_weight_elems(64, 16, 16, 16, 3, 3) == 2 * 1 * 9 * 1024      # 2 groups per filter block, one channel block
    # groups of whole channel blocks with a multiple of 32 filters also carry the tensor-core sections (TF32 part and
    # residual): [F_C/32][taps][G*K][32]
    assert B.small_group_conv_weight_elems(128, 32, 32, 32, 3, 3) == 4 * 1 * 9 * 1024 + 2 * (1 * 9 * 128 * 32)
    assert B.small_group_conv_weight_elems(64, 64, 1, 8, 1, 1) == 1 * 2 * 1024            # one group: the dense size
    assert B.small_group_conv_weight_elems(40, 1, 1, 1, 3, 3) == 2 * 1 * 9 * 1024         # depthwise as a group convolution
    assert B.small_group_conv_weight_elems(96, 48, 48, 20, 1, 1) == 2 * 3 * 1024          # filter block 0 spans both groups
    assert B.small_group_conv_weight_elems(10, 4, 4, 2, 3, 3) == 0


def test_status_strings_and_null_context(lib):
    for s in range(0, 10):
        assert len(lib.small_strerror(s)) > 0
    assert lib.small_strerror(99) == b"unknown status"
    # a NULL context is rejected before anything else is looked at
    assert lib.small_relu(None, None, None, 1, 1, 1, 1, None) == 9
    assert lib.small_conv2d(None, None, None, None, None, 1, 1, 1, 1, 1, 1, 1, 1, 0, 0, 0, 0, 0, None) == 9
    assert lib.small_shutdown(None) == 9
    assert lib.small_init(0, None) == 1


def test_workspace_plan_matches_memory_model(lib):
    # Section 5.3: intermediate buffers are shared; with slots assigned by liveness the residual CNN needs three
    # buffers of the largest activation (two for a layer's input/output pair plus the live shortcut)
    from paper_2303_04769_b200.net import assign_slots
    from synth import configs
    net = configs.residual_cnn()
    slot_of, n_slots = assign_slots(net["layers"])
    assert n_slots == 3
    assert slot_of["in"] == B.SLOT_INPUT and slot_of["out"] == B.SLOT_OUTPUT
    # no layer reads and writes the same slot unless it accumulates into it
    for L in net["layers"]:
        assert slot_of[L["src"]] != slot_of[L["dst"]]
    # a chain needs three: a slot is reused two layers on, so that a pair of layers run as one fused layer never
    # writes the tensor it reads
    assert assign_slots(configs.dwsep_cnn()["layers"])[1] == 3
    # descriptors -> bytes: one conv 16->16 on 32x32 at N=2 from slot 0 to slot 1
    L = B.small_layer()
    L.op, L.C, L.K, L.H, L.W, L.FH, L.FW, L.stride = B.OP_CONV, 16, 16, 32, 32, 3, 3, 1
    L.pad_t = L.pad_b = L.pad_l = L.pad_r = 1
    L.src, L.dst = 0, 1
    arr = (B.small_layer * 1)(L)
    assert B.small_net_workspace_bytes(arr, 2) == 2 * (2 * 32 * 32 * 32 * 4)
    L.pad_t = 3   # pad >= window: malformed
    arr = (B.small_layer * 1)(L)
    assert B.small_net_workspace_bytes(arr, 2) == 0
