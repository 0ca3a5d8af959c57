"""Workload descriptions: shapes and layer lists only, no arithmetic.

A network is a list of layer dicts over named tensors.  Keys:
  op        "conv" | "dwconv" | "pool" | "fc"
  name      label used in reports
  src, dst  tensor names ("in" is the network input, "out" the result)
  C, K      input / output channels (K == C for dwconv and pool)
  FH, FW    window; stride; pad = (top, bottom, left, right)
  relu      apply max(x, 0) to the result
  accumulate  dst already holds a tensor of the output's shape; the layer adds
              its result to it (the residual join) before the optional ReLU
  pool      "max" | "avg" (op == "pool"); FH = FW = 0 means the whole plane
Spatial sizes are not stored: they follow from the input size and the
window / stride / pad of each layer.

The four networks take the tensor shapes of the MLPerf-Tiny models the paper
evaluates (Section 5.1.1) as sized by this project's workload list; weights are
synthetic (He-normal), never trained values.
"""
from __future__ import annotations

from . import he_normal, normal, uniform, DEFAULT_SEED

P0 = (0, 0, 0, 0)
P1 = (1, 1, 1, 1)


def _conv(name, src, dst, C, K, F, stride, pad, relu, accumulate=False):
    fh, fw = (F, F) if isinstance(F, int) else F
    return dict(op="conv", name=name, src=src, dst=dst, C=C, K=K, FH=fh, FW=fw, stride=stride,
                pad=tuple(pad), relu=relu, accumulate=accumulate)


def _dw(name, src, dst, C, stride, relu=True):
    return dict(op="dwconv", name=name, src=src, dst=dst, C=C, K=C, FH=3, FW=3, stride=stride,
                pad=P1, relu=relu, accumulate=False)


def _gap(name, src, dst, C):
    return dict(op="pool", name=name, src=src, dst=dst, C=C, K=C, FH=0, FW=0, stride=1, pad=P0,
                relu=False, accumulate=False, pool="avg")


def _fc(name, src, dst, J, K, relu=False):
    return dict(op="fc", name=name, src=src, dst=dst, C=J, K=K, FH=1, FW=1, stride=1, pad=P0,
                relu=relu, accumulate=False)


def single_conv_pool():
    """3x3 conv + bias + ReLU on 1x16x32x32, then 2x2 stride-2 max pool (the small parity case)."""
    layers = [
        _conv("conv3x3", "in", "a", 16, 16, 3, 1, P1, True),
        dict(op="pool", name="maxpool2x2", src="a", dst="out", C=16, K=16, FH=2, FW=2, stride=2, pad=P0,
             relu=False, accumulate=False, pool="max"),
    ]
    return dict(name="single_conv_pool", batch=1, input=(16, 32, 32), input_dist=("uniform", -1.0, 1.0),
                weight_dist="uniform", layers=layers)


def residual_cnn(batch=256):
    """8-layer residual CNN on 3x32x32 (the ResNet-shaped model, Section 5.1.1): a 3x3 stem, three
    stages of two 3x3 convolutions whose second one joins the stage input (identity, or a 1x1
    stride-2 convolution when the size changes), global average pool, FC 64->10."""
    L = [_conv("stem", "in", "x1", 3, 16, 3, 1, P1, True)]
    # stage 1: identity shortcut, join in place on the stage input
    L += [_conv("s1a", "x1", "a1", 16, 16, 3, 1, P1, True),
          _conv("s1b", "a1", "x1", 16, 16, 3, 1, P1, True, accumulate=True)]
    # stage 2: 16 -> 32, stride 2
    L += [_conv("s2a", "x1", "a2", 16, 32, 3, 2, P1, True),
          _conv("s2sc", "x1", "x2", 16, 32, 1, 2, P0, False),
          _conv("s2b", "a2", "x2", 32, 32, 3, 1, P1, True, accumulate=True)]
    # stage 3: 32 -> 64, stride 2
    L += [_conv("s3a", "x2", "a3", 32, 64, 3, 2, P1, True),
          _conv("s3sc", "x2", "x3", 32, 64, 1, 2, P0, False),
          _conv("s3b", "a3", "x3", 64, 64, 3, 1, P1, True, accumulate=True)]
    L += [_gap("gap", "x3", "g", 64), _fc("fc", "g", "out", 64, 10)]
    return dict(name="residual_cnn", batch=batch, input=(3, 32, 32), input_dist=("uniform", 0.0, 1.0),
                weight_dist="he_normal", layers=L)


def dwsep_cnn(batch=64):
    """Depthwise-separable CNN on 3x96x96 (the MobileNet-shaped model at quarter width)."""
    outs = [16, 32, 32, 64, 64, 128, 128, 128, 128, 128, 128, 256, 256]
    stride2 = {2, 4, 6, 12}
    L = [_conv("stem", "in", "p0", 3, 8, 3, 2, P1, True)]
    c, cur = 8, "p0"
    for i, k in enumerate(outs, 1):
        L.append(_dw(f"b{i}dw", cur, f"d{i}", c, 2 if i in stride2 else 1))
        L.append(_conv(f"b{i}pw", f"d{i}", f"p{i}", c, k, 1, 1, P0, True))
        c, cur = k, f"p{i}"
    L += [_gap("gap", cur, "g", c), _fc("fc", "g", "out", c, 2)]
    return dict(name="dwsep_cnn", batch=batch, input=(3, 96, 96), input_dist=("uniform", 0.0, 1.0),
                weight_dist="he_normal", layers=L)


def kws_cnn(batch=1024):
    """Keyword-spotting-shaped depthwise-separable CNN on 1x49x10 (the DS-CNN-shaped model).
    The 10x4 stride-2 stem uses 'same' padding: 49x10 -> 25x5 needs pads top 4, bottom 5, left 1, right 1."""
    L = [_conv("stem", "in", "p0", 1, 64, (10, 4), 2, (4, 5, 1, 1), True)]
    cur = "p0"
    for i in range(1, 5):
        L.append(_dw(f"b{i}dw", cur, f"d{i}", 64, 1))
        L.append(_conv(f"b{i}pw", f"d{i}", f"p{i}", 64, 64, 1, 1, P0, True))
        cur = f"p{i}"
    L += [_gap("gap", cur, "g", 64), _fc("fc", "g", "out", 64, 12)]
    return dict(name="kws_cnn", batch=batch, input=(1, 49, 10), input_dist=("normal", 0.0, 1.0),
                weight_dist="he_normal", layers=L)


def autoencoder_fc(batch=4096):
    """Fully-connected autoencoder on 640 features (the Deep-Autoencoder-shaped model, Section 5.1.1): an encoder of
    four 128-wide layers, an 8-wide bottleneck, a mirrored decoder; ReLU after every layer but the last (normalisation
    folded into the biases).  Every layer is a full reduction (Table 1) over a 1x1 plane."""
    widths = [640, 128, 128, 128, 128, 8, 128, 128, 128, 128, 640]
    L, cur = [], "in"
    for i in range(1, len(widths)):
        last = i == len(widths) - 1
        dst = "out" if last else f"h{i}"
        L.append(_fc(f"fc{i}", cur, dst, widths[i - 1], widths[i], relu=not last))
        cur = dst
    return dict(name="autoencoder_fc", batch=batch, input=(640, 1, 1), input_dist=("normal", 0.0, 1.0),
                weight_dist="he_normal", layers=L)


NETWORKS = {"single_conv_pool": single_conv_pool, "residual_cnn": residual_cnn,
            "dwsep_cnn": dwsep_cnn, "kws_cnn": kws_cnn, "autoencoder_fc": autoencoder_fc}

# GPU-scale layer sweep: batch 128, C = K, square planes, stride 1 (conv3x3 / depthwise pad 1, conv1x1 pad 0)
SWEEP_BATCH = 128
SWEEP_SIZES = [(64, 56), (128, 28), (256, 14), (512, 7)]
SWEEP_KINDS = ["conv3x3", "conv1x1", "dw3x3", "maxpool2x2", "relu"]


def weight_shape(layer):
    if layer["op"] == "conv":
        return (layer["K"], layer["C"], layer["FH"], layer["FW"])
    if layer["op"] == "dwconv":
        return (layer["C"], layer["FH"], layer["FW"])
    if layer["op"] == "fc":
        return (layer["K"], layer["C"])
    return None


def fan_in(layer):
    if layer["op"] == "conv":
        return layer["C"] * layer["FH"] * layer["FW"]
    if layer["op"] == "dwconv":
        return layer["FH"] * layer["FW"]
    return layer["C"]


def make_params(net, seed=DEFAULT_SEED):
    """Per-layer (weights, bias) in the natural NCHW-side shapes; None for layers without weights.
    Every weighted layer gets a bias (uniform[-0.1, 0.1]; uniform[-1, 1] for the single-conv case)."""
    params = []
    for i, layer in enumerate(net["layers"]):
        shp = weight_shape(layer)
        if shp is None:
            params.append((None, None))
            continue
        if net["weight_dist"] == "uniform":
            w = uniform(shp, -1.0, 1.0, 10 + 4 * i, seed)
            b = uniform((layer["K"],), -1.0, 1.0, 11 + 4 * i, seed)
        else:
            w = he_normal(shp, fan_in(layer), 10 + 4 * i, seed)
            b = uniform((layer["K"],), -0.1, 0.1, 11 + 4 * i, seed)
        params.append((w, b))
    return params


def make_input(net, batch=None, seed=DEFAULT_SEED):
    n = net["batch"] if batch is None else batch
    shape = (n,) + tuple(net["input"])
    kind, a, b = net["input_dist"]
    if kind == "uniform":
        return uniform(shape, a, b, 1, seed)
    return normal(shape, a, b, 1, seed)
