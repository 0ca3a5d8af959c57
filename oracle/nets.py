"""Runs a synth.configs network through the CPU oracle, layer by layer, in NCHW.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  Returns every named tensor so that
tests can compare intermediates as well as the final result.
"""
from __future__ import annotations

import numpy as np

from . import conv2d, dwconv2d, fc, pool2d, out_size


def run_net(net, params, x, keep_all=True, f32acc=False, init=None):
    """x: [N][C][H][W] float32.  Returns dict name -> NCHW array ('out' is the result;
    an FC result is [N][K][1][1]).  init: named tensors that exist before the first layer
    (the target of an accumulating layer when a sub-list of a network is run)."""
    t = {"in": np.ascontiguousarray(x, dtype=np.float32)}
    if init:
        t.update({k: np.ascontiguousarray(v, dtype=np.float32) for k, v in init.items()})
    for layer, (w, b) in zip(net["layers"], params):
        src = t[layer["src"]]
        op = layer["op"]
        if op == "conv":
            acc = t[layer["dst"]] if layer["accumulate"] else None
            y = conv2d(src, w, b, layer["stride"], layer["pad"], layer["relu"], accumulate_into=acc, f32acc=f32acc)
        elif op == "dwconv":
            y = dwconv2d(src, w, b, layer["stride"], layer["pad"], layer["relu"])
        elif op == "pool":
            fh, fw = layer["FH"], layer["FW"]
            if fh == 0:
                fh, fw = src.shape[2], src.shape[3]
            y = pool2d(src, fh, fw, layer["stride"], layer["pad"], layer["pool"])
        elif op == "fc":
            y = fc(src, w, b, layer["relu"]).reshape(src.shape[0], layer["K"], 1, 1)
        else:
            raise ValueError(op)
        t[layer["dst"]] = y
        if not keep_all and layer["src"] not in ("in",) and layer["src"] != layer["dst"]:
            pass
    return t


def shapes(net, batch=None):
    """Per-layer (C, H, W) -> (K, OH, OW), from the oracle's own size rule."""
    n = net["batch"] if batch is None else batch
    dims = {"in": tuple(net["input"])}
    rows = []
    for layer in net["layers"]:
        c, h, w = dims[layer["src"]]
        fh, fw = layer["FH"], layer["FW"]
        if layer["op"] == "pool" and fh == 0:
            fh, fw = h, w
        if layer["op"] == "fc":
            oh = ow = 1
        else:
            pt, pb, pl, pr = layer["pad"]
            oh, ow = out_size(h, fh, layer["stride"], pt, pb), out_size(w, fw, layer["stride"], pl, pr)
        dims[layer["dst"]] = (layer["K"], oh, ow)
        rows.append(dict(name=layer["name"], op=layer["op"], N=n, inp=(c, h, w), out=(layer["K"], oh, ow), F=(fh, fw)))
    return rows


def buffer_plan(net):
    """Section 5.3's float memory model on one image: (parameter count incl. biases excluded,
    largest input+output element pair over the layers, model input elements)."""
    rows = shapes(net, 1)
    largest = max(int(np.prod(r["inp"])) + int(np.prod(r["out"])) for r in rows)
    weights = 0
    biases = 0
    for layer in net["layers"]:
        if layer["op"] == "conv":
            weights += layer["K"] * layer["C"] * layer["FH"] * layer["FW"]
            biases += layer["K"]
        elif layer["op"] == "dwconv":
            weights += layer["C"] * layer["FH"] * layer["FW"]
            biases += layer["C"]
        elif layer["op"] == "fc":
            weights += layer["K"] * layer["C"]
            biases += layer["K"]
    return dict(weights=weights, biases=biases, largest_pair=largest, model_input=int(np.prod(net["input"])))
