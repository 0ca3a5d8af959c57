"""Turns a layer list (dicts with op / src / dst / C / K / FH / FW / stride / pad / relu / accumulate / pool) into
the small_layer descriptors of small_run_net: packs the filters once through the library, assigns named tensors
to workspace slots and allocates the workspace with torch.  Host-side bookkeeping only."""
from __future__ import annotations

import torch

from . import binding as B


def assign_slots(layers):
    """Greedy slot reuse by liveness: a tensor's slot is free again one layer after its last reader (so the output of the
    layer behind it never lands on it: the library may run those two layers as one fused layer, which must not write the
    tensor it reads); a layer never writes the slot it reads (only accumulate updates its destination in place).
    'in' / 'out' are the caller's."""
    last_use = {}
    for i, L in enumerate(layers):
        last_use[L["src"]] = i
        if L.get("accumulate"):
            last_use[L["dst"]] = i
    slot_of, free, pending, n_slots = {"in": B.SLOT_INPUT, "out": B.SLOT_OUTPUT}, [], [], 0
    for i, L in enumerate(layers):
        dst = L["dst"]
        if dst not in slot_of:
            if free:
                slot_of[dst] = free.pop(0)
            else:
                slot_of[dst] = n_slots
                n_slots += 1
        free += pending                       # slots whose last reader was the previous layer
        pending = []
        name = L["src"]
        if last_use.get(name) == i and slot_of.get(name, -1) >= 0 and name != dst:
            pending.append(slot_of[name])
    return slot_of, n_slots


class Net:
    """A network resident on the device: packed filters, plain layer descriptors and workspace.  Which neighbouring
    layers run as one fused layer is the library's decision inside small_run_net; fuse_dwpw (True: where it pays, "all":
    wherever the fused kernel takes the shape, False: never) and fuse_convpool only select the library's fusion setting
    for this network's runs."""

    def __init__(self, ctx, net, params, batch=None, math="fp32", device="cuda", fuse_dwpw=True, fuse_convpool=True, fuse_fc_chain=True, fuse_poolfc=True):
        self.ctx = ctx
        self.N = net["batch"] if batch is None else batch
        self.in_shape = tuple(net["input"])
        self.math = B.MATH[math]
        self.fusion = ((B.FUSE_DWPW_ALWAYS if fuse_dwpw == "all" else B.FUSE_DWPW if fuse_dwpw else 0)
                       | (B.FUSE_CONVPOOL if fuse_convpool else 0) | (B.FUSE_FC_CHAIN if fuse_fc_chain else 0)
                       | (B.FUSE_POOLFC if fuse_poolfc else 0))
        self.keep = []            # device tensors the descriptors point into
        self._offsets = None
        layers_in = net["layers"]
        slot_of, _ = assign_slots(layers_in)
        self.slot_of = slot_of
        dims = {"in": self.in_shape}
        descs = []
        self.layer_rows = []
        for li, (L, (w, b)) in enumerate(zip(layers_in, params)):
            c, h, wd = dims[L["src"]]
            fh, fw = L["FH"], L["FW"]
            if L["op"] == "pool" and fh == 0:
                fh, fw = h, wd
            pt, pb, pl, pr = L["pad"]
            d = B.small_layer()
            d.C, d.K, d.H, d.W, d.FH, d.FW, d.stride = L["C"], L["K"], h, wd, fh, fw, L["stride"]
            d.pad_t, d.pad_b, d.pad_l, d.pad_r = pt, pb, pl, pr
            d.src, d.dst, d.src2 = slot_of[L["src"]], slot_of.get(L["dst"], 0), 0
            flags = (B.RELU if L["relu"] else 0) | (B.ACCUMULATE if L.get("accumulate") else 0)
            wt = None if w is None else torch.from_numpy(w).to(device)
            bt = None if b is None else torch.from_numpy(b).to(device)
            oh, ow = B.small_out_size(h, fh, L["stride"], pt, pb), B.small_out_size(wd, fw, L["stride"], pl, pr)
            if L["op"] == "conv":
                d.op = B.OP_CONV
                flags |= self.math
                wb = torch.empty(B.small_conv_weight_elems(L["C"], L["K"], fh, fw, self.math), device=device)
                B.small_pack_conv_weights(ctx, wt, wb, L["C"], L["K"], fh, fw, self.math)
            elif L["op"] == "dwconv":
                d.op = B.OP_DWCONV
                wb = torch.empty(B.small_dw_weight_elems(L["C"], fh, fw), device=device)
                B.small_pack_dw_weights(ctx, wt, wb, L["C"], fh, fw)
            elif L["op"] == "pool":
                d.op = B.OP_POOL
                d.pool_mode = B.POOL_MAX if L["pool"] == "max" else B.POOL_AVG
                wb = None
            elif L["op"] == "fc":
                d.op = B.OP_FC
                flags |= self.math
                wb = torch.empty(B.small_fc_weight_elems(L["C"], L["K"], self.math), device=device)
                B.small_pack_fc_weights(ctx, wt, wb, L["C"], L["K"], self.math)
                oh = ow = 1
            else:
                raise ValueError(L["op"])
            d.flags = flags
            d.w_blk = None if wb is None else wb.data_ptr()
            d.bias = None if bt is None else bt.data_ptr()
            self.keep += [wb, bt, wt]
            dims[L["dst"]] = (L["K"], oh, ow)
            self.layer_rows.append(dict(name=L["name"], op=L["op"], C=L["C"], K=L["K"], H=h, W=wd, FH=fh, FW=fw,
                                        stride=L["stride"], pad=L["pad"], OH=oh, OW=ow, dst=L["dst"], first=li, upto=li + 1))
            descs.append(d)
        torch.cuda.synchronize()
        self.dims = dims
        self.out_shape = dims["out"]
        self.layers = (B.small_layer * len(descs))(*descs)
        self.ws_bytes = B.small_net_workspace_bytes(self.layers, self.N)
        c, h, w = self.in_shape
        oc, oh, ow = self.out_shape
        self.stage_bytes = B.small_net_host_staging_bytes(self.N, c, h, w, oc, oh, ow)
        self.workspace = torch.empty(self.ws_bytes + self.stage_bytes + 256, dtype=torch.uint8, device=device)
        assert self.workspace.data_ptr() % 256 == 0
        self.out_blk = torch.empty(B.small_packed_elems(self.N, oc, oh, ow), device=device)

    def launches(self):
        """Kernel launches of one run under this network's fusion setting."""
        B.small_set_net_fusion(self.ctx, self.fusion)
        try:
            return B.small_net_launches(self.ctx, self.layers, self.N)
        finally:
            B.small_set_net_fusion(self.ctx, B.FUSE_DEFAULT)

    def run(self, in_blk, out_blk=None, stream=None, n_layers=None):
        """Runs all layers (or the first n_layers, to inspect an intermediate)."""
        out_blk = self.out_blk if out_blk is None else out_blk
        layers = self.layers if n_layers is None else (B.small_layer * n_layers)(*self.layers[:n_layers])
        B.small_set_net_fusion(self.ctx, self.fusion)
        try:
            B.small_run_net(self.ctx, layers, self.N, in_blk, out_blk, self.workspace, self.ws_bytes, stream)
        finally:
            B.small_set_net_fusion(self.ctx, B.FUSE_DEFAULT)
        return out_blk

    def run_host(self, in_host, out_host, stream=None):
        c, h, w = self.in_shape
        oc, oh, ow = self.out_shape
        B.small_set_net_fusion(self.ctx, self.fusion)
        try:
            B.small_run_net_host(self.ctx, self.layers, self.N, in_host, c, h, w, out_host, oc, oh, ow,
                                 self.workspace, self.ws_bytes + self.stage_bytes, stream)
        finally:
            B.small_set_net_fusion(self.ctx, B.FUSE_DEFAULT)

    def slot_ptr(self, slot, in_blk, out_blk):
        if slot == B.SLOT_INPUT:
            return in_blk.data_ptr()
        if slot == B.SLOT_OUTPUT:
            return out_blk.data_ptr()
        if self._offsets is None:
            self._offsets = self.slot_offsets()
        return self.workspace.data_ptr() + self._offsets[slot]

    def run_layer(self, i, in_blk, out_blk=None, stream=None):
        """Launches layer i alone through its own entry point, on the same buffers small_run_net would use."""
        out_blk = self.out_blk if out_blk is None else out_blk
        L, N = self.layers[i], self.N
        src, dst = self.slot_ptr(L.src, in_blk, out_blk), self.slot_ptr(L.dst, in_blk, out_blk)
        pad = (L.pad_t, L.pad_b, L.pad_l, L.pad_r)
        if L.op == B.OP_CONV:
            B.small_conv2d(self.ctx, src, L.w_blk, L.bias, dst, N, L.C, L.K, L.H, L.W, L.FH, L.FW, L.stride, pad, L.flags, stream)
        elif L.op == B.OP_DWCONV:
            B.small_dwconv2d(self.ctx, src, L.w_blk, L.bias, dst, N, L.C, L.H, L.W, L.FH, L.FW, L.stride, pad, L.flags, stream)
        elif L.op == B.OP_POOL:
            B.small_pool2d(self.ctx, src, dst, None, N, L.C, L.H, L.W, L.FH, L.FW, L.stride, pad, L.pool_mode, stream)
        elif L.op == B.OP_FC:
            B.small_fc(self.ctx, src, L.w_blk, L.bias, dst, N, L.C, L.K, L.flags, stream)
        elif L.op == B.OP_DWPW:
            B.small_dwpw_conv2d(self.ctx, src, L.w_blk, L.bias, L.w_blk2, L.bias2, dst, None, N, L.C, L.K, L.H, L.W, L.stride, pad,
                                L.flags, stream)
        elif L.op == B.OP_CONVPOOL:
            B.small_conv_maxpool2d(self.ctx, src, L.w_blk, L.bias, dst, None, N, L.C, L.K, L.H, L.W, L.FH, L.FW, L.stride, pad, L.flags, stream)
        else:
            raise ValueError(L.op)

    def slot_offsets(self):
        """Byte offset of every slot, by the library's rule: sizes rounded up to 256 bytes, back to back."""
        sizes = {}
        for L, row in zip(self.layers, self.layer_rows):
            if L.src >= 0:
                sizes[L.src] = max(sizes.get(L.src, 0), 4 * B.small_packed_elems(self.N, L.C, L.H, L.W))
            if L.dst >= 0:
                sizes[L.dst] = max(sizes.get(L.dst, 0), 4 * B.small_packed_elems(self.N, row["K"], row["OH"], row["OW"]))
        offs, off = {}, 0
        for s in range(max(sizes) + 1 if sizes else 0):
            offs[s] = off
            off += ((sizes.get(s, 0) + 255) // 256) * 256
        return offs

    def slot_tensor(self, name):
        """View of a named intermediate inside the workspace (valid right after the layer that wrote it)."""
        slot = self.slot_of[name]
        c, h, w = self.dims[name]
        n = B.small_packed_elems(self.N, c, h, w)
        off = self.slot_offsets()[slot]
        return self.workspace[off:off + 4 * n].view(torch.float32)
