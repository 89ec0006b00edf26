"""Run a layer stack (dsq_inputs.Stack) through the C-ABI library.

Marshalling only: weights are packed once with dsq_pack_weights, every tensor
is a pre-allocated packed-code buffer, and a forward pass is one
dsq_quantize_act followed by one dsq_conv2d / dsq_dwconv2d / dsq_maxpool2x2
call per layer on the current stream.  No fp32 activation tensor is written
between layers.  The call sequence can be captured in a CUDA graph.
"""
import numpy as np
import torch

from . import binding as B


def _delta_f32(bits, lo, hi):
    return (np.float32(hi) - np.float32(lo)) / np.float32(2 ** bits - 1)


class GpuStack:
    def __init__(self, st, params, batch=None, w_offset=0.5, device="cuda",
                 keep_debug=False):
        self.st, self.bits, self.w_offset = st, st.bits, w_offset
        self.batch = st.batch if batch is None else batch
        self.device = device
        self.keep_debug = keep_debug
        self.ws = B.new_workspace(device)
        bits = self.bits
        shapes = st.tensor_shapes()
        self.shapes = shapes
        self.ranges = {"in": (st.in_lo, st.in_hi)}
        self.codes = {}
        for name, (H, W, Cc) in shapes.items():
            self.codes[name] = torch.zeros(
                (self.batch, H, W, B.dsq_row_pitch(Cc, bits)),
                dtype=torch.uint8, device=device)
        self.layers = []
        for L in st.layers:
            if L.kind == "pool":
                self.ranges[L.dst] = self.ranges[L.src]
                self.layers.append((L, None))
                continue
            p = params[L.name]
            a_lo, a_hi = self.ranges[L.src]
            w = torch.from_numpy(p["w"]).to(device)
            per_ch = p["w_hi"].size > 1
            if per_ch:
                lo = torch.from_numpy(p["w_lo"]).to(device)
                hi = torch.from_numpy(p["w_hi"]).to(device)
            else:
                lo, hi = float(p["w_lo"][0]), float(p["w_hi"][0])
            blob, conv = B.dsq_pack_weights(w, bits, lo, hi, self.ws,
                                            depthwise=(L.kind == "dw"),
                                            stride=L.stride, pad=L.pad)
            da = _delta_f32(bits, a_lo, a_hi)
            w_lo = np.broadcast_to(p["w_lo"], (L.cout,)).astype(np.float32)
            w_hi = np.broadcast_to(p["w_hi"], (L.cout,)).astype(np.float32)
            dw = ((w_hi - w_lo) / np.float32(2 ** bits - 1)).astype(np.float32)
            scale = torch.from_numpy((da * dw).astype(np.float32)).to(device)
            bias = torch.from_numpy(p["bias"]).to(device)
            self.ranges[L.dst] = (L.out_lo, L.out_hi)
            self.layers.append((L, dict(blob=blob, conv=conv, scale=scale,
                                        bias=bias)))
        B.check_workspace(self.ws, "dsq_pack_weights")
        self.debug = {}

    def forward(self, x):
        """x: fp32 NHWC CUDA tensor, or None to run the layers on the input
        codes already in place.  Returns the packed codes of st.out."""
        st, bits = self.st, self.bits
        if x is not None:
            B.dsq_quantize_act(x, bits, st.in_lo, st.in_hi, out=self.codes["in"])
        for L, w in self.layers:
            H, W, Cc = self.shapes[L.src]
            shape = (self.batch, H, W, Cc)
            src = self.codes[L.src]
            if L.kind == "pool":
                B.dsq_maxpool2x2(src, shape, bits, out=self.codes[L.dst])
                continue
            a_lo, a_hi = self.ranges[L.src]
            res = res_q = None
            if L.residual is not None:
                res = self.codes[L.residual]
                res_q = (bits,) + tuple(self.ranges[L.residual])
            kw = dict(w_offset=self.w_offset, residual=res, residual_q=res_q,
                      requant=(bits, L.out_lo, L.out_hi),
                      want_f32=self.keep_debug, want_acc=self.keep_debug,
                      out_codes=self.codes[L.dst])
            if L.kind == "dw":
                _, y, acc = B.dsq_dwconv2d(src, shape, (bits, a_lo, a_hi),
                                           w["blob"], w["conv"], w["scale"],
                                           w["bias"], **kw)
            else:
                _, y, acc = B.dsq_conv2d(src, shape, (bits, a_lo, a_hi),
                                         w["blob"], w["conv"], w["scale"],
                                         w["bias"], self.ws, **kw)
            if self.keep_debug:
                self.debug["y:" + L.name] = y
                self.debug["acc:" + L.name] = acc
        return self.codes[st.out]

    def n_launches(self):
        """Kernels launched by one forward pass."""
        return 1 + len(self.layers)

    def unpack(self, name):
        """int8 codes [batch, H, W, C] of a tensor (test aid)."""
        H, W, Cc = self.shapes[name]
        rows = self.batch * H * W
        return B.dsq_unpack(self.codes[name].view(rows, -1), rows, Cc,
                            self.bits, False).view(self.batch, H, W, Cc)

    def check(self):
        B.check_workspace(self.ws, "stack forward")
