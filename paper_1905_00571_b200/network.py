"""Marshalling helpers: turn a synthetic model description (workloads.models.Model)
into packed layers, device-resident epilogue vectors and a cadnn_net.  No layer
arithmetic happens here; every op runs inside the CUDA library."""
import numpy as np
import torch

from . import binding as B


def desc_for(op, dtype, batch_hint=1, autotune=False):
    if op.kind == "fc":
        return B.make_desc(op.c_in, op.c_out, 1, 1, 1, 0, 1, 1, 1, batch_hint, dtype, autotune=autotune)
    kh, kw = int(op.w.shape[1]), int(op.w.shape[2])   # rectangular kernels carry their own shape
    return B.make_desc(op.c_in, op.c_out, kh, kw, op.stride, op.pad, op.groups,
                       op.in_hw[0], op.in_hw[1], batch_hint, dtype, autotune=autotune, pad_w=getattr(op, "pad_w", -1),
                       fmt=B.FMT_GROUPED if getattr(op, "fmt", "auto") == "grouped" else 0)


def pack_op(op, dtype, batch_hint=1, autotune=False):
    dtype = "s8" if op.w.dtype == np.int8 else "f32"   # (an int8 network may end in float layers)
    d = desc_for(op, dtype, batch_hint, autotune)
    if op.w.dtype == np.int8:
        return B.cadnn_pack_q8(d, op.w, op.mask)
    return B.cadnn_pack(d, op.w, op.mask)


class PackedModel:
    """Packed weights + device epilogue vectors + cadnn_net for one batch size."""

    def __init__(self, model, batch=1, device="cuda:0", autotune=False):
        self.model = model
        self.batch = batch
        self.device = torch.device(device)
        self.weights = {}
        self.vecs = {}
        ops = []
        with torch.cuda.device(self.device):
            for i, op in enumerate(model.ops):
                if op.kind in ("conv", "fc"):
                    w = pack_op(op, model.dtype, batch, autotune)
                    self.weights[i] = w
                    sc = None if op.scale is None else torch.from_numpy(op.scale).to(self.device)
                    bi = None if op.bias is None else torch.from_numpy(op.bias).to(self.device)
                    self.vecs[i] = (sc, bi)
                    ops.append(B.Op(B.OP_CONV if op.kind == "conv" else B.OP_FC, w.handle, op.src, op.dst, op.res,
                                    None if sc is None else sc.data_ptr(), None if bi is None else bi.data_ptr(),
                                    B.ACT[op.act], B.DTYPE[op.out], 0, 0, 0, float(op.res_scale), op.dst_off, op.dst_total))
                elif op.kind in ("maxpool", "avgpool"):
                    ops.append(B.Op(B.OP_MAXPOOL if op.kind == "maxpool" else B.OP_AVGPOOL, None, op.src, op.dst, -1, None, None,
                                    0, B.DTYPE[model.dtype], op.k, op.stride, op.pad, 0.0, op.dst_off, op.dst_total))
                elif op.kind == "gavgpool":
                    ops.append(B.Op(B.OP_GAVGPOOL, None, op.src, op.dst, -1, None, None, 0, B.F32, 0, 0, 0, 0.0, 0, 0))
                else:
                    raise ValueError(op.kind)
            h, w_, c = model.in_shape
            self.ops = ops
            self.net = B.cadnn_net_create(ops, batch, h, w_, c, model.dtype, keep=(self.weights, self.vecs))
        last = model.ops[-1]
        self.out_shape = (batch, last.c_out) if last.kind in ("fc", "gavgpool") else (batch, last.out_hw[0], last.out_hw[1], last.c_out)
        self.out_dtype = {"f32": torch.float32, "s8": torch.int8, "s32": torch.int32}[last.out]

    def new_output(self):
        return torch.empty(self.out_shape, dtype=self.out_dtype, device=self.device)

    def forward(self, x, y=None, use_graph=True, stream=None):
        if y is None:
            y = self.new_output()
        return B.cadnn_forward(self.net, x, y, use_graph, stream)

    def forward_static(self, x, y, stream=None):
        """Same layers through cadnn_forward_static (no allocation; any batch that fits the fixed workspace)."""
        return B.cadnn_forward_static(self.ops, x, y, self.model.dtype, stream)

    def forward_host(self, x_host, y_host, use_graph=True, stream=None):
        return B.cadnn_forward_host(self.net, x_host, y_host, use_graph, stream)

    def launches_per_forward(self):
        """Kernel launches one forward issues (cadnn_net_info)."""
        return B.cadnn_net_info(self.net)["launches"]

    def layer_times(self, x, y, flush_l2=False, reps=1):
        return B.cadnn_net_layer_times(self.net, x, y, len(self.model.ops), flush_l2, reps)
