"""Whole-network walker of the CPU oracle (test infrastructure only).

Chains the plain C layer routines over an op list (``workloads.models.Model``),
feeding its own outputs forward, and keeps every intermediate tensor so that a
single layer of the CUDA library can be checked on oracle-produced inputs.

Pins (tests/test_oracle_pins.py): a hand-worked literal network
(tests/golden/walker_handworked.json) and float / int8 multi-op models whose every
slot equals the composition of the layer routines written out call by call.
"""
import numpy as np
from . import ref


def _pad(op):
    pw = getattr(op, "pad_w", -1)
    return op.pad if pw is None or pw < 0 else (op.pad, pw)


def run_op(op, x, residual=None):
    """Apply one op to numpy input x (NHWC, or [n,k] for fc)."""
    if op.kind == "conv":
        if op.w.dtype == np.int8:
            return ref.conv2d_s8(x, op.w, op.mask, op.stride, op.pad, op.groups,
                                 op.scale, op.bias, op.act, op.out,
                                 residual, getattr(op, "res_scale", 0.0))
        return ref.conv2d_f32(x, op.w, op.mask, op.stride, _pad(op), op.groups,
                              op.scale, op.bias, residual, op.act)
    if op.kind == "fc":
        n = x.shape[0]
        x2 = x.reshape(n, -1)
        w2 = op.w.reshape(op.c_out, -1)
        m2 = None if op.mask is None else op.mask.reshape(op.c_out, -1)
        if op.w.dtype == np.int8:
            return ref.fc_s8(x2, w2, m2, op.scale, op.bias, op.act, op.out)
        return ref.fc_f32(x2, w2, m2, op.scale, op.bias, residual, op.act)
    if op.kind == "maxpool":
        return ref.maxpool(x, op.k, op.stride, op.pad)
    if op.kind == "avgpool":
        return ref.avgpool(x, op.k, op.stride, op.pad)
    if op.kind == "gavgpool":
        return ref.gavgpool(x)
    raise ValueError(op.kind)


def forward(model, x):
    """Returns (output of the last op, {slot: tensor}).

    An op with ``dst_total > 0`` writes channels [dst_off, dst_off + c) of a slot
    that has dst_total channels: the channel concatenation of an Inception
    module is several ops writing windows of one slot."""
    slots = {0: x}
    y = x
    for op in model.ops:
        res = slots[op.res] if op.res >= 0 else None
        y = run_op(op, slots[op.src], res)
        total = getattr(op, "dst_total", 0)
        if total:
            if op.dst not in slots:
                slots[op.dst] = np.zeros(y.shape[:-1] + (total,), y.dtype)
            off = op.dst_off
            assert slots[op.dst].shape[:-1] == y.shape[:-1] and off + y.shape[-1] <= total
            slots[op.dst][..., off:off + y.shape[-1]] = y
            y = slots[op.dst]
        else:
            slots[op.dst] = y
    return y, slots
