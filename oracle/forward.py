"""Whole-network walker of the CPU oracle (test infrastructure only).

Chains the plain C layer routines over an op list (``workloads.models.Model``),
feeding its own outputs forward, and keeps every intermediate tensor so that a
single layer of the CUDA library can be checked on oracle-produced inputs.
"""
import numpy as np
from . import ref


def run_op(op, x, residual=None):
    """Apply one op to numpy input x (NHWC, or [n,k] for fc)."""
    if op.kind == "conv":
        if op.w.dtype == np.int8:
            return ref.conv2d_s8(x, op.w, op.mask, op.stride, op.pad, op.groups,
                                 op.scale, op.bias, op.act, op.out)
        return ref.conv2d_f32(x, op.w, op.mask, op.stride, op.pad, op.groups,
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
    if op.kind == "gavgpool":
        return ref.gavgpool(x)
    raise ValueError(op.kind)


def forward(model, x, keep=True):
    """Returns (output of the last op, {slot: tensor})."""
    slots = {0: x}
    y = x
    for op in model.ops:
        res = slots[op.res] if op.res >= 0 else None
        y = run_op(op, slots[op.src], res)
        slots[op.dst] = y
        if not keep:
            live = {o.src for o in model.ops} | {o.res for o in model.ops}
            # drop tensors no later op reads
            pass
    return y, slots
