"""Thin ctypes binding of the C ABI declared in include/cadnn.h.

Same names as the C entry points; argument marshalling only - every step of a
layer or network runs inside the CUDA library.  torch supplies device memory
and streams.  Importing this module fails if the library has not been built:
there is no fallback path.
"""
import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcadnn.so")
if not os.path.exists(LIB_PATH):
    raise ImportError("libcadnn.so is missing: run `python -m paper_1905_00571_b200.build` "
                      "(or __graft_entry__.build()) first; there is no fallback implementation")
_lib = ctypes.CDLL(LIB_PATH)

OK = 0
F32, S8, S32 = 0, 1, 2
DTYPE = {"f32": F32, "s8": S8, "s32": S32}
ACT = {"none": 0, "relu": 1, "relu6": 2, None: 0}
PACK_HOST_ONLY = 1
PACK_AUTOTUNE = 2
OP_CONV, OP_FC, OP_MAXPOOL, OP_GAVGPOOL, OP_AVGPOOL = 0, 1, 2, 3, 4
FMT_NAMES = {1: "tiled_csr", 2: "row_csr", 3: "dense_dw", 4: "dense_smallc", 5: "grouped"}
FMT_GROUPED = 5
KIND_NAMES = {1: "sconv_spatial", 2: "sconv_linear", 3: "fc_spmv", 4: "dw", 5: "dense_smallc"}


class LayerDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("c_in", "c_out", "kh", "kw", "stride", "pad", "groups", "in_h", "in_w",
                 "batch_hint", "dtype", "fmt", "flags", "pad_w")]


class Epilogue(ctypes.Structure):
    _fields_ = [("scale", ctypes.c_void_p), ("bias", ctypes.c_void_p), ("residual", ctypes.c_void_p),
                ("act", ctypes.c_int), ("out_dtype", ctypes.c_int), ("out_c_total", ctypes.c_int),
                ("out_c_off", ctypes.c_int), ("residual_scale", ctypes.c_float)]


class Op(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("w", ctypes.c_void_p), ("src", ctypes.c_int), ("dst", ctypes.c_int),
                ("res", ctypes.c_int), ("scale", ctypes.c_void_p), ("bias", ctypes.c_void_p),
                ("act", ctypes.c_int), ("out_dtype", ctypes.c_int), ("pool_k", ctypes.c_int),
                ("pool_stride", ctypes.c_int), ("pool_pad", ctypes.c_int), ("res_scale", ctypes.c_float),
                ("dst_c_off", ctypes.c_int), ("dst_c_total", ctypes.c_int)]


_vp, _i, _i64p = ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int64)
_SIGS = {
    "cadnn_pack": (_i, [ctypes.POINTER(LayerDesc), _vp, _vp, _vp, ctypes.POINTER(_vp)]),
    "cadnn_pack_q8": (_i, [ctypes.POINTER(LayerDesc), _vp, _vp, ctypes.POINTER(_vp)]),
    "cadnn_weights_info": (_i, [_vp, _i64p, _i64p, ctypes.POINTER(_i)]),
    "cadnn_weights_schedule": (_i, [_vp, ctypes.POINTER(_i)]),
    "cadnn_weights_planar_schedule": (_i, [_vp, ctypes.POINTER(_i)]),
    "cadnn_weights_warp_loads": (_i, [_vp, _i64p, _i, ctypes.POINTER(_i)]),
    "cadnn_weights_unpack": (_i, [_vp, _vp, _vp]),
    "cadnn_weights_free": (None, [_vp]),
    "cadnn_free_weights": (None, [_vp]),
    "cadnn_conv2d": (_i, [_vp, _vp, _i, _i, _i, _vp, ctypes.POINTER(Epilogue), _vp]),
    "cadnn_weights_workspace_bytes": (_i, [_vp, _i, _i64p]),
    "cadnn_conv2d_workspace": (_i, [_vp, _vp, _i, _i, _i, _vp, ctypes.POINTER(Epilogue), _vp, ctypes.c_int64, _vp]),
    "cadnn_weights_block_info": (_i, [_vp, ctypes.POINTER(_i), _i64p]),
    "cadnn_conv2d_planar": (_i, [_vp, _vp, _i, _vp, ctypes.POINTER(Epilogue), _vp]),
    "cadnn_fc": (_i, [_vp, _vp, _i, _vp, ctypes.POINTER(Epilogue), _vp]),
    "cadnn_maxpool2d": (_i, [_vp, _i, _i, _i, _i, _i, _i, _i, _i, _vp, _vp]),
    "cadnn_pool2d": (_i, [_vp, _i, _i, _i, _i, _i, _i, _i, _i, _i, _vp, _i, _i, _vp]),
    "cadnn_global_avgpool": (_i, [_vp, _i, _i, _i, _i, _vp, _vp]),
    "cadnn_net_create": (_i, [ctypes.POINTER(Op), _i, _i, _i, _i, _i, _i, ctypes.POINTER(_vp)]),
    "cadnn_forward": (_i, [_vp, _vp, _vp, _i, _vp]),
    "cadnn_forward_host": (_i, [_vp, _vp, _vp, _i, _vp]),
    "cadnn_forward_static": (_i, [ctypes.POINTER(Op), _i, _i, _i, _i, _i, _i, _vp, _vp, _vp]),
    "cadnn_net_info": (_i, [_vp, ctypes.POINTER(_i), _i64p]),
    "cadnn_net_layout": (_i, [_vp, ctypes.POINTER(_i), ctypes.POINTER(_i)]),
    "cadnn_net_parity_layers": (_i, [_vp, ctypes.POINTER(_i), ctypes.POINTER(_i), _i]),
    "cadnn_weights_parity_form": (_i, [_vp, ctypes.POINTER(_vp)]),
    "cadnn_net_layer_times": (_i, [_vp, _vp, _vp, _i, _i, ctypes.POINTER(ctypes.c_float), _vp]),
    "cadnn_net_layer_time": (_i, [_vp, _i, _vp, _vp, _i, _i, ctypes.POINTER(ctypes.c_float), _vp]),
    "cadnn_debug_set_device_status": (_i, [_i, _i]),
    "cadnn_measure_alu_peak": (_i, [_i, ctypes.POINTER(ctypes.c_double), _vp]),
    "cadnn_net_persistent_plan": (_i, [_vp, _i, ctypes.POINTER(_i)]),
    "cadnn_net_persistent_profile": (_i, [_vp, _i] + [ctypes.POINTER(ctypes.c_float)] * 5 + [ctypes.POINTER(_i)]),
    "cadnn_net_slot": (_i, [_vp, _i, ctypes.POINTER(_vp), _i64p]),
    "cadnn_net_free": (None, [_vp]),
    "cadnn_device_status": (_i, [ctypes.POINTER(_i)]),
    "cadnn_status_str": (ctypes.c_char_p, [_i]),
    "cadnn_last_cuda_error": (ctypes.c_char_p, []),
}
for _name, (_res, _args) in _SIGS.items():
    _fn = getattr(_lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args

EXPORTED = tuple(_SIGS)


class CadnnError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = "%s: %s" % (where, _lib.cadnn_status_str(status).decode())
        if status == 6:
            msg += " (%s)" % _lib.cadnn_last_cuda_error().decode()
        super().__init__(msg)


def _check(st, where):
    if st != OK:
        raise CadnnError(st, where)


def _np_ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _dev_ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if hasattr(stream, "cuda_stream"):
        return ctypes.c_void_p(stream.cuda_stream)
    return ctypes.c_void_p(int(stream))


class Weights:
    """Owner of a cadnn_weights handle."""

    def __init__(self, handle, desc):
        self.handle = handle
        self.desc = desc

    def free(self):
        if self.handle:
            _lib.cadnn_weights_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def make_desc(c_in, c_out, kh=1, kw=1, stride=1, pad=0, groups=1, in_h=1, in_w=1, batch_hint=1,
              dtype="f32", host_only=False, autotune=False, pad_w=-1, fmt=0):
    flags = (PACK_HOST_ONLY if host_only else 0) | (PACK_AUTOTUNE if autotune else 0)
    return LayerDesc(c_in, c_out, kh, kw, stride, pad, groups, in_h, in_w, batch_hint, DTYPE[dtype], fmt, flags, pad_w)


def cadnn_pack(desc, w_ohwi, mask=None, w_scale=None):
    w = np.ascontiguousarray(w_ohwi, dtype=np.float32)
    m = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    s = None if w_scale is None else np.ascontiguousarray(w_scale, dtype=np.float32)
    expect = desc.c_out * desc.kh * desc.kw * (desc.c_in // max(1, desc.groups))
    if w.size != expect or (m is not None and m.size != expect) or (s is not None and s.size != desc.c_out):
        raise ValueError("weight / mask / scale size does not match the layer description")
    out = ctypes.c_void_p()
    _check(_lib.cadnn_pack(ctypes.byref(desc), _np_ptr(w), _np_ptr(m), _np_ptr(s), ctypes.byref(out)), "cadnn_pack")
    return Weights(out, desc)


def cadnn_pack_q8(desc, q_ohwi, mask=None):
    q = np.ascontiguousarray(q_ohwi, dtype=np.int8)
    m = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    expect = desc.c_out * desc.kh * desc.kw * (desc.c_in // max(1, desc.groups))
    if q.size != expect or (m is not None and m.size != expect):
        raise ValueError("weight / mask size does not match the layer description")
    out = ctypes.c_void_p()
    _check(_lib.cadnn_pack_q8(ctypes.byref(desc), _np_ptr(q), _np_ptr(m), ctypes.byref(out)), "cadnn_pack_q8")
    return Weights(out, desc)


def cadnn_weights_info(w):
    nnz, pb, fmt = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int()
    _check(_lib.cadnn_weights_info(w.handle, ctypes.byref(nnz), ctypes.byref(pb), ctypes.byref(fmt)), "cadnn_weights_info")
    return {"nnz": nnz.value, "packed_bytes": pb.value, "fmt": fmt.value}


def cadnn_weights_schedule(w):
    arr = (ctypes.c_int * 16)()
    _check(_lib.cadnn_weights_schedule(w.handle, arr), "cadnn_weights_schedule")
    keys = ("kind", "T", "RPW", "G", "CIc", "TH", "TW", "pitch", "NW", "stages", "ksplit", "chunks", "smem",
            "TBX", "TBY", "max_entries")
    return dict(zip(keys, list(arr)))


def cadnn_weights_planar_schedule(w):
    arr = (ctypes.c_int * 16)()
    _check(_lib.cadnn_weights_planar_schedule(w.handle, arr), "cadnn_weights_planar_schedule")
    keys = ("variant", "T", "RPW", "NW", "KS", "G", "CIc", "stages", "chunks", "tiles", "smem", "max_entries",
            "staged_us_x100", "direct_us_x100", "tma", "KC")
    return dict(zip(keys, list(arr)))


def cadnn_device_status():
    n = ctypes.c_int()
    _check(_lib.cadnn_device_status(ctypes.byref(n)), "cadnn_device_status")
    return {"copy_timeouts": n.value}


def cadnn_weights_warp_loads(w):
    n = ctypes.c_int()
    _check(_lib.cadnn_weights_warp_loads(w.handle, None, 0, ctypes.byref(n)), "cadnn_weights_warp_loads")
    buf = (ctypes.c_int64 * max(1, n.value))()
    _check(_lib.cadnn_weights_warp_loads(w.handle, buf, n.value, ctypes.byref(n)), "cadnn_weights_warp_loads")
    return np.array(buf[: n.value], dtype=np.int64)


def cadnn_weights_unpack(w):
    d = w.desc
    shape = (d.c_out, d.kh, d.kw, d.c_in // max(1, d.groups))
    dense = np.empty(shape, np.float32)
    mask = np.empty(shape, np.uint8)
    _check(_lib.cadnn_weights_unpack(w.handle, _np_ptr(dense), _np_ptr(mask)), "cadnn_weights_unpack")
    return dense, mask


def _epilogue(scale, bias, residual, act, out_dtype, out_c_total=0, out_c_off=0, residual_scale=0.0):
    return Epilogue(None if scale is None else scale.data_ptr(), None if bias is None else bias.data_ptr(),
                    None if residual is None else residual.data_ptr(), ACT[act] if not isinstance(act, int) else act,
                    DTYPE[out_dtype] if not isinstance(out_dtype, int) else out_dtype, out_c_total, out_c_off,
                    float(residual_scale))


def cadnn_conv2d(w, x, y, scale=None, bias=None, residual=None, act="none", out_dtype=None, stream=None,
                 out_c_total=0, out_c_off=0, residual_scale=0.0):
    """x, y: torch CUDA tensors, NHWC contiguous; y is written in place (channels [out_c_off, out_c_off + c_out)
    of it when out_c_total > 0)."""
    n, h, wd = int(x.shape[0]), int(x.shape[1]), int(x.shape[2])
    if out_dtype is None:
        out_dtype = w.desc.dtype
    ep = _epilogue(scale, bias, residual, act, out_dtype, out_c_total, out_c_off, residual_scale)
    _check(_lib.cadnn_conv2d(w.handle, _dev_ptr(x), n, h, wd, _dev_ptr(y), ctypes.byref(ep), _stream(stream)),
           "cadnn_conv2d")
    return y


def cadnn_weights_workspace_bytes(w, n):
    b = ctypes.c_int64()
    _check(_lib.cadnn_weights_workspace_bytes(w.handle, int(n), ctypes.byref(b)), "cadnn_weights_workspace_bytes")
    return int(b.value)


def cadnn_weights_block_info(w):
    nb, nz = ctypes.c_int(), ctypes.c_int64()
    _check(_lib.cadnn_weights_block_info(w.handle, ctypes.byref(nb), ctypes.byref(nz)), "cadnn_weights_block_info")
    return {"blocks": nb.value, "block_nnz": nz.value}


def cadnn_conv2d_workspace(w, x, y, workspace, scale=None, bias=None, residual=None, act="none", out_dtype=None, stream=None,
                           residual_scale=0.0):
    """cadnn_conv2d for a layer packed as FMT_GROUPED: workspace is a torch CUDA tensor of at least
    cadnn_weights_workspace_bytes(w, n) bytes (None for other formats)."""
    n, h, wd = int(x.shape[0]), int(x.shape[1]), int(x.shape[2])
    if out_dtype is None:
        out_dtype = w.desc.dtype
    ep = _epilogue(scale, bias, residual, act, out_dtype, 0, 0, residual_scale)
    nbytes = 0 if workspace is None else int(workspace.numel() * workspace.element_size())
    _check(_lib.cadnn_conv2d_workspace(w.handle, _dev_ptr(x), n, h, wd, _dev_ptr(y), ctypes.byref(ep), _dev_ptr(workspace),
                                       nbytes, _stream(stream)), "cadnn_conv2d_workspace")
    return y


def cadnn_conv2d_planar(w, x, y, scale=None, bias=None, residual=None, act="none", stream=None):
    """x [n, c_in, pitch(h, w)], y [n, c_out, pitch(ho, wo)]: float CUDA tensors of channel planes, each
    (h+2) x (w+2) with a zero one-pixel border, followed by padding to pitch = a multiple of 4 floats."""
    ep = _epilogue(scale, bias, residual, act, F32)
    _check(_lib.cadnn_conv2d_planar(w.handle, _dev_ptr(x), int(x.shape[0]), _dev_ptr(y), ctypes.byref(ep), _stream(stream)),
           "cadnn_conv2d_planar")
    return y


def cadnn_fc(w, x, y, scale=None, bias=None, residual=None, act="none", out_dtype=None, stream=None):
    if out_dtype is None:
        out_dtype = w.desc.dtype
    ep = _epilogue(scale, bias, residual, act, out_dtype)
    _check(_lib.cadnn_fc(w.handle, _dev_ptr(x), int(x.shape[0]), _dev_ptr(y), ctypes.byref(ep), _stream(stream)),
           "cadnn_fc")
    return y


def cadnn_maxpool2d(x, y, k, stride, pad=0, stream=None):
    import torch
    n, h, wd, c = (int(v) for v in x.shape)
    dt = S8 if x.dtype == torch.int8 else F32
    _check(_lib.cadnn_maxpool2d(_dev_ptr(x), n, h, wd, c, k, stride, pad, dt, _dev_ptr(y), _stream(stream)),
           "cadnn_maxpool2d")
    return y


def cadnn_pool2d(x, y, k, stride, pad=0, kind="max", out_c_total=0, out_c_off=0, stream=None):
    """Max / average pool of x (NHWC) into y, or into channels [out_c_off, out_c_off + c) of a wider y."""
    import torch
    n, h, wd, c = (int(v) for v in x.shape)
    dt = S8 if x.dtype == torch.int8 else F32
    _check(_lib.cadnn_pool2d(_dev_ptr(x), n, h, wd, c, k, stride, pad, dt, 1 if kind == "avg" else 0, _dev_ptr(y),
                             out_c_total, out_c_off, _stream(stream)), "cadnn_pool2d")
    return y


def cadnn_global_avgpool(x, y, stream=None):
    n, h, wd, c = (int(v) for v in x.shape)
    _check(_lib.cadnn_global_avgpool(_dev_ptr(x), n, h, wd, c, _dev_ptr(y), _stream(stream)), "cadnn_global_avgpool")
    return y


class Net:
    def __init__(self, handle, keep):
        self.handle = handle
        self._keep = keep   # objects the C side borrows (weights, scale / bias tensors)

    def free(self):
        if self.handle:
            _lib.cadnn_net_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def cadnn_net_create(ops, n, h, w, c, in_dtype, keep=None):
    """ops: list of binding.Op."""
    arr = (Op * len(ops))(*ops)
    out = ctypes.c_void_p()
    _check(_lib.cadnn_net_create(arr, len(ops), n, h, w, c, DTYPE[in_dtype] if not isinstance(in_dtype, int) else in_dtype,
                                 ctypes.byref(out)), "cadnn_net_create")
    return Net(out, keep)


def cadnn_forward(net, x, y, use_graph=True, stream=None):
    _check(_lib.cadnn_forward(net.handle, _dev_ptr(x), _dev_ptr(y), 1 if use_graph else 0, _stream(stream)),
           "cadnn_forward")
    return y


def cadnn_forward_host(net, x_host, y_host, use_graph=True, stream=None):
    """x_host, y_host: CPU torch tensors (pinned recommended) or numpy arrays; blocks until y_host is filled."""
    xp = x_host.data_ptr() if hasattr(x_host, "data_ptr") else x_host.ctypes.data
    yp = y_host.data_ptr() if hasattr(y_host, "data_ptr") else y_host.ctypes.data
    _check(_lib.cadnn_forward_host(net.handle, ctypes.c_void_p(xp), ctypes.c_void_p(yp), 1 if use_graph else 0,
                                   _stream(stream)), "cadnn_forward_host")
    return y_host


STATIC_WORKSPACE_BYTES = 32 << 20


def cadnn_forward_static(ops, x, y, in_dtype, stream=None):
    """Run the op list on x (NHWC torch CUDA tensor) into y without allocating: intermediates live
    in the library's fixed device workspace (STATIC_WORKSPACE_BYTES); see include/cadnn.h."""
    arr = (Op * len(ops))(*ops)
    n, h, w, c = (int(v) for v in x.shape)
    _check(_lib.cadnn_forward_static(arr, len(ops), n, h, w, c, DTYPE[in_dtype] if not isinstance(in_dtype, int) else in_dtype,
                                     _dev_ptr(x), _dev_ptr(y), _stream(stream)), "cadnn_forward_static")
    return y


def cadnn_net_info(net):
    nl, ws = ctypes.c_int(), ctypes.c_int64()
    _check(_lib.cadnn_net_info(net.handle, ctypes.byref(nl), ctypes.byref(ws)), "cadnn_net_info")
    return {"launches": nl.value, "workspace_bytes": ws.value}


def cadnn_net_parity_layers(net, ops=False):
    """Number of stride-2 layers run in their parity-plane form (ops=True: their op indices)."""
    c = ctypes.c_int()
    _check(_lib.cadnn_net_parity_layers(net.handle, ctypes.byref(c), None, 0), "cadnn_net_parity_layers")
    if not ops:
        return c.value
    buf = (ctypes.c_int * max(1, c.value))()
    _check(_lib.cadnn_net_parity_layers(net.handle, ctypes.byref(c), buf, c.value), "cadnn_net_parity_layers")
    return list(buf[: c.value])


class _Borrowed:
    """A handle owned by another object (never freed here)."""

    def __init__(self, handle, desc):
        self.handle = handle
        self.desc = desc


def cadnn_weights_parity_form(w):
    """The stride-1 form of a stride-2 layer over the parity planes of its input (None if the layer has none):
    4 c_in input channels (plane-major) for a 3x3 layer, c_in for a 1x1 layer, maps of ceil(h / 2) x ceil(w / 2)."""
    out = ctypes.c_void_p()
    _check(_lib.cadnn_weights_parity_form(w.handle, ctypes.byref(out)), "cadnn_weights_parity_form")
    if not out.value:
        return None
    d = w.desc
    dc = LayerDesc(4 * d.c_in if d.kh == 3 else d.c_in, d.c_out, d.kh, d.kw, 1, d.pad, d.groups, (d.in_h + 1) // 2,
                   (d.in_w + 1) // 2, d.batch_hint, d.dtype, d.fmt, d.flags, d.pad_w)
    return _Borrowed(out, dc)


def cadnn_net_layout(net):
    pl, po = ctypes.c_int(), ctypes.c_int()
    _check(_lib.cadnn_net_layout(net.handle, ctypes.byref(pl), ctypes.byref(po)), "cadnn_net_layout")
    return {"planar": bool(pl.value), "persistent_ops": po.value}


def cadnn_net_layer_times(net, x, y, n_ops, flush_l2=False, reps=1, stream=None):
    ms = (ctypes.c_float * n_ops)()
    _check(_lib.cadnn_net_layer_times(net.handle, _dev_ptr(x), _dev_ptr(y), 1 if flush_l2 else 0, int(reps), ms,
                                      _stream(stream)),
           "cadnn_net_layer_times")
    return [float(v) for v in ms]


def cadnn_net_layer_time(net, op, x, y, flush_l2=False, reps=1, stream=None):
    ms = ctypes.c_float()
    _check(_lib.cadnn_net_layer_time(net.handle, int(op), _dev_ptr(x), _dev_ptr(y), 1 if flush_l2 else 0, int(reps),
                                     ctypes.byref(ms), _stream(stream)), "cadnn_net_layer_time")
    return float(ms.value)


def cadnn_debug_set_device_status(copy_timeouts, barrier_timeouts):
    _check(_lib.cadnn_debug_set_device_status(int(copy_timeouts), int(barrier_timeouts)), "cadnn_debug_set_device_status")


def cadnn_free_weights(w):
    """Alias of Weights.free (the C ABI exports both names)."""
    w.free()


def cadnn_measure_alu_peak(dtype="f32", stream=None):
    """Measured multiply-add rate of the plain ALUs, operations per second (a multiply-add counts 2)."""
    v = ctypes.c_double()
    _check(_lib.cadnn_measure_alu_peak(DTYPE[dtype], ctypes.byref(v), _stream(stream)), "cadnn_measure_alu_peak")
    return float(v.value)


def cadnn_net_persistent_plan(net, op):
    """Planner's choice for op `op` of the persistent run, or None if the op is not part of one."""
    arr = (ctypes.c_int * 12)()
    st = _lib.cadnn_net_persistent_plan(net.handle, int(op), arr)
    if st == 4:
        return None
    _check(st, "cadnn_net_persistent_plan")
    keys = ("TB", "T", "G", "tiles", "groups", "L", "CIc", "cpp", "passes", "strided", "est_clk", "phase")
    return dict(zip(keys, list(arr)))


def cadnn_net_persistent_profile(net, cap=256):
    """Per phase of the persistent kernel's last launch: (wall clocks, longest block clocks, mean block clocks,
    mean clocks until the tile copies were issued, until they had landed)."""
    arrs = [(ctypes.c_float * cap)() for _ in range(5)]
    n = ctypes.c_int()
    _check(_lib.cadnn_net_persistent_profile(net.handle, cap, *arrs, ctypes.byref(n)), "cadnn_net_persistent_profile")
    k = min(cap, n.value)
    return [tuple(float(a[i]) for a in arrs) for i in range(k)]


def cadnn_net_slot(net, slot):
    ptr, b = ctypes.c_void_p(), ctypes.c_int64()
    _check(_lib.cadnn_net_slot(net.handle, slot, ctypes.byref(ptr), ctypes.byref(b)), "cadnn_net_slot")
    return ptr.value, b.value
