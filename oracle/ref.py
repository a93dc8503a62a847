"""ctypes front end of the C oracle (``cadnn_ref.c``): numpy arrays in, numpy arrays out.

TEST INFRASTRUCTURE ONLY.  Every function here forwards to the plain C loops;
no arithmetic of the method lives in this file except shape bookkeeping.
The shared object is compiled on first use with
``gcc -O2 -ffp-contract=off -fopenmp`` (contraction off so that the single
``fmaf`` of the int8 requantization is the only fused operation).
"""
import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cadnn_ref.c")
_SO = os.path.join(_HERE, "libcadnn_ref.so")

ACT = {"none": 0, "relu": 1, "relu6": 2, None: 0}
OUT = {"s8": 0, "s32": 1, "f32": 2}
_OUT_NP = {"s8": np.int8, "s32": np.int32, "f32": np.float32}


def build(force=False):
    """Compile the oracle if the shared object is missing or older than its source."""
    if (not force and os.path.exists(_SO)
            and os.path.getmtime(_SO) >= os.path.getmtime(_SRC)):
        return _SO
    tmp = _SO + ".tmp%d" % os.getpid()
    cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
           "-o", tmp, _SRC, "-lm"]
    subprocess.check_call(cmd)
    os.replace(tmp, _SO)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.ref_requant_f32.restype = ctypes.c_float
        _lib.ref_requant_f32.argtypes = [ctypes.c_int32, ctypes.c_float, ctypes.c_float, ctypes.c_int]
        _lib.ref_requant_s8.restype = ctypes.c_int8
        _lib.ref_requant_s8.argtypes = [ctypes.c_int32, ctypes.c_float, ctypes.c_float, ctypes.c_int]
        _lib.ref_requant_res_f32.restype = ctypes.c_float
        _lib.ref_requant_res_f32.argtypes = [ctypes.c_int32, ctypes.c_float, ctypes.c_float, ctypes.c_int8,
                                             ctypes.c_float, ctypes.c_int]
        _lib.ref_requant_res_s8.restype = ctypes.c_int8
        _lib.ref_requant_res_s8.argtypes = [ctypes.c_int32, ctypes.c_float, ctypes.c_float, ctypes.c_int8,
                                            ctypes.c_float, ctypes.c_int]
    return _lib


def num_threads():
    return int(lib().ref_num_threads())


def set_threads(t):
    lib().ref_set_threads(int(t))


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dt):
    return None if a is None else np.ascontiguousarray(a, dtype=dt)


def out_hw(h, w, k, stride, pad):
    return (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1


def _pads(pad):
    """pad may be one int (both axes) or a (pad_h, pad_w) pair."""
    if isinstance(pad, (tuple, list)):
        return int(pad[0]), int(pad[1])
    return int(pad), int(pad)


def conv2d_f32(x, wt, mask=None, stride=1, pad=0, groups=1, scale=None, bias=None,
               residual=None, act="none"):
    """x [n,h,w,c_in] float32, wt [c_out,kh,kw,c_in/groups] float32 -> y [n,ho,wo,c_out].
    pad: int, or (pad_h, pad_w) for rectangular kernels."""
    x = _c(x, np.float32); wt = _c(wt, np.float32); mask = _c(mask, np.uint8)
    scale = _c(scale, np.float32); bias = _c(bias, np.float32); residual = _c(residual, np.float32)
    n, h, w, c_in = x.shape
    c_out, kh, kw, cg = wt.shape
    assert cg * groups == c_in, "weight shape does not match c_in/groups"
    ph, pw = _pads(pad)
    ho, wo = (h + 2 * ph - kh) // stride + 1, (w + 2 * pw - kw) // stride + 1
    y = np.empty((n, ho, wo, c_out), np.float32)
    if residual is not None:
        assert residual.shape == y.shape
    rc = lib().ref_conv2d_f32_hw(_p(x), n, h, w, c_in, _p(wt), _p(mask), c_out, kh, kw,
                                 stride, ph, pw, groups, _p(scale), _p(bias), _p(residual),
                                 ACT[act], _p(y))
    if rc != 0:
        raise ValueError("ref_conv2d_f32 rejected the shape")
    return y


def fc_f32(x, wt, mask=None, scale=None, bias=None, residual=None, act="none"):
    """x [n,k], wt [c_out,k] -> y [n,c_out]."""
    x = _c(x, np.float32); wt = _c(wt, np.float32); mask = _c(mask, np.uint8)
    scale = _c(scale, np.float32); bias = _c(bias, np.float32); residual = _c(residual, np.float32)
    n, k = x.shape
    c_out = wt.shape[0]
    assert wt.size == c_out * k
    y = np.empty((n, c_out), np.float32)
    lib().ref_fc_f32(_p(x), n, k, _p(wt), _p(mask), c_out, _p(scale), _p(bias), _p(residual),
                     ACT[act], _p(y))
    return y


def quantize_weights(wt, s_w):
    wt = _c(wt, np.float32); s_w = _c(s_w, np.float32)
    c_out = wt.shape[0]
    q = np.empty(wt.shape, np.int8)
    lib().ref_quantize_weights(_p(wt), _p(s_w), c_out, wt.size // c_out, _p(q))
    return q


def requant_s8(acc, m, b, act="none"):
    return int(lib().ref_requant_s8(int(acc), float(np.float32(m)), float(np.float32(b)), ACT[act]))


def requant_f32(acc, m, b, act="none"):
    return np.float32(lib().ref_requant_f32(int(acc), float(np.float32(m)), float(np.float32(b)), ACT[act]))


def requant_res_s8(acc, m, b, r, rs, act="none"):
    return int(lib().ref_requant_res_s8(int(acc), float(np.float32(m)), float(np.float32(b)), int(r),
                                        float(np.float32(rs)), ACT[act]))


def requant_res_f32(acc, m, b, r, rs, act="none"):
    return np.float32(lib().ref_requant_res_f32(int(acc), float(np.float32(m)), float(np.float32(b)), int(r),
                                                float(np.float32(rs)), ACT[act]))


def conv2d_s8(x, wq, mask=None, stride=1, pad=0, groups=1, m=None, b=None, act="none", out="s8",
              residual=None, residual_scale=0.0):
    """Int8 layer; residual (int8, y's shape) joins the requantization as a second fmaf."""
    x = _c(x, np.int8); wq = _c(wq, np.int8); mask = _c(mask, np.uint8)
    m = _c(m, np.float32); b = _c(b, np.float32); residual = _c(residual, np.int8)
    n, h, w, c_in = x.shape
    c_out, kh, kw, cg = wq.shape
    assert cg * groups == c_in
    ho, wo = (h + 2 * pad - kh) // stride + 1, (w + 2 * pad - kw) // stride + 1
    y = np.empty((n, ho, wo, c_out), _OUT_NP[out])
    if residual is not None:
        assert residual.shape == y.shape
    rc = lib().ref_conv2d_s8_res(_p(x), n, h, w, c_in, _p(wq), _p(mask), c_out, kh, kw, stride, pad,
                                 groups, _p(m), _p(b), _p(residual), ctypes.c_float(float(residual_scale)),
                                 ACT[act], OUT[out], _p(y))
    if rc != 0:
        raise ValueError("ref_conv2d_s8 rejected the arguments")
    return y


def fc_s8(x, wq, mask=None, m=None, b=None, act="none", out="s8"):
    x = _c(x, np.int8); wq = _c(wq, np.int8); mask = _c(mask, np.uint8)
    m = _c(m, np.float32); b = _c(b, np.float32)
    n, k = x.shape
    c_out = wq.shape[0]
    assert wq.size == c_out * k
    y = np.empty((n, c_out), _OUT_NP[out])
    rc = lib().ref_fc_s8(_p(x), n, k, _p(wq), _p(mask), c_out, _p(m), _p(b), ACT[act], OUT[out], _p(y))
    if rc != 0:
        raise ValueError("ref_fc_s8 rejected the arguments")
    return y


def maxpool(x, k, stride, pad=0):
    n, h, w, c = x.shape
    ho, wo = out_hw(h, w, k, stride, pad)
    if x.dtype == np.int8:
        x = _c(x, np.int8); y = np.empty((n, ho, wo, c), np.int8)
        rc = lib().ref_maxpool_s8(_p(x), n, h, w, c, k, stride, pad, _p(y))
    else:
        x = _c(x, np.float32); y = np.empty((n, ho, wo, c), np.float32)
        rc = lib().ref_maxpool_f32(_p(x), n, h, w, c, k, stride, pad, _p(y))
    if rc != 0:
        raise ValueError("ref_maxpool rejected the arguments")
    return y


def avgpool(x, k, stride, pad=0):
    """k x k average pool; padded taps count as zeros, divisor k*k."""
    x = _c(x, np.float32)
    n, h, w, c = x.shape
    ho, wo = out_hw(h, w, k, stride, pad)
    y = np.empty((n, ho, wo, c), np.float32)
    rc = lib().ref_avgpool_f32(_p(x), n, h, w, c, k, stride, pad, _p(y))
    if rc != 0:
        raise ValueError("ref_avgpool rejected the arguments")
    return y


def gavgpool(x):
    x = _c(x, np.float32)
    n, h, w, c = x.shape
    y = np.empty((n, c), np.float32)
    lib().ref_gavgpool_f32(_p(x), n, h, w, c, _p(y))
    return y
