"""Pins for the CPU oracle: each test ties it to something other than itself
(hand-worked literals, closed forms, invariants, library routines, exact
rational arithmetic), chosen so that a dropped term, a flipped kernel, a wrong
padding/stride convention, a transposed operand or a wrong rounding mode fails
at least one of them."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import ref

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "conv_handworked.json")))
R = np.random.default_rng(1234)


def _x33():
    return np.array(GOLD["x_3x3"], np.float32).reshape(1, 3, 3, 1)


def _w22():
    return np.array(GOLD["w_2x2"], np.float32).reshape(1, 2, 2, 1)


def test_handworked_valid_conv_is_cross_correlation():
    y = ref.conv2d_f32(_x33(), _w22())
    assert y.shape == (1, 2, 2, 1)
    np.testing.assert_array_equal(y[0, :, :, 0], np.array(GOLD["valid_s1_p0"], np.float32))
    assert y[0, 0, 0, 0] != GOLD["flipped_kernel_would_give_y00"]


def test_handworked_stride2_pad1():
    y = ref.conv2d_f32(_x33(), _w22(), stride=2, pad=1)
    np.testing.assert_array_equal(y[0, :, :, 0], np.array(GOLD["s2_p1"], np.float32))


def test_handworked_mask_and_epilogue():
    mask = np.ones((1, 2, 2, 1), np.uint8)
    mask[0, 0, 1, 0] = 0
    y = ref.conv2d_f32(_x33(), _w22(), mask)
    np.testing.assert_array_equal(y[0, :, :, 0], np.array(GOLD["mask_drop_w01_s1_p0"], np.float32))
    sc, bi = np.array([2.0], np.float32), np.array([-20.0], np.float32)
    y = ref.conv2d_f32(_x33(), _w22(), scale=sc, bias=bi, act="relu")
    np.testing.assert_array_equal(y[0, :, :, 0], np.array(GOLD["scale2_bias_m20_relu"], np.float32))
    res = np.full((1, 2, 2, 1), 0.5, np.float32)
    y = ref.conv2d_f32(_x33(), _w22(), scale=sc, bias=bi, residual=res, act="relu")
    np.testing.assert_array_equal(y[0, :, :, 0], np.array(GOLD["scale2_bias_m20_res_half_relu"], np.float32))
    y = ref.conv2d_f32(_x33(), _w22(), scale=sc, bias=bi, residual=res, act="relu6")
    np.testing.assert_array_equal(y[0, :, :, 0], np.array(GOLD["scale2_bias_m20_res_half_relu6"], np.float32))


def _brute_conv(x, w, mask, stride, pad, groups):
    """Gather-form brute force over an explicitly zero-padded copy, float64."""
    n, h, wd, c_in = x.shape
    c_out, kh, kw, cg = w.shape
    og = c_out // groups
    xp = np.zeros((n, h + 2 * pad, wd + 2 * pad, c_in), np.float64)
    xp[:, pad:pad + h, pad:pad + wd, :] = x
    we = w.astype(np.float64) * (1 if mask is None else mask)
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (wd + 2 * pad - kw) // stride + 1
    y = np.zeros((n, ho, wo, c_out), np.float64)
    for co in range(c_out):
        g = co // og
        for oy in range(ho):
            for ox in range(wo):
                patch = xp[:, oy * stride:oy * stride + kh, ox * stride:ox * stride + kw, g * cg:(g + 1) * cg]
                y[:, oy, ox, co] = np.tensordot(patch, we[co], axes=([1, 2, 3], [0, 1, 2]))
    return y


@pytest.mark.parametrize("k,stride,pad", [(1, 1, 0), (2, 1, 0), (3, 1, 1), (3, 2, 1), (3, 2, 0), (2, 2, 1), (1, 2, 0)])
@pytest.mark.parametrize("groups", [1, 3])
def test_brute_force_tiny(k, stride, pad, groups):
    n, h, w, c_in, c_out = 2, 5, 6, 3, 6
    x = R.standard_normal((n, h, w, c_in)).astype(np.float32)
    wt = R.standard_normal((c_out, k, k, c_in // groups)).astype(np.float32)
    mask = (R.random(wt.shape) < 0.5).astype(np.uint8)
    y = ref.conv2d_f32(x, wt, mask, stride, pad, groups)
    want = _brute_conv(x, wt, mask, stride, pad, groups)
    assert y.shape == want.shape
    # the oracle rounds a float64 sum once to float32
    np.testing.assert_allclose(y, want.astype(np.float32), rtol=0, atol=1e-6)


@pytest.mark.parametrize("k,stride,pad,groups", [(3, 1, 1, 1), (3, 2, 1, 1), (7, 2, 3, 1), (1, 1, 0, 1), (3, 1, 1, 8), (5, 1, 2, 2)])
def test_against_float64_library_convolution(k, stride, pad, groups):
    n, h, w, c_in, c_out = 2, 11, 9, 8, 16
    x = R.standard_normal((n, h, w, c_in)).astype(np.float32)
    wt = R.standard_normal((c_out, k, k, c_in // groups)).astype(np.float32)
    mask = (R.random(wt.shape) < 0.3).astype(np.uint8)
    y = ref.conv2d_f32(x, wt, mask, stride, pad, groups)
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    wtt = torch.from_numpy((wt * mask).astype(np.float64)).permute(0, 3, 1, 2)
    want = torch.nn.functional.conv2d(xt, wtt, None, stride, pad, 1, groups).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(y, want.astype(np.float32), rtol=0, atol=2e-6)


def test_mask_none_equals_all_ones_and_density_one():
    x = R.standard_normal((1, 6, 6, 4)).astype(np.float32)
    wt = R.standard_normal((5, 3, 3, 4)).astype(np.float32)
    a = ref.conv2d_f32(x, wt, None, 1, 1)
    b = ref.conv2d_f32(x, wt, np.ones(wt.shape, np.uint8), 1, 1)
    np.testing.assert_array_equal(a, b)


def test_masked_out_value_is_ignored_even_if_nonzero():
    x = R.standard_normal((1, 4, 4, 2)).astype(np.float32)
    wt = R.standard_normal((3, 3, 3, 2)).astype(np.float32)
    mask = (R.random(wt.shape) < 0.5).astype(np.uint8)
    a = ref.conv2d_f32(x, wt, mask, 1, 1)
    b = ref.conv2d_f32(x, wt * mask, None, 1, 1)
    np.testing.assert_array_equal(a, b)


def test_identity_1x1_is_a_copy():
    x = R.standard_normal((2, 5, 7, 6)).astype(np.float32)
    wt = np.eye(6, dtype=np.float32).reshape(6, 1, 1, 6)
    np.testing.assert_array_equal(ref.conv2d_f32(x, wt), x)
    xq = R.integers(-127, 128, size=(2, 5, 7, 6)).astype(np.int8)
    wq = np.eye(6, dtype=np.int8).reshape(6, 1, 1, 6)
    np.testing.assert_array_equal(ref.conv2d_s8(xq, wq, m=np.ones(6, np.float32), b=np.zeros(6, np.float32)), xq)


@pytest.mark.parametrize("ky,kx", [(0, 0), (0, 2), (1, 1), (2, 0), (2, 1)])
@pytest.mark.parametrize("stride", [1, 2])
def test_single_tap_filter_is_a_shift_with_zero_fill(ky, kx, stride):
    h, w = 7, 6
    x = R.standard_normal((1, h, w, 1)).astype(np.float32)
    wt = np.zeros((1, 3, 3, 1), np.float32)
    wt[0, ky, kx, 0] = 1.0
    y = ref.conv2d_f32(x, wt, None, stride, 1)
    ho, wo = (h + 2 - 3) // stride + 1, (w + 2 - 3) // stride + 1
    assert y.shape == (1, ho, wo, 1)
    for oy in range(ho):
        for ox in range(wo):
            iy, ix = oy * stride + ky - 1, ox * stride + kx - 1
            want = x[0, iy, ix, 0] if (0 <= iy < h and 0 <= ix < w) else 0.0
            assert y[0, oy, ox, 0] == want


def test_1x1_conv_is_a_matrix_product_and_fc_is_matvec():
    x = R.standard_normal((2, 4, 5, 7)).astype(np.float32)
    wt = R.standard_normal((9, 1, 1, 7)).astype(np.float32)
    mask = (R.random(wt.shape) < 0.4).astype(np.uint8)
    y = ref.conv2d_f32(x, wt, mask)
    a = x.reshape(-1, 7).astype(np.float64)
    b = (wt * mask).reshape(9, 7).astype(np.float64)
    want = (a @ b.T).astype(np.float32).reshape(2, 4, 5, 9)
    np.testing.assert_allclose(y, want, rtol=0, atol=1e-6)
    xf = R.standard_normal((3, 7)).astype(np.float32)
    yf = ref.fc_f32(xf, wt.reshape(9, 7), mask.reshape(9, 7))
    np.testing.assert_allclose(yf, (xf.astype(np.float64) @ b.T).astype(np.float32), rtol=0, atol=1e-6)
    # fc equals a 1x1 convolution on a 1x1 image, bit for bit (same sum order)
    yc = ref.conv2d_f32(xf.reshape(3, 1, 1, 7), wt, mask).reshape(3, 9)
    np.testing.assert_array_equal(yf, yc)


def test_linearity_and_mask_additivity_and_channel_permutation():
    x1 = R.standard_normal((1, 6, 6, 3)).astype(np.float32)
    x2 = R.standard_normal((1, 6, 6, 3)).astype(np.float32)
    wt = R.standard_normal((4, 3, 3, 3)).astype(np.float32)
    f = lambda x, m=None: ref.conv2d_f32(x, wt, m, 1, 1).astype(np.float64)
    np.testing.assert_allclose(f(2 * x1 + 4 * x2), 2 * f(x1) + 4 * f(x2), rtol=0, atol=2e-5)
    m1 = (R.random(wt.shape) < 0.5).astype(np.uint8)
    m2 = ((1 - m1) * (R.random(wt.shape) < 0.5)).astype(np.uint8)
    np.testing.assert_allclose(f(x1, m1) + f(x1, m2), f(x1, m1 | m2), rtol=0, atol=2e-6)
    perm = R.permutation(4)
    yp = ref.conv2d_f32(x1, wt[perm], m1[perm], 1, 1)
    np.testing.assert_array_equal(yp, ref.conv2d_f32(x1, wt, m1, 1, 1)[..., perm])
    # exact in the integer path
    xq = R.integers(-127, 128, size=(1, 6, 6, 3)).astype(np.int8)
    wq = R.integers(-127, 128, size=(4, 3, 3, 3)).astype(np.int8)
    g = lambda m: ref.conv2d_s8(xq, wq, m, 1, 1, out="s32")
    np.testing.assert_array_equal(g(m1) + g(m2), g(m1 | m2))


def test_int8_accumulator_against_int64_matrix_product():
    xq = R.integers(-127, 128, size=(2, 5, 5, 6)).astype(np.int8)
    wq = R.integers(-127, 128, size=(7, 3, 3, 6)).astype(np.int8)
    mask = (R.random(wq.shape) < 0.3).astype(np.uint8)
    y = ref.conv2d_s8(xq, wq, mask, 1, 1, out="s32")
    xt = torch.from_numpy(xq.astype(np.int64)).permute(0, 3, 1, 2)
    wt = torch.from_numpy((wq.astype(np.int64) * mask)).permute(0, 3, 1, 2)
    want = torch.nn.functional.conv2d(xt.double(), wt.double(), None, 1, 1).permute(0, 2, 3, 1).numpy()
    np.testing.assert_array_equal(y, want.astype(np.int64))
    xf = R.integers(-127, 128, size=(3, 50)).astype(np.int8)
    wf = R.integers(-127, 128, size=(11, 50)).astype(np.int8)
    mf = (R.random(wf.shape) < 0.5).astype(np.uint8)
    want = xf.astype(np.int64) @ (wf.astype(np.int64) * mf).T
    np.testing.assert_array_equal(ref.fc_s8(xf, wf, mf, out="s32"), want)


def _round_half_even(fr):
    fl = fr.numerator // fr.denominator
    rem = fr - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        return fl + 1
    return fl


def _to_f32_exact(fr):
    """Round an exact rational to the nearest float32, ties to even (normal range)."""
    if fr == 0:
        return Fraction(0)
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = 0
    while a >= 2 ** 24:
        a /= 2; e += 1
    while a < 2 ** 23:
        a *= 2; e -= 1
    q = _round_half_even(a)
    return sign * Fraction(q) * (Fraction(2) ** e)


def _requant_exact(acc, m, b, act):
    accf = _to_f32_exact(Fraction(acc))
    t = _to_f32_exact(accf * Fraction(float(np.float32(m))) + Fraction(float(np.float32(b))))
    if act == "relu" and t < 0:
        t = Fraction(0)
    tf = t
    t = min(max(t, Fraction(-127)), Fraction(127))
    return _round_half_even(t), tf


def test_requant_literals():
    for c in GOLD["requant_cases"]:
        assert ref.requant_s8(c["acc"], c["m"], c["b"], c["act"]) == c["q"], c


def test_requant_against_exact_rational_arithmetic():
    accs = [0, 1, -1, 2, 3, 5, 7, 127, 128, 255, 2 ** 24 - 1, 2 ** 24, 2 ** 24 + 1, 2 ** 24 + 3,
            -(2 ** 24) - 1, -(2 ** 24) - 3, 33554431, 33554433, 400000001, -400000003, 2 ** 31 - 1, -(2 ** 31)]
    accs += [int(v) for v in R.integers(-2 ** 31, 2 ** 31 - 1, size=300)]
    accs += [int(v) for v in R.integers(-3000, 3000, size=300)]
    ms = [0.5, 0.25, 1.0, 3.0517578125e-05, 1e-3, 0.0123456, 1.0 / 3.0, 2.3e-7]
    bs = [0.0, 0.5, -0.5, 1.25, -3.3, 17.0]
    for acc in accs:
        for m in ms:
            for b in bs[: (6 if abs(acc) < 5000 else 2)]:
                for act in ("none", "relu"):
                    q, tf = _requant_exact(acc, m, b, act)
                    assert ref.requant_s8(acc, m, b, act) == q, (acc, m, b, act)
                    assert Fraction(float(ref.requant_f32(acc, m, b, act))) == tf, (acc, m, b, act)


def test_weight_quantization_round_half_even_and_clamp():
    s = np.array([0.5, 2.0], np.float32)
    w = np.array([[0.25, 0.75, 1.25, -0.25, -0.75, 100.0, -100.0, 0.3],
                  [1.0, 3.0, 5.0, -1.0, -3.0, 253.0, 255.0, -300.0]], np.float32)
    q = ref.quantize_weights(w, s)
    want = np.array([[0, 2, 2, 0, -2, 127, -127, 1], [0, 2, 2, 0, -2, 126, 127, -127]], np.int8)
    np.testing.assert_array_equal(q, want)


def test_int8_conv_output_kinds_are_consistent():
    xq = R.integers(-127, 128, size=(1, 5, 5, 4)).astype(np.int8)
    wq = R.integers(-127, 128, size=(6, 3, 3, 4)).astype(np.int8)
    m = (R.random(6) * 1e-3 + 1e-4).astype(np.float32)
    b = R.standard_normal(6).astype(np.float32)
    acc = ref.conv2d_s8(xq, wq, None, 1, 1, out="s32")
    yf = ref.conv2d_s8(xq, wq, None, 1, 1, m=m, b=b, act="relu", out="f32")
    yq = ref.conv2d_s8(xq, wq, None, 1, 1, m=m, b=b, act="relu", out="s8")
    for idx in np.ndindex(acc.shape):
        co = idx[-1]
        assert yq[idx] == ref.requant_s8(int(acc[idx]), m[co], b[co], "relu")
        assert yf[idx] == ref.requant_f32(int(acc[idx]), m[co], b[co], "relu")


def test_pools_against_library_routines():
    x = R.standard_normal((2, 9, 10, 5)).astype(np.float32)
    xt = torch.from_numpy(x).permute(0, 3, 1, 2)
    for k, s, p in [(3, 2, 1), (2, 2, 0), (3, 1, 1)]:
        want = torch.nn.functional.max_pool2d(xt, k, s, p).permute(0, 2, 3, 1).numpy()
        np.testing.assert_array_equal(ref.maxpool(x, k, s, p), want)
    # padding never counts as zero: an all-negative map keeps negative maxima
    neg = -np.abs(x) - 1.0
    assert ref.maxpool(neg, 3, 2, 1).max() < 0
    xq = R.integers(-128, 128, size=(2, 8, 8, 3)).astype(np.int8)
    want = xq.reshape(2, 4, 2, 4, 2, 3).max(axis=(2, 4))
    np.testing.assert_array_equal(ref.maxpool(xq, 2, 2, 0), want)
    np.testing.assert_allclose(ref.gavgpool(x), x.astype(np.float64).mean(axis=(1, 2)).astype(np.float32), rtol=0, atol=1e-7)


def test_relu_of_negative_zero_and_relu6():
    x = np.array([-1.0, -0.0, 0.0, 3.0, 7.0], np.float32).reshape(1, 1, 5, 1)
    wt = np.ones((1, 1, 1, 1), np.float32)
    y = ref.conv2d_f32(x, wt, act="relu").reshape(-1)
    np.testing.assert_array_equal(y, np.array([0, 0, 0, 3, 7], np.float32))
    assert not np.signbit(y[1])
    y6 = ref.conv2d_f32(x, wt, act="relu6").reshape(-1)
    np.testing.assert_array_equal(y6, np.array([0, 0, 0, 3, 6], np.float32))


def test_empty_row_gives_epilogue_of_zero():
    x = R.standard_normal((1, 4, 4, 3)).astype(np.float32)
    wt = R.standard_normal((2, 3, 3, 3)).astype(np.float32)
    mask = np.ones(wt.shape, np.uint8)
    mask[1] = 0
    bias = np.array([0.1, 0.7], np.float32)
    y = ref.conv2d_f32(x, wt, mask, 1, 1, bias=bias, act="relu")
    np.testing.assert_array_equal(y[..., 1], np.full((1, 4, 4), 0.7, np.float32))


# ---- the network walker (oracle/forward.py) ----

def _op(kind, src, dst, **kw):
    from workloads.models import Op
    return Op(kind, kw.pop("name", kind), src, dst, **kw)


def _model(ops, dtype, in_shape):
    from workloads.models import Model
    return Model("pin", dtype, in_shape, ops=ops, n_slots=max(o.dst for o in ops) + 1)


def test_walker_handworked_network():
    from oracle import forward as F
    G = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "walker_handworked.json")))
    one = lambda v: np.array(v, np.float32)
    ops = [
        _op("conv", 0, 1, c_in=1, c_out=1, k=2, act="relu", w=_w22(), scale=one([2.0]), bias=one([-20.0])),
        _op("conv", 1, 2, res=1, c_in=1, c_out=1, k=1, act="relu", w=one([0.5]).reshape(1, 1, 1, 1), bias=one([1.0])),
        _op("conv", 2, 3, res=1, c_in=1, c_out=1, k=1, act="none", w=one([-1.0]).reshape(1, 1, 1, 1)),
        _op("gavgpool", 3, 4, c_in=1, c_out=1),
        _op("fc", 4, 5, c_in=1, c_out=2, w=one([[2.0], [-1.0]]).reshape(2, 1, 1, 1), bias=one([0.25, 0.5])),
    ]
    y, slots = F.forward(_model(ops, "f32", (3, 3, 1)), _x33())
    np.testing.assert_array_equal(slots[1][0, :, :, 0], one(G["slot1"]))
    np.testing.assert_array_equal(slots[2][0, :, :, 0], one(G["slot2"]))
    np.testing.assert_array_equal(slots[3][0, :, :, 0], one(G["slot3"]))
    np.testing.assert_array_equal(slots[4].reshape(-1), one(G["slot4"]))
    np.testing.assert_array_equal(y.reshape(-1), one(G["logits"]))
    assert y is slots[5]


def test_walker_equals_the_composition_of_pinned_layer_calls_f32():
    """conv A -> conv B (+ the network input as residual) -> max pool -> fc, plus a side conv C that
    reads A's output and lands in a channel window beside a pooled copy: every slot equals the layer
    routines called one by one with explicitly named tensors."""
    from oracle import forward as F
    g = np.random.default_rng(77)
    rn = lambda *s: g.standard_normal(s).astype(np.float32)
    x = rn(2, 6, 6, 4)
    wa, wb, wc, wf = rn(4, 3, 3, 4), rn(4, 3, 3, 4), rn(3, 1, 3, 4), rn(5, 1, 1, 3 * 3 * 4)
    ma, mb = (g.random(wa.shape) < 0.5).astype(np.uint8), (g.random(wb.shape) < 0.5).astype(np.uint8)
    mf = (g.random(wf.shape) < 0.5).astype(np.uint8)
    sa, ba, sb, bb, sf, bf = rn(4), rn(4), rn(4), rn(4), rn(5), rn(5)
    ops = [
        _op("conv", 0, 1, c_in=4, c_out=4, k=3, pad=1, act="relu", w=wa, mask=ma, scale=sa, bias=ba),
        _op("conv", 1, 2, res=0, c_in=4, c_out=4, k=3, pad=1, act="relu6", w=wb, mask=mb, scale=sb, bias=bb),
        _op("maxpool", 2, 3, k=2, stride=2, pad=0, c_in=4, c_out=4),
        # a concatenation: slot 4 = [conv C of slot 1 (3 channels, 1x3 kernel, pad (0,1)) | avg pool of slot 2 (4 channels)]
        _op("conv", 1, 4, c_in=4, c_out=3, k=3, pad=0, pad_w=1, act="none", w=wc, dst_off=0, dst_total=7),
        _op("avgpool", 2, 4, k=3, stride=1, pad=1, c_in=4, c_out=4, dst_off=3, dst_total=7),
        _op("fc", 3, 5, c_in=36, c_out=5, w=wf, mask=mf, scale=sf, bias=bf),
    ]
    y, slots = F.forward(_model(ops, "f32", (6, 6, 4)), x)
    a = ref.conv2d_f32(x, wa, ma, 1, 1, 1, sa, ba, None, "relu")
    b = ref.conv2d_f32(a, wb, mb, 1, 1, 1, sb, bb, x, "relu6")
    p = ref.maxpool(b, 2, 2, 0)
    c = ref.conv2d_f32(a, wc, None, 1, (0, 1))
    q = ref.avgpool(b, 3, 1, 1)
    f = ref.fc_f32(p.reshape(2, -1), wf.reshape(5, -1), mf.reshape(5, -1), sf, bf)
    np.testing.assert_array_equal(slots[1], a)
    np.testing.assert_array_equal(slots[2], b)
    np.testing.assert_array_equal(slots[3], p)
    np.testing.assert_array_equal(slots[4], np.concatenate([c, q], axis=-1))
    np.testing.assert_array_equal(y, f)
    # the residual matters and comes from slot 0, not from the layer's own input
    assert not np.array_equal(b, ref.conv2d_f32(a, wb, mb, 1, 1, 1, sb, bb, a, "relu6"))
    assert not np.array_equal(b, ref.conv2d_f32(a, wb, mb, 1, 1, 1, sb, bb, None, "relu6"))


def test_walker_equals_the_composition_of_pinned_layer_calls_int8():
    from oracle import forward as F
    g = np.random.default_rng(78)
    ri = lambda *s: g.integers(-127, 128, size=s).astype(np.int8)
    x = ri(2, 6, 6, 4)
    wa, wb, wf = ri(4, 3, 3, 4), ri(4, 3, 3, 4), ri(5, 1, 1, 36)
    ma = (g.random(wa.shape) < 0.5).astype(np.uint8)
    m_a = np.full(4, 2e-3, np.float32); b_a = g.standard_normal(4).astype(np.float32)
    m_b = np.full(4, 3e-3, np.float32); b_b = g.standard_normal(4).astype(np.float32)
    m_f = np.full(5, 1e-3, np.float32); b_f = g.standard_normal(5).astype(np.float32)
    ops = [
        _op("conv", 0, 1, c_in=4, c_out=4, k=3, pad=1, act="relu", w=wa, mask=ma, scale=m_a, bias=b_a, out="s8"),
        _op("conv", 1, 2, res=0, res_scale=0.75, c_in=4, c_out=4, k=3, pad=1, act="relu", w=wb, scale=m_b, bias=b_b, out="s8"),
        _op("maxpool", 2, 3, k=2, stride=2, pad=0, c_in=4, c_out=4, out="s8"),
        _op("fc", 3, 4, c_in=36, c_out=5, w=wf, scale=m_f, bias=b_f, out="f32"),
    ]
    y, slots = F.forward(_model(ops, "s8", (6, 6, 4)), x)
    a = ref.conv2d_s8(x, wa, ma, 1, 1, 1, m_a, b_a, "relu", "s8")
    b = ref.conv2d_s8(a, wb, None, 1, 1, 1, m_b, b_b, "relu", "s8", x, 0.75)
    p = ref.maxpool(b, 2, 2, 0)
    f = ref.fc_s8(p.reshape(2, -1), wf.reshape(5, -1), None, m_f, b_f, "none", "f32")
    for got, want in ((slots[1], a), (slots[2], b), (slots[3], p), (y, f)):
        assert got.dtype == want.dtype
        np.testing.assert_array_equal(got, want)
    assert not np.array_equal(b, ref.conv2d_s8(a, wb, None, 1, 1, 1, m_b, b_b, "relu", "s8"))


# ---- corners ----

@pytest.mark.parametrize("k,s,p", [(3, 2, 1), (3, 1, 1), (2, 2, 1), (5, 3, 2)])
def test_padded_max_pools_against_int64_window_max(k, s, p):
    xq = R.integers(-128, 128, size=(2, 9, 7, 3)).astype(np.int8)
    n, h, w, c = xq.shape
    ho, wo = (h + 2 * p - k) // s + 1, (w + 2 * p - k) // s + 1
    lo = np.iinfo(np.int64).min
    xp = np.full((n, h + 2 * p, w + 2 * p, c), lo, np.int64)
    xp[:, p:p + h, p:p + w] = xq
    want = np.empty((n, ho, wo, c), np.int64)
    for oy in range(ho):
        for ox in range(wo):
            want[:, oy, ox] = xp[:, oy * s:oy * s + k, ox * s:ox * s + k].max(axis=(1, 2))
    got = ref.maxpool(xq, k, s, p)
    assert got.dtype == np.int8
    np.testing.assert_array_equal(got.astype(np.int64), want)
    # all-negative input: a padded tap must never win as a zero
    neg = (-np.abs(xq.astype(np.int16)) - 1).clip(-128, -1).astype(np.int8)
    assert ref.maxpool(neg, k, s, p).max() < 0


@pytest.mark.parametrize("groups", [2, 4])
def test_grouped_int8_convolution_against_brute_force(groups):
    xq = R.integers(-127, 128, size=(2, 5, 6, 8)).astype(np.int8)
    wq = R.integers(-127, 128, size=(8, 3, 3, 8 // groups)).astype(np.int8)
    mask = (R.random(wq.shape) < 0.6).astype(np.uint8)
    got = ref.conv2d_s8(xq, wq, mask, 2, 1, groups, out="s32")
    want = _brute_conv(xq.astype(np.float64), wq.astype(np.float64), mask, 2, 1, groups)
    np.testing.assert_array_equal(got.astype(np.int64), want.astype(np.int64))


@pytest.mark.parametrize("kh,kw,ph,pw,stride", [(1, 7, 0, 3, 1), (7, 1, 3, 0, 1), (1, 3, 0, 1, 1), (3, 1, 1, 0, 2), (5, 5, 2, 2, 1), (3, 3, 0, 0, 2)])
def test_rectangular_kernels_against_float64_library_convolution(kh, kw, ph, pw, stride):
    x = R.standard_normal((2, 10, 9, 6)).astype(np.float32)
    wt = R.standard_normal((5, kh, kw, 6)).astype(np.float32)
    mask = (R.random(wt.shape) < 0.4).astype(np.uint8)
    y = ref.conv2d_f32(x, wt, mask, stride, (ph, pw))
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    wtt = torch.from_numpy((wt * mask).astype(np.float64)).permute(0, 3, 1, 2)
    want = torch.nn.functional.conv2d(xt, wtt, None, stride, (ph, pw)).permute(0, 2, 3, 1).numpy()
    assert y.shape == want.shape
    np.testing.assert_allclose(y, want.astype(np.float32), rtol=0, atol=2e-6)
    # a single tap at (ky, kx) is a shift: pins which axis pad_h and pad_w belong to
    one = np.zeros((1, kh, kw, 1), np.float32)
    one[0, kh - 1, 0, 0] = 1.0
    xs = R.standard_normal((1, 10, 9, 1)).astype(np.float32)
    ys = ref.conv2d_f32(xs, one, None, 1, (ph, pw))
    for oy in range(ys.shape[1]):
        for ox in range(ys.shape[2]):
            iy, ix = oy + kh - 1 - ph, ox - pw
            want1 = xs[0, iy, ix, 0] if (0 <= iy < 10 and 0 <= ix < 9) else 0.0
            assert ys[0, oy, ox, 0] == want1


@pytest.mark.parametrize("k,s,p", [(3, 1, 1), (3, 2, 0), (5, 3, 2), (2, 2, 0)])
def test_average_pool_against_library_routine(k, s, p):
    x = R.standard_normal((2, 9, 8, 3)).astype(np.float32)
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    want = torch.nn.functional.avg_pool2d(xt, k, s, p, count_include_pad=True).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(ref.avgpool(x, k, s, p), want.astype(np.float32), rtol=0, atol=1e-7)
    # constant map: a corner window of a padded 3x3 pool sees 4 of 9 taps
    if (k, s, p) == (3, 1, 1):
        c = ref.avgpool(np.ones((1, 4, 4, 1), np.float32), 3, 1, 1)
        assert c[0, 0, 0, 0] == np.float32(4.0 / 9.0) and c[0, 1, 1, 0] == 1.0 and c[0, 0, 1, 0] == np.float32(6.0 / 9.0)


def _requant_res_exact(acc, m, b, r, rs, act):
    accf = _to_f32_exact(Fraction(acc))
    t = _to_f32_exact(accf * Fraction(float(np.float32(m))) + Fraction(float(np.float32(b))))
    t = _to_f32_exact(Fraction(int(r)) * Fraction(float(np.float32(rs))) + t)
    if act == "relu" and t < 0:
        t = Fraction(0)
    tf = t
    t = min(max(t, Fraction(-127)), Fraction(127))
    return _round_half_even(t), tf


def test_requant_with_int8_residual_against_exact_rational_arithmetic():
    accs = [0, 1, -1, 3, 5, 127, 255, 2 ** 24 + 1, -(2 ** 24) - 3, 33554433, 400000001]
    accs += [int(v) for v in R.integers(-40000, 40000, size=150)]
    for acc in accs:
        for m in (0.5, 1e-3, 0.0123456, 1.0 / 3.0):
            for b in (0.0, 0.5, -3.3):
                for r in (-127, -1, 0, 1, 3, 127):
                    for rs in (0.5, 0.75, 1.0 / 3.0, 1.37):
                        for act in ("none", "relu"):
                            q, tf = _requant_res_exact(acc, m, b, r, rs, act)
                            assert ref.requant_res_s8(acc, m, b, r, rs, act) == q, (acc, m, b, r, rs, act)
                            assert Fraction(float(ref.requant_res_f32(acc, m, b, r, rs, act))) == tf
    # literals: halves round to even AFTER the residual joined (0.5*1 + 0 + 0.5*2 = 1.5 -> 2; 2.5 -> 2)
    assert ref.requant_res_s8(1, 0.5, 0.0, 2, 0.5, "none") == 2
    assert ref.requant_res_s8(3, 0.5, 0.0, 2, 0.5, "none") == 2
    assert ref.requant_res_s8(-9, 0.5, 0.0, 2, 0.5, "relu") == 0
    assert ref.requant_res_s8(100, 1.0, 0.0, 127, 1.0, "none") == 127


def test_int8_conv_with_residual_is_the_scalar_rule_per_element():
    xq = R.integers(-127, 128, size=(1, 5, 5, 4)).astype(np.int8)
    wq = R.integers(-127, 128, size=(6, 3, 3, 4)).astype(np.int8)
    rq = R.integers(-127, 128, size=(1, 5, 5, 6)).astype(np.int8)
    m = (R.random(6) * 1e-3 + 1e-4).astype(np.float32)
    b = R.standard_normal(6).astype(np.float32)
    acc = ref.conv2d_s8(xq, wq, None, 1, 1, out="s32")
    yq = ref.conv2d_s8(xq, wq, None, 1, 1, m=m, b=b, act="relu", out="s8", residual=rq, residual_scale=0.6)
    yf = ref.conv2d_s8(xq, wq, None, 1, 1, m=m, b=b, act="none", out="f32", residual=rq, residual_scale=0.6)
    for idx in np.ndindex(acc.shape):
        co = idx[-1]
        assert yq[idx] == ref.requant_res_s8(int(acc[idx]), m[co], b[co], int(rq[idx]), 0.6, "relu")
        assert yf[idx] == ref.requant_res_f32(int(acc[idx]), m[co], b[co], int(rq[idx]), 0.6, "none")
