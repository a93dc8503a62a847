"""GPU parity, layer by layer: the CUDA library (through its C ABI) against the CPU
oracle on the same seeded inputs.  Sizes span several tiles and ragged tails."""
import numpy as np
import pytest
import torch

from oracle import ref
from workloads import gen, models
from parity import assert_close_f32, assert_exact

pytestmark = pytest.mark.gpu

B = pytest.importorskip("paper_1905_00571_b200.binding") if torch.cuda.is_available() else None
DEV = "cuda:0"
TORCH_DT = {"f32": torch.float32, "s8": torch.int8, "s32": torch.int32}


def _seed(case):
    import zlib
    return zlib.crc32(repr(case).encode()) % (2 ** 31)


def _dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def run_conv(x, w, mask, stride, pad, groups=1, scale=None, bias=None, residual=None, act="none",
             dtype="f32", out="f32", batch_hint=None, q8=False):
    n, h, wd, c_in = x.shape
    c_out, kh, kw, _ = w.shape
    d = B.make_desc(c_in, c_out, kh, kw, stride, pad, groups, h, wd, batch_hint or n, dtype)
    wh = B.cadnn_pack_q8(d, w, mask) if q8 else B.cadnn_pack(d, w, mask)
    ho, wo = (h + 2 * pad - kh) // stride + 1, (wd + 2 * pad - kw) // stride + 1
    y = torch.empty((n, ho, wo, c_out), dtype=TORCH_DT[out], device=DEV)
    y.fill_(0)
    B.cadnn_conv2d(wh, _dev(x), y, _dev(scale), _dev(bias), _dev(residual), act, out)
    torch.cuda.synchronize()
    res = y.cpu().numpy()
    wh.free()
    return res


CONV_CASES = [
    # n, h, w, c_in, c_out, k, stride, pad, density, act
    (1, 56, 56, 64, 64, 3, 1, 1, 0.10, "relu"),
    (2, 28, 28, 32, 48, 3, 1, 1, 0.125, "relu"),
    (1, 28, 28, 32, 40, 3, 2, 1, 0.125, "relu"),
    (3, 14, 14, 24, 20, 3, 1, 1, 0.3, "none"),
    (2, 7, 7, 96, 64, 3, 1, 1, 0.125, "relu6"),
    (1, 13, 17, 5, 7, 3, 1, 1, 0.5, "relu"),      # odd sizes, c_in not a multiple of 4
    (1, 13, 17, 6, 9, 3, 2, 0, 0.5, "relu"),
    (1, 9, 9, 8, 8, 5, 1, 2, 0.2, "none"),
    (1, 40, 300, 8, 16, 3, 1, 1, 0.2, "relu"),    # wider than one tile
    (1, 32, 32, 3, 16, 7, 2, 3, 1.0, "relu"),     # stem-like dense layer
    (1, 12, 12, 16, 16, 3, 1, 1, 1.0, "none"),    # density 1.0
    (1, 12, 12, 16, 16, 3, 1, 1, 0.0, "relu"),    # one kept weight in the whole layer
    (2, 20, 20, 130, 70, 3, 1, 1, 0.05, "relu"),  # several channel chunks, ragged
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_sparse_conv_f32(case):
    n, h, w, c_in, c_out, k, stride, pad, density, act = case
    g = gen.rng(_seed(case))
    x = gen.relu_normal_input(g, (n, h, w, c_in))
    wt = gen.he_weights(g, c_out, k, k, c_in)
    mask = None if density >= 1.0 else gen.random_mask(g, wt.shape, density)
    scale, bias = gen.folded_bn(g, c_out)
    ho, wo = ref.out_hw(h, w, k, stride, pad)
    residual = gen.normal_input(g, (n, ho, wo, c_out))
    want = ref.conv2d_f32(x, wt, mask, stride, pad, 1, scale, bias, residual, act)
    got = run_conv(x, wt, mask, stride, pad, 1, scale, bias, residual, act)
    assert_close_f32(got, want, str(case))
    # no epilogue at all
    want = ref.conv2d_f32(x, wt, mask, stride, pad)
    got = run_conv(x, wt, mask, stride, pad)
    assert_close_f32(got, want, str(case) + " bare")


@pytest.mark.parametrize("batch_hint", [1, 8, 128])
def test_schedule_hint_does_not_change_results(batch_hint):
    g = gen.rng(77)
    x = gen.relu_normal_input(g, (2, 28, 28, 64))
    wt = gen.he_weights(g, 64, 3, 3, 64)
    mask = gen.magnitude_mask(wt, 0.125)
    want = ref.conv2d_f32(x, wt, mask, 1, 1, act="relu")
    got = run_conv(x, wt, mask, 1, 1, act="relu", batch_hint=batch_hint)
    assert_close_f32(got, want)


def test_skewed_and_empty_filters():
    g = gen.rng(5)
    x = gen.relu_normal_input(g, (1, 14, 14, 64))
    wt = gen.he_weights(g, 50, 3, 3, 64)
    mask = gen.skewed_mask(g, wt.shape, 0.15, skew=8.0)
    mask[3] = 0
    mask[17] = 0
    bias = gen.normal_input(g, (50,))
    want = ref.conv2d_f32(x, wt, mask, 1, 1, bias=bias, act="relu")
    got = run_conv(x, wt, mask, 1, 1, bias=bias, act="relu")
    assert_close_f32(got, want)
    np.testing.assert_array_equal(got[..., 3], np.full((1, 14, 14), max(bias[3], 0.0), np.float32))


ONE_BY_ONE = [
    (1, 56, 56, 64, 256, 1, 0.125, "relu"),
    (2, 28, 28, 256, 64, 1, 0.125, "none"),
    (1, 28, 28, 64, 96, 2, 0.125, "none"),   # strided downsample branch
    (3, 7, 7, 160, 100, 1, 0.25, "relu6"),
    (1, 9, 11, 10, 6, 1, 0.4, "relu"),
    (2, 9, 11, 10, 6, 2, 0.4, "relu"),
]


@pytest.mark.parametrize("case", ONE_BY_ONE)
def test_sparse_1x1_conv_f32(case):
    n, h, w, c_in, c_out, stride, density, act = case
    g = gen.rng(_seed(case))
    x = gen.normal_input(g, (n, h, w, c_in))
    wt = gen.he_weights(g, c_out, 1, 1, c_in)
    mask = gen.magnitude_mask(wt, density)
    scale, bias = gen.folded_bn(g, c_out)
    ho, wo = ref.out_hw(h, w, 1, stride, 0)
    residual = gen.normal_input(g, (n, ho, wo, c_out))
    want = ref.conv2d_f32(x, wt, mask, stride, 0, 1, scale, bias, residual, act)
    got = run_conv(x, wt, mask, stride, 0, 1, scale, bias, residual, act)
    assert_close_f32(got, want, str(case))


def test_identity_1x1_is_a_copy_on_gpu():
    g = gen.rng(9)
    x = gen.normal_input(g, (2, 6, 5, 12))
    wt = np.eye(12, dtype=np.float32).reshape(12, 1, 1, 12)
    got = run_conv(x, wt, (wt != 0).astype(np.uint8), 1, 0)
    np.testing.assert_array_equal(got, x)


def run_fc(x, w, mask, scale, bias, act, dtype, out, batch_hint, q8=False):
    n, k = x.shape
    c_out = w.shape[0]
    d = B.make_desc(k, c_out, batch_hint=batch_hint, dtype=dtype)
    wh = B.cadnn_pack_q8(d, w, mask) if q8 else B.cadnn_pack(d, w, mask)
    y = torch.zeros((n, c_out), dtype=TORCH_DT[out], device=DEV)
    B.cadnn_fc(wh, _dev(x), y, _dev(scale), _dev(bias), None, act, out)
    torch.cuda.synchronize()
    info = B.cadnn_weights_schedule(wh)
    wh.free()
    return y.cpu().numpy(), info


@pytest.mark.parametrize("n,hint", [(1, 1), (3, 1), (8, 8), (11, 1), (16, 16), (40, 64)])
def test_sparse_fc_f32(n, hint):
    g = gen.rng(100 + n)
    k, c_out = 2048, 1000
    x = gen.relu_normal_input(g, (n, k))
    wt = gen.he_weights(g, c_out, 1, 1, k)
    mask = gen.magnitude_mask(wt, 0.10)
    scale, bias = gen.folded_bn(g, c_out)
    want = ref.fc_f32(x, wt.reshape(c_out, k), mask.reshape(c_out, k), scale, bias, None, "none")
    got, info = run_fc(x, wt, mask, scale, bias, "none", "f32", "f32", hint)
    assert info["kind"] == (3 if hint <= 8 else 2)
    assert_close_f32(got, want, "fc n=%d" % n)


@pytest.mark.parametrize("n,hint", [(1, 1), (5, 4), (16, 16)])
@pytest.mark.parametrize("out", ["s8", "s32", "f32"])
def test_sparse_fc_s8_bit_exact(n, hint, out):
    g = gen.rng(200 + n)
    k, c_out = 3000, 515
    x = gen.int8_relu_activation(g, (n, k))
    wq = gen.int8_weights(g, (c_out, 1, 1, k))
    mask = gen.random_mask(g, wq.shape, 0.04)
    m = (g.uniform(0.5, 2.0, size=c_out) * 1e-3).astype(np.float32)
    b = (g.standard_normal(c_out) * 4).astype(np.float32)
    act = "relu" if out == "s8" else "none"
    want = ref.fc_s8(x, wq.reshape(c_out, k), mask.reshape(c_out, k), m, b, act, out)
    got, _ = run_fc(x, wq, mask, m, b, act, "s8", out, hint, q8=True)
    assert_exact(got, want, "fc s8 n=%d out=%s" % (n, out))


S8_CASES = [
    (1, 28, 28, 64, 64, 3, 1, 1, 0.08),
    (2, 14, 14, 128, 72, 3, 1, 1, 0.08),
    (1, 32, 32, 3, 64, 3, 1, 1, 0.08),      # K = 27: some filters keep nothing
    (1, 17, 13, 6, 10, 3, 2, 1, 0.5),
    (1, 10, 10, 16, 12, 1, 1, 0, 0.3),
    (1, 224, 16, 8, 8, 3, 1, 1, 0.2),
]


@pytest.mark.parametrize("case", S8_CASES)
@pytest.mark.parametrize("out", ["s8", "s32", "f32"])
def test_sparse_conv_s8_bit_exact(case, out):
    n, h, w, c_in, c_out, k, stride, pad, density = case
    g = gen.rng(_seed(case))
    x = gen.int8_image(g, (n, h, w, c_in))
    wq = gen.int8_weights(g, (c_out, k, k, c_in))
    mask = gen.random_mask(g, wq.shape, density)
    m = (g.uniform(0.5, 2.0, size=c_out) * 2e-3).astype(np.float32)
    b = (g.standard_normal(c_out) * 4).astype(np.float32)
    act = "relu" if out != "s32" else "none"
    want = ref.conv2d_s8(x, wq, mask, stride, pad, 1, m, b, act, out)
    got = run_conv(x, wq, mask, stride, pad, 1, m, b, None, act, "s8", out, q8=True)
    assert_exact(got, want, str(case) + out)


def test_int8_pack_from_float_weights_matches_oracle_quantizer():
    g = gen.rng(31)
    wt = gen.normal_weights(g, (16, 3, 3, 8), 1.0)
    s_w = (np.abs(wt).reshape(16, -1).max(1) / 127.0).astype(np.float32)
    mask = gen.random_mask(g, wt.shape, 0.3)
    x = gen.int8_image(g, (1, 9, 9, 8))
    q = ref.quantize_weights(wt, s_w)
    want = ref.conv2d_s8(x, q, mask, 1, 1, out="s32")
    d = B.make_desc(8, 16, 3, 3, 1, 1, 1, 9, 9, 1, "s8")
    wh = B.cadnn_pack(d, wt, mask, s_w)
    y = torch.zeros((1, 9, 9, 16), dtype=torch.int32, device=DEV)
    B.cadnn_conv2d(wh, _dev(x), y, out_dtype="s32")
    torch.cuda.synchronize()
    assert_exact(y.cpu().numpy(), want)


DW_CASES = [(1, 112, 112, 32, 1), (2, 56, 56, 96, 2), (1, 14, 14, 384, 1), (1, 7, 7, 960, 1), (3, 9, 11, 10, 2)]


@pytest.mark.parametrize("case", DW_CASES)
def test_depthwise_f32(case):
    n, h, w, c, stride = case
    g = gen.rng(_seed(case))
    x = gen.relu_normal_input(g, (n, h, w, c))
    wt = gen.he_weights(g, c, 3, 3, 1)
    scale, bias = gen.folded_bn(g, c)
    want = ref.conv2d_f32(x, wt, None, stride, 1, c, scale, bias, None, "relu6")
    got = run_conv(x, wt, None, stride, 1, c, scale, bias, None, "relu6")
    assert_close_f32(got, want, str(case))


def test_pools():
    g = gen.rng(3)
    x = gen.normal_input(g, (2, 112, 112, 64))
    y = torch.empty((2, 56, 56, 64), device=DEV)
    B.cadnn_maxpool2d(_dev(x), y, 3, 2, 1)
    assert_exact(y.cpu().numpy(), ref.maxpool(x, 3, 2, 1))
    xq = gen.int8_image(g, (2, 30, 30, 24))
    yq = torch.empty((2, 15, 15, 24), dtype=torch.int8, device=DEV)
    B.cadnn_maxpool2d(_dev(xq), yq, 2, 2, 0)
    assert_exact(yq.cpu().numpy(), ref.maxpool(xq, 2, 2, 0))
    xa = gen.normal_input(g, (3, 7, 7, 2048))
    ya = torch.empty((3, 2048), device=DEV)
    B.cadnn_global_avgpool(_dev(xa), ya)
    assert_close_f32(ya.cpu().numpy(), ref.gavgpool(xa))


def test_argument_errors_are_reported_not_raised_as_faults():
    d = B.make_desc(8, 8, 3, 3, 1, 1, 1, 10, 10, 1, "f32")
    wt = np.zeros((8, 3, 3, 8), np.float32)
    wh = B.cadnn_pack(d, wt)
    x = torch.zeros((1, 12, 10, 8), device=DEV)
    y = torch.zeros((1, 12, 10, 8), device=DEV)
    with pytest.raises(B.CadnnError) as e:
        B.cadnn_conv2d(wh, x, y)
    assert e.value.status == 2
    x = torch.zeros((1, 10, 10, 8), device=DEV)
    with pytest.raises(B.CadnnError) as e:
        B.cadnn_conv2d(wh, x, x)
    assert e.value.status == 1
    with pytest.raises(B.CadnnError) as e:
        B.cadnn_conv2d(wh, x, y, out_dtype="s8")
    assert e.value.status == 3
