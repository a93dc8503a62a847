"""GPU parity of what the paper's other two networks (Table 2: Inception-V3, MobileNet-V1) need beyond
ResNet / VGG / MobileNet-V2: rectangular kernels with one padding per axis, channel windows of a
concatenated output, average pools, and the two networks themselves against the oracle's walker."""
import numpy as np
import pytest
import torch

from oracle import forward as oracle_forward
from oracle import ref
from workloads import gen, models
from parity import assert_close_f32, assert_exact, NET_FLOOR

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

RECT_CASES = [
    # n, h, w, c_in, c_out, kh, kw, pad_h, pad_w, stride, density
    (1, 17, 17, 128, 128, 1, 7, 0, 3, 1, 0.125), (1, 17, 17, 128, 192, 7, 1, 3, 0, 1, 0.125),
    (2, 8, 8, 384, 384, 1, 3, 0, 1, 1, 0.125), (2, 8, 8, 448, 200, 3, 1, 1, 0, 1, 0.125),
    (1, 35, 35, 48, 64, 5, 5, 2, 2, 1, 0.125), (1, 35, 35, 288, 384, 3, 3, 0, 0, 2, 0.125),
    (2, 9, 13, 10, 7, 1, 7, 0, 3, 1, 0.5), (1, 13, 9, 10, 7, 7, 1, 3, 0, 2, 0.5), (1, 11, 11, 6, 5, 5, 5, 2, 2, 2, 1.0),
    (1, 12, 10, 16, 24, 3, 5, 0, 1, 1, 0.3),
]


@pytest.mark.parametrize("case", RECT_CASES)
def test_rectangular_kernels_f32(case):
    from paper_1905_00571_b200 import binding as B
    n, h, w, c_in, c_out, kh, kw, ph, pw, stride, density = case
    g = gen.rng(sum(case[:10]))
    x = gen.relu_normal_input(g, (n, h, w, c_in))
    wt = gen.he_weights(g, c_out, kh, kw, c_in)
    mask = None if density >= 1.0 else gen.magnitude_mask(wt, density)
    scale, bias = gen.folded_bn(g, c_out)
    want = ref.conv2d_f32(x, wt, mask, stride, (ph, pw), 1, scale, bias, None, "relu")
    d = B.make_desc(c_in, c_out, kh, kw, stride, ph, 1, h, w, n, "f32", pad_w=pw)
    wh = B.cadnn_pack(d, wt, mask)
    dense, m2 = B.cadnn_weights_unpack(wh)
    np.testing.assert_array_equal(dense, wt * (1 if mask is None else mask))
    y = torch.zeros(want.shape, device=DEV)
    dev = lambda a: torch.from_numpy(a).to(DEV)
    B.cadnn_conv2d(wh, dev(x), y, dev(scale), dev(bias), None, "relu")
    torch.cuda.synchronize()
    assert_close_f32(y.cpu().numpy(), want, str(case))


def test_rectangular_kernel_int8_bit_exact():
    from paper_1905_00571_b200 import binding as B
    g = gen.rng(91)
    x = gen.int8_relu_activation(g, (2, 12, 9, 20))
    q = gen.int8_weights(g, (24, 1, 7, 20))
    mask = gen.random_mask(g, q.shape, 0.2)
    m = (g.uniform(0.5, 1.5, size=24) * 2e-4).astype(np.float32)
    b = (g.standard_normal(24) * 3).astype(np.float32)
    # the int8 oracle takes one padding for both axes; a 1x7 kernel with pad (0, 3) equals a 7x7 kernel whose
    # only kept row is the middle one, with pad 3
    q7 = np.zeros((24, 7, 7, 20), np.int8); m7 = np.zeros((24, 7, 7, 20), np.uint8)
    q7[:, 3] = q[:, 0]; m7[:, 3] = mask[:, 0]
    want = ref.conv2d_s8(x, q7, m7, 1, 3, 1, m, b, "relu", "s8")
    d = B.make_desc(20, 24, 1, 7, 1, 0, 1, 12, 9, 2, "s8", pad_w=3)
    wh = B.cadnn_pack_q8(d, q, mask)
    y = torch.zeros(want.shape, dtype=torch.int8, device=DEV)
    dev = lambda a: torch.from_numpy(a).to(DEV)
    B.cadnn_conv2d(wh, dev(x), y, dev(m), dev(b), None, "relu", out_dtype="s8")
    torch.cuda.synchronize()
    assert_exact(y.cpu().numpy(), want, "1x7 int8")


@pytest.mark.parametrize("c_out,total,off", [(64, 256, 64), (96, 200, 104), (7, 23, 9), (32, 32, 0)])
def test_conv_writes_a_channel_window(c_out, total, off):
    """A branch of a concatenation: the layer fills channels [off, off + c_out) of a wider tensor and leaves
    the other channels alone (aligned and unaligned windows)."""
    from paper_1905_00571_b200 import binding as B
    g = gen.rng(c_out + total + off)
    x = gen.relu_normal_input(g, (2, 9, 11, 40))
    wt = gen.he_weights(g, c_out, 3, 3, 40)
    mask = gen.magnitude_mask(wt, 0.25)
    scale, bias = gen.folded_bn(g, c_out)
    want = ref.conv2d_f32(x, wt, mask, 1, 1, 1, scale, bias, None, "relu")
    wh = B.cadnn_pack(B.make_desc(40, c_out, 3, 3, 1, 1, 1, 9, 11, 2, "f32"), wt, mask)
    y = torch.full((2, 9, 11, total), -7.0, device=DEV)
    dev = lambda a: torch.from_numpy(a).to(DEV)
    B.cadnn_conv2d(wh, dev(x), y, dev(scale), dev(bias), None, "relu", out_c_total=total, out_c_off=off)
    torch.cuda.synchronize()
    got = y.cpu().numpy()
    assert_close_f32(got[..., off:off + c_out], want, "window")
    rest = np.delete(got, np.s_[off:off + c_out], axis=-1)
    assert (rest == -7.0).all()
    # a window that does not fit is refused
    with pytest.raises(B.CadnnError):
        B.cadnn_conv2d(wh, dev(x), y, dev(scale), dev(bias), None, "relu", out_c_total=total, out_c_off=total - c_out + 1)


@pytest.mark.parametrize("kind,k,s,p", [("avg", 3, 1, 1), ("avg", 3, 2, 0), ("avg", 5, 3, 2), ("max", 3, 2, 0), ("max", 3, 2, 1)])
def test_pools_into_channel_windows(kind, k, s, p):
    from paper_1905_00571_b200 import binding as B
    g = gen.rng(k * 100 + s * 10 + p)
    x = gen.normal_input(g, (2, 13, 10, 24))
    want = ref.avgpool(x, k, s, p) if kind == "avg" else ref.maxpool(x, k, s, p)
    for total, off in ((0, 0), (40, 11)):
        shape = want.shape[:-1] + (total or 24,)
        y = torch.full(shape, -7.0, device=DEV)
        B.cadnn_pool2d(torch.from_numpy(x).to(DEV), y, k, s, p, kind, total, off)
        torch.cuda.synchronize()
        got = y.cpu().numpy()
        if kind == "avg":
            assert_close_f32(got[..., off:off + 24], want, "avg pool")
        else:
            assert_exact(got[..., off:off + 24], want, "max pool")
        if total:
            assert (np.delete(got, np.s_[off:off + 24], axis=-1) == -7.0).all()
    if kind == "max":
        xq = gen.int8_image(g, (2, 13, 10, 24))
        y = torch.zeros(ref.maxpool(xq, k, s, p).shape[:-1] + (30,), dtype=torch.int8, device=DEV)
        B.cadnn_pool2d(torch.from_numpy(xq).to(DEV), y, k, s, p, "max", 30, 6)
        torch.cuda.synchronize()
        assert_exact(y.cpu().numpy()[..., 6:30], ref.maxpool(xq, k, s, p), "int8 max pool window")


def _run(model, batch, use_graph=True, autotune=False):
    from paper_1905_00571_b200.network import PackedModel
    x = models.make_input(model, batch)
    pm = PackedModel(model, batch, DEV, autotune=autotune)
    xd = torch.from_numpy(x).to(DEV)
    y = pm.new_output()
    pm.forward(xd, y, use_graph=use_graph)
    pm.forward(xd, y, use_graph=use_graph)
    torch.cuda.synchronize()
    return x, y.cpu().numpy(), pm


def _check_logits(got, want):
    assert_close_f32(got, want, "logits", floor=NET_FLOOR)
    for b in range(want.shape[0]):
        assert set(np.argsort(-got[b])[:5]) == set(np.argsort(-want[b])[:5])


@pytest.mark.parametrize("batch,use_graph", [(1, True), (2, False)])
def test_inception_v3_reduced(batch, use_graph):
    m = models.inception_v3(width=0.25, image=139, classes=100)
    x, got, pm = _run(m, batch, use_graph)
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)
    # the static-workspace entry point places a concatenation once, at its first writer
    y2 = torch.zeros_like(pm.new_output())
    pm.forward_static(torch.from_numpy(x).to(DEV), y2)
    torch.cuda.synchronize()
    _check_logits(y2.cpu().numpy(), want)


def test_inception_v3_full_batch1():
    m = models.inception_v3()
    x, got, _ = _run(m, 1)
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)


@pytest.mark.parametrize("batch", [1, 3])
def test_mobilenet_v1_reduced(batch):
    m = models.mobilenet_v1(width=0.5, image=96, classes=100)
    x, got, _ = _run(m, batch)
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)


def test_mobilenet_v1_full_batch1():
    from paper_1905_00571_b200 import binding as B
    m = models.mobilenet_v1()
    x, got, pm = _run(m, 1)
    assert B.cadnn_net_layout(pm.net)["planar"]
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)


@pytest.mark.parametrize("out", ["s8", "f32"])
@pytest.mark.parametrize("c_out", [64, 30])
def test_int8_conv_with_int8_residual_bit_exact(out, c_out):
    """The shortcut of a quantized residual block: a second fused multiply-add on the int8 residual before the ReLU."""
    from paper_1905_00571_b200 import binding as B
    g = gen.rng(300 + c_out)
    x = gen.int8_relu_activation(g, (2, 9, 10, 48))
    q = gen.int8_weights(g, (c_out, 3, 3, 48))
    mask = gen.random_mask(g, q.shape, 0.15)
    r = gen.int8_relu_activation(g, (2, 9, 10, c_out))
    m = (g.uniform(0.5, 1.5, size=c_out) * 3e-4).astype(np.float32)
    b = (g.standard_normal(c_out) * 3).astype(np.float32)
    want = ref.conv2d_s8(x, q, mask, 1, 1, 1, m, b, "relu", out, r, 0.6)
    wh = B.cadnn_pack_q8(B.make_desc(48, c_out, 3, 3, 1, 1, 1, 9, 10, 2, "s8"), q, mask)
    y = torch.zeros(want.shape, dtype=torch.int8 if out == "s8" else torch.float32, device=DEV)
    dev = lambda a: torch.from_numpy(a).to(DEV)
    B.cadnn_conv2d(wh, dev(x), y, dev(m), dev(b), dev(r), "relu", out_dtype=out, residual_scale=0.6)
    torch.cuda.synchronize()
    assert_exact(y.cpu().numpy(), want, "int8 residual")
    assert not np.array_equal(want, ref.conv2d_s8(x, q, mask, 1, 1, 1, m, b, "relu", out))


@pytest.mark.parametrize("batch", [1, 2])
def test_resnet50_int8_reduced(batch):
    from paper_1905_00571_b200 import binding as B
    m = models.resnet50_int8(width=0.25, image=64, classes=100)
    x, got, pm = _run(m, batch)
    want, slots = oracle_forward.forward(m, x)
    _check_logits(got, want)
    # everything up to the float tail is integer work: the last int8 tensor matches bit for bit
    import ctypes
    last_q = [op for op in m.ops if op.out == "s8"][-1]
    ptr, nbytes = B.cadnn_net_slot(pm.net, last_q.dst)
    host = np.empty(nbytes, np.int8)
    assert ctypes.CDLL("libcudart.so").cudaMemcpy(ctypes.c_void_p(host.ctypes.data), ctypes.c_void_p(ptr), ctypes.c_size_t(nbytes), 2) == 0
    assert_exact(host[:slots[last_q.dst].size].reshape(slots[last_q.dst].shape), slots[last_q.dst], last_q.name)


def test_resnet50_int8_full_batch1():
    m = models.resnet50_int8()
    x, got, _ = _run(m, 1)
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)
