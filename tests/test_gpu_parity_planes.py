"""GPU parity of the stride-2 layers that run as stride-1 layers over parity planes of their input (the layer
before them stores its output a second time, split by row and column parity): whole networks and every tensor in
between against the oracle's walker, odd and rectangular map sizes included."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import forward as oracle_forward
from workloads import gen, models
from parity import assert_close_f32, NET_FLOOR

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _slot_to_host(B, net, slot):
    ptr, nbytes = B.cadnn_net_slot(net, slot)
    host = np.empty(nbytes // 4, np.float32)
    rt = ctypes.CDLL("libcudart.so")
    assert rt.cudaMemcpy(ctypes.c_void_p(host.ctypes.data), ctypes.c_void_p(ptr), ctypes.c_size_t(nbytes), 2) == 0
    return host


def _planes_to_nhwc(raw, shape):
    n, h, w, c = shape
    pitch = ((h + 2) * (w + 2) + 3) // 4 * 4
    planes = raw[:n * c * pitch].reshape(n, c, pitch)
    grid = planes[:, :, :(h + 2) * (w + 2)].reshape(n, c, h + 2, w + 2)
    border = grid.copy()
    border[:, :, 1:h + 1, 1:w + 1] = 0
    assert not border.any(), "a plane's border was written"
    return grid[:, :, 1:h + 1, 1:w + 1].transpose(0, 2, 3, 1)


def _run_and_compare(m, batch, expect_layers, monkeypatch, autotune=False):
    from paper_1905_00571_b200 import binding as B
    from paper_1905_00571_b200.network import PackedModel
    monkeypatch.setenv("CADNN_FORCE_PLANAR", "1")
    monkeypatch.setenv("CADNN_FORCE_PARITY_PLANES", "1")
    monkeypatch.setenv("CADNN_PERSIST", "0")
    x = models.make_input(m, batch)
    pm = PackedModel(m, batch, DEV, autotune=autotune)
    assert B.cadnn_net_layout(pm.net)["planar"]
    assert B.cadnn_net_parity_layers(pm.net) == expect_layers
    xd = torch.from_numpy(x).to(DEV)
    y = pm.new_output()
    for use_graph in (False, True, True):
        y.zero_()
        pm.forward(xd, y, use_graph=use_graph)
    torch.cuda.synchronize()
    assert B.cadnn_device_status()["copy_timeouts"] == 0
    want, slots = oracle_forward.forward(m, x)
    for op in m.ops[:-1]:
        ref_t = slots[op.dst]
        if ref_t.ndim != 4:
            continue
        got = _planes_to_nhwc(_slot_to_host(B, pm.net, op.dst), ref_t.shape)
        assert_close_f32(got, ref_t, "output of %s" % op.name, floor=NET_FLOOR)
    assert_close_f32(y.cpu().numpy(), want, "logits", floor=NET_FLOOR)


@pytest.mark.parametrize("batch,image", [(1, 64), (3, 72), (2, 96)])
def test_reduced_resnet50_with_parity_plane_layers(batch, image, monkeypatch):
    """The three 3x3 and three 1x1 stride-2 layers of ResNet-50 v1.5 in their stride-1 form; image 72 gives the odd
    plane sizes 9 and 5."""
    _run_and_compare(models.resnet50(width=0.25, image=image, classes=100), batch, 6, monkeypatch)


def _conv(m, g, name, src, c_in, c_out, k, stride, pad, hw, act, density, res=-1):
    w = gen.he_weights(g, c_out, k, k, c_in)
    mask = None if density >= 1.0 else gen.random_mask(g, w.shape, density)
    scale, bias = gen.folded_bn(g, c_out, gain=1.0 / np.sqrt(max(density, 1e-3)))
    ho = ((hw[0] + 2 * pad - k) // stride + 1, (hw[1] + 2 * pad - k) // stride + 1)
    dst = m.new_slot()
    m.ops.append(models.Op("conv", name, src, dst, res, c_in, c_out, k, stride, pad, 1, act, w, mask, scale, bias,
                           "f32", density, hw, ho))
    return dst, ho


@pytest.mark.parametrize("in_hw", [(26, 34), (25, 33), (12, 40)])
def test_rectangular_odd_maps_at_stride_2(in_hw, monkeypatch):
    """13 x 17 (and 13 x 17 from an odd image, 6 x 20) maps: a 3x3 stride-2 layer over four parity planes and a 1x1
    stride-2 layer over the (even, even) plane of another tensor, joined as a residual."""
    g = gen.rng(41)
    m = models.Model("odd_maps", "f32", (in_hw[0], in_hw[1], 3), seed=41)
    stem, hw = _conv(m, g, "stem", 0, 3, 16, 3, 2, 1, in_hw, "relu", 1.0)
    a, _ = _conv(m, g, "a", stem, 16, 32, 1, 1, 0, hw, "relu", 0.3)
    b, _ = _conv(m, g, "b", a, 32, 48, 1, 1, 0, hw, "relu", 0.3)
    ds, hw2 = _conv(m, g, "ds", a, 32, 64, 1, 2, 0, hw, "none", 0.3)
    c2, hw2b = _conv(m, g, "c2", b, 48, 48, 3, 2, 1, hw, "relu", 0.2)
    assert hw2 == hw2b
    c3, _ = _conv(m, g, "c3", c2, 48, 64, 1, 1, 0, hw2, "relu", 0.3, res=ds)
    pool = m.new_slot()
    m.ops.append(models.Op("gavgpool", "pool", c3, pool, c_in=64, c_out=64, in_hw=hw2, out_hw=(1, 1)))
    w = gen.he_weights(g, 10, 1, 1, 64)
    m.ops.append(models.Op("fc", "fc", pool, m.new_slot(), -1, 64, 10, 1, 1, 0, 1, "none", w, None,
                           np.ones(10, np.float32), np.zeros(10, np.float32), "f32", 1.0, (1, 1), (1, 1)))
    _run_and_compare(m, 2, 2, monkeypatch)


def test_full_resnet50_takes_the_faster_form(monkeypatch):
    """With timed schedules the net picks per layer; whatever it picks matches the oracle."""
    from paper_1905_00571_b200 import binding as B
    from paper_1905_00571_b200.network import PackedModel
    monkeypatch.setenv("CADNN_PERSIST", "0")
    m = models.resnet50()
    x = models.make_input(m, 1)
    pm = PackedModel(m, 1, DEV, autotune=True)
    assert B.cadnn_net_layout(pm.net)["planar"]
    assert 0 <= B.cadnn_net_parity_layers(pm.net) <= 6
    y = pm.new_output()
    pm.forward(torch.from_numpy(x).to(DEV), y)
    torch.cuda.synchronize()
    want, _ = oracle_forward.forward(m, x)
    assert_close_f32(y.cpu().numpy(), want, "logits", floor=NET_FLOOR)
