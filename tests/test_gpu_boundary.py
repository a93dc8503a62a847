"""GPU checks of boundary conventions: the device status word surfaces as
CADNN_E_DEVICE_STATUS at the net's synchronization points (driven from the host: no kernel is
made to wait), an op list whose residual is not a planar tensor falls back to NHWC, graph
replays read fresh inputs, and the alias names work."""
import numpy as np
import pytest
import torch

from oracle import forward as oracle_forward
from oracle import ref
from workloads import gen, models
from parity import assert_close_f32, NET_FLOOR

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_device_status_word_is_surfaced_at_sync_points():
    from paper_1905_00571_b200 import binding as B
    from paper_1905_00571_b200.network import PackedModel
    m = models.resnet50(width=0.25, image=64, classes=100)
    pm = PackedModel(m, 1, DEV)
    x = models.make_input(m, 1)
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.empty((1, 100)).pin_memory()
    want, _ = oracle_forward.forward(m, x)
    base = B.cadnn_device_status()["copy_timeouts"]
    assert base == 0
    pm.forward_host(xh, yh)                      # clean run: OK
    assert_close_f32(yh.numpy(), want, "host forward", floor=NET_FLOOR)
    try:
        B.cadnn_debug_set_device_status(3, 0)    # as if three waits on a copy barrier had run out
        with pytest.raises(B.CadnnError) as e:
            pm.forward_host(xh, yh)
        assert e.value.status == 7
        assert B.cadnn_device_status()["copy_timeouts"] == 3
        pm.forward_host(xh, yh)                  # nothing moved since the net last looked: OK again
        xd = torch.from_numpy(x).to(DEV)
        yd = pm.new_output()
        B.cadnn_debug_set_device_status(4, 0)
        with pytest.raises(B.CadnnError) as e:
            B.cadnn_net_layer_time(pm.net, 0, xd, yd)
        assert e.value.status == 7
        t = B.cadnn_net_layer_time(pm.net, 0, xd, yd, reps=4)
        assert 0.0 < t < 10.0
        assert len(pm.layer_times(xd, yd)) == len(m.ops)
    finally:
        B.cadnn_debug_set_device_status(0, 0)
    assert B.cadnn_device_status()["copy_timeouts"] == 0


def test_residual_from_the_network_input_keeps_the_net_nhwc():
    """conv(x) + x: the residual is slot 0, an NHWC tensor, so the planar kernels must not be chosen."""
    from paper_1905_00571_b200 import binding as B
    g = gen.rng(5)
    c = 16
    x = gen.relu_normal_input(g, (2, 10, 10, c))
    w1 = gen.he_weights(g, c, 3, 3, c); m1 = gen.random_mask(g, w1.shape, 0.3)
    wf = gen.he_weights(g, 7, 1, 1, c); mf = gen.random_mask(g, wf.shape, 0.5)
    h1 = B.cadnn_pack(B.make_desc(c, c, 3, 3, 1, 1, 1, 10, 10, 2, "f32"), w1, m1)
    hf = B.cadnn_pack(B.make_desc(c, 7, 1, 1, 1, 0, 1, 1, 1, 2, "f32"), wf, mf)
    ops = [B.Op(B.OP_CONV, h1.handle, 0, 1, 0, None, None, B.ACT["relu"], B.F32, 0, 0, 0),
           B.Op(B.OP_GAVGPOOL, None, 1, 2, -1, None, None, 0, B.F32, 0, 0, 0),
           B.Op(B.OP_FC, hf.handle, 2, 3, -1, None, None, 0, B.F32, 0, 0, 0)]
    net = B.cadnn_net_create(ops, 2, 10, 10, c, "f32", keep=(h1, hf))
    assert B.cadnn_net_layout(net)["planar"] is False
    a = ref.conv2d_f32(x, w1, m1, 1, 1, residual=x, act="relu")
    want = ref.fc_f32(ref.gavgpool(a), wf.reshape(7, -1), mf.reshape(7, -1))
    y = torch.zeros((2, 7), device=DEV)
    B.cadnn_forward(net, torch.from_numpy(x).to(DEV), y, True, None)
    torch.cuda.synchronize()
    assert_close_f32(y.cpu().numpy(), want, "residual from slot 0")
    B.cadnn_free_weights(h1)
    assert h1.handle is None


def test_graph_replays_read_fresh_input_contents():
    """The same x buffer is overwritten between replays of the captured graph (layers launched as
    programmatic dependents): every replay must see the new contents."""
    from paper_1905_00571_b200.network import PackedModel
    for m in (models.resnet50(width=0.25, image=64, classes=100), models.mobilenet_v2(width=0.5, image=64, classes=100)):
        pm = PackedModel(m, 1, DEV)
        xd = torch.empty((1,) + tuple(m.in_shape), device=DEV)
        y = pm.new_output()
        for seed in (11, 12, 13):
            x = models.make_input(m, 1, seed=seed)
            xd.copy_(torch.from_numpy(x))
            pm.forward(xd, y, use_graph=True)
            torch.cuda.synchronize()
            want, _ = oracle_forward.forward(m, x)
            assert_close_f32(y.cpu().numpy(), want, "%s replay with seed %d" % (m.name, seed), floor=NET_FLOOR)
