"""GPU parity, whole networks: cadnn_forward against the oracle's network walker."""
import numpy as np
import pytest
import torch

from oracle import forward as oracle_forward
from workloads import models
from parity import assert_close_f32, assert_exact, NET_FLOOR

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run(model, batch, use_graph=True):
    from paper_1905_00571_b200.network import PackedModel
    x = models.make_input(model, batch)
    pm = PackedModel(model, batch, DEV)
    xd = torch.from_numpy(x).to(DEV)
    y = pm.new_output()
    pm.forward(xd, y, use_graph=use_graph)
    pm.forward(xd, y, use_graph=use_graph)   # second call replays the captured graph
    torch.cuda.synchronize()
    return x, y.cpu().numpy()


def _check_logits(got, want):
    assert_close_f32(got, want, "logits", floor=NET_FLOOR)
    for b in range(want.shape[0]):
        assert set(np.argsort(-got[b])[:5]) == set(np.argsort(-want[b])[:5])


@pytest.mark.parametrize("batch,use_graph", [(1, True), (3, False)])
def test_resnet50_reduced(batch, use_graph):
    m = models.resnet50(width=0.25, image=64, classes=100)
    x, got = _run(m, batch, use_graph)
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)


def test_resnet50_full_batch1():
    m = models.resnet50()
    x, got = _run(m, 1)
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)


@pytest.mark.parametrize("batch", [1, 2])
def test_mobilenet_v2_reduced(batch):
    m = models.mobilenet_v2(width=0.5, image=96, classes=100)
    x, got = _run(m, batch)
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)


def test_mobilenet_v2_full_batch1():
    m = models.mobilenet_v2()
    x, got = _run(m, 1)
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)


@pytest.mark.parametrize("batch", [1, 2])
def test_vgg16_int8_reduced_bit_exact(batch):
    m = models.vgg16(width=0.25, image=64, classes=100, fc_width=256)
    x, got = _run(m, batch)
    want, _ = oracle_forward.forward(m, x)
    assert_exact(got, want, "vgg logits")


def test_vgg16_int8_full_batch1_bit_exact():
    m = models.vgg16()
    x, got = _run(m, 1)
    want, _ = oracle_forward.forward(m, x)
    assert_exact(got, want, "vgg logits")


def test_graph_with_parallel_branches_matches_layer_by_layer():
    """A hand-made op list with a branch read later as a residual and a branch nobody reads: the captured
    graph (forked branches, joined where read or at the end) gives the oracle's result, as does the
    plain launch order."""
    from paper_1905_00571_b200 import binding as B
    from oracle import ref
    from workloads import gen
    g = gen.rng(77)
    c = 16
    x = gen.relu_normal_input(g, (2, 12, 12, c))
    ws, masks, handles = [], [], []
    for _ in range(5):
        w = gen.he_weights(g, c, 3, 3, c)
        m = gen.random_mask(g, w.shape, 0.3)
        d = B.make_desc(c, c, 3, 3, 1, 1, 1, 12, 12, 2, "f32")
        ws.append(w); masks.append(m); handles.append(B.cadnn_pack(d, w, m))
    # slots: 0 input; A: 0->1; B: 1->2 (read only by D, as residual); C: 1->3; D: 3->4 (+2); E: 1->5 (never read); F: 4->6
    plan = [(0, 0, 1, -1), (1, 1, 2, -1), (2, 1, 3, -1), (3, 3, 4, 2), (4, 1, 5, -1), (0, 4, 6, -1)]
    ops = [B.Op(B.OP_CONV, handles[wi].handle, src, dst, res, None, None, B.ACT["relu"], B.DTYPE["f32"], 0, 0, 0)
           for wi, src, dst, res in plan]
    vals = {0: x}
    for wi, src, dst, res in plan:
        vals[dst] = ref.conv2d_f32(vals[src], ws[wi], masks[wi], 1, 1, residual=vals[res] if res >= 0 else None, act="relu")
    net = B.cadnn_net_create(ops, 2, 12, 12, c, "f32", keep=handles)
    xd = torch.from_numpy(x).to(DEV)
    for use_graph in (True, True, False):
        y = torch.zeros((2, 12, 12, c), device=DEV)
        B.cadnn_forward(net, xd, y, use_graph, None)
        torch.cuda.synchronize()
        assert_close_f32(y.cpu().numpy(), vals[6], "forked graph" if use_graph else "stream order")


@pytest.mark.parametrize("image,batch", [(80, 3), (72, 1)])
def test_mobilenet_v2_runs_channel_planar(image, batch, monkeypatch):
    """Depthwise layers have a planar kernel: the whole MobileNet-V2 keeps planar feature maps (odd map
    sizes at stride 2 included) and matches the oracle; the NHWC route gives the same logits."""
    from paper_1905_00571_b200 import binding as B
    from paper_1905_00571_b200.network import PackedModel
    m = models.mobilenet_v2(width=0.5, image=image, classes=100)
    x = models.make_input(m, batch)
    want, _ = oracle_forward.forward(m, x)
    xd = torch.from_numpy(x).to(DEV)
    outs = []
    for planar in (True, False):
        if planar:
            monkeypatch.delenv("CADNN_NO_PLANAR_DW", raising=False)
        else:
            monkeypatch.setenv("CADNN_NO_PLANAR_DW", "1")
        pm = PackedModel(m, batch, DEV)
        assert B.cadnn_net_layout(pm.net)["planar"] == planar
        y = pm.new_output()
        pm.forward(xd, y)
        pm.forward(xd, y, use_graph=False)
        torch.cuda.synchronize()
        _check_logits(y.cpu().numpy(), want)
        outs.append(y.cpu().numpy())
    assert_close_f32(outs[0], outs[1], "planar vs NHWC", floor=NET_FLOOR)


@pytest.mark.parametrize("name", ["resnet50", "mobilenet_v2", "resnet50_int8"])
def test_general_graph_scheduler_on_residual_networks(name, monkeypatch):
    """The lane scheduler that captures independent branches as parallel graph branches (the default for networks with
    concatenations) forced on residual networks: three replays with the input buffer overwritten in between - a missing
    dependency would let a layer read a tensor of the previous replay - against the oracle."""
    from paper_1905_00571_b200.network import PackedModel
    monkeypatch.setenv("CADNN_GRAPH_LANES", "1")
    monkeypatch.setenv("CADNN_FORCE_PARITY_PLANES", "1")
    if name == "resnet50":
        m = models.resnet50(width=0.25, image=64, classes=100)
    elif name == "mobilenet_v2":
        m = models.mobilenet_v2(width=0.5, image=64, classes=100)
    else:
        m = models.resnet50_int8(width=0.25, image=64, classes=100)
    pm = PackedModel(m, 2, DEV)
    y = pm.new_output()
    xd = None
    for seed in (11, 12, 13):
        x = models.make_input(m, 2, seed=seed)
        if xd is None:
            xd = torch.from_numpy(x).to(DEV)
        else:
            xd.copy_(torch.from_numpy(x))
        pm.forward(xd, y)
        torch.cuda.synchronize()
        want, _ = oracle_forward.forward(m, x)
        got = y.cpu().numpy()
        _check_logits(got, want)   # (the int8 network's pooled vector and classifier are float: close, not bit-equal)
