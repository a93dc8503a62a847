"""GPU parity of the persistent whole-network kernel (one cooperative launch for the run of
sparse convs, grid barriers between layers) against the oracle's network walker, and against
the layer-by-layer path of the same library."""
import numpy as np
import pytest
import torch

from oracle import forward as oracle_forward
from workloads import models
from parity import assert_close_f32, NET_FLOOR

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run(model, batch, use_graph, persistent, monkeypatch, calls=2):
    from paper_1905_00571_b200 import binding as B
    from paper_1905_00571_b200.network import PackedModel
    if persistent:
        monkeypatch.setenv("CADNN_PERSIST", "1")
    else:
        monkeypatch.setenv("CADNN_PERSIST", "0")
    x = models.make_input(model, batch)
    pm = PackedModel(model, batch, DEV)
    info = B.cadnn_net_info(pm.net)
    xd = torch.from_numpy(x).to(DEV)
    y = pm.new_output()
    for _ in range(calls):   # the second call replays the captured graph; barrier words must be back at zero
        y.zero_()
        pm.forward(xd, y, use_graph=use_graph)
    torch.cuda.synchronize()
    assert B.cadnn_device_status()["copy_timeouts"] == 0
    return x, y.cpu().numpy(), info


def _check_logits(got, want):
    assert_close_f32(got, want, "logits", floor=NET_FLOOR)
    for b in range(want.shape[0]):
        assert set(np.argsort(-got[b])[:5]) == set(np.argsort(-want[b])[:5])


@pytest.mark.parametrize("batch,use_graph", [(1, True), (1, False), (3, True), (2, False)])
def test_resnet50_reduced_persistent(batch, use_graph, monkeypatch):
    m = models.resnet50(width=0.25, image=64, classes=100)
    x, got, info = _run(m, batch, use_graph, True, monkeypatch, calls=3)
    assert info["launches"] < len(m.ops) - 40, info   # the 52 sparse convs are one launch
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)
    _, layered, info2 = _run(m, batch, use_graph, False, monkeypatch)
    assert info2["launches"] == len(m.ops)
    assert_close_f32(got, layered, "persistent vs layer-by-layer", floor=NET_FLOOR)


def test_resnet50_full_batch1_persistent(monkeypatch):
    m = models.resnet50()
    x, got, info = _run(m, 1, True, True, monkeypatch, calls=3)
    assert info["launches"] == len(m.ops) - 51, info
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)


@pytest.mark.parametrize("T,ksw", [(1, 1), (2, 8), (8, 2), (4, 4)])
def test_persistent_task_shapes(T, ksw, monkeypatch):
    """Every (bands per lane, warps per filter) shape of the task loop, ragged tiles included."""
    monkeypatch.setenv("CADNN_PERSIST_T", str(T))
    monkeypatch.setenv("CADNN_PERSIST_KSW", str(ksw))
    m = models.resnet50(width=0.25, image=64, classes=100)
    x, got, info = _run(m, 2, True, True, monkeypatch)
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)
