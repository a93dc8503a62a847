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
