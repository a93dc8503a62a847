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


@pytest.mark.parametrize("tb,grid,tile_kb", [(1, 0, 0), (2, 0, 0), (3, 40, 0), (4, 0, 0), (6, 0, 0), (8, 0, 0),
                                             (0, 0, 16), (2, 33, 24), (1, 5, 0)])
def test_persistent_item_shapes(tb, grid, tile_kb, monkeypatch):
    """Every tile size of the item planner (ragged last tiles included), fewer blocks than items
    (several items per block and phase), and a tile buffer so small that the input channels are
    taken in several passes with partial sums parked in shared memory."""
    if tb:
        monkeypatch.setenv("CADNN_PERSIST_TB", str(tb))
    if grid:
        monkeypatch.setenv("CADNN_PERSIST_GRID", str(grid))
    if tile_kb:
        monkeypatch.setenv("CADNN_PERSIST_TILE_KB", str(tile_kb))
    m = models.resnet50(width=0.25, image=64, classes=100)
    x, got, info = _run(m, 2, True, True, monkeypatch)
    if tb not in (6, 8):   # (tiles of 6 or 8 bands exceed what a stride-2 layer of this net can stage: no plan, layered run)
        assert info["launches"] < len(m.ops) - 40, info
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)


@pytest.mark.parametrize("no_parity", [False, True])
def test_persistent_stride2_layouts(no_parity, monkeypatch):
    """Stride-2 layers read parity planes written by their producer (default), or stage whole input rows
    and address them with a lane stride (the fallback when the producer is not part of the run)."""
    if no_parity:
        monkeypatch.setenv("CADNN_PERSIST_NO_PARITY", "1")
    m = models.resnet50(width=0.5, image=96, classes=100)
    x, got, info = _run(m, 2, True, True, monkeypatch)
    assert info["launches"] < len(m.ops) - 40, info
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)


def test_persistent_odd_map_sizes(monkeypatch):
    """Odd plane sizes at stride 2 (image 72: 18 -> 9 -> 5 -> 3) through the persistent kernel."""
    m = models.resnet50(width=0.25, image=72, classes=100)
    x, got, info = _run(m, 1, True, True, monkeypatch)
    want, _ = oracle_forward.forward(m, x)
    _check_logits(got, want)
