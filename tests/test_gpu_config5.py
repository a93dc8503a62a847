"""GPU parity beyond batch 1 and below the logits: the pruned ResNet-50 of the batch sweep at batch 8
(full size) and batch 32 (reduced), images first / middle / last against the oracle, and every
intermediate tensor of the full-size channel-planar network against the oracle's slots."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import forward as oracle_forward
from workloads import models
from parity import assert_close_f32, NET_FLOOR, REL_TOL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _check_images(model, batch, autotune, picks):
    from paper_1905_00571_b200.network import PackedModel
    x = models.make_input(model, batch)
    pm = PackedModel(model, batch, DEV, autotune=autotune)
    xd = torch.from_numpy(x).to(DEV)
    y = pm.new_output()
    pm.forward(xd, y)
    pm.forward(xd, y)
    torch.cuda.synchronize()
    got = y.cpu().numpy()
    for b in picks:
        want, _ = oracle_forward.forward(model, x[b:b + 1])
        assert_close_f32(got[b:b + 1], want, "image %d of %d" % (b, batch), floor=NET_FLOOR)
        assert set(np.argsort(-got[b])[:5]) == set(np.argsort(-want[0])[:5])
    # every image of the batch got its own result (no image computed twice, none skipped)
    assert len({got[b].tobytes() for b in range(batch)}) == batch


def test_resnet50_full_size_batch8_with_timed_schedules():
    _check_images(models.resnet50(), 8, True, (0, 4, 7))


def test_resnet50_reduced_batch32_with_timed_schedules():
    _check_images(models.resnet50(width=0.25, image=64, classes=100), 32, True, (0, 15, 31))


@pytest.mark.parametrize("density", [0.05, 0.5, 1.0])
def test_resnet50_reduced_density_sweep_batch8(density):
    """The other densities of the sweep (masks nested by magnitude), schedules from the time model."""
    _check_images(models.resnet50(width=0.25, image=64, classes=100, density=density,
                                  fc_density=0.10 if density < 1.0 else 1.0), 8, False, (0, 3, 7))


def _slot_to_host(B, net, slot):
    ptr, nbytes = B.cadnn_net_slot(net, slot)
    if not ptr:
        return None
    host = np.empty(nbytes // 4, np.float32)
    rt = ctypes.CDLL("libcudart.so")
    rc = rt.cudaMemcpy(ctypes.c_void_p(host.ctypes.data), ctypes.c_void_p(ptr), ctypes.c_size_t(nbytes), 2)
    assert rc == 0
    return host


def test_every_intermediate_tensor_of_the_planar_resnet50():
    """Walks the slots of the full-size network (channel planes with a zero border) and compares each with
    the oracle's tensor of the same slot; the assertion names the first layer out of tolerance."""
    from paper_1905_00571_b200 import binding as B
    from paper_1905_00571_b200.network import PackedModel
    m = models.resnet50()
    x = models.make_input(m, 1)
    pm = PackedModel(m, 1, DEV, autotune=True)
    assert B.cadnn_net_layout(pm.net)["planar"]
    y = pm.new_output()
    pm.forward(torch.from_numpy(x).to(DEV), y)
    torch.cuda.synchronize()
    want, slots = oracle_forward.forward(m, x)
    checked = 0
    for op in m.ops[:-1]:
        ref_t = slots[op.dst]
        raw = _slot_to_host(B, pm.net, op.dst)
        assert raw is not None, op.name
        if ref_t.ndim == 2:                      # the pooled vector that feeds the classifier
            got = raw[:ref_t.size].reshape(ref_t.shape)
        else:
            n, h, w, c = ref_t.shape
            pitch = ((h + 2) * (w + 2) + 3) // 4 * 4
            planes = raw[:n * c * pitch].reshape(n, c, pitch)
            grid = planes[:, :, :(h + 2) * (w + 2)].reshape(n, c, h + 2, w + 2)
            border = grid.copy()
            border[:, :, 1:h + 1, 1:w + 1] = 0
            assert not border.any() and not planes[:, :, (h + 2) * (w + 2):].any(), "border of %s was written" % op.name
            got = grid[:, :, 1:h + 1, 1:w + 1].transpose(0, 2, 3, 1)
        # rounding compounds layer by layer: the whole-network floor applies from the first layer on
        assert_close_f32(got, ref_t, "slot %d, output of %s" % (op.dst, op.name), floor=NET_FLOOR)
        checked += 1
    assert checked == len(m.ops) - 1
    assert_close_f32(y.cpu().numpy(), want, "logits", floor=NET_FLOOR)
