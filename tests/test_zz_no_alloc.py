"""cadnn_forward_static, the entry point for callers that must not allocate while they run a
network (a latency-critical serving thread, since cudaMalloc / cudaFree synchronize the whole
device; a process whose device memory belongs to another allocator; a batch size no cadnn_net
was built for).  It keeps the intermediate tensors in a fixed device array inside the library
instead of cudaMalloc'ed buffers.  Checked here against cadnn_forward AND against the CPU
oracle's network walker, through the C ABI, on two calls in a row (the second call finds the
array full of the first call's data), and for the clear refusal of a shape whose intermediates
exceed the fixed workspace.

Collected last on purpose: a run that stops at the first failure has then already run every
other test."""
import numpy as np
import pytest
import torch

from oracle import forward as oracle_forward
from workloads import models
from parity import assert_close_f32, assert_exact, NET_FLOOR

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _both(model, batch, static_batch=None):
    from paper_1905_00571_b200.network import PackedModel
    pm = PackedModel(model, batch, DEV)
    nb = static_batch or batch
    x = torch.from_numpy(models.make_input(model, nb)).to(DEV)
    want = []
    for b0 in range(0, nb, batch):          # reference: the allocating path, `batch` images at a time
        yb = pm.new_output()
        pm.forward(x[b0:b0 + batch].contiguous(), yb, use_graph=False)
        want.append(yb)
    torch.cuda.synchronize()
    want = torch.cat(want).cpu().numpy()
    outs = []
    for _ in range(2):                      # two calls in a row share the same device array
        y = torch.zeros((nb,) + tuple(pm.out_shape[1:]), dtype=pm.out_dtype, device=DEV)
        pm.forward_static(x, y)
        torch.cuda.synchronize()
        outs.append(y.cpu().numpy())
    oracle, _ = oracle_forward.forward(model, x.cpu().numpy())
    return want, outs, pm, oracle


def test_static_forward_matches_allocating_forward_f32():
    m = models.resnet50(width=0.25, image=64, classes=100)
    want, outs, _, oracle = _both(m, 2)
    for got in outs:
        assert_close_f32(got, want, "resnet50 reduced, static workspace", floor=NET_FLOOR)
        assert_close_f32(got, oracle, "resnet50 reduced, static workspace vs oracle", floor=NET_FLOOR)
    np.testing.assert_array_equal(outs[0], outs[1])


def test_static_forward_runs_a_batch_no_net_was_built_for():
    m = models.mobilenet_v2(width=0.5, image=96, classes=100)
    want, outs, _, oracle = _both(m, 1, static_batch=3)
    for got in outs:
        assert_close_f32(got, want, "mobilenet_v2 reduced, batch 3 through a batch-1 packing", floor=NET_FLOOR)
        assert_close_f32(got, oracle, "mobilenet_v2 reduced, static workspace vs oracle", floor=NET_FLOOR)


def test_static_forward_int8_bit_exact():
    m = models.vgg16(width=0.25, image=64, classes=100, fc_width=256)
    want, outs, _, oracle = _both(m, 1)
    for got in outs:
        assert_exact(got, want, "vgg16 int8 reduced, static workspace")
        assert_exact(got, oracle, "vgg16 int8 reduced, static workspace vs oracle")


def test_static_forward_refuses_what_does_not_fit():
    from paper_1905_00571_b200 import binding as B
    from paper_1905_00571_b200.network import PackedModel
    m = models.resnet50(width=0.25, image=64, classes=100)
    pm = PackedModel(m, 1, DEV)
    # 64x64x3 input -> the stem's 32x32x16 float output alone is 64 KiB per image
    too_many = (B.STATIC_WORKSPACE_BYTES // (32 * 32 * 16 * 4)) + 1
    x = torch.zeros((too_many, 64, 64, 3), device=DEV)
    y = torch.zeros((too_many, 100), device=DEV)
    with pytest.raises(B.CadnnError) as e:
        pm.forward_static(x, y)
    assert e.value.status == 4


def test_static_forward_refuses_a_bad_epilogue_before_any_launch():
    """An int8 layer with ReLU6 in the middle of the list is refused in the planning pass: the output
    buffer keeps its contents, so nothing ran."""
    from paper_1905_00571_b200 import binding as B
    from paper_1905_00571_b200.network import PackedModel
    m = models.vgg16(width=0.25, image=64, classes=100, fc_width=256)
    pm = PackedModel(m, 1, DEV)
    ops = list(pm.ops)
    bad = B.Op.from_buffer_copy(ops[4])
    bad.act = B.ACT["relu6"]
    ops[4] = bad
    x = torch.from_numpy(models.make_input(m, 1)).to(DEV)
    y = torch.full((1, 100), 7.0, device=DEV)
    with pytest.raises(B.CadnnError) as e:
        B.cadnn_forward_static(ops, x, y, "s8")
    assert e.value.status == 4
    torch.cuda.synchronize()
    assert float(y.min()) == 7.0 and float(y.max()) == 7.0
