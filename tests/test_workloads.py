"""Synthetic workload generators: counts match the architectures the paper's
Table 2 / Section 3 name, masks are exact-k, and the oracle's activations stay in
a sane range through the synthetic networks (so parity tests compare real signal)."""
import numpy as np

from workloads import gen, models
from oracle import forward


def test_masks_are_exact_k_and_deterministic():
    g = gen.rng(1)
    m = gen.random_mask(g, (64, 3, 3, 64), 0.10)
    assert int(m.sum()) == 3686
    m2 = gen.random_mask(gen.rng(1), (64, 3, 3, 64), 0.10)
    np.testing.assert_array_equal(m, m2)
    w = gen.he_weights(gen.rng(5), 32, 3, 3, 16)
    mm = gen.magnitude_mask(w, 0.125)
    assert int(mm.sum()) == gen.keep_count(0.125, w.size)
    assert np.abs(w[mm == 1]).min() >= np.abs(w[mm == 0]).max()
    assert gen.magnitude_mask(w, 1.0).all()
    sk = gen.skewed_mask(gen.rng(3), (32, 3, 3, 16), 0.2, skew=6.0)
    per = sk.reshape(32, -1).sum(1)
    assert per.max() > 2 * per.min()


def test_single_layer_config():
    m = models.single_layer()
    op = m.ops[0]
    assert op.w.shape == (64, 3, 3, 64) and op.nnz == 3686 and op.act == "relu"
    x = models.make_input(m, 1)
    assert x.shape == (1, 56, 56, 64) and x.min() == 0.0


def test_resnet50_counts_and_activation_health():
    m = models.resnet50()
    convs = [o for o in m.ops if o.kind == "conv"]
    assert len(convs) == 53 and sum(o.kind == "fc" for o in m.ops) == 1
    assert sum(o.w.size for o in m.weight_ops()) == 25502912
    assert m.ops[0].mask is None and m.ops[0].w.shape == (64, 7, 7, 3)
    assert m.ops[-1].nnz == 204800
    assert sum(o.nnz for o in m.weight_ops()) == 3144896
    s2 = [o for o in convs if o.stride == 2 and o.k == 3]
    assert [o.name for o in s2] == ["s3b0.c2", "s4b0.c2", "s5b0.c2"]
    y, slots = forward.forward(m, models.make_input(m, 1))
    for op in m.ops:
        sd = float(slots[op.dst].std())
        assert 0.1 < sd < 10.0, (op.name, sd)
    assert np.isfinite(y).all() and y.shape == (1, 1000)


def test_mobilenet_v2_counts_and_health():
    m = models.mobilenet_v2()
    assert sum(o.w.size for o in m.weight_ops()) == 3469760
    dw = [o for o in m.ops if o.kind == "conv" and o.groups > 1]
    assert len(dw) == 17 and all(o.mask is None for o in dw)
    assert len([o for o in m.ops if o.kind == "conv" and o.k == 1]) == 34
    y, slots = forward.forward(m, models.make_input(m, 1))
    for op in m.ops:
        sd = float(slots[op.dst].std())
        assert 0.1 < sd < 10.0, (op.name, sd)


def test_vgg16_reduced_health_and_full_counts():
    small = models.vgg16(width=0.25, image=64, classes=100, fc_width=256)
    y, slots = forward.forward(small, models.make_input(small, 2))
    for op in small.ops:
        a = slots[op.dst]
        if a.dtype == np.int8:
            assert 0.05 < float((a > 0).mean()) < 0.9, op.name
            assert float((a >= 127).mean()) < 0.05, op.name
    assert y.dtype == np.float32 and np.isfinite(y).all()
    # conv1 has K = 27 at 8 %: some filters keep nothing at all
    c1 = models.vgg16(width=1.0, image=32, classes=10, fc_width=64).ops[0]
    assert (c1.mask.reshape(64, -1).sum(1) == 0).any()


def test_mobilenet_v1_counts_and_health():
    m = models.mobilenet_v1()
    # 4.23 M parameters without BatchNorm vectors: stem 864, depthwise 13 layers, pointwise 13 layers, fc 1.024 M
    assert sum(o.w.size for o in m.weight_ops()) == 4209088
    dw = [o for o in m.ops if o.kind == "conv" and o.groups > 1]
    pw = [o for o in m.ops if o.kind == "conv" and o.k == 1]
    assert len(dw) == 13 and all(o.mask is None for o in dw) and len(pw) == 13
    assert [o.stride for o in dw].count(2) == 4
    y, slots = forward.forward(m, models.make_input(m, 1))
    for op in m.ops:
        sd = float(slots[op.dst].std())
        assert 0.1 < sd < 10.0, (op.name, sd)
    assert y.shape == (1, 1000) and np.isfinite(y).all()


def test_inception_v3_counts_and_health():
    m = models.inception_v3()
    convs = [o for o in m.ops if o.kind == "conv"]
    assert len(convs) == 94 and sum(o.kind == "fc" for o in m.ops) == 1
    assert sum(o.w.size for o in m.weight_ops()) == 23799136
    shapes = {(o.w.shape[1], o.w.shape[2]) for o in convs}
    assert {(1, 7), (7, 1), (1, 3), (3, 1), (5, 5), (3, 3), (1, 1)} <= shapes
    assert sum(o.kind == "avgpool" for o in m.ops) == 9 and sum(o.kind == "maxpool" for o in m.ops) == 4
    # every concatenated slot is covered exactly once by its writers' windows
    cover = {}
    for o in m.ops:
        if o.dst_total:
            cover.setdefault(o.dst, []).append((o.dst_off, o.c_out, o.dst_total))
    assert len(cover) == 11
    for dst, wins in cover.items():
        wins.sort()
        assert wins[0][0] == 0 and all(a[0] + a[1] == b[0] for a, b in zip(wins, wins[1:])) and wins[-1][0] + wins[-1][1] == wins[-1][2]
    y, slots = forward.forward(m, models.make_input(m, 1))
    for op in m.ops:
        sd = float(slots[op.dst].std())
        assert 0.05 < sd < 20.0, (op.name, sd)
    assert slots[m.ops[-3].dst].shape == (1, 8, 8, 2048) and y.shape == (1, 1000) and np.isfinite(y).all()
