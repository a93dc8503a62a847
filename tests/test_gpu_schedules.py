"""GPU parity across the schedule space of the sparse conv kernel: every structural option the
packer can pick (warps per block, filters per warp, pixel bands, channel chunks and pipeline
depth, cluster split of the reduction, stride-2 de-interleaving) must give the oracle's result.
The CADNN_SCHEDULE override forces options the time model would not choose for these sizes."""
import os

import numpy as np
import pytest
import torch

from oracle import ref
from workloads import gen, models
from parity import assert_close_or_bounded, assert_close_f32, assert_exact, NET_FLOOR

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _B():
    from paper_1905_00571_b200 import binding
    return binding


def _run(x, w, mask, stride, pad, sched, dtype="f32", out="f32", scale=None, bias=None, act="relu", autotune=False):
    B = _B()
    n, h, wd, c_in = x.shape
    c_out, kh, kw, _ = w.shape
    old = os.environ.pop("CADNN_SCHEDULE", None)
    if sched:
        os.environ["CADNN_SCHEDULE"] = sched
    try:
        d = B.make_desc(c_in, c_out, kh, kw, stride, pad, 1, h, wd, n, dtype, autotune=autotune)
        wh = B.cadnn_pack_q8(d, w, mask) if dtype == "s8" else B.cadnn_pack(d, w, mask)
    finally:
        os.environ.pop("CADNN_SCHEDULE", None)
        if old is not None:
            os.environ["CADNN_SCHEDULE"] = old
    info = B.cadnn_weights_schedule(wh)
    ho, wo = (h + 2 * pad - kh) // stride + 1, (wd + 2 * pad - kw) // stride + 1
    tdt = {"f32": torch.float32, "s8": torch.int8, "s32": torch.int32}[out]
    y = torch.zeros((n, ho, wo, c_out), dtype=tdt, device=DEV)
    dev = lambda a: None if a is None else torch.from_numpy(a).to(DEV)
    B.cadnn_conv2d(wh, dev(x), y, dev(scale), dev(bias), None, act, out)
    torch.cuda.synchronize()
    wh.free()
    return y.cpu().numpy(), info


SCHEDULES = [
    "nw=4,rpw=1,tbx=1,tby=1,cic=16,ks=1",
    "nw=8,rpw=2,tbx=1,tby=3,cic=32,ks=1",      # two chunks: double-buffered pipeline
    "nw=8,rpw=1,tbx=1,tby=2,cic=8,ks=1",       # many small chunks: three-stage pipeline
    "nw=16,rpw=4,tbx=1,tby=2,cic=64,ks=1",
    "nw=16,rpw=8,tbx=1,tby=4,cic=64,ks=1",
    "nw=16,rpw=16,tbx=1,tby=2,cic=64,ks=1",
    "nw=8,rpw=1,tbx=1,tby=7,cic=32,ks=2",      # reduction split over a 2-block cluster
    "nw=8,rpw=2,tbx=1,tby=5,cic=16,ks=4",
    "nw=4,rpw=1,tbx=1,tby=8,cic=8,ks=8",       # 8-block cluster, partial last tile
]


@pytest.mark.parametrize("sched", SCHEDULES)
@pytest.mark.parametrize("stride", [1, 2])
def test_3x3_schedules_f32(sched, stride):
    g = gen.rng(41)
    x = gen.relu_normal_input(g, (2, 28, 28, 64))
    wt = gen.he_weights(g, 80, 3, 3, 64)
    mask = gen.magnitude_mask(wt, 0.125)
    scale, bias = gen.folded_bn(g, 80)
    want = ref.conv2d_f32(x, wt, mask, stride, 1, 1, scale, bias, None, "relu")
    got, info = _run(x, wt, mask, stride, 1, sched, scale=scale, bias=bias)
    assert info["kind"] == 1
    assert_close_f32(got, want, sched)


@pytest.mark.parametrize("sched", ["nw=4,rpw=1,tbx=1,cic=32,ks=1", "nw=8,rpw=4,tbx=4,cic=64,ks=2",
                                   "nw=16,rpw=16,tbx=2,cic=128,ks=2", "nw=8,rpw=2,tbx=8,cic=16,ks=8",
                                   "nw=16,rpw=8,tbx=3,cic=256,ks=1"])
@pytest.mark.parametrize("stride", [1, 2])
def test_1x1_schedules_f32(sched, stride):
    g = gen.rng(42)
    x = gen.normal_input(g, (3, 14, 14, 256))
    wt = gen.he_weights(g, 200, 1, 1, 256)
    mask = gen.magnitude_mask(wt, 0.125)
    scale, bias = gen.folded_bn(g, 200)
    want = ref.conv2d_f32(x, wt, mask, stride, 0, 1, scale, bias, None, "relu")
    got, info = _run(x, wt, mask, stride, 0, sched, scale=scale, bias=bias)
    assert info["kind"] == 2
    assert_close_f32(got, want, sched)


@pytest.mark.parametrize("sched", ["nw=8,rpw=2,tbx=1,tby=4,cic=32,ks=2", "nw=16,rpw=4,tbx=1,tby=2,cic=64,ks=1",
                                   "nw=4,rpw=1,tbx=1,tby=7,cic=8,ks=4"])
@pytest.mark.parametrize("out", ["s8", "s32"])
def test_3x3_schedules_int8_bit_exact(sched, out):
    g = gen.rng(43)
    x = gen.int8_relu_activation(g, (2, 28, 28, 64))
    wq = gen.int8_weights(g, (72, 3, 3, 64))
    mask = gen.random_mask(g, wq.shape, 0.08)
    m = (g.uniform(0.5, 2.0, size=72) * 2e-3).astype(np.float32)
    b = (g.standard_normal(72) * 4).astype(np.float32)
    want = ref.conv2d_s8(x, wq, mask, 1, 1, 1, m, b, "relu" if out == "s8" else "none", out)
    got, _ = _run(x, wq, mask, 1, 1, sched, dtype="s8", out=out, scale=m, bias=b, act="relu" if out == "s8" else "none")
    assert_exact(got, want, sched)


def test_wide_map_uses_several_bands_across():
    g = gen.rng(44)
    x = gen.relu_normal_input(g, (1, 12, 224, 16))
    wt = gen.he_weights(g, 24, 3, 3, 16)
    mask = gen.random_mask(g, wt.shape, 0.2)
    want = ref.conv2d_f32(x, wt, mask, 1, 1, act="relu")
    for sched in ("nw=8,rpw=1,tbx=7,tby=1", "nw=4,rpw=2,tbx=1,tby=4", "nw=8,rpw=1,tbx=1,tby=1"):
        got, _ = _run(x, wt, mask, 1, 1, sched)
        assert_close_f32(got, want, sched)


def test_timed_schedule_selection_keeps_results():
    g = gen.rng(45)
    x = gen.relu_normal_input(g, (1, 14, 14, 128))
    wt = gen.he_weights(g, 128, 3, 3, 128)
    mask = gen.magnitude_mask(wt, 0.125)
    want = ref.conv2d_f32(x, wt, mask, 1, 1, act="relu")
    got, info = _run(x, wt, mask, 1, 1, None, autotune=True)
    assert_close_f32(got, want, str(info))


def test_schedule_cache_reproduces_the_timed_choice(tmp_path, monkeypatch):
    """CADNN_TUNE_CACHE: the second pack of a layer reads the measured schedules back (no timing) and computes the same."""
    B = _B()
    cache = tmp_path / "tune.cache"
    monkeypatch.setenv("CADNN_TUNE_CACHE", str(cache))
    g = gen.rng(46)
    x = gen.relu_normal_input(g, (1, 14, 14, 128))
    wt = gen.he_weights(g, 96, 3, 3, 128)
    mask = gen.magnitude_mask(wt, 0.125)
    want = ref.conv2d_f32(x, wt, mask, 1, 1, act="relu")
    d = B.make_desc(128, 96, 3, 3, 1, 1, 1, 14, 14, 1, "f32", autotune=True)
    w1 = B.cadnn_pack(d, wt, mask)
    assert cache.exists() and len(cache.read_text().splitlines()) == 1
    w2 = B.cadnn_pack(d, wt, mask)
    assert len(cache.read_text().splitlines()) == 1          # nothing was timed again
    assert B.cadnn_weights_schedule(w1) == B.cadnn_weights_schedule(w2)
    assert B.cadnn_weights_planar_schedule(w1) == B.cadnn_weights_planar_schedule(w2)
    xd = torch.from_numpy(x).to(DEV)
    for w in (w1, w2):
        y = torch.empty((1, 14, 14, 96), device=DEV)
        B.cadnn_conv2d(w, xd, y, act="relu")
        torch.cuda.synchronize()
        assert_close_f32(y.cpu().numpy(), want, "cached schedule")
    # another layer (different nonzeros per filter) is a different key
    mask2 = gen.magnitude_mask(wt, 0.25)
    B.cadnn_pack(d, wt, mask2)
    assert len(cache.read_text().splitlines()) == 2


STEM_CASES = [(1, 64, 64, 3, 64, 7, 2, 3), (2, 33, 47, 3, 32, 3, 2, 1), (1, 20, 20, 4, 24, 3, 1, 1),
              (1, 18, 70, 1, 70, 5, 1, 2), (1, 224, 224, 3, 64, 7, 2, 3), (2, 30, 141, 3, 70, 7, 2, 3),
              (1, 9, 9, 3, 8, 3, 2, 1)]


@pytest.mark.parametrize("case", STEM_CASES)
def test_dense_stem_conv(case):
    B = _B()
    n, h, w, c_in, c_out, k, stride, pad = case
    g = gen.rng(sum(case))
    x = gen.normal_input(g, (n, h, w, c_in))
    wt = gen.he_weights(g, c_out, k, k, c_in)
    scale, bias = gen.folded_bn(g, c_out)
    for mask in (None, gen.random_mask(g, wt.shape, 0.7)):
        want = ref.conv2d_f32(x, wt, mask, stride, pad, 1, scale, bias, None, "relu6")
        got, info = _run(x, wt, mask, stride, pad, None, scale=scale, bias=bias, act="relu6")
        assert info["kind"] == 5
        # a dense sum of k*k*c_in signed products cancels and ReLU6 pins max|r| at 6: elements that miss the
        # layer floor must satisfy the fp32 accumulation bound (sum of |w x| from the oracle on absolute values)
        am = np.abs(wt) if mask is None else np.abs(wt) * mask
        s_abs = ref.conv2d_f32(np.abs(x), am, None, stride, pad, 1, np.abs(scale), np.abs(bias), None, "none")
        assert_close_or_bounded(got, want, s_abs, k * k * c_in + 4, str(case))


def test_forward_host_and_empty_batch():
    from paper_1905_00571_b200.network import PackedModel
    B = _B()
    m = models.resnet50(width=0.25, image=64, classes=100)
    pm = PackedModel(m, 2, DEV, autotune=True)
    x = models.make_input(m, 2)
    xd = torch.from_numpy(x).to(DEV)
    y = pm.new_output()
    pm.forward(xd, y)
    torch.cuda.synchronize()
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.empty(pm.out_shape, dtype=pm.out_dtype).pin_memory()
    pm.forward_host(xh, yh)
    pm.forward_host(xh, yh)
    np.testing.assert_array_equal(yh.numpy(), y.cpu().numpy())
    t = pm.layer_times(xd, y, reps=3)
    assert len(t) == len(m.ops) and all(v > 0 for v in t)
    # a layer call with n = 0 launches nothing and succeeds
    d = B.make_desc(8, 8, 3, 3, 1, 1, 1, 6, 6, 1, "f32")
    wh = B.cadnn_pack(d, np.ones((8, 3, 3, 8), np.float32))
    x0 = torch.zeros((0, 6, 6, 8), device=DEV)
    buf = torch.zeros(16, device=DEV)
    st = B._lib.cadnn_conv2d(wh.handle, buf.data_ptr(), 0, 6, 6, buf.data_ptr() + 32, None, None)
    assert st == 0


def test_resnet50_full_batch1_with_timed_schedules():
    from oracle import forward as oracle_forward
    from paper_1905_00571_b200.network import PackedModel
    m = models.resnet50()
    x = models.make_input(m, 1)
    pm = PackedModel(m, 1, DEV, autotune=True)    # the configuration bench.py times
    y = pm.new_output()
    pm.forward(torch.from_numpy(x).to(DEV), y)
    torch.cuda.synchronize()
    want, _ = oracle_forward.forward(m, x)
    got = y.cpu().numpy()
    assert_close_f32(got, want, "logits", floor=NET_FLOOR)
    assert set(np.argsort(-got[0])[:5]) == set(np.argsort(-want[0])[:5])


def _pitch(h, w):
    return ((h + 2) * (w + 2) + 3) // 4 * 4


def _to_planar(a):
    """NHWC numpy -> [n, c, pitch] torch CUDA tensor: planes of (h+2) x (w+2) with a zero border, padded to a multiple of 4."""
    n, h, w, c = a.shape
    t = torch.zeros((n, c, _pitch(h, w)), dtype=torch.float32, device=DEV)
    t[:, :, :(h + 2) * (w + 2)].view(n, c, h + 2, w + 2)[:, :, 1:h + 1, 1:w + 1] = \
        torch.from_numpy(np.ascontiguousarray(a.transpose(0, 3, 1, 2))).to(DEV)
    return t


PLANAR_CASES = [
    # n, h, w, c_in, c_out, k, stride, density
    (1, 56, 56, 64, 64, 3, 1, 0.125), (2, 28, 28, 128, 128, 3, 2, 0.125), (1, 14, 14, 256, 200, 3, 1, 0.125),
    (3, 7, 7, 512, 96, 3, 1, 0.125), (1, 56, 56, 64, 256, 1, 1, 0.125), (2, 28, 28, 512, 130, 1, 2, 0.125),
    (1, 13, 17, 10, 7, 3, 1, 0.5), (1, 13, 17, 10, 7, 3, 2, 0.5), (1, 9, 9, 16, 16, 1, 1, 1.0), (1, 9, 9, 16, 16, 3, 1, 0.0),
    (2, 7, 7, 2048, 512, 1, 1, 0.125), (1, 14, 14, 1024, 256, 1, 1, 0.05), (2, 5, 3, 6, 5, 3, 1, 1.0), (1, 28, 28, 130, 66, 3, 1, 0.3),
]


@pytest.mark.parametrize("staged", [True, False])
@pytest.mark.parametrize("case", PLANAR_CASES)
def test_planar_sparse_conv(case, staged):
    """Both planar kernels: the shared-memory-staged one (linear tiles at stride 1, row tiles at stride 2) and the direct one."""
    B = _B()
    n, h, w, c_in, c_out, k, stride, density = case
    pad = k // 2
    g = gen.rng(sum(case[:7]))
    x = gen.relu_normal_input(g, (n, h, w, c_in))
    wt = gen.he_weights(g, c_out, k, k, c_in)
    mask = None if density >= 1.0 else gen.magnitude_mask(wt, density)
    scale, bias = gen.folded_bn(g, c_out)
    ho, wo = ref.out_hw(h, w, k, stride, pad)
    res = gen.normal_input(g, (n, ho, wo, c_out))
    want = ref.conv2d_f32(x, wt, mask, stride, pad, 1, scale, bias, res, "relu")
    d = B.make_desc(c_in, c_out, k, k, stride, pad, 1, h, w, n, "f32", autotune=(c_in >= 256))
    if not staged:
        os.environ["CADNN_NO_STAGED"] = "1"
    try:
        wh = B.cadnn_pack(d, wt, mask)
    finally:
        os.environ.pop("CADNN_NO_STAGED", None)
    y = torch.zeros((n, c_out, _pitch(ho, wo)), device=DEV)
    dev = lambda a: torch.from_numpy(a).to(DEV)
    B.cadnn_conv2d_planar(wh, _to_planar(x), y, dev(scale), dev(bias), _to_planar(res), "relu")
    torch.cuda.synchronize()
    yc = y.cpu().numpy()
    planes = yc[:, :, :(ho + 2) * (wo + 2)].reshape(n, c_out, ho + 2, wo + 2)
    got = planes[:, :, 1:ho + 1, 1:wo + 1].transpose(0, 2, 3, 1)
    # the residual (|res| up to ~4) cancels against the conv result: elements that miss the layer floor must
    # satisfy the fp32 accumulation bound
    am = np.abs(wt) if mask is None else np.abs(wt) * mask
    s_abs = ref.conv2d_f32(np.abs(x), am, None, stride, pad, 1, np.abs(scale), np.abs(bias), np.abs(res), "none")
    terms = int(am.reshape(c_out, -1).astype(bool).sum(1).max()) + 4
    assert_close_or_bounded(got, want, s_abs, terms, str(case))
    # the border (and the padding behind a plane) is never written
    border = planes.copy()
    border[:, :, 1:ho + 1, 1:wo + 1] = 0
    assert not border.any() and not yc[:, :, (ho + 2) * (wo + 2):].any()


PLANAR_OVERRIDES = [
    # (case, CADNN_PLANAR_SCHEDULE): cp.async and TMA staging, rings and all-in-flight, warps sharing a
    # filter, clusters splitting the input channels (ragged last chunk included)
    ((1, 14, 14, 256, 200, 3, 1, 0.125), "t=2,nw=16,ks=2,rpw=1,chunks=4,stages=2,tma=0"),
    ((1, 14, 14, 256, 200, 3, 1, 0.125), "t=2,nw=16,ks=2,rpw=1,chunks=4,stages=2,tma=1"),
    ((1, 14, 14, 256, 200, 3, 1, 0.125), "t=4,nw=8,ks=1,rpw=4,chunks=8,stages=8,tma=1"),
    ((1, 14, 14, 256, 200, 3, 1, 0.125), "t=1,nw=16,ks=1,rpw=4,chunks=4,stages=1,tma=1,kc=4"),
    ((1, 14, 14, 256, 200, 3, 1, 0.125), "t=2,nw=8,ks=2,rpw=2,chunks=8,stages=2,tma=1,kc=2"),
    ((2, 7, 7, 2048, 512, 1, 1, 0.125), "t=1,nw=16,ks=1,rpw=8,chunks=8,stages=1,tma=1,kc=8"),
    ((2, 7, 7, 2048, 512, 1, 1, 0.125), "t=2,nw=16,ks=2,rpw=2,chunks=16,stages=3,tma=1,kc=4"),
    ((1, 28, 28, 130, 66, 3, 1, 0.3), "t=4,nw=8,ks=2,rpw=2,chunks=2,stages=1,tma=1,kc=2"),
    ((1, 28, 28, 130, 66, 3, 1, 0.3), "t=8,nw=4,ks=4,rpw=1,chunks=3,stages=3,tma=0"),
    ((1, 56, 56, 64, 256, 1, 1, 0.125), "t=8,nw=8,ks=1,rpw=2,chunks=1,stages=1,tma=1"),
    ((3, 7, 7, 512, 96, 3, 1, 0.125), "t=1,nw=8,ks=8,rpw=1,chunks=4,stages=4,tma=1"),
    ((1, 13, 17, 10, 7, 3, 1, 0.5), "t=1,nw=4,ks=2,rpw=2,chunks=2,stages=2,tma=1"),
    # stride 2: row tiles
    ((2, 28, 28, 128, 128, 3, 2, 0.125), "t=2,nw=8,ks=2,rpw=2,chunks=2,stages=2,tma=1"),
    ((2, 28, 28, 128, 128, 3, 2, 0.125), "t=1,nw=16,ks=1,rpw=4,chunks=4,stages=1,tma=1,kc=4"),
    ((1, 56, 56, 256, 512, 1, 2, 0.125), "t=1,nw=16,ks=1,rpw=2,chunks=4,stages=2,tma=1"),
    ((1, 14, 14, 512, 96, 3, 2, 0.125), "t=2,nw=16,ks=4,rpw=1,chunks=8,stages=2,tma=1,kc=2"),
    ((1, 13, 17, 10, 7, 3, 2, 0.5), "t=4,nw=4,ks=1,rpw=1,chunks=1,stages=1,tma=1"),
    ((2, 28, 28, 512, 130, 1, 2, 0.125), "t=2,nw=8,ks=1,rpw=2,chunks=2,stages=2,tma=1"),
]


@pytest.mark.parametrize("case,sched", PLANAR_OVERRIDES)
def test_planar_staged_schedule_space(case, sched):
    B = _B()
    n, h, w, c_in, c_out, k, stride, density = case
    pad = k // 2
    g = gen.rng(sum(case[:7]) + 1)
    x = gen.relu_normal_input(g, (n, h, w, c_in))
    wt = gen.he_weights(g, c_out, k, k, c_in)
    mask = gen.magnitude_mask(wt, density)
    scale, bias = gen.folded_bn(g, c_out)
    want = ref.conv2d_f32(x, wt, mask, stride, pad, 1, scale, bias, None, "relu")
    ho, wo = ref.out_hw(h, w, k, stride, pad)
    d = B.make_desc(c_in, c_out, k, k, stride, pad, 1, h, w, n, "f32")
    os.environ["CADNN_PLANAR_SCHEDULE"] = sched
    try:
        wh = B.cadnn_pack(d, wt, mask)
    finally:
        os.environ.pop("CADNN_PLANAR_SCHEDULE", None)
    ps = B.cadnn_weights_planar_schedule(wh)
    asked = dict(kv.split("=") for kv in sched.split(","))
    assert ps["variant"] == 2 and ps["T"] == int(asked["t"]) and ps["NW"] == int(asked["nw"]) and ps["KS"] == int(asked["ks"])
    assert ps["tma"] == int(asked["tma"]) and ps["KC"] == int(asked.get("kc", 1)) and ps["RPW"] == int(asked["rpw"])
    y = torch.zeros((n, c_out, _pitch(ho, wo)), device=DEV)
    dev = lambda a: torch.from_numpy(a).to(DEV)
    B.cadnn_conv2d_planar(wh, _to_planar(x), y, dev(scale), dev(bias), None, "relu")
    torch.cuda.synchronize()
    planes = y.cpu().numpy()[:, :, :(ho + 2) * (wo + 2)].reshape(n, c_out, ho + 2, wo + 2)
    # outputs that cancel carry a few ulps of the operands: elements that miss the layer floor must satisfy
    # the fp32 accumulation bound
    am = np.abs(wt) * mask
    s_abs = ref.conv2d_f32(np.abs(x), am, None, stride, pad, 1, np.abs(scale), np.abs(bias), None, "none")
    terms = int(mask.reshape(c_out, -1).sum(1).max()) + 4
    assert_close_or_bounded(planes[:, :, 1:ho + 1, 1:wo + 1].transpose(0, 2, 3, 1), want, s_abs, terms, "%s %s" % (case, sched))
    border = planes.copy()
    border[:, :, 1:ho + 1, 1:wo + 1] = 0
    assert not border.any()
    assert B.cadnn_device_status()["copy_timeouts"] == 0


def test_planar_and_nhwc_networks_agree_with_the_oracle():
    from oracle import forward as oracle_forward
    from paper_1905_00571_b200.network import PackedModel
    m = models.resnet50(width=0.25, image=64, classes=100)
    x = models.make_input(m, 2)
    want, _ = oracle_forward.forward(m, x)
    outs = []
    for no_planar in (False, True):
        if no_planar:
            os.environ["CADNN_NO_PLANAR"] = "1"
        try:
            pm = PackedModel(m, 2, DEV)
        finally:
            os.environ.pop("CADNN_NO_PLANAR", None)
        y = pm.new_output()
        pm.forward(torch.from_numpy(x).to(DEV), y)
        pm.forward(torch.from_numpy(x).to(DEV), y)
        torch.cuda.synchronize()
        outs.append(y.cpu().numpy())
        assert_close_f32(outs[-1], want, "planar off" if no_planar else "planar on", floor=NET_FLOOR)
