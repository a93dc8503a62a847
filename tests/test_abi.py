"""CPU-side checks of the C ABI: the library loads, exports every symbol the header
declares, and the host-only packer round-trips and balances (no GPU needed)."""
import os
import re

import numpy as np
import pytest

from workloads import gen, models

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_1905_00571_b200 import build
    build.build()
    from paper_1905_00571_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(B):
    import ctypes
    hdr = open(os.path.join(ROOT, "include", "cadnn.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(cadnn_[a-z0-9_]+)\s*\(", hdr))
    assert len(names) >= 19
    lib = ctypes.CDLL(B.LIB_PATH)
    for n in sorted(names):
        assert hasattr(lib, n), n
    assert names == set(B.EXPORTED)


def _host_pack(B, w, mask, in_hw, stride=1, pad=1, dtype="f32", hint=1, q8=False, scale=None):
    c_out, kh, kw, c_in = w.shape
    d = B.make_desc(c_in, c_out, kh, kw, stride, pad, 1, in_hw, in_hw, hint, dtype, host_only=True)
    return B.cadnn_pack_q8(d, w, mask) if q8 else B.cadnn_pack(d, w, mask, scale)


@pytest.mark.parametrize("shape,hw,density", [((64, 3, 3, 64), 56, 0.1), ((70, 3, 3, 130), 20, 0.05),
                                               ((256, 1, 1, 64), 56, 0.125), ((16, 7, 7, 3), 224, 1.0),
                                               ((32, 3, 3, 16), 14, 0.0)])
@pytest.mark.parametrize("hint", [1, 64])
def test_pack_unpack_round_trip(B, shape, hw, density, hint):
    g = gen.rng(11)
    w = gen.he_weights(g, *shape)
    mask = None if density >= 1.0 else gen.random_mask(g, shape, density)
    pad = shape[1] // 2
    wh = _host_pack(B, w, mask, hw, 1, pad, hint=hint)
    dense, m2 = B.cadnn_weights_unpack(wh)
    want_mask = np.ones(shape, np.uint8) if mask is None else mask
    np.testing.assert_array_equal(m2, want_mask)
    np.testing.assert_array_equal(dense, w * want_mask)
    info = B.cadnn_weights_info(wh)
    assert info["nnz"] == int(want_mask.sum())
    # compressed formats: at least value + 16-bit offset per stored nonzero; dense formats: 4 bytes per weight
    assert info["packed_bytes"] >= (4 if info["fmt"] in (3, 4) else 6) * info["nnz"]


def test_pack_keeps_masked_in_zero_values(B):
    w = np.zeros((8, 1, 1, 8), np.float32)
    mask = np.eye(8, dtype=np.uint8).reshape(8, 1, 1, 8)
    wh = _host_pack(B, w, mask, 4, 1, 0)
    assert B.cadnn_weights_info(wh)["nnz"] == 8
    _, m2 = B.cadnn_weights_unpack(wh)
    np.testing.assert_array_equal(m2, mask)


def test_fc_row_csr_round_trip_and_s8(B):
    g = gen.rng(12)
    q = gen.int8_weights(g, (100, 1, 1, 3000))
    mask = gen.random_mask(g, q.shape, 0.04)
    d = B.make_desc(3000, 100, batch_hint=1, dtype="s8", host_only=True)
    wh = B.cadnn_pack_q8(d, q, mask)
    assert B.cadnn_weights_info(wh)["fmt"] == 2
    dense, m2 = B.cadnn_weights_unpack(wh)
    np.testing.assert_array_equal(m2, mask)
    np.testing.assert_array_equal(dense, (q * mask).astype(np.float32))


def test_float_to_int8_quantization_in_the_packer(B):
    w = np.array([0.25, 0.75, 1.25, -0.75, 100.0, -100.0, 0.3, 0.0], np.float32).reshape(1, 1, 1, 8)
    s = np.array([0.5], np.float32)
    d = B.make_desc(8, 1, in_h=2, in_w=2, dtype="s8", host_only=True)
    wh = B.cadnn_pack(d, w, None, s)
    dense, _ = B.cadnn_weights_unpack(wh)
    np.testing.assert_array_equal(dense.reshape(-1), np.array([0, 2, 2, -2, 127, -127, 1, 0], np.float32))


def test_regrouping_balances_warp_loads_on_a_skewed_mask(B):
    g = gen.rng(13)
    shape = (256, 3, 3, 64)
    w = gen.he_weights(g, *shape)
    mask = gen.skewed_mask(g, shape, 0.125, skew=8.0)
    wh = _host_pack(B, w, mask, 28, hint=64)
    s = B.cadnn_weights_schedule(wh)
    assert s["RPW"] >= 2
    loads = B.cadnn_weights_warp_loads(wh).reshape(-1, 8)          # [block][warp]
    per_row = mask.reshape(256, -1).sum(1)
    naive = per_row.reshape(-1, 8, s["RPW"]).sum(2)                 # consecutive filters per warp
    spread = lambda a: float((a.max(1) / np.maximum(a.mean(1), 1)).mean())
    assert loads.sum() == mask.sum()
    assert spread(loads) < spread(naive)
    assert spread(loads) < 1.25


def test_pack_rejects_bad_arguments(B):
    w = np.zeros((8, 3, 3, 8), np.float32)
    d = B.make_desc(8, 8, 3, 3, 1, 1, 2, 10, 10, 1, "f32", host_only=True)      # grouped, not depthwise
    with pytest.raises(B.CadnnError) as e:
        B.cadnn_pack(d, np.zeros((8, 3, 3, 4), np.float32))
    assert e.value.status == 4
    d = B.make_desc(8, 8, 3, 3, 0, 1, 1, 10, 10, 1, "f32", host_only=True)      # stride 0
    with pytest.raises(B.CadnnError) as e:
        B.cadnn_pack(d, w)
    assert e.value.status == 1
    d = B.make_desc(8, 8, 3, 3, 1, 1, 1, 10, 10, 1, "s8", host_only=True)       # int8 without scale
    with pytest.raises(B.CadnnError) as e:
        B.cadnn_pack(d, w)
    assert e.value.status == 1
    d = B.make_desc(140000, 4, dtype="s8", host_only=True)                       # int32 sum could overflow
    with pytest.raises(B.CadnnError) as e:
        B.cadnn_pack_q8(d, np.zeros((4, 1, 1, 140000), np.int8))
    assert e.value.status == 4


def test_compute_without_device_image_is_refused(B):
    d = B.make_desc(8, 8, 1, 1, in_h=4, in_w=4, host_only=True)
    wh = B.cadnn_pack(d, np.zeros((8, 1, 1, 8), np.float32))
    import ctypes
    ep = None
    st = B._lib.cadnn_conv2d(wh.handle, ctypes.c_void_p(256), 1, 4, 4, ctypes.c_void_p(512), ep, None)
    assert st == 1


def test_grouped_format_finds_the_dense_blocks_and_round_trips(B, monkeypatch):
    """Block-structured int8 layer, host-only pack: the blocks the mask keeps (nearly) whole are found, the
    remainder stays sparse, and unpacking gives back exactly the kept weights and the mask."""
    g = gen.rng(21)
    shape = (128, 3, 3, 192)
    q = gen.int8_weights(g, shape)
    mask = gen.block_mask(g, shape, 0.25, sprinkle=0.02)
    # one block at 60 % (taken at the default threshold of 0.5) and one at 30 % (left to the sparse image)
    mask[0:64, 0, 0, 0:64] = (g.random((64, 64)) < 0.6)
    mask[64:128, 2, 2, 128:192] = (g.random((64, 64)) < 0.3)
    blocks_whole = 0
    for nt in range(2):
        for ky in range(3):
            for kx in range(3):
                for ck in range(3):
                    blocks_whole += int(mask[nt * 64:nt * 64 + 64, ky, kx, ck * 64:ck * 64 + 64].mean() >= 0.5)
    d = B.make_desc(192, 128, 3, 3, 1, 1, 1, 20, 20, 1, "s8", host_only=True, fmt=B.FMT_GROUPED)
    wh = B.cadnn_pack_q8(d, q, mask)
    info = B.cadnn_weights_info(wh)
    bi = B.cadnn_weights_block_info(wh)
    assert info["fmt"] == B.FMT_GROUPED and info["nnz"] == int(mask.sum())
    assert bi["blocks"] == blocks_whole and 0 < bi["block_nnz"] < info["nnz"]
    dense, m2 = B.cadnn_weights_unpack(wh)
    np.testing.assert_array_equal(m2, mask)
    np.testing.assert_array_equal(dense, q.astype(np.float32) * mask)
    assert B.cadnn_weights_workspace_bytes(wh, 2) == 2 * 20 * 20 * 128 * 4
    # a threshold of 1.0 leaves the 60 % block to the sparse image as well
    monkeypatch.setenv("CADNN_BLOCK_DENSITY", "1.0")
    wh2 = B.cadnn_pack_q8(d, q, mask)
    assert B.cadnn_weights_block_info(wh2)["blocks"] == blocks_whole - 1
    # shapes the format does not cover are refused
    with pytest.raises(B.CadnnError):
        B.cadnn_pack_q8(B.make_desc(96, 128, 3, 3, 1, 1, 1, 20, 20, 1, "s8", host_only=True, fmt=B.FMT_GROUPED),
                        gen.int8_weights(g, (128, 3, 3, 96)), None)


@pytest.mark.parametrize("k,h,w", [(3, 13, 17), (3, 14, 14), (3, 7, 8), (1, 13, 17), (1, 14, 14)])
def test_parity_form_of_a_stride2_layer_is_the_same_layer(B, k, h, w):
    """The packer's second form of a stride-2 layer - a stride-1 layer over the input split by row and column parity -
    computes what the layer computes: the oracle's convolution of the split input with the rearranged weights equals
    its stride-2 convolution of the input with the original ones."""
    from oracle import ref
    g = np.random.default_rng(100 * k + h + w)
    c_in, c_out, pad = 6, 5, (1 if k == 3 else 0)
    wt = g.standard_normal((c_out, k, k, c_in)).astype(np.float32)
    mask = (g.random(wt.shape) < 0.4).astype(np.uint8)
    d = B.make_desc(c_in, c_out, k, k, 2, pad, 1, h, w, 1, "f32", host_only=True)
    wh = B.cadnn_pack(d, wt, mask)
    form = B.cadnn_weights_parity_form(wh)
    assert form is not None
    w2, m2 = B.cadnn_weights_unpack(form)
    assert int(m2.sum()) == int(mask.sum())
    x = g.standard_normal((2, h, w, c_in)).astype(np.float32)
    h2, wd2 = (h + 1) // 2, (w + 1) // 2
    planes = np.zeros((2, h2, wd2, (4 if k == 3 else 1) * c_in), np.float32)
    for py in range(2 if k == 3 else 1):
        for px in range(2 if k == 3 else 1):
            sub = x[:, py::2, px::2, :]
            par = py * 2 + px
            planes[:, :sub.shape[1], :sub.shape[2], par * c_in:(par + 1) * c_in] = sub
    want = ref.conv2d_f32(x, wt, mask, 2, pad)
    got = ref.conv2d_f32(planes, w2, m2, 1, pad)
    assert got.shape == want.shape
    np.testing.assert_allclose(got, want, rtol=1e-6, atol=1e-6)
