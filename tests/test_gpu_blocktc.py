"""GPU parity of the block-structured int8 format: dense 64 x 64 blocks on the tensor cores (tcgen05), the
remaining nonzeros in the sparse kernel, sums added in int32 - bit-exact against the oracle's plain
definition over the dense masked weights."""
import numpy as np
import pytest
import torch

from oracle import forward as oracle_forward
from oracle import ref
from workloads import gen, models
from parity import assert_exact

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CASES = [
    # n, h, w, c_in, c_out, k, pad, block_density, sprinkle, out
    (1, 20, 20, 64, 64, 3, 1, 0.5, 0.0, "s32"),
    (1, 20, 20, 64, 64, 3, 1, 0.5, 0.02, "s8"),
    (2, 28, 28, 128, 192, 3, 1, 0.25, 0.02, "s8"),
    (1, 14, 14, 256, 128, 1, 0, 0.5, 0.05, "s8"),
    (3, 9, 23, 128, 64, 3, 1, 1.0, 0.0, "f32"),
    (1, 56, 56, 128, 128, 3, 1, 0.25, 0.01, "s8"),
    (1, 17, 33, 192, 64, 5, 2, 0.1, 0.01, "s8"),
    (2, 8, 8, 64, 128, 3, 1, 0.0, 0.03, "s8"),
]


@pytest.mark.parametrize("case", CASES)
def test_block_structured_int8_layer_bit_exact(case):
    from paper_1905_00571_b200 import binding as B
    n, h, w, c_in, c_out, k, pad, bd, sp, out = case
    g = gen.rng(sum(v for v in case if isinstance(v, int)))
    x = gen.int8_image(g, (n, h, w, c_in))
    q = gen.int8_weights(g, (c_out, k, k, c_in))
    mask = gen.block_mask(g, q.shape, bd, sp) if bd > 0 else (g.random(q.shape) < sp).astype(np.uint8)
    m = (g.uniform(0.5, 1.5, size=c_out) * 2e-5).astype(np.float32)
    b = (g.standard_normal(c_out) * 3).astype(np.float32)
    want = ref.conv2d_s8(x, q, mask, 1, pad, 1, m, b, "relu", out)
    d = B.make_desc(c_in, c_out, k, k, 1, pad, 1, h, w, n, "s8", fmt=B.FMT_GROUPED)
    wh = B.cadnn_pack_q8(d, q, mask)
    bi = B.cadnn_weights_block_info(wh)
    assert (bi["blocks"] > 0) == (bd > 0)
    ws = torch.empty(B.cadnn_weights_workspace_bytes(wh, n), dtype=torch.uint8, device=DEV)
    tdt = {"s8": torch.int8, "s32": torch.int32, "f32": torch.float32}[out]
    dev = lambda a: torch.from_numpy(a).to(DEV)
    for _ in range(2):
        y = torch.zeros(want.shape, dtype=tdt, device=DEV)
        B.cadnn_conv2d_workspace(wh, dev(x), y, ws, dev(m), dev(b), None, "relu", out_dtype=out)
        torch.cuda.synchronize()
        assert B.cadnn_device_status()["copy_timeouts"] == 0
        assert_exact(y.cpu().numpy(), want, str(case))
    y2 = torch.zeros(want.shape, dtype=tdt, device=DEV)
    if ws.numel() > 0:
        # the plain entry point refuses a layer that needs a workspace
        with pytest.raises(B.CadnnError):
            B.cadnn_conv2d(wh, dev(x), y2, dev(m), dev(b), None, "relu", out_dtype=out)
    else:
        # every kept weight sits in a dense block: the tensor-core kernel applies the epilogue itself
        assert sp == 0.0 and bd > 0
        B.cadnn_conv2d(wh, dev(x), y2, dev(m), dev(b), None, "relu", out_dtype=out)
        torch.cuda.synchronize()
        assert_exact(y2.cpu().numpy(), want, str(case) + " plain entry")


@pytest.mark.parametrize("out,c_total,c_off,act", [("s8", 0, 0, "relu"), ("f32", 0, 0, "none"), ("s8", 160, 32, "none"),
                                                   ("s8", 131, 3, "relu"), ("f32", 132, 4, "relu"), ("f32", 131, 3, "none")])
def test_block_only_layer_epilogue_residual_and_window(out, c_total, c_off, act):
    """A layer made of dense blocks only: requantization, int8 residual (whole-tensor outputs) or channel window
    inside the tensor-core kernel, against the oracle."""
    from paper_1905_00571_b200 import binding as B
    n, h, w, c_in, c_out, k, pad = 2, 13, 21, 128, 128, 3, 1
    g = gen.rng(900 + c_total + c_off)
    x = gen.int8_image(g, (n, h, w, c_in))
    q = gen.int8_weights(g, (c_out, k, k, c_in))
    mask = gen.block_mask(g, q.shape, 0.4, 0.0)
    m = (g.uniform(0.5, 1.5, size=c_out) * 2e-5).astype(np.float32)
    b = (g.standard_normal(c_out) * 3).astype(np.float32)
    r = gen.int8_image(g, (n, h, w, c_out)) if c_total == 0 else None
    rs = np.float32(0.0371 if c_total == 0 else 0.0)
    want = ref.conv2d_s8(x, q, mask, 1, pad, 1, m, b, act, out, residual=r, residual_scale=rs)
    d = B.make_desc(c_in, c_out, k, k, 1, pad, 1, h, w, n, "s8", fmt=B.FMT_GROUPED)
    wh = B.cadnn_pack_q8(d, q, mask)
    assert B.cadnn_weights_workspace_bytes(wh, n) == 0
    tdt = {"s8": torch.int8, "f32": torch.float32}[out]
    dev = lambda a: torch.from_numpy(a).to(DEV)
    ct = c_total if c_total else c_out
    fill = 77
    y = torch.full((n, h, w, ct), fill, dtype=tdt, device=DEV)
    B.cadnn_conv2d(wh, dev(x), y, dev(m), dev(b), dev(r) if r is not None else None, act, out_dtype=out, out_c_total=c_total, out_c_off=c_off,
                   residual_scale=float(rs))
    torch.cuda.synchronize()
    assert B.cadnn_device_status()["copy_timeouts"] == 0
    got = y.cpu().numpy()
    assert_exact(got[..., c_off:c_off + c_out], want, "window")
    rest = np.delete(got, np.s_[c_off:c_off + c_out], axis=3)
    assert (rest == fill).all()


@pytest.mark.parametrize("batch", [1, 2])
def test_vgg16_block_pruned_reduced_bit_exact(batch):
    from paper_1905_00571_b200 import binding as B
    from paper_1905_00571_b200.network import PackedModel
    m = models.vgg16_block(width=1.0, image=32, classes=100, fc_width=256)
    assert sum(getattr(o, "fmt", "auto") == "grouped" for o in m.ops) == 12
    x = models.make_input(m, batch)
    pm = PackedModel(m, batch, DEV)
    xd = torch.from_numpy(x).to(DEV)
    y = pm.new_output()
    pm.forward(xd, y)
    pm.forward(xd, y)
    torch.cuda.synchronize()
    assert B.cadnn_device_status()["copy_timeouts"] == 0
    want, _ = oracle_forward.forward(m, x)
    assert_exact(y.cpu().numpy(), want, "block-pruned vgg logits")
