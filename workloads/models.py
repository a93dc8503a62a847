"""Synthetic networks shaped like the paper's workloads (Section 5, Table 2, and
the VGGNet named in Section 3): ResNet-50 v1.5, VGG-16, MobileNet-V2, MobileNet-V1.

A network is plain data: an ordered list of ops over numbered tensor slots
(slot 0 is the input image).  Both the CPU oracle's network walker and the CUDA
library's binding consume this list; nothing here computes a layer.

Gains.  With random weights, activations would vanish or explode over ~50
layers, so each layer's folded BatchNorm scale is multiplied by a gain derived
from summary statistics of the generated tensors (kept weight energy), and
int8 layers get a requantization multiplier derived from the row's sum of
squared integer weights.  These are recipes for synthetic inputs only.
"""
from dataclasses import dataclass, field
from typing import List, Optional, Tuple
import numpy as np

from . import gen


@dataclass
class Op:
    kind: str                      # 'conv' | 'fc' | 'maxpool' | 'avgpool' | 'gavgpool'
    name: str
    src: int
    dst: int
    res: int = -1                  # residual slot added in the epilogue, -1 = none
    c_in: int = 0
    c_out: int = 0
    k: int = 1
    stride: int = 1
    pad: int = 0
    groups: int = 1
    act: str = "none"              # 'none' | 'relu' | 'relu6'
    w: Optional[np.ndarray] = None     # f32: float32 OHWI; s8: int8 codes OHWI
    mask: Optional[np.ndarray] = None  # uint8, same shape; None = dense
    scale: Optional[np.ndarray] = None  # f32: folded BN scale; s8: multiplier M
    bias: Optional[np.ndarray] = None   # f32: folded BN bias;  s8: offset B
    out: str = "f32"               # 'f32' | 's8' | 's32'
    density: float = 1.0
    in_hw: Tuple[int, int] = (0, 0)
    out_hw: Tuple[int, int] = (0, 0)
    pad_w: int = -1                # padding along the width when it differs from `pad` (rectangular kernels)
    res_scale: float = 0.0         # int8 residual: s_r / s_y
    dst_off: int = 0               # first channel of dst this op writes (channel concatenation)
    dst_total: int = 0             # channels of the dst slot; 0 = the op's own c_out
    fmt: str = "auto"              # 'grouped': ask the packer for the block-structured int8 format

    @property
    def nnz(self):
        if self.w is None:
            return 0
        return int(self.w.size if self.mask is None else int(self.mask.sum()))


@dataclass
class Model:
    name: str
    dtype: str                     # 'f32' | 's8'
    in_shape: Tuple[int, int, int]  # (h, w, c)
    ops: List[Op] = field(default_factory=list)
    seed: int = 0
    n_slots: int = 1

    def new_slot(self):
        s = self.n_slots
        self.n_slots += 1
        return s

    def weight_ops(self):
        return [o for o in self.ops if o.kind in ("conv", "fc")]


def _hw_out(h, k, s, p):
    return (h + 2 * p - k) // s + 1


_GAMMA_RMS = np.sqrt(1.0 + 1.0 / 12.0)   # rms of U(0.5, 1.5)


def _f32_conv(m, g, name, src, c_in, c_out, k, stride, pad, h, act, density,
              groups=1, res=-1, gain=1.0, prune="magnitude", kw=None, pad_w=None, dst=None, dst_off=0, dst_total=0):
    """One float conv op (square k x k kernel unless kw is given; pad_w pads the columns when it
    differs from pad).  dst / dst_off / dst_total: write a channel window of an existing slot."""
    cg = c_in // groups
    kw = k if kw is None else kw
    w = gen.he_weights(g, c_out, k, kw, cg)
    if density >= 1.0:
        mask = None
        kept = 1.0
    else:
        mask = gen.magnitude_mask(w, density) if prune == "magnitude" else gen.random_mask(g, w.shape, density)
        kept = gen.kept_energy(w, mask)
    # He-initialised weights double the second moment; a ReLU halves it again.
    layer_gain = gain / (_GAMMA_RMS * np.sqrt(kept))
    if act == "none":
        layer_gain /= np.sqrt(2.0)
    scale, bias = gen.folded_bn(g, c_out, gain=layer_gain)
    if dst is None:
        dst = m.new_slot()
    ho = _hw_out(h, k, stride, pad)
    wo = _hw_out(h, kw, stride, pad if pad_w is None else pad_w)
    m.ops.append(Op("conv", name, src, dst, res, c_in, c_out, k, stride, pad, groups, act,
                    w, mask, scale, bias, "f32", density, (h, h), (ho, wo),
                    pad_w=-1 if pad_w is None else pad_w, dst_off=dst_off, dst_total=dst_total))
    return dst, ho


def _f32_fc(m, g, name, src, k_in, c_out, density):
    w = gen.he_weights(g, c_out, 1, 1, k_in)
    mask = None if density >= 1.0 else gen.magnitude_mask(w, density)
    kept = 1.0 if mask is None else gen.kept_energy(w, mask)
    scale = np.full(c_out, 1.0 / np.sqrt(2.0 * kept), np.float32)
    bias = (g.standard_normal(c_out) * 0.1).astype(np.float32)
    dst = m.new_slot()
    m.ops.append(Op("fc", name, src, dst, -1, k_in, c_out, 1, 1, 0, 1, "none",
                    w, mask, scale, bias, "f32", density, (1, 1), (1, 1)))
    return dst


def single_layer(seed=1, c_in=64, c_out=64, hw=56, k=3, stride=1, pad=1, density=0.10):
    """One 3x3 conv layer: N(0, 0.05^2) weights, exactly-k uniform random mask,
    max(0, N(0,1)) input, no bias, ReLU."""
    g = gen.rng(seed)
    m = Model("single_conv", "f32", (hw, hw, c_in), seed=seed)
    w = gen.normal_weights(g, (c_out, k, k, c_in), 0.05)
    mask = None if density >= 1.0 else gen.random_mask(g, w.shape, density)
    ho = _hw_out(hw, k, stride, pad)
    m.ops.append(Op("conv", "conv", 0, m.new_slot(), -1, c_in, c_out, k, stride, pad, 1, "relu",
                    w, mask, None, None, "f32", density, (hw, hw), (ho, ho)))
    return m


def resnet50(seed=2, density=0.125, fc_density=0.10, width=1.0, image=224, classes=1000):
    """ResNet-50 v1.5: stride 2 sits on the 3x3 conv of the first block of stages
    3 to 5.  The 7x7 stem stays dense; every other conv is magnitude-pruned per
    layer to `density`; the classifier to `fc_density`."""
    g = gen.rng(seed)
    m = Model("resnet50", "f32", (image, image, 3), seed=seed)
    ch = lambda c: max(8, int(round(c * width)))
    cur, h = _f32_conv(m, g, "conv1", 0, 3, ch(64), 7, 2, 3, image, "relu", 1.0)
    dst = m.new_slot()
    ho = _hw_out(h, 3, 2, 1)
    m.ops.append(Op("maxpool", "pool1", cur, dst, k=3, stride=2, pad=1, c_in=ch(64), c_out=ch(64),
                    in_hw=(h, h), out_hw=(ho, ho)))
    cur, h, c_in = dst, ho, ch(64)
    for si, (mid, blocks, stride) in enumerate([(64, 3, 1), (128, 4, 2), (256, 6, 2), (512, 3, 2)]):
        mid = ch(mid)
        out = mid * 4
        for b in range(blocks):
            s = stride if b == 0 else 1
            nm = "s%db%d" % (si + 2, b)
            if b == 0:
                short, _ = _f32_conv(m, g, nm + ".ds", cur, c_in, out, 1, s, 0, h, "none", density)
            else:
                short = cur
            t, _ = _f32_conv(m, g, nm + ".c1", cur, c_in, mid, 1, 1, 0, h, "relu", density)
            t, h2 = _f32_conv(m, g, nm + ".c2", t, mid, mid, 3, s, 1, h, "relu", density)
            cur, _ = _f32_conv(m, g, nm + ".c3", t, mid, out, 1, 1, 0, h2, "relu", density,
                               res=short, gain=0.4)
            h, c_in = h2, out
    dst = m.new_slot()
    m.ops.append(Op("gavgpool", "avgpool", cur, dst, c_in=c_in, c_out=c_in, in_hw=(h, h), out_hw=(1, 1)))
    _f32_fc(m, g, "fc", dst, c_in, classes, fc_density)
    return m


def mobilenet_v2(seed=4, density=0.25, width=1.0, image=224, classes=1000):
    """MobileNet-V2 (width 1.0): stem 3x3 s2 and all depthwise 3x3 dense; pointwise
    1x1 convs, the 1x1 head and the classifier magnitude-pruned to `density`.
    ReLU6 after expand and depthwise, no activation after project."""
    g = gen.rng(seed)
    m = Model("mobilenet_v2", "f32", (image, image, 3), seed=seed)
    ch = lambda c: max(8, int(round(c * width / 8.0)) * 8)
    c_in = ch(32)
    cur, h = _f32_conv(m, g, "stem", 0, 3, c_in, 3, 2, 1, image, "relu6", 1.0)
    cfg = [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2), (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)]
    for t, c, n, s in cfg:
        c = ch(c)
        for b in range(n):
            st = s if b == 0 else 1
            nm = "ir%d_%d" % (c, b)
            hid = c_in * t
            x_in = cur
            tcur = cur
            if t != 1:
                tcur, _ = _f32_conv(m, g, nm + ".expand", tcur, c_in, hid, 1, 1, 0, h, "relu6", density)
            tcur, h2 = _f32_conv(m, g, nm + ".dw", tcur, hid, hid, 3, st, 1, h, "relu6", 1.0, groups=hid)
            use_res = (st == 1 and c_in == c)
            cur, _ = _f32_conv(m, g, nm + ".project", tcur, hid, c, 1, 1, 0, h2, "none", density,
                               res=x_in if use_res else -1, gain=0.7 if use_res else 1.0)
            h, c_in = h2, c
    head = ch(1280)
    cur, _ = _f32_conv(m, g, "head", cur, c_in, head, 1, 1, 0, h, "relu6", density)
    dst = m.new_slot()
    m.ops.append(Op("gavgpool", "avgpool", cur, dst, c_in=head, c_out=head, in_hw=(h, h), out_hw=(1, 1)))
    _f32_fc(m, g, "fc", dst, head, classes, density)
    return m


def mobilenet_v1(seed=5, density=0.25, width=1.0, image=224, classes=1000):
    """MobileNet-V1 (Table 2 of the paper lists it next to V2): stem 3x3 s2 and the 13 depthwise 3x3
    convs dense, the 13 pointwise 1x1 convs and the classifier magnitude-pruned to `density`;
    ReLU after every conv."""
    g = gen.rng(seed)
    m = Model("mobilenet_v1", "f32", (image, image, 3), seed=seed)
    ch = lambda c: max(8, int(round(c * width / 8.0)) * 8)
    c_in = ch(32)
    cur, h = _f32_conv(m, g, "stem", 0, 3, c_in, 3, 2, 1, image, "relu", 1.0)
    cfg = [(64, 1), (128, 2), (128, 1), (256, 2), (256, 1), (512, 2), (512, 1), (512, 1), (512, 1), (512, 1), (512, 1),
           (1024, 2), (1024, 1)]
    for i, (c, st) in enumerate(cfg):
        c = ch(c)
        cur, h = _f32_conv(m, g, "b%d.dw" % (i + 1), cur, c_in, c_in, 3, st, 1, h, "relu", 1.0, groups=c_in)
        cur, _ = _f32_conv(m, g, "b%d.pw" % (i + 1), cur, c_in, c, 1, 1, 0, h, "relu", density)
        c_in = c
    dst = m.new_slot()
    m.ops.append(Op("gavgpool", "avgpool", cur, dst, c_in=c_in, c_out=c_in, in_hw=(h, h), out_hw=(1, 1)))
    _f32_fc(m, g, "fc", dst, c_in, classes, density)
    return m


def inception_v3(seed=6, density=0.125, fc_density=0.10, width=1.0, image=299, classes=1000):
    """Inception-V3 (Table 2 of the paper): the 3x3 s2 stem conv dense, the other 93 convs (1x1, 3x3,
    5x5, 1x7, 7x1, 1x3, 3x1) magnitude-pruned to `density`, the classifier to `fc_density`; every conv is
    Conv + folded BatchNorm + ReLU.  The branches of a module write their channel windows of one
    concatenated tensor; average pools count padded taps as zeros (divisor k*k)."""
    g = gen.rng(seed)
    m = Model("inception_v3", "f32", (image, image, 3), seed=seed)
    ch = lambda c: max(8, int(round(c * width / 8.0)) * 8)

    def conv(name, src, c_in, c_out, h, k=1, stride=1, pad=0, kw=None, pad_w=None, dens=density, **kwargs):
        return _f32_conv(m, g, name, src, c_in, c_out, k, stride, pad, h, "relu", dens, kw=kw, pad_w=pad_w, **kwargs)

    def pool(kind, name, src, c, h, k, stride, pad, dst=None, dst_off=0, dst_total=0):
        if dst is None:
            dst = m.new_slot()
        ho = _hw_out(h, k, stride, pad)
        m.ops.append(Op(kind, name, src, dst, k=k, stride=stride, pad=pad, c_in=c, c_out=c, in_hw=(h, h), out_hw=(ho, ho),
                        dst_off=dst_off, dst_total=dst_total))
        return dst, ho

    cur, h = conv("conv1a", 0, 3, ch(32), image, 3, 2, 0, dens=1.0)
    cur, h = conv("conv2a", cur, ch(32), ch(32), h, 3, 1, 0)
    cur, h = conv("conv2b", cur, ch(32), ch(64), h, 3, 1, 1)
    cur, h = pool("maxpool", "pool1", cur, ch(64), h, 3, 2, 0)
    cur, h = conv("conv3b", cur, ch(64), ch(80), h, 1)
    cur, h = conv("conv4a", cur, ch(80), ch(192), h, 3, 1, 0)
    cur, h = pool("maxpool", "pool2", cur, ch(192), h, 3, 2, 0)
    c_in = ch(192)

    def module_a(nm, src, c_in, h, pool_features):
        total = ch(64) + ch(64) + ch(96) + ch(pool_features)
        out = m.new_slot()
        off = 0
        conv(nm + ".b1", src, c_in, ch(64), h, dst=out, dst_off=off, dst_total=total); off += ch(64)
        t, _ = conv(nm + ".b5a", src, c_in, ch(48), h)
        conv(nm + ".b5b", t, ch(48), ch(64), h, 5, 1, 2, dst=out, dst_off=off, dst_total=total); off += ch(64)
        t, _ = conv(nm + ".b3a", src, c_in, ch(64), h)
        t, _ = conv(nm + ".b3b", t, ch(64), ch(96), h, 3, 1, 1)
        conv(nm + ".b3c", t, ch(96), ch(96), h, 3, 1, 1, dst=out, dst_off=off, dst_total=total); off += ch(96)
        t, _ = pool("avgpool", nm + ".pool", src, c_in, h, 3, 1, 1)
        conv(nm + ".bp", t, c_in, ch(pool_features), h, dst=out, dst_off=off, dst_total=total)
        return out, total

    def module_b(nm, src, c_in, h):
        total = ch(384) + ch(96) + c_in
        out = m.new_slot()
        _, ho = conv(nm + ".b3", src, c_in, ch(384), h, 3, 2, 0, dst=out, dst_off=0, dst_total=total)
        t, _ = conv(nm + ".bda", src, c_in, ch(64), h)
        t, _ = conv(nm + ".bdb", t, ch(64), ch(96), h, 3, 1, 1)
        conv(nm + ".bdc", t, ch(96), ch(96), h, 3, 2, 0, dst=out, dst_off=ch(384), dst_total=total)
        pool("maxpool", nm + ".pool", src, c_in, h, 3, 2, 0, dst=out, dst_off=ch(384) + ch(96), dst_total=total)
        return out, total, ho

    def module_c(nm, src, c_in, h, c7):
        c7 = ch(c7)
        total = 4 * ch(192)
        out = m.new_slot()
        conv(nm + ".b1", src, c_in, ch(192), h, dst=out, dst_off=0, dst_total=total)
        t, _ = conv(nm + ".b7a", src, c_in, c7, h)
        t, _ = conv(nm + ".b7b", t, c7, c7, h, 1, 1, 0, kw=7, pad_w=3)
        conv(nm + ".b7c", t, c7, ch(192), h, 7, 1, 3, kw=1, pad_w=0, dst=out, dst_off=ch(192), dst_total=total)
        t, _ = conv(nm + ".bda", src, c_in, c7, h)
        t, _ = conv(nm + ".bdb", t, c7, c7, h, 7, 1, 3, kw=1, pad_w=0)
        t, _ = conv(nm + ".bdc", t, c7, c7, h, 1, 1, 0, kw=7, pad_w=3)
        t, _ = conv(nm + ".bdd", t, c7, c7, h, 7, 1, 3, kw=1, pad_w=0)
        conv(nm + ".bde", t, c7, ch(192), h, 1, 1, 0, kw=7, pad_w=3, dst=out, dst_off=2 * ch(192), dst_total=total)
        t, _ = pool("avgpool", nm + ".pool", src, c_in, h, 3, 1, 1)
        conv(nm + ".bp", t, c_in, ch(192), h, dst=out, dst_off=3 * ch(192), dst_total=total)
        return out, total

    def module_d(nm, src, c_in, h):
        total = ch(320) + ch(192) + c_in
        out = m.new_slot()
        t, _ = conv(nm + ".b3a", src, c_in, ch(192), h)
        _, ho = conv(nm + ".b3b", t, ch(192), ch(320), h, 3, 2, 0, dst=out, dst_off=0, dst_total=total)
        t, _ = conv(nm + ".b7a", src, c_in, ch(192), h)
        t, _ = conv(nm + ".b7b", t, ch(192), ch(192), h, 1, 1, 0, kw=7, pad_w=3)
        t, _ = conv(nm + ".b7c", t, ch(192), ch(192), h, 7, 1, 3, kw=1, pad_w=0)
        conv(nm + ".b7d", t, ch(192), ch(192), h, 3, 2, 0, dst=out, dst_off=ch(320), dst_total=total)
        pool("maxpool", nm + ".pool", src, c_in, h, 3, 2, 0, dst=out, dst_off=ch(320) + ch(192), dst_total=total)
        return out, total, ho

    def module_e(nm, src, c_in, h):
        total = ch(320) + 4 * ch(384) + ch(192)
        out = m.new_slot()
        off = 0
        conv(nm + ".b1", src, c_in, ch(320), h, dst=out, dst_off=off, dst_total=total); off += ch(320)
        t, _ = conv(nm + ".b3a", src, c_in, ch(384), h)
        conv(nm + ".b3b", t, ch(384), ch(384), h, 1, 1, 0, kw=3, pad_w=1, dst=out, dst_off=off, dst_total=total); off += ch(384)
        conv(nm + ".b3c", t, ch(384), ch(384), h, 3, 1, 1, kw=1, pad_w=0, dst=out, dst_off=off, dst_total=total); off += ch(384)
        t, _ = conv(nm + ".bda", src, c_in, ch(448), h)
        t, _ = conv(nm + ".bdb", t, ch(448), ch(384), h, 3, 1, 1)
        conv(nm + ".bdc", t, ch(384), ch(384), h, 1, 1, 0, kw=3, pad_w=1, dst=out, dst_off=off, dst_total=total); off += ch(384)
        conv(nm + ".bdd", t, ch(384), ch(384), h, 3, 1, 1, kw=1, pad_w=0, dst=out, dst_off=off, dst_total=total); off += ch(384)
        t, _ = pool("avgpool", nm + ".pool", src, c_in, h, 3, 1, 1)
        conv(nm + ".bp", t, c_in, ch(192), h, dst=out, dst_off=off, dst_total=total)
        return out, total

    cur, c_in = module_a("m5b", cur, c_in, h, 32)
    cur, c_in = module_a("m5c", cur, c_in, h, 64)
    cur, c_in = module_a("m5d", cur, c_in, h, 64)
    cur, c_in, h = module_b("m6a", cur, c_in, h)
    for nm, c7 in (("m6b", 128), ("m6c", 160), ("m6d", 160), ("m6e", 192)):
        cur, c_in = module_c(nm, cur, c_in, h, c7)
    cur, c_in, h = module_d("m7a", cur, c_in, h)
    cur, c_in = module_e("m7b", cur, c_in, h)
    cur, c_in = module_e("m7c", cur, c_in, h)
    dst = m.new_slot()
    m.ops.append(Op("gavgpool", "avgpool", cur, dst, c_in=c_in, c_out=c_in, in_hw=(h, h), out_hw=(1, 1)))
    _f32_fc(m, g, "fc", dst, c_in, classes, fc_density)
    return m


# Target rms of the requantized pre-activation, and the input second moments the
# multiplier recipe assumes (image codes; post-ReLU codes; post-ReLU codes after a
# 2x2 max pool).  Synthetic-input recipe only.
_T_RMS = 127.0 / 3.0
_M2_IMAGE = _T_RMS ** 2
_M2_RELU = 0.5 * _T_RMS ** 2
_M2_POOLED = 1.3 * _T_RMS ** 2


def _s8_layer(m, g, kind, name, src, c_in, c_out, k, pad, h, act, density, m2_in, out="s8", stride=1, res=-1,
              res_scale=0.0, gain=1.0):
    shape = (c_out, k, k, c_in)
    q = gen.int8_weights(g, shape)
    mask = None if density >= 1.0 else gen.random_mask(g, shape, density)
    qq = q.astype(np.float64) ** 2
    if mask is not None:
        qq = qq * mask
    row_energy = qq.reshape(c_out, -1).sum(axis=1)
    mult = np.where(row_energy > 0, _T_RMS / np.sqrt(np.maximum(row_energy, 1.0) * m2_in), 1.0)
    mult = (mult * gain * g.uniform(0.8, 1.25, size=c_out)).astype(np.float32)
    offs = (g.standard_normal(c_out) * 0.1 * _T_RMS).astype(np.float32)
    dst = m.new_slot()
    ho = _hw_out(h, k, stride, pad)
    m.ops.append(Op(kind, name, src, dst, res, c_in, c_out, k, stride, pad, 1, act, q, mask,
                    mult, offs, out, density, (h, h), (ho, ho), res_scale=res_scale))
    return dst


def vgg16_block(seed=8, block_density=0.25, sprinkle=0.01, width=1.0, image=224, classes=1000, fc_width=4096):
    """VGG-16, int8, with BLOCK-structured pruning of the convs from conv2 on: of the 64 output channels x 64
    input channels x one tap blocks of a layer exactly round(block_density * blocks) are kept whole, and a
    further `sprinkle` of the remaining positions is kept at random (so that the sparse kernel has a
    remainder to add).  conv1 (3 input channels) and the FC layers are pruned as in vgg16()."""
    g = gen.rng(seed)
    base = vgg16(seed=seed, width=width, image=image, classes=classes, fc_width=fc_width)
    base.name = "vgg16_block"
    for op in base.ops:
        if op.kind != "conv" or op.c_in % 64 or op.c_out % 64:
            continue
        op.mask = gen.block_mask(g, op.w.shape, block_density, sprinkle)
        op.density = float(op.mask.mean())
        op.fmt = "grouped"
        qq = (op.w.astype(np.float64) ** 2) * op.mask
        row_energy = qq.reshape(op.c_out, -1).sum(axis=1)
        mult = np.where(row_energy > 0, _T_RMS / np.sqrt(np.maximum(row_energy, 1.0) * _M2_RELU), 1.0)
        op.scale = (mult * g.uniform(0.8, 1.25, size=op.c_out)).astype(np.float32)
    return base


def vgg16(seed=3, density=0.08, fc_density=0.04, width=1.0, image=224, classes=1000, fc_width=4096):
    """VGG-16 with int8 weights and activations: 13 convs at `density`, 3 FC layers
    at `fc_density`, exactly-k uniform random masks, five int8 2x2 max pools.
    The last layer returns fmaf(acc, M, B) as float32 without rounding."""
    g = gen.rng(seed)
    m = Model("vgg16", "s8", (image, image, 3), seed=seed)
    cfg = [64, 64, "M", 128, 128, "M", 256, 256, 256, "M", 512, 512, 512, "M", 512, 512, 512, "M"]
    cur, h, c_in, i = 0, image, 3, 0
    m2 = _M2_IMAGE
    for c in cfg:
        if c == "M":
            dst = m.new_slot()
            m.ops.append(Op("maxpool", "pool%d" % i, cur, dst, k=2, stride=2, pad=0, c_in=c_in, c_out=c_in,
                            in_hw=(h, h), out_hw=(h // 2, h // 2), out="s8"))
            cur, h, m2 = dst, h // 2, _M2_POOLED
            continue
        i += 1
        c = max(8, int(round(c * width)))
        cur = _s8_layer(m, g, "conv", "conv%d" % i, cur, c_in, c, 3, 1, h, "relu", density, m2)
        c_in, m2 = c, _M2_RELU
    # FC input is the NHWC flatten (h, w, c order) of the last feature map.
    k_in = h * h * c_in
    cur = _s8_layer(m, g, "fc", "fc6", cur, k_in, fc_width, 1, 0, 1, "relu", fc_density, _M2_POOLED)
    cur = _s8_layer(m, g, "fc", "fc7", cur, fc_width, fc_width, 1, 0, 1, "relu", fc_density, _M2_RELU)
    _s8_layer(m, g, "fc", "fc8", cur, fc_width, classes, 1, 0, 1, "none", fc_density, _M2_RELU, out="f32")
    return m


def resnet50_int8(seed=7, density=0.125, fc_density=0.10, width=1.0, image=224, classes=1000):
    """ResNet-50 v1.5 with int8 weights and activations (the int8 counterpart of the pruned ResNet-50): dense
    int8 7x7 stem, every other conv an exactly-k random mask at `density`, an int8 3x3 max pool, the shortcut of
    a block joining the last conv's requantization as an int8 residual (two fused multiply-adds, then ReLU).
    The last block stores float32 (no rounding), which feeds a float global average pool and a pruned
    float classifier."""
    g = gen.rng(seed)
    m = Model("resnet50_int8", "s8", (image, image, 3), seed=seed)
    ch = lambda c: max(8, int(round(c * width)))
    cur = _s8_layer(m, g, "conv", "conv1", 0, 3, ch(64), 7, 3, image, "relu", 1.0, _M2_IMAGE, stride=2)
    h = _hw_out(image, 7, 2, 3)
    dst = m.new_slot()
    ho = _hw_out(h, 3, 2, 1)
    m.ops.append(Op("maxpool", "pool1", cur, dst, k=3, stride=2, pad=1, c_in=ch(64), c_out=ch(64),
                    in_hw=(h, h), out_hw=(ho, ho), out="s8"))
    cur, h, c_in = dst, ho, ch(64)
    m2 = _M2_POOLED
    stages = [(64, 3, 1), (128, 4, 2), (256, 6, 2), (512, 3, 2)]
    for si, (mid, blocks, stride) in enumerate(stages):
        mid = ch(mid)
        out = mid * 4
        for b in range(blocks):
            s = stride if b == 0 else 1
            nm = "s%db%d" % (si + 2, b)
            last = si == len(stages) - 1 and b == blocks - 1
            if b == 0:
                short = _s8_layer(m, g, "conv", nm + ".ds", cur, c_in, out, 1, 0, h, "none", density, m2, stride=s)
            else:
                short = cur
            t = _s8_layer(m, g, "conv", nm + ".c1", cur, c_in, mid, 1, 0, h, "relu", density, m2)
            t = _s8_layer(m, g, "conv", nm + ".c2", t, mid, mid, 3, 1, h, "relu", density, _M2_RELU, stride=s)
            h2 = _hw_out(h, 3, s, 1)
            cur = _s8_layer(m, g, "conv", nm + ".c3", t, mid, out, 1, 0, h2, "relu", density, _M2_RELU,
                            out="f32" if last else "s8", res=short, res_scale=0.6, gain=0.6)
            h, c_in, m2 = h2, out, 1.1 * _T_RMS ** 2
    dst = m.new_slot()
    m.ops.append(Op("gavgpool", "avgpool", cur, dst, c_in=c_in, c_out=c_in, in_hw=(h, h), out_hw=(1, 1)))
    # float classifier on the pooled float features (in code units: ~T_RMS)
    w = gen.he_weights(g, classes, 1, 1, c_in)
    mask = None if fc_density >= 1.0 else gen.magnitude_mask(w, fc_density)
    kept = 1.0 if mask is None else gen.kept_energy(w, mask)
    scale = np.full(classes, 1.0 / (_T_RMS * np.sqrt(2.0 * kept)), np.float32)
    bias = (g.standard_normal(classes) * 0.1).astype(np.float32)
    out_slot = m.new_slot()
    m.ops.append(Op("fc", "fc", dst, out_slot, -1, c_in, classes, 1, 1, 0, 1, "none", w, mask, scale, bias, "f32",
                    fc_density, (1, 1), (1, 1)))
    return m


def make_input(model, batch=1, seed=None):
    g = gen.rng(model.seed * 1000003 + 17 if seed is None else seed)
    h, w, c = model.in_shape
    if model.dtype == "s8":
        return gen.int8_image(g, (batch, h, w, c))
    if model.name == "single_conv":
        return gen.relu_normal_input(g, (batch, h, w, c))
    return gen.normal_input(g, (batch, h, w, c))
