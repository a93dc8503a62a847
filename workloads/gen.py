"""Seeded synthetic tensors: weights, pruning masks, inputs, folded BatchNorm vectors.

This module serves both the CPU oracle's tests and the CUDA library's tests and
benchmark.  It holds no layer arithmetic: it only draws random numbers, ranks
magnitudes to build masks, and computes summary statistics of the tensors it
generated so that synthetic networks keep sane activation ranges.

Stand-in for the paper's workloads: the paper (Section 5, Table 2) evaluates
ImageNet models pruned by ADMM (Section 3).  Neither the data nor the trained
weights are available, so every tensor here is random with the shape, density
and value distribution of those workloads.
"""
import numpy as np


def rng(seed):
    return np.random.Generator(np.random.PCG64(int(seed)))


def keep_count(density, numel):
    """Number of weights a layer keeps: round(density * numel), at least 1."""
    return max(1, min(int(numel), int(np.floor(density * numel + 0.5))))


def random_mask(g, shape, density):
    """Exactly-k uniform random unstructured mask (k = keep_count), uint8."""
    numel = int(np.prod(shape))
    k = keep_count(density, numel)
    m = np.zeros(numel, np.uint8)
    if k >= numel:
        m[:] = 1
    else:
        m[g.choice(numel, size=k, replace=False)] = 1
    return m.reshape(shape)


def magnitude_mask(w, density):
    """Keep exactly k weights of largest |w| over the whole layer (the Euclidean
    projection onto the cardinality constraint of Section 3); ties go to the
    lower flat index."""
    numel = w.size
    k = keep_count(density, numel)
    m = np.zeros(numel, np.uint8)
    if k >= numel:
        m[:] = 1
    else:
        order = np.argsort(-np.abs(w.reshape(-1)), kind="stable")
        m[order[:k]] = 1
    return m.reshape(w.shape)


def skewed_mask(g, shape, density, skew=4.0):
    """Unstructured mask whose per-filter density varies by a factor of about
    `skew` between the sparsest and densest filter (load-balance stress case)."""
    c_out = shape[0]
    per = int(np.prod(shape[1:]))
    rel = np.exp(g.uniform(0.0, np.log(skew), size=c_out))
    rel *= density * c_out / rel.sum()
    m = np.zeros((c_out, per), np.uint8)
    for co in range(c_out):
        k = min(per, int(round(rel[co] * per)))
        if k > 0:
            m[co, g.choice(per, size=k, replace=False)] = 1
    return m.reshape(shape)


def block_mask(g, shape, block_density, sprinkle=0.0, bm=64, bk=64):
    """Block-structured mask for OHWI weights [c_out, kh, kw, c_in]: the tensor is cut into blocks of bm output
    channels x bk input channels at one tap; exactly keep_count(block_density, blocks) blocks are kept whole,
    and of the positions outside them a fraction `sprinkle` is kept at random."""
    c_out, kh, kw, c_in = shape
    nb_o, nb_i = c_out // bm, c_in // bk
    blocks = nb_o * kh * kw * nb_i
    k = keep_count(block_density, blocks)
    pick = np.zeros(blocks, np.uint8)
    pick[g.choice(blocks, size=k, replace=False)] = 1
    pick = pick.reshape(nb_o, kh, kw, nb_i)
    m = np.repeat(np.repeat(pick, bm, axis=0), bk, axis=3)
    full = np.zeros(shape, np.uint8)
    full[:nb_o * bm, :, :, :nb_i * bk] = m
    if sprinkle > 0.0:
        full |= ((g.random(shape) < sprinkle) & (full == 0)).astype(np.uint8)
    return full


def normal_weights(g, shape, std):
    return (g.standard_normal(shape) * std).astype(np.float32)


def he_weights(g, c_out, kh, kw, cg):
    """N(0, 2 / fan_in) weights, OHWI [c_out][kh][kw][c_in/groups]."""
    fan_in = kh * kw * cg
    return normal_weights(g, (c_out, kh, kw, cg), np.sqrt(2.0 / fan_in))


def relu_normal_input(g, shape):
    """max(0, N(0,1)) activations, like a post-ReLU feature map."""
    return np.maximum(g.standard_normal(shape), 0.0).astype(np.float32)


def normal_input(g, shape):
    return g.standard_normal(shape).astype(np.float32)


def int8_image(g, shape):
    """Symmetric int8 image: round(N(0,1) * 127/3) clipped to [-127, 127]."""
    v = np.rint(g.standard_normal(shape) * (127.0 / 3.0))
    return np.clip(v, -127, 127).astype(np.int8)


def int8_relu_activation(g, shape):
    """Int8 feature map as a ReLU + requantize layer leaves it: values in [0, 127]."""
    v = np.rint(np.maximum(g.standard_normal(shape), 0.0) * (127.0 / 3.0))
    return np.clip(v, 0, 127).astype(np.int8)


def int8_weights(g, shape, std=40.0):
    """Integer weight codes in [-127, 127]."""
    v = np.rint(g.standard_normal(shape) * std)
    return np.clip(v, -127, 127).astype(np.int8)


def folded_bn(g, c_out, gain=1.0, bias_std=0.1):
    """Synthetic BatchNorm folded to per-channel (scale, bias): gamma ~ U(0.5, 1.5)
    times `gain`, beta ~ N(0, bias_std^2), running mean 0 and variance 1."""
    scale = (g.uniform(0.5, 1.5, size=c_out) * gain).astype(np.float32)
    bias = (g.standard_normal(c_out) * bias_std).astype(np.float32)
    return scale, bias


def kept_energy(w, mask):
    """Fraction of the layer's sum of squares that survives the mask (a summary
    statistic of the generated tensors, used only to pick the synthetic gain)."""
    tot = float(np.sum(np.square(w, dtype=np.float64)))
    if tot == 0.0:
        return 1.0
    kept = float(np.sum(np.square(w, dtype=np.float64) * (mask != 0)))
    return max(kept / tot, 1e-12)
