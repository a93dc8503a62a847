"""Comparison rules shared by the GPU parity tests.

Float layers: elementwise |g - r| <= 1e-4 * max(|r|, tau) with the floor
tau = 1e-3 * max|r| of the tensor (pure relative error is ill-posed where a ReLU
or cancellation drives r to 0).  The bound follows from fp32 accumulation in any
order of at most a few thousand terms against a float64 sum rounded once.
Integer layers: bit-exact.
"""
import numpy as np

REL_TOL = 1e-4
FLOOR = 1e-3


NET_FLOOR = 1e-2   # whole-network logits: rounding compounds over ~55 layers and logits cancel


def assert_close_f32(got, ref, what="", floor=FLOOR):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), what
    peak = float(np.abs(ref).max()) if ref.size else 0.0
    denom = np.maximum(np.abs(ref), floor * peak)
    if peak == 0.0:
        assert float(np.abs(got).max() if got.size else 0.0) == 0.0, what
        return 0.0
    rel = np.abs(got - ref) / denom
    worst = float(rel.max()) if rel.size else 0.0
    assert worst <= REL_TOL, "%s: max rel err %.3e at %s (got %r ref %r), %d violations" % (
        what, worst, np.unravel_index(int(rel.argmax()), rel.shape), got.flat[int(rel.argmax())],
        ref.flat[int(rel.argmax())], int((rel > REL_TOL).sum()))
    return worst


def assert_exact(got, ref, what=""):
    got = np.asarray(got)
    ref = np.asarray(ref)
    assert got.shape == ref.shape and got.dtype == ref.dtype, (what, got.shape, ref.shape, got.dtype, ref.dtype)
    bad = int((got != ref).sum())
    assert bad == 0, "%s: %d of %d elements differ" % (what, bad, got.size)


def assert_close_or_bounded(got, ref, abs_sum, terms, what=""):
    """Float layers whose outputs cancel (a residual, or a dense sum of signed products, against a
    ReLU / ReLU6 that pins max|r|): first the plain rule at the layer floor; an element that misses it
    must still satisfy the bound that fp32 accumulation in any order obeys,
        |g - r| <= 1e-4 |r| + terms * 2^-24 * S,   S = sum |w x| |scale| + |bias| + |residual|
    (`abs_sum`, from a second oracle call on the absolute values; `terms` = multiply-adds per output
    plus the epilogue's operations).  Returns (worst relative error at the layer floor, elements that
    needed the bound)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    abs_sum = np.asarray(abs_sum, dtype=np.float64)
    assert got.shape == ref.shape == abs_sum.shape, (what, got.shape, ref.shape, abs_sum.shape)
    assert np.isfinite(got).all(), what
    peak = float(np.abs(ref).max()) if ref.size else 0.0
    err = np.abs(got - ref)
    denom = np.maximum(np.abs(ref), FLOOR * max(peak, 1e-30))
    rel = err / denom
    worst = float(rel.max()) if rel.size else 0.0
    miss = rel > REL_TOL
    bound = REL_TOL * np.abs(ref) + float(terms) * 2.0 ** -24 * abs_sum
    bad = miss & (err > bound)
    assert not bad.any(), "%s: %d elements beyond both the floor rule (worst %.3e) and the fp32 bound; first at %s: got %r ref %r bound %.3e" % (
        what, int(bad.sum()), worst, np.unravel_index(int(bad.argmax()), bad.shape), got.flat[int(bad.argmax())],
        ref.flat[int(bad.argmax())], bound.flat[int(bad.argmax())])
    return worst, int(miss.sum())
