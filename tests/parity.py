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
