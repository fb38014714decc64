"""Helpers shared by the GPU parity tests."""
import numpy as np


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def bf16_ulp(x):
    """Spacing of bfloat16 numbers at |x| (8 significand bits)."""
    ax = np.maximum(np.abs(np.asarray(x, dtype=np.float64)), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


def assert_bf16_close(got, want, what, tol_rel=2e-3, min_equal=0.98):
    """Same operands on both sides: the two bf16 results may differ only where the fp32
    value sat next to a rounding boundary, i.e. by at most one bf16 spacing, rarely."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64).reshape(got.shape)
    r = rel_l2(got, want)
    assert r <= tol_rel, "%s: relative L2 error %.3e > %.1e" % (what, r, tol_rel)
    # absolute part: fp32 accumulation error of the contraction (a few 1e-6 of a typical
    # element) also moves elements whose own magnitude, hence bf16 spacing, is tiny
    rms = float(np.sqrt(np.mean(want * want))) if want.size else 0.0
    slack = bf16_ulp(want) * 1.01 + 3e-5 * rms
    bad = np.abs(got - want) > slack
    assert not bad.any(), "%s: %d elements differ by more than one bf16 spacing" % (what, int(bad.sum()))
    eq = float((got == want).mean()) if want.size else 1.0
    assert eq >= min_equal, "%s: only %.4f of the elements are bit-equal" % (what, eq)
    return r
