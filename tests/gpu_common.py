"""Helpers shared by the GPU parity tests."""
import numpy as np

_CHUNK = 1 << 24      # elements compared at a time (keeps the float64 temporaries of huge tensors small)


def _chunks(a, b):
    a = np.asarray(a).reshape(-1)
    b = np.asarray(b).reshape(-1)
    assert a.size == b.size, (a.size, b.size)
    for i in range(0, max(a.size, 1), _CHUNK):
        yield a[i:i + _CHUNK].astype(np.float64), b[i:i + _CHUNK].astype(np.float64)


def rel_l2(a, b):
    num = den = 0.0
    for x, y in _chunks(a, b):
        d = x - y
        num += float(d @ d)
        den += float(y @ y)
    return float(np.sqrt(num) / max(np.sqrt(den), 1e-300))


def bf16_ulp(x):
    """Spacing of bfloat16 numbers at |x| (8 significand bits)."""
    ax = np.maximum(np.abs(np.asarray(x, dtype=np.float64)), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


def assert_bf16_close(got, want, what, tol_rel=2e-3, min_equal=0.98, k_terms=1024):
    """Same operands on both sides: the two bf16 results may differ only where the fp32
    value sat next to a rounding boundary, i.e. by at most one bf16 spacing, rarely.
    k_terms = length of the contraction behind the tensor: the fp32 accumulation error that the
    absolute part of the bound allows grows like its square root (3e-5 of the tensor's rms up to
    1024 terms: the worst element of 1e7 sits about five standard deviations out)."""
    got = np.asarray(got)
    want = np.asarray(want).reshape(got.shape)
    r = rel_l2(got, want)
    assert r <= tol_rel, "%s: relative L2 error %.3e > %.1e" % (what, r, tol_rel)
    # absolute part: fp32 accumulation error of the contraction (a few 1e-6 of a typical
    # element) also moves elements whose own magnitude, hence bf16 spacing, is tiny
    sq = sum(float(y @ y) for _, y in _chunks(got, want))
    rms = float(np.sqrt(sq / want.size)) if want.size else 0.0
    n_bad = n_eq = 0
    acc_slack = 3e-5 * rms * max(1.0, float(np.sqrt(k_terms / 1024.0)))
    worst = []
    for x, y in _chunks(got, want):
        slack = bf16_ulp(y) * 1.01 + acc_slack
        bad = np.abs(x - y) > slack
        if bad.any():
            for i in np.flatnonzero(bad)[:3]:
                worst.append((float(x[i]), float(y[i]), float(slack[i])))
        n_bad += int(bad.sum())
        n_eq += int((x == y).sum())
    assert n_bad == 0, "%s: %d elements differ by more than one bf16 spacing (got, want, allowed: %s; rms %.3e)" % (
        what, n_bad, worst[:6], rms)
    eq = n_eq / want.size if want.size else 1.0
    assert eq >= min_equal, "%s: only %.4f of the elements are bit-equal" % (what, eq)
    return r
