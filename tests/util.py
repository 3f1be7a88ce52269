"""Helpers shared by the GPU parity tests: transfers and the error metrics of the tolerance."""
import numpy as np

# relative L2 error allowed against the fp64 oracle, per accuracy class, and the
# max-abs bound as a fraction of max|y_ref|
TOL_REL_L2 = {0: 1e-3, 1: 1e-2}
TOL_MAX_ABS_FRAC = 2e-2


def rel_l2(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref.ravel())
    return float(np.linalg.norm((got - ref).ravel()) / den) if den > 0 else float(np.linalg.norm(got.ravel()))


def max_abs_frac(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    m = np.abs(ref).max()
    return float(np.abs(got - ref).max() / m) if m > 0 else float(np.abs(got).max())


def assert_close(got, ref, precision_class, what=""):
    e, a = rel_l2(got, ref), max_abs_frac(got, ref)
    assert np.isfinite(np.asarray(got)).all(), what + ": non-finite output"
    assert e <= TOL_REL_L2[precision_class], "%s: relL2 %.3e > %.1e" % (what, e, TOL_REL_L2[precision_class])
    assert a <= TOL_MAX_ABS_FRAC, "%s: max-abs %.3e of max|y_ref|" % (what, a)
    return e, a


def to_dev(torch, a, device="cuda:0"):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(device)
