"""Shared test plumbing: run a compiled plan on numpy buffers through the library's host interpreter."""
import numpy as np

from paper_2608_00358_b200 import binding as hb

SENTINEL = 0xA5


def np_dtype(dt):
    return np.float32 if dt == hb.FP32 else np.uint16


def interpret(plan, X, seed=0, fill=SENTINEL):
    """X: per-rank numpy arrays (any dtype, C-contiguous). Returns per-rank uint8 receive buffers."""
    info = plan.info()
    Y = []
    for r in range(info.R):
        s, v = plan.extents(r)
        assert X[r].nbytes >= s, (r, X[r].nbytes, s)
        Y.append(np.full(v, fill, dtype=np.uint8))
    scratch = np.full(max(info.scratch_bytes, 1), fill, dtype=np.uint8)
    rc = plan.interpret_host([x.ctypes.data for x in X], [y.ctypes.data for y in Y], scratch.ctypes.data, 0, seed)
    assert rc == hb.OK, hb.status_string(rc)
    return Y


def assert_reduction_close(dt, got, exact_f64, oracle_rounded, what=""):
    """Acceptance rule: fp32 within 1e-5 relative + 1e-6 absolute of the FP64 sum; 16-bit within 1 ulp of
    the directly rounded FP64 sum."""
    from oracle import oracle as orc
    if got.size == 0:
        assert exact_f64.size == 0
        return
    if dt == hb.FP32:
        err = np.abs(got.astype(np.float64) - exact_f64)
        tol = 1e-5 * np.abs(exact_f64) + 1e-6
        assert np.all(err <= tol), (what, float((err - tol).max()))
    else:
        d = orc.ulp_distance(dt, got, oracle_rounded)
        assert d.max() <= 1, (what, int(d.max()), int((d > 1).sum()))
