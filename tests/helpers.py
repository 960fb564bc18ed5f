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


def count_beyond_rule(dt, got, exact_f64, oracle_rounded):
    """Elements of `got` outside the acceptance rule: fp32 within 1e-5 relative + 1e-6 absolute of the FP64 sum,
    16-bit within 1 ulp of the directly rounded FP64 sum. Returns (boolean mask, absolute errors)."""
    from oracle import oracle as orc
    from paper_2608_00358_b200 import synth
    if dt == hb.FP32:
        err = np.abs(got.astype(np.float64) - exact_f64)
        return err > 1e-5 * np.abs(exact_f64) + 1e-6, err
    err = np.abs(synth.from_bits(got, dt) - exact_f64)
    return orc.ulp_distance(dt, got, oracle_rounded) > 1, err


def assert_reduction_close(dt, got, exact_f64, oracle_rounded, what="", X=None, max_beyond=0):
    """The acceptance rule, counted, not widened: the number of elements outside it must not exceed
    `max_beyond`, which is 0 unless the calling test names a reason and a figure of its own. Elements that
    are outside (possible only where the test allows some) must still satisfy the error bound of FP32
    recursive summation, (R-1) * 2^-24 * sum_q |x_q| plus half an ulp of the stored result: the method
    prescribes FP32 adds (Sec. II-A.2), and that is what cancellation to a tiny result can cost.
    Returns the count."""
    from paper_2608_00358_b200 import synth
    if got.size == 0:
        assert exact_f64.size == 0
        return 0
    miss, err = count_beyond_rule(dt, got, exact_f64, oracle_rounded)
    beyond = int(miss.sum())
    assert beyond <= max_beyond, (what, "elements outside the rule: %d, allowed: %d" % (beyond, max_beyond), float(err[miss].max()))
    if beyond:
        assert X is not None, what
        idx = np.nonzero(miss)[0]
        abs_sum = sum(np.abs(synth.from_bits(x[idx], dt)) for x in X)
        g = synth.from_bits(got[idx], dt)
        half_ulp = np.maximum(np.abs(g), 2.0 ** -126) * 2.0 ** -(24 if dt == hb.FP32 else (8 if dt == hb.BF16 else 11))
        bound = half_ulp + (len(X) - 1) * 2.0 ** -24 * abs_sum
        assert np.all(err[idx] <= bound), (what, float((err[idx] - bound).max()))
    return beyond
