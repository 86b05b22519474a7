"""Acceptance rules for comparing CUDA results with the oracle (test helpers)."""
import numpy as np


def ordered16(bits):
    """Map binary16 bit patterns to integers that are monotone in value (+0 == -0)."""
    b = np.asarray(bits).astype(np.int32)
    mag = b & 0x7FFF
    return np.where(b & 0x8000, -mag, mag)


def half_value(bits):
    return np.asarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


def gemm_accept(got_bits, ref_bits, K=None, absdot=None, exact=None):
    """Element-wise acceptance of an FP16 result computed with FP32 accumulation in an
    unspecified order against the oracle's ascending-order FP32 sum.  Passes if any holds:
    same non-finite class; <= 2 FP16 ulp apart; within 1e-2 relative; (cancellation
    near zero) within the a-priori bound 2*K*2^-23*sum|a*b| that holds for any FP32
    summation order; or (overflow on the store) one side is the largest finite FP16 value and the
    other the infinity of the same sign, which is what two FP32 sums on either side of the
    rounding threshold 65520 give - accepted only when the caller passes the exact sum and that
    sum lies within the same a-priori bound of 65520 (so that both results are roundings of sums
    an FP32 summation order can legitimately produce), and the two results are neighbours in the
    ordering of FP16 values.  Returns (ok mask, stats dict)."""
    g = np.asarray(got_bits, dtype=np.uint16)
    r = np.asarray(ref_bits, dtype=np.uint16)
    gv, rv = half_value(g), half_value(r)
    g_nan, r_nan = np.isnan(gv), np.isnan(rv)
    g_inf, r_inf = np.isinf(gv), np.isinf(rv)
    same_nonfinite = (g_nan & r_nan) | (g_inf & r_inf & (np.sign(gv) == np.sign(rv)))
    finite = ~(g_nan | r_nan | g_inf | r_inf)
    ulp = np.abs(ordered16(g) - ordered16(r))
    with np.errstate(invalid="ignore"):
        c_ulp = finite & (ulp <= 2)
        c_rel = finite & (np.abs(gv - rv) <= 1e-2 * np.abs(rv))
        if absdot is not None and K is not None:
            c_abs = finite & (np.abs(gv - rv) <= 2.0 * K * 2.0 ** -23 * np.asarray(absdot) + 2.0 ** -24)
        else:
            c_abs = np.zeros_like(finite)
    # 0x7BFF (65504) against 0x7C00 (inf), same sign: adjacent codes, and the exact sum close
    # enough to the rounding threshold for a change of summation order to cross it
    if exact is not None and absdot is not None and K is not None:
        near = np.abs(np.abs(np.asarray(exact, dtype=np.float64)) - 65520.0) <= 2.0 * K * 2.0 ** -23 * np.asarray(absdot)
        edge = (g_inf ^ r_inf) & ~(g_nan | r_nan) & (ulp == 1) & near
    else:
        edge = np.zeros_like(finite)
    ok = same_nonfinite | c_ulp | c_rel | c_abs | edge
    stats = dict(n=int(g.size), exact=int((g == r).sum()), max_ulp=int(ulp[finite].max()) if finite.any() else 0,
                 by_ulp=int(c_ulp.sum()), by_rel_only=int((c_rel & ~c_ulp).sum()),
                 by_abs_only=int((c_abs & ~c_ulp & ~c_rel).sum()), overflow_edge=int(edge.sum()), failed=int((~ok).sum()))
    return ok, stats
