"""Comparators of the GPU parity tests for the two places where a result is not unique: a code
that follows an order-dependent floating-point reduction (LayerNorm statistics, softmax sums)
may legitimately land on either side of a rounding boundary.  Everything else is compared byte
for byte, stage by stage, each stage fed the GPU's own upstream bytes (stage isolation).

near_tie_codes      : codes differ by at most one, and only where the fp64 pre-rounding value lies
                      within tau of a half-integer.
attention_codes_valid: the fused attention kernels never materialise P = round(127 p).  Every P code
                      whose fp64 value 127 p lies within tau of a half-integer may be either
                      neighbour; all others are fixed.  The INT32 sums P.V that such a family of P
                      matrices can produce form, per output element, an interval (each ambiguous
                      code moves the sum by +-V); Eq. 2 and the final rounding are monotone, so the
                      valid output codes are an interval too, and the GPU's code must lie in it.
"""
import numpy as np

import oracle

TAU_LN = 127 * 2.0 ** -16    # fp32 LayerNorm statistics in another summation order
TAU_P = 127 * 2.0 ** -18     # fp32 exp / row sum in another order and with another exp routine


def near_tie_codes(q_gpu, q_or, v64, tau, what="codes"):
    """v64: the exact (fp64) value whose rounding the codes are, same shape.  Returns the fraction
    of codes that differ (all of them within tau of a tie, else the assertion fails)."""
    q_gpu = np.asarray(q_gpu).astype(np.int32)
    q_or = np.asarray(q_or).astype(np.int32)
    diff = q_gpu != q_or
    if not diff.any():
        return 0.0
    assert np.abs(q_gpu - q_or).max() <= 1, "%s differ by more than one" % what
    v = np.asarray(v64, np.float64)[diff]
    dist = np.abs(np.abs(v - np.floor(v)) - 0.5)
    assert np.all(dist <= tau), "%s: a code differs %.3g away from a rounding boundary (tau %.3g)" % (what, dist.max(), tau)
    # and the GPU's code is one of the two neighbours of the exact value
    assert np.all(np.abs(q_gpu[diff] - np.asarray(v64, np.float64)[diff]) <= 0.5 + tau)
    return float(diff.mean())


def ln_codes_near_tie(q_gpu, q_or, x, gamma_hat, beta_hat, eps, delta, what="LayerNorm codes"):
    """q_gpu against the oracle's codes q_or, ties judged on the fp64 LayerNorm of x divided by the
    step (delta: scalar or one step per row)."""
    y64 = oracle.ln_f64(x, np.asarray(gamma_hat, np.float64), None if beta_hat is None else np.asarray(beta_hat, np.float64), eps)
    d = np.asarray(delta, np.float64).reshape(-1)
    v = y64 / (d[:, None] if d.size == y64.shape[0] and d.size > 1 else float(d[0]))
    vc = np.clip(v, -127.0, 127.0)  # saturated values are nowhere near a tie
    return near_tie_codes(q_gpu, q_or, vc, TAU_LN, what)


def _softmax_rows_f64(scores, visible):
    """fp64 softmax of each row over its first visible[i] keys (plain definition)."""
    s = np.asarray(scores, np.float64)
    n_rows, n_keys = s.shape
    mask = np.arange(n_keys)[None, :] < np.asarray(visible)[:, None]
    s = np.where(mask, s, -np.inf)
    e = np.exp(s - s.max(axis=1, keepdims=True))
    return e / e.sum(axis=1, keepdims=True)


def attention_codes_valid(got, scores, visible, V, alpha_pv, requant_mul=None, out_dtype=None, tau=TAU_P, P_oracle=None):
    """got [rows, d]: the kernel's output for one (sequence, head); scores [rows, keys]: the exact
    fp32 scores (INT32 accumulators times alpha_qk, from the oracle on the same codes); visible[i]:
    keys row i attends over; V [keys, d] INT8.  Output either INT8 codes (requant_mul given) or
    16-bit floats (out_dtype).  P_oracle: the oracle's P codes of the same rows, cross-checked.
    Returns (fraction of P codes that are ambiguous, fraction of output elements with more than one
    valid value, fraction of outputs that differ from the oracle's own)."""
    p64 = _softmax_rows_f64(scores, visible)
    v127 = 127.0 * p64
    lo = np.floor(v127)
    near = np.abs((v127 - lo) - 0.5) <= tau
    P_or = np.rint(v127).astype(np.int64)           # the fixed codes; at ambiguous positions one of the two neighbours
    if P_oracle is not None:  # the oracle's own (fp32) codes agree with the definition wherever the definition is unambiguous
        assert np.array_equal(np.asarray(P_oracle).astype(np.int64)[~near], P_or[~near])
    alt = np.where(P_or == lo, lo + 1, lo).astype(np.int64)
    delta = np.where(near, alt - P_or, 0)            # +-1 where the other neighbour is valid too
    # integer sums through float64 matrix products: every partial sum is an integer below 2^53, so they are exact
    V64 = np.asarray(V).astype(np.float64)
    acc0 = np.rint(P_or.astype(np.float64) @ V64).astype(np.int64)
    vp, vn = np.maximum(V64, 0), np.maximum(-V64, 0)
    dp, dn = (delta > 0).astype(np.float64), (delta < 0).astype(np.float64)
    up = np.rint(dp @ vp + dn @ vn).astype(np.int64)
    down = np.rint(dp @ vn + dn @ vp).astype(np.int64)
    acc_lo, acc_hi = (acc0 - down).astype(np.int32), (acc0 + up).astype(np.int32)

    def finish(acc):
        y = oracle.scale_acc(acc, float(alpha_pv))
        return oracle.requant(y, requant_mul).astype(np.float64) if requant_mul is not None else oracle.round_to(y, out_dtype).astype(np.float64)
    out_lo, out_hi, out0 = finish(acc_lo), finish(acc_hi), finish(acc0.astype(np.int32))
    g = np.asarray(got, np.float64)
    bad = (g < out_lo) | (g > out_hi)
    assert not bad.any(), "%d of %d attention outputs outside the valid interval (worst by %.3g)" % (
        bad.sum(), bad.size, np.maximum(out_lo - g, g - out_hi).max())
    return float(near.mean()), float((out_lo != out_hi).mean()), float((g != out0).mean())
