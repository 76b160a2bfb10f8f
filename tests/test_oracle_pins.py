"""Pins for the CPU oracle: everything here checks the oracle against something that is
NOT the oracle -- hand-evaluated values, closed forms, invariants the paper states, library
routines (torch CPU in fp64) and brute force written independently in this file."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, val = line.split(":", 1)
            rows = [[float(v) for v in r.split()] for r in val.split(";")]
            out[key.strip()] = np.array(rows if len(rows) > 1 else rows[0])
    return out


# --------------------------------------------------------------------------- #
# Worked example (Eq. 3, Eq. 4 at alpha = 0.5, Eq. 1 per token)
# --------------------------------------------------------------------------- #
def test_worked_example_alpha05():
    g = _read_golden("worked_example_alpha05.txt")
    X = g["X"].astype(np.float32)
    W_stored = g["W"].T.astype(np.float32).copy()  # stored [C_o, C_i]
    ax = oracle.calib_absmax(X)
    aw = oracle.calib_absmax(W_stored)
    assert np.array_equal(ax, g["act_absmax"])
    assert np.array_equal(aw, g["w_absmax"])
    s = oracle.smooth_scales(ax, aw, 0.5)
    assert np.array_equal(s, g["s"])
    Xh = X / s
    assert np.array_equal(Xh, g["X_hat"])
    # W_hat through the weight quantiser's folding: dequantised codes reproduce diag(s) W
    Wq, ws = oracle.quant_weight(W_stored, s, "per_channel")
    What = g["W_hat"].T  # stored orientation
    assert np.allclose(Wq * ws[:, None], What, atol=np.abs(What).max() / 127 / 2 + 1e-6)
    assert np.array_equal(oracle.calib_absmax(Xh), g["smoothed_absmax"])
    assert np.array_equal(np.abs(What).max(axis=0), g["smoothed_absmax"])
    assert np.array_equal(oracle.linear_f64(Xh, What), g["Y"])
    assert np.array_equal(oracle.linear_f64(X, W_stored), g["Y"])
    q, d = oracle.quant_act(Xh, "per_token")
    assert np.array_equal(q, g["X_hat_q"].astype(np.int8))
    assert np.allclose(d, np.array([4.0, 3.0]) / 127.0, rtol=1e-7)


# --------------------------------------------------------------------------- #
# Eq. 3: smoothing is an exact identity
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("alpha", [0.0, 0.3, 0.5, 0.75, 1.0])
def test_smoothing_equivalence_fp64(alpha):
    rng = np.random.default_rng(7)
    X = rng.standard_normal((9, 33))
    X[:, [3, 17]] *= 60.0
    W = rng.standard_normal((21, 33)) * 0.02
    s = oracle.smooth_scales(np.abs(X).max(0), np.abs(W).max(0), alpha).astype(np.float64)
    Y = oracle.linear_f64(X, W)
    Ys = oracle.linear_f64(X / s, W * s)
    assert np.abs(Ys - Y).max() / np.abs(Y).max() <= 1e-10


# --------------------------------------------------------------------------- #
# Eq. 4: closed forms at the end points and at alpha = 0.5
# --------------------------------------------------------------------------- #
def test_smooth_scales_closed_forms():
    rng = np.random.default_rng(11)
    X = rng.standard_normal((64, 48)).astype(np.float32)
    X[:, 5] *= 70
    W = (rng.standard_normal((40, 48)) * 0.02).astype(np.float32)
    ax, aw = np.abs(X).max(0), np.abs(W).max(0)
    # alpha = 1: s_j = max|X_j|  -> every smoothed activation channel has maximum 1
    s1 = oracle.smooth_scales(ax, aw, 1.0)
    assert np.array_equal(s1, ax)
    assert np.allclose(np.abs(X / s1).max(0), 1.0, rtol=1e-6)
    # alpha = 0: s_j = 1 / max|W_j|  -> every smoothed weight input channel has maximum 1
    s0 = oracle.smooth_scales(ax, aw, 0.0)
    assert np.allclose(s0, 1.0 / aw.astype(np.float64), rtol=1e-7)
    assert np.allclose(np.abs(W * s0).max(0), 1.0, rtol=1e-6)
    # alpha = 0.5: both sides share sqrt(ax * aw); pow pinned against sqrt
    sh = oracle.smooth_scales(ax, aw, 0.5)
    ref = np.sqrt(ax.astype(np.float64) / aw.astype(np.float64))
    assert np.allclose(sh, ref, rtol=1e-7)
    both = np.sqrt(ax.astype(np.float64) * aw)
    assert np.allclose(np.abs(X / sh).max(0), both, rtol=1e-6)
    assert np.allclose(np.abs(W * sh).max(0), both, rtol=1e-6)
    # general alpha: max|X_hat_j| = ax^(1-a) aw^(1-a), max|W_hat_j| = ax^a aw^a
    a = 0.75
    sa = oracle.smooth_scales(ax, aw, a).astype(np.float64)
    assert np.allclose(ax / sa, ax.astype(np.float64) ** (1 - a) * aw.astype(np.float64) ** (1 - a),
                       rtol=1e-6)
    assert np.allclose(aw * sa, ax.astype(np.float64) ** a * aw.astype(np.float64) ** a, rtol=1e-6)


def test_smooth_scales_floor_and_range():
    s = oracle.smooth_scales(np.array([0.0, 4.0], np.float32), np.array([4.0, 0.0], np.float32), 0.5)
    assert np.all(np.isfinite(s)) and np.all(s > 0)
    assert np.allclose(s, [np.sqrt(1e-5 / 4.0), np.sqrt(4.0 / 1e-5)], rtol=1e-6)
    with pytest.raises(ValueError):
        oracle.smooth_scales(np.ones(2, np.float32), np.ones(2, np.float32), 1.5)


# --------------------------------------------------------------------------- #
# Eq. 1: the quantiser
# --------------------------------------------------------------------------- #
def test_quantizer_ties_and_clamp():
    # Delta = 1 exactly when the maximum is 127: ties go to the even neighbour
    v = np.array([[127, 62.5, 0.5, -0.5, 1.5, -2.5, 63.5, -126.5]], np.float32)
    q, d = oracle.quant_act(v, "per_token")
    assert d[0] == 1.0
    assert q.tolist() == [[127, 62, 0, 0, 2, -2, 64, -126]]
    # static step calibrated at half the runtime maximum saturates at +-127
    q2, _ = oracle.quant_act(np.array([[254.0, -300.0, 63.4]], np.float32), "per_tensor_static",
                             static_scale=np.float32(1.0))
    assert q2.tolist() == [[127, -127, 63]]


def test_quantizer_properties():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((37, 129)).astype(np.float32)
    x[:, 9] *= 55
    q, d = oracle.quant_act(x, "per_token")
    # the maximum element of every row maps to +-127, zero to zero, odd symmetry
    idx = np.abs(x).argmax(1)
    assert np.all(np.abs(q[np.arange(37), idx]) == 127)
    assert np.all(np.abs(q) <= 127)
    qn, dn = oracle.quant_act(-x, "per_token")
    assert np.array_equal(qn, -q) and np.array_equal(dn, d)
    z, _ = oracle.quant_act(np.zeros((2, 8), np.float32), "per_token")
    assert not z.any()
    # rounding error is at most half a step
    err = np.abs(x.astype(np.float64) - q.astype(np.float64) * d[:, None].astype(np.float64))
    assert np.all(err <= d[:, None] / 2 * (1 + 1e-5))
    # idempotence: quantising the dequantised codes with the same step returns the codes
    deq = (q.astype(np.float32) * d[:, None]).astype(np.float32)
    assert np.array_equal(oracle.quantize(deq, d, True), q)
    # independent restatement of Eq. 1 in fp64 agrees except at (rare) near-ties, by one code
    lit = oracle.quantize_f64_literal(x, d, True)
    diff = (lit.astype(np.int32) - q.astype(np.int32))
    assert np.abs(diff).max() <= 1 and (diff != 0).mean() < 1e-3
    # and against numpy written out here
    ref = np.clip(np.rint(x.astype(np.float64) / d[:, None].astype(np.float64)), -127, 127)
    assert np.array_equal(lit, ref.astype(np.int8))


def test_granularity_cross_checks():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((16, 64)).astype(np.float32)
    # static step calibrated on the same tensor == per-tensor dynamic
    qd, dd = oracle.quant_act(x, "per_tensor_dynamic")
    qs, ds = oracle.quant_act(x, "per_tensor_static", static_scale=np.float32(np.abs(x).max()) / np.float32(127))
    assert np.array_equal(qd, qs) and dd[0] == ds[0]
    assert dd[0] == np.float32(np.abs(x).max()) / np.float32(127)
    # per-token == per-tensor when every row has the same maximum
    x2 = x.copy()
    x2[:, 0] = 9.0
    qt, dt = oracle.quant_act(x2, "per_token")
    qp, dp = oracle.quant_act(x2, "per_tensor_dynamic")
    assert np.array_equal(qt, qp) and np.all(dt == dp[0])
    # per-channel weight == per-tensor weight when all rows of W_hat share one maximum
    w = (rng.standard_normal((8, 64)) * 0.02).astype(np.float32)
    w[:, 3] = 0.5
    qc, dc = oracle.quant_weight(w, None, "per_channel")
    qt2, dt2 = oracle.quant_weight(w, None, "per_tensor")
    assert np.array_equal(qc, qt2) and np.all(dc == dt2[0])
    # explicit per-channel multiplier == pre-multiplied input
    cm = rng.uniform(0.1, 2.0, 64).astype(np.float32)
    qa, da = oracle.quant_act(x, "per_token", col_mul=cm)
    qb, db = oracle.quant_act((x * cm).astype(np.float32), "per_token")
    assert np.array_equal(qa, qb) and np.array_equal(da, db)


def test_calib_absmax_running_max_and_fold():
    rng = np.random.default_rng(13)
    batches = [rng.standard_normal((10, 24)).astype(np.float32) for _ in range(4)]
    a = None
    for b in batches:
        a = oracle.calib_absmax(b, a)
    assert np.array_equal(a, np.abs(np.concatenate(batches)).max(0))
    # fold: gamma/s and beta/s, rounded to the parameter dtype
    gamma = (1 + 0.1 * rng.standard_normal(24)).astype(np.float16).astype(np.float32)
    beta = (0.1 * rng.standard_normal(24)).astype(np.float16).astype(np.float32)
    s = rng.uniform(0.5, 9.0, 24).astype(np.float32)
    gh, bh = oracle.fold_ln_weight(gamma, beta, s, "f16")
    assert np.array_equal(gh, (gamma / s).astype(np.float16).astype(np.float32))
    assert np.array_equal(bh, (beta / s).astype(np.float16).astype(np.float32))
    gb, _ = oracle.fold_ln_weight(gamma, None, s, "bf16")
    t = torch.from_numpy(gamma / s).to(torch.bfloat16).float().numpy()
    assert np.array_equal(gb, t)


def test_round_to_bf16_is_rne_on_bits():
    # re-derive bf16 RNE on the bit pattern, independent of the library cast
    rng = np.random.default_rng(17)
    y = (rng.standard_normal(4096) * 37).astype(np.float32)
    y[:4] = [1.00390625, 1.01171875, -1.00390625, 3.0]  # exact ties: 1+2^-8 -> 1, 1+3*2^-8 -> 1+2^-6
    u = y.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    ref = r.astype(np.uint32).view(np.float32)
    assert np.array_equal(oracle.round_to(y, "bf16"), ref)


# --------------------------------------------------------------------------- #
# LayerNorm and its folding
# --------------------------------------------------------------------------- #
def test_layernorm_against_torch_fp64():
    rng = np.random.default_rng(19)
    x = rng.standard_normal((12, 96)).astype(np.float32)
    x[:, 7] *= 40
    gamma = 1 + 0.1 * rng.standard_normal(96)
    beta = 0.1 * rng.standard_normal(96)
    y = oracle.ln_f64(x, gamma, beta, 1e-5)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x).double(), (96,),
                                         torch.from_numpy(gamma), torch.from_numpy(beta), 1e-5)
    assert np.abs(y - ref.numpy()).max() <= 1e-12
    # folding: LN(x; gamma/s, beta/s) = LN(x; gamma, beta) / s
    s = rng.uniform(0.3, 8.0, 96)
    yf = oracle.ln_f64(x, gamma / s, beta / s, 1e-5)
    assert np.abs(yf - y / s).max() <= 1e-12
    # normative fp32 element-wise path stays within fp32 rounding of the fp64 result
    mu, rstd = oracle.ln_stats(x, 1e-5)
    y32 = oracle.ln_apply(x, mu.astype(np.float32), rstd.astype(np.float32),
                          gamma.astype(np.float32), beta.astype(np.float32))
    assert np.abs(y32 - y).max() <= 1e-4 * max(1.0, np.abs(y).max())
    # ln_quant == quant_act(ln_apply)
    q, d, yy = oracle.ln_quant(x, gamma.astype(np.float32), beta.astype(np.float32), 1e-5, "per_token")
    q2, d2 = oracle.quant_act(y32, "per_token")
    assert np.array_equal(q, q2) and np.array_equal(d, d2) and np.array_equal(yy, y32)


@pytest.mark.parametrize("mean_over_sigma", [0.0, 10.0, 100.0])
def test_ln_apply_error_bound_on_rows_with_a_large_mean(mean_over_sigma):
    """The normative fp32 element-wise LayerNorm is n = fma(x, rstd, -(mu * rstd)), y = fma(n, g, b).
    Its rounding error against the same expression in exact arithmetic is bounded, per element, by
        2^-24 * [ (|mu * rstd| + |n|) * |g| + |y| ]            (one rounding each: the product mu * rstd,
                                                                n, and y)
    which grows with |mu| / sigma.  Pinned here on rows whose mean is 0, 10 and 100 standard deviations
    away from zero, (a) against fp64 evaluation with the SAME fp32 statistics (isolates the element-wise
    path), (b) against the fp64 LayerNorm with its own fp64 statistics, where the fp32 rounding of mu and
    rstd alone may contribute (|mu * rstd| + |n|) * |g| * 2^-24 more.  A wrong sign, a dropped shift or
    a swapped operand is off by ~|mu| / sigma and fails at once."""
    rng = np.random.default_rng(1905 + int(mean_over_sigma))
    C = 512
    sigma = 0.75
    x = (mean_over_sigma * sigma + sigma * rng.standard_normal((24, C))).astype(np.float16).astype(np.float32)
    g = (1 + 0.1 * rng.standard_normal(C)).astype(np.float16).astype(np.float32)
    b = (0.1 * rng.standard_normal(C)).astype(np.float16).astype(np.float32)
    mu, rstd = oracle.ln_stats(x, 1e-5)
    mu32, rstd32 = mu.astype(np.float32), rstd.astype(np.float32)
    assert abs(np.abs(mu * rstd).mean() - mean_over_sigma) <= 0.1 * mean_over_sigma + 0.2  # the rows are what they claim
    y32 = oracle.ln_apply(x, mu32, rstd32, g, b).astype(np.float64)
    u = 2.0 ** -24
    x64, g64, b64 = x.astype(np.float64), g.astype(np.float64), b.astype(np.float64)
    # (a) same fp32 statistics, exact arithmetic
    m64, r64 = mu32.astype(np.float64)[:, None], rstd32.astype(np.float64)[:, None]
    n_same = x64 * r64 - m64 * r64
    y_same = n_same * g64 + b64
    bound_a = 1.01 * u * ((np.abs(m64 * r64) + np.abs(n_same)) * np.abs(g64) + np.abs(y_same))
    assert np.all(np.abs(y32 - y_same) <= bound_a)
    # (b) the fp64 LayerNorm (own statistics): add the rounding of mu and rstd to fp32
    y_true = oracle.ln_f64(x, g64, b64, 1e-5)
    n_true = (x64 - mu[:, None]) * rstd[:, None]
    bound_b = bound_a + 1.01 * u * (np.abs(mu * rstd)[:, None] + 2 * np.abs(n_true)) * np.abs(g64)
    assert np.all(np.abs(y32 - y_true) <= bound_b)
    # the bound is what it says: of the order of (1 + |mu| / sigma) * 2^-24, far below a quantisation step
    assert bound_b.max() <= (mean_over_sigma + 8) * 4 * u
    # in code units: even at |mu| / sigma = 100 the error moves a value by < 1e-3 of a quantisation step
    step = np.abs(y_true).max(axis=1, keepdims=True) / 127.0
    assert (np.abs(y32 - y_true) / step).max() <= 1e-3


# --------------------------------------------------------------------------- #
# INT8 GEMM
# --------------------------------------------------------------------------- #
def test_gemm_i32_brute_force_and_closed_forms():
    rng = np.random.default_rng(23)
    Xq = rng.integers(-127, 128, (7, 50), dtype=np.int8)
    Wq = rng.integers(-127, 128, (11, 50), dtype=np.int8)
    acc = oracle.gemm_i32(Xq, Wq)
    ref = np.zeros((7, 11), np.int64)
    for t in range(7):
        for o in range(11):
            for j in range(50):
                ref[t, o] += int(Xq[t, j]) * int(Wq[o, j])
    assert np.array_equal(acc, ref)
    # library routine (int64 matmul)
    assert np.array_equal(acc, Xq.astype(np.int64) @ Wq.astype(np.int64).T)
    # not symmetric in its operands: a transposed-operand mistake fails here
    assert acc.shape == (7, 11)
    # B stored [K, N]
    assert np.array_equal(oracle.gemm_i32_bt(Xq, np.ascontiguousarray(Wq.T)), ref)
    # all-127 inputs: acc = 16129 K ; W = 127 I: acc = 127 X
    K = 512
    ones = np.full((3, K), 127, np.int8)
    assert np.all(oracle.gemm_i32(ones, np.full((5, K), 127, np.int8)) == 16129 * K)
    eye = (127 * np.eye(50)).astype(np.int8)
    assert np.array_equal(oracle.gemm_i32(Xq, eye), 127 * Xq.astype(np.int32))
    # largest supported K keeps |acc| inside int32; one more block of K would not
    Kmax = 133144
    big = oracle.gemm_i32(np.full((1, Kmax), 127, np.int8), np.full((1, Kmax), -127, np.int8))
    assert big[0, 0] == -16129 * Kmax
    with pytest.raises(OverflowError):
        oracle.gemm_i32(np.full((1, Kmax + 16), 127, np.int8), np.full((1, Kmax + 16), 127, np.int8))


# --------------------------------------------------------------------------- #
# Eq. 2: dequantisation
# --------------------------------------------------------------------------- #
def test_dequant_exact_grid():
    # X = sx_t * A, W = sw_o * B with integer A, B in [-127, 127] and a +-127 in every row:
    # quantisation is lossless and Y = sx_t sw_o (A B^T) exactly
    rng = np.random.default_rng(29)
    A = rng.integers(-127, 128, (6, 40)).astype(np.int64)
    B = rng.integers(-127, 128, (9, 40)).astype(np.int64)
    A[:, 0] = 127
    B[:, 1] = -127
    sx = np.array([2.0 ** -k for k in range(6)])  # powers of two keep X exactly representable
    sw = np.array([2.0 ** -(k + 3) for k in range(9)])
    X = (A * sx[:, None]).astype(np.float32)
    W = (B * sw[:, None]).astype(np.float32)
    Xq, dx = oracle.quant_act(X, "per_token")
    Wq, dw = oracle.quant_weight(W, None, "per_channel")
    assert np.array_equal(Xq, A.astype(np.int8)) and np.array_equal(Wq, B.astype(np.int8))
    bias = rng.standard_normal(9).astype(np.float32)
    acc, y = oracle.w8a8_linear(Xq, dx, Wq, dw, bias=bias, out_dtype="f32")
    assert np.array_equal(acc, A @ B.T)
    truth = (A @ B.T) * sx[:, None] * sw[None, :] + bias[None, :]
    assert np.abs(y - truth).max() <= 1e-6 * np.abs(truth).max()
    # ReLU and the order of the outer scalings (rows get Delta_x, columns get Delta_w)
    _, yr = oracle.w8a8_linear(Xq, dx, Wq, dw, bias=bias, relu=True, out_dtype="f32")
    assert np.array_equal(yr, np.maximum(y, 0))
    y_nob = oracle.dequant(acc, dx, dw)
    assert np.allclose(y_nob, acc * dx[:, None].astype(np.float64) * dw[None, :], rtol=1e-6)


def test_dequant_error_bound_generic():
    # |Y_q - Y_fp| <= sum_j (|x_j| Dw/2 + |w_j| Dx/2 + Dx Dw/4) for unclamped rounding
    rng = np.random.default_rng(31)
    X = rng.standard_normal((8, 200)).astype(np.float32)
    X[:, 4] *= 50
    W = (rng.standard_normal((12, 200)) * 0.02).astype(np.float32)
    Xq, dx = oracle.quant_act(X, "per_token")
    Wq, dw = oracle.quant_weight(W, None, "per_channel")
    _, y = oracle.w8a8_linear(Xq, dx, Wq, dw, out_dtype="f32")
    truth = oracle.linear_f64(X, W)
    bound = (np.abs(X).sum(1)[:, None] * dw[None, :] / 2 + np.abs(W).sum(1)[None, :] * dx[:, None] / 2
             + 200 * dx[:, None] * dw[None, :] / 4)
    assert np.all(np.abs(y - truth) <= bound * (1 + 1e-4) + 1e-6)
    # requant: codes of y with a static multiplier
    r = np.float32(3.7)
    assert np.array_equal(oracle.requant(y, r), np.clip(np.rint(y * r), -127, 127).astype(np.int8))


def test_smoothing_helps_quantisation_error():
    # The method's point (Section 4): with outlier channels, W8A8 error after smoothing is far
    # below the unsmoothed error.  A sign or direction mistake in Eq. 3/4 reverses this.
    rng = np.random.default_rng(37)
    X = rng.standard_normal((32, 256)).astype(np.float32)
    X[:, [10, 99, 200]] *= 80
    W = (rng.standard_normal((64, 256)) * 0.02).astype(np.float32)
    truth = oracle.linear_f64(X, W)

    def w8a8(Xi, Wi):
        Xq, dx = oracle.quant_act(Xi, "per_tensor_dynamic")
        Wq, dw = oracle.quant_weight(Wi, None, "per_tensor")
        return oracle.w8a8_linear(Xq, dx, Wq, dw, out_dtype="f32")[1]

    e_naive = np.abs(w8a8(X, W) - truth).mean()
    s = oracle.smooth_scales(oracle.calib_absmax(X), oracle.calib_absmax(W), 0.5)
    e_smooth = np.abs(w8a8((X / s).astype(np.float32), (W * s).astype(np.float32)) - truth).mean()
    assert e_smooth < 0.35 * e_naive


# --------------------------------------------------------------------------- #
# Attention plumbing
# --------------------------------------------------------------------------- #
def test_softmax_causal_and_bmm():
    rng = np.random.default_rng(41)
    S = (rng.standard_normal((16, 16)) * 3).astype(np.float16).astype(np.float32)
    P = oracle.softmax_causal(S)
    assert np.allclose(P.sum(1), 1.0, atol=1e-6)
    assert not np.triu(P, 1).any()
    mask = torch.full((16, 16), float("-inf"), dtype=torch.float64).triu(1)
    ref = torch.softmax(torch.from_numpy(S).double() + mask, -1).numpy()
    assert np.abs(oracle.softmax_causal_f64(S) - ref).max() <= 1e-14
    assert np.abs(P - ref).max() <= 1e-6
    Pq, _ = oracle.softmax_quant_p(S)
    assert np.abs(Pq - np.rint(ref * 127)).max() <= 1 and Pq[0, 0] == 127
    # batched products against int64 einsum
    A = rng.integers(-127, 128, (2, 3, 8, 32), dtype=np.int8)
    B = rng.integers(-127, 128, (2, 3, 10, 32), dtype=np.int8)
    acc, out = oracle.w8a8_bmm(A, B, 0.001, out_dtype="f16")
    assert np.array_equal(acc, np.einsum("bhik,bhjk->bhij", A.astype(np.int64), B.astype(np.int64)))
    assert np.array_equal(out, (acc.astype(np.float32) * np.float32(0.001)).astype(np.float16).astype(np.float32))
    V = rng.integers(-127, 128, (2, 3, 32, 12), dtype=np.int8)
    acc2, q2 = oracle.w8a8_bmm(A, V, 0.002, b_is_kn=True, requant_mul=np.float32(1.5))
    ref2 = np.einsum("bhik,bhkj->bhij", A.astype(np.int64), V.astype(np.int64))
    assert np.array_equal(acc2, ref2)
    y = (ref2.astype(np.float32) * np.float32(0.002)) * np.float32(1.5)
    assert np.array_equal(q2, np.clip(np.rint(y), -127, 127).astype(np.int8))


# --------------------------------------------------------------------------- #
# Generation-stage attention over an INT8 KV cache
# --------------------------------------------------------------------------- #
def test_softmax_prefix_reduces_to_causal_and_to_library_softmax():
    rng = np.random.default_rng(43)
    S = (rng.standard_normal((12, 12)) * 4).astype(np.float32)
    assert np.array_equal(oracle.softmax_prefix(S, 1), oracle.softmax_causal(S))
    # one row that sees every key = the last row of the causal softmax = a plain softmax
    last = oracle.softmax_prefix(S[-1:], 12)
    assert np.array_equal(last[0], oracle.softmax_causal(S)[-1])
    ref = torch.softmax(torch.from_numpy(S[-1:]).double(), -1).numpy()
    assert np.abs(last - ref).max() <= 1e-6
    # a shorter prefix leaves the tail at zero and still sums to one
    P5 = oracle.softmax_prefix(S[:1], 5)
    assert not P5[0, 5:].any() and abs(P5.sum() - 1.0) <= 1e-6
    # softmax is invariant under a common shift of the scores
    assert np.abs(oracle.softmax_prefix(S[:1] + 3.0, 12) - oracle.softmax_prefix(S[:1], 12)).max() <= 1e-6


def test_kv_decode_attention_is_the_last_row_of_prompt_attention():
    """Incremental decoding must give what the prompt pass gives for its last token: the same q,
    the same keys and values, every position visible."""
    rng = np.random.default_rng(44)
    B, H, L, d = 2, 3, 37, 16
    q = rng.integers(-100, 101, (B, H, L, d), dtype=np.int8)
    K = rng.integers(-100, 101, (B, H, L, d), dtype=np.int8)
    V = rng.integers(-100, 101, (B, H, L, d), dtype=np.int8)
    a_qk, a_pv, r = np.float32(0.004), np.float32(0.01 / 127), np.float32(1 / 0.004)
    _, scores = oracle.w8a8_bmm(q, K, a_qk, out_dtype="f32")
    want = np.empty((B, H, d), np.int8)
    for b in range(B):
        for h in range(H):
            Pq, _ = oracle.softmax_quant_p(scores[b, h])
            _, o = oracle.w8a8_bmm(Pq, V[b, h], a_pv, b_is_kn=True, requant_mul=r)
            want[b, h] = o[-1]
    got, _ = oracle.kv_decode_attention(q[:, :, -1], K, V, [L, L], a_qk, a_pv, requant_mul=r)
    assert np.array_equal(got, want)
    # a shorter valid length ignores everything stored beyond it
    got_short, _ = oracle.kv_decode_attention(q[:, :, -1], K, V, [20, 9], a_qk, a_pv, requant_mul=r)
    K2, V2 = K.copy(), V.copy()
    K2[0, :, 20:], V2[0, :, 20:], K2[1, :, 9:], V2[1, :, 9:] = 99, -99, -99, 99
    got_short2, _ = oracle.kv_decode_attention(q[:, :, -1], K2, V2, [20, 9], a_qk, a_pv, requant_mul=r)
    assert np.array_equal(got_short, got_short2) and not np.array_equal(got_short, got)


def test_kv_decode_attention_closed_forms_and_error_bound():
    rng = np.random.default_rng(45)
    B, H, L, d = 1, 2, 50, 8
    q = rng.integers(-90, 91, (B, H, d), dtype=np.int8)
    V = rng.integers(-127, 128, (B, H, L, d), dtype=np.int8)
    K = rng.integers(-90, 91, (B, H, L, d), dtype=np.int8)
    a_qk, d_v = np.float32(0.002), np.float32(0.03)
    a_pv = np.float32(d_v / np.float32(127.0))
    # one cached position: p = 1, P_bar = 127, out = 127 * v * (d_v / 127)
    out1, Ps = oracle.kv_decode_attention(q, K, V, [1], a_qk, a_pv, out_dtype="f32")
    assert all(P[0] == 127 and P.size == 1 for P in Ps)
    assert np.array_equal(out1, (V[:, :, 0].astype(np.float32) * np.float32(127.0)) * a_pv)
    # identical keys: uniform p = 1/L, so every P_bar = round(127 / L) and out = P_bar * sum(v) * alpha
    Ku = np.broadcast_to(K[:, :, :1], K.shape).copy()
    outu, Ps = oracle.kv_decode_attention(q, Ku, V, [L], a_qk, a_pv, out_dtype="f32")
    pb = int(np.rint(127.0 / L))
    assert all((P == pb).all() for P in Ps)
    assert np.array_equal(outu, (pb * V.astype(np.int64).sum(2)).astype(np.float32) * a_pv)
    # against the unquantised-probability result in fp64: each P_bar/127 is within 0.5/127 of p
    out, _ = oracle.kv_decode_attention(q, K, V, [L], a_qk, a_pv, out_dtype="f32")
    s = np.einsum("bhd,bhld->bhl", q.astype(np.float64), K.astype(np.float64)) * float(a_qk)
    p = np.exp(s - s.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    truth = np.einsum("bhl,bhld->bhd", p, V.astype(np.float64)) * float(d_v)
    bound = (0.5 / 127) * np.abs(V.astype(np.float64)).sum(2) * float(d_v)
    assert np.all(np.abs(out - truth) <= bound * (1 + 1e-5) + 1e-6)
    assert np.abs(out - truth).max() > 0  # the bound is not vacuous: quantising p does move the result


def test_decode_block_continues_the_prompt_block_exactly():
    """The generation-stage block fed with the prompt's last token and a cache holding the earlier
    tokens' k, v codes reproduces the prompt block's last row bit for bit, at every stage."""
    rng = np.random.default_rng(46)
    B, S, H, d, ffn = 2, 9, 2, 8, 32
    hid = H * d
    x = (rng.standard_normal((B * S, hid)) * 2).astype(np.float16).astype(np.float32)
    p = {"g1": (1 + 0.1 * rng.standard_normal(hid)).astype(np.float16).astype(np.float32),
         "b1": (0.1 * rng.standard_normal(hid)).astype(np.float16).astype(np.float32),
         "g2": (1 + 0.1 * rng.standard_normal(hid)).astype(np.float16).astype(np.float32),
         "b2": (0.1 * rng.standard_normal(hid)).astype(np.float16).astype(np.float32),
         "d_ln1": 0.03, "d_q": 0.02, "d_k": 0.02, "d_v": 0.015, "d_attn": 0.012, "d_ln2": 0.03, "d_fc1": 0.02}
    for n, (N, K) in {"qkv": (3 * hid, hid), "out_proj": (hid, hid), "fc1": (ffn, hid), "fc2": (hid, ffn)}.items():
        p[n] = {"Wq": rng.integers(-127, 128, (N, K), dtype=np.int8),
                "w_scale": rng.uniform(5e-4, 2e-3, N).astype(np.float32),
                "bias": (0.05 * rng.standard_normal(N)).astype(np.float16).astype(np.float32)}
    prompt = oracle.decoder_block_static(x, p, B, S, H, d, "f16", score_dtype="f32")
    qkv = prompt["qkv"].reshape(B, S, 3, H, d)
    L_max = 12
    Kc = np.zeros((B, H, L_max, d), np.int8)
    Vc = np.zeros((B, H, L_max, d), np.int8)
    Kc[:, :, :S - 1] = qkv[:, :S - 1, 1].transpose(0, 2, 1, 3)
    Vc[:, :, :S - 1] = qkv[:, :S - 1, 2].transpose(0, 2, 1, 3)
    x_last = x.reshape(B, S, hid)[:, -1]
    dec = oracle.decoder_block_static_decode(x_last, p, Kc, Vc, [S - 1, S - 1], H, d, "f16")
    for key in ("x1q", "qkv", "attn", "proj", "h", "x2q", "f1q", "fc2", "y"):
        want = prompt[key].reshape(B, S, -1)[:, -1]
        assert np.array_equal(dec[key], want), key
    assert np.array_equal(Kc[:, :, S - 1], qkv[:, S - 1, 1]) and np.array_equal(Vc[:, :, S - 1], qkv[:, S - 1, 2])
    assert np.abs(prompt["attn"]).max() > 10 and np.abs(prompt["y"]).max() > 0.5  # not a vacuous comparison


# --------------------------------------------------------------------------- #
# Static-step calibration with the largest tokens clipped
# --------------------------------------------------------------------------- #
def test_clipped_absmax_pins():
    rng = np.random.default_rng(47)
    v = np.arange(1, 101, dtype=np.float32)
    rng.shuffle(v)
    assert oracle.clip_count(100, 0.02) == 2 and oracle.clip_count(100, np.float32(0.02)) == 2
    assert oracle.clip_count(65536, 0.02) == 1311 and oracle.clip_count(7, 0.0) == 0
    assert oracle.clipped_absmax(v, 0) == 100.0                   # nothing clipped: the plain maximum
    assert oracle.clipped_absmax(v, 2) == 98.0                    # the two largest of 100 tokens set aside
    assert oracle.clipped_absmax(v, 50) == 50.0
    assert oracle.clipped_absmax(v, 100) == 1.0 and oracle.clipped_absmax(v, 1000) == 1.0   # never empties the set
    assert oracle.clipped_absmax(np.array([5, 5, 5, 1], np.float32), 1) == 5.0              # ties
    x = np.abs(rng.standard_normal(4099)).astype(np.float32) * 7
    for k in (0, 4, 82, 1230):
        want = np.partition(x, x.size - 1 - k)[x.size - 1 - k]    # library selection
        assert oracle.clipped_absmax(x, k) == want
        assert oracle.clipped_absmax(rng.permutation(x), k) == want
        assert (x > want).sum() <= k                               # at most k tokens lie above the result
    # on the outlier-token model, clipping the few huge tokens shrinks the static step a lot
    X = rng.standard_normal((1000, 64)).astype(np.float32)
    X[::100] *= 50.0                                               # 1 % of the tokens are outliers
    ta = oracle.row_absmax(X)
    assert oracle.clipped_absmax(ta, oracle.clip_count(1000, 0.02)) < 0.1 * oracle.clipped_absmax(ta, 0)
    assert oracle.clipped_absmax(ta, 0) == oracle.calib_absmax(X).max()


def test_decoder_block_static_tracks_the_float_block():
    """The W8A8 block (static steps taken from the float block's own maxima) stays within a few
    per cent of the same block computed in fp64 with library routines -- a dropped residual, a
    transposed weight, a missing 1/sqrt(d) or a wrong mask would be off by far more."""
    rng = np.random.default_rng(48)
    B, S, H, d, ffn = 2, 24, 2, 16, 64
    hid = H * d
    f16 = lambda a: a.astype(np.float16).astype(np.float32)
    x = f16(rng.standard_normal((B * S, hid)))
    g1, b1 = f16(1 + 0.1 * rng.standard_normal(hid)), f16(0.1 * rng.standard_normal(hid))
    g2, b2 = f16(1 + 0.1 * rng.standard_normal(hid)), f16(0.1 * rng.standard_normal(hid))
    shapes = {"qkv": (3 * hid, hid), "out_proj": (hid, hid), "fc1": (ffn, hid), "fc2": (hid, ffn)}
    p = {"g1": g1, "b1": b1, "g2": g2, "b2": b2}
    Wf, bias = {}, {}
    for n, (N, K) in shapes.items():
        W = f16(rng.standard_normal((N, K)) / np.sqrt(K))
        Wq, ws = oracle.quant_weight(W, None, "per_channel")
        bias[n] = f16(0.05 * rng.standard_normal(N))
        p[n] = {"Wq": Wq, "w_scale": ws, "bias": bias[n]}
        Wf[n] = torch.from_numpy(Wq.astype(np.float64) * ws[:, None].astype(np.float64))  # the weights the block really uses
    # the float block, fp64, library routines
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    X = t(x)
    ln1 = torch.nn.functional.layer_norm(X, (hid,), t(g1), t(b1), 1e-5)
    qkv = ln1 @ Wf["qkv"].T + t(bias["qkv"])
    q, k, v = (qkv[:, i * hid:(i + 1) * hid].reshape(B, S, H, d).permute(0, 2, 1, 3) for i in range(3))
    sc = q @ k.transpose(-1, -2) / np.sqrt(d)
    sc = sc + torch.full((S, S), float("-inf"), dtype=torch.float64).triu(1)
    att = (torch.softmax(sc, -1) @ v).permute(0, 2, 1, 3).reshape(B * S, hid)
    h = X + att @ Wf["out_proj"].T + t(bias["out_proj"])
    ln2 = torch.nn.functional.layer_norm(h, (hid,), t(g2), t(b2), 1e-5)
    f1 = torch.relu(ln2 @ Wf["fc1"].T + t(bias["fc1"]))
    y = h + f1 @ Wf["fc2"].T + t(bias["fc2"])
    step = lambda a: float(a.abs().max()) / 127.0
    p.update(d_ln1=step(ln1), d_q=step(qkv[:, :hid]), d_k=step(qkv[:, hid:2 * hid]), d_v=step(qkv[:, 2 * hid:]),
             d_attn=step(att), d_ln2=step(ln2), d_fc1=step(f1))
    out = oracle.decoder_block_static(x, p, B, S, H, d, "f16")
    rel = lambda a, b: float(np.linalg.norm(np.asarray(a, np.float64) - b.numpy()) / np.linalg.norm(b.numpy()))
    assert rel(out["h"], h) < 0.02
    assert rel(out["y"], y) < 0.03
    assert rel(out["attn"].astype(np.float64) * p["d_attn"], att) < 0.06
    # and the error is not zero: the block does quantise
    assert rel(out["y"], y) > 1e-4
