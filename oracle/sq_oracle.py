"""CPU ORACLE for the SmoothQuant W8A8 hot path -- test infrastructure only.

Thin numpy front end over oracle/sq_oracle.c.  Every function names the part
of the paper it restates.  Nothing here is imported by, or imports, the CUDA
library or its Python binding; only tests, the smoke check and the benchmark's
CPU-baseline leg call it.

Conventions
-----------
* fp16/bf16 tensors are passed as float32 numpy arrays whose values are exactly
  representable in that type ("A-valued float32").  `round_to(y, dtype)` rounds
  an fp32 array to fp16/bf16 (round-to-nearest-even, library cast) and returns
  it as A-valued float32 again.
* Stored weights are W[C_o, C_i] row-major, the transpose of the paper's
  W in R^{C_i x C_o}; "W_j" of Eq. 4 is therefore column j of the stored W.
* Granularities (Fig. 3 / Table 2): "per_token" (O1), "per_tensor_dynamic"
  (O2), "per_tensor_static" (O3) for activations; "per_channel" (= per output
  channel) and "per_tensor" for weights.

Parity unpinned: nothing in this module.
"""
import ctypes
import os

import numpy as np

from . import build as _build

_lib = ctypes.CDLL(_build.build())

_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)
_i8p = ctypes.POINTER(ctypes.c_int8)
_i32p = ctypes.POINTER(ctypes.c_int32)
_i64 = ctypes.c_int64

_lib.sqo_step_size.restype = ctypes.c_float
_lib.sqo_step_size.argtypes = [ctypes.c_float]
_lib.sqo_gemm_i32.restype = _i64
_lib.sqo_gemm_i32_bt.restype = _i64
_lib.sqo_num_threads.restype = ctypes.c_int


def _p(a, ty):
    return a.ctypes.data_as(ty) if a is not None else None


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i8(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.int8
    return a


def num_threads() -> int:
    """Threads the brute-force GEMM spreads its rows over."""
    return int(_lib.sqo_num_threads())


def round_to(y, dtype: str):
    """Round fp32 values to fp16 / bf16 (RNE) and return them widened to fp32."""
    y = _f32(y)
    if dtype == "f16":
        return y.astype(np.float16).astype(np.float32)
    if dtype == "bf16":
        import torch
        return torch.from_numpy(y).to(torch.bfloat16).to(torch.float32).numpy()
    if dtype == "f32":
        return y
    raise ValueError(dtype)


# --------------------------------------------------------------------------- #
# Offline transform (Section 4)
# --------------------------------------------------------------------------- #
def calib_absmax(X, absmax=None):
    """Section 4: per-input-channel max|X_j| over all calibration tokens (running max)."""
    X = _f32(X)
    rows, cols = X.shape
    a = np.zeros(cols, np.float32) if absmax is None else _f32(absmax).copy()
    _lib.sqo_col_absmax(_p(X, _f32p), _i64(rows), _i64(cols), _i64(cols), _p(a, _f32p))
    return a


def row_absmax(X):
    X = _f32(X)
    m = np.empty(X.shape[0], np.float32)
    _lib.sqo_row_absmax(_p(X, _f32p), _i64(X.shape[0]), _i64(X.shape[1]), _i64(X.shape[1]),
                        _p(m, _f32p))
    return m


def clip_count(T: int, clip_frac: float) -> int:
    """Number of tokens a clipping fraction sets aside: clip_frac * T rounded to the nearest integer."""
    return int(np.floor(float(clip_frac) * T + 0.5))


def clipped_absmax(token_absmax, n_clip: int):
    """Calibration of a static step with the largest tokens set aside (Section 5.2: for GLM-130B
    the top 2 % of tokens are clipped when the static step sizes are calibrated).  Of the T
    per-token absolute maxima (row_absmax over every calibration token), the n_clip largest are
    dropped and the largest of the rest is returned; the static step is step_size() of it.
    n_clip = 0 is the plain maximum; at least one token is always kept."""
    a = np.sort(np.ascontiguousarray(token_absmax, np.float32).reshape(-1))  # library sort, ascending
    T = a.size
    k = max(0, min(int(n_clip), T - 1))
    return np.float32(a[T - 1 - k])


def smooth_scales(act_absmax, w_absmax, alpha: float):
    """Eq. 4: s_j = max|X_j|^alpha / max|W_j|^(1-alpha)."""
    if not (0.0 <= alpha <= 1.0):
        raise ValueError("alpha must lie in [0, 1]")
    ax, aw = _f32(act_absmax), _f32(w_absmax)
    s = np.empty_like(ax)
    _lib.sqo_smooth_scales(_p(ax, _f32p), _p(aw, _f32p), _i64(ax.size), ctypes.c_float(alpha),
                           _p(s, _f32p))
    return s


def smooth_scales_inv(s):
    """The explicit activation-side factor of Eq. 3, 1/s_j, as one fp32 division."""
    s = _f32(s)
    o = np.empty_like(s)
    one = np.ones_like(s)
    _lib.sqo_div_by_s(_p(one, _f32p), _p(s, _f32p), _i64(s.size), _p(o, _f32p))
    return o


def fold_ln_weight(gamma, beta, s, dtype: str):
    """Eq. 3 folded offline into the preceding LayerNorm: gamma/s, beta/s, stored in `dtype`."""
    s = _f32(s)
    outs = []
    for p in (gamma, beta):
        if p is None:
            outs.append(None)
            continue
        p = _f32(p)
        o = np.empty_like(p)
        _lib.sqo_div_by_s(_p(p, _f32p), _p(s, _f32p), _i64(p.size), _p(o, _f32p))
        outs.append(round_to(o, dtype))
    return outs[0], outs[1]


def step_size(absmax: float) -> float:
    """Eq. 1: Delta = max|X| / 127."""
    return float(_lib.sqo_step_size(ctypes.c_float(absmax)))


def quantize(V, delta, per_row: bool):
    """Eq. 1 with given step size(s): clamp(round(V / Delta)) to [-127, 127], RNE."""
    V = _f32(V)
    d = _f32(np.atleast_1d(delta))
    Q = np.empty(V.shape, np.int8)
    _lib.sqo_quantize(_p(V, _f32p), _i64(V.shape[0]), _i64(V.shape[1]), _i64(V.shape[1]),
                      _p(d, _f32p), ctypes.c_int(1 if per_row else 0), _p(Q, _i8p))
    return Q


def quantize_f64_literal(V, delta, per_row: bool):
    """Eq. 1 taken literally (true division, fp64): diagnostic only."""
    V = _f32(V)
    d = _f32(np.atleast_1d(delta))
    Q = np.empty(V.shape, np.int8)
    _lib.sqo_quantize_f64_literal(_p(V, _f32p), _i64(V.shape[0]), _i64(V.shape[1]),
                                  _i64(V.shape[1]), _p(d, _f32p),
                                  ctypes.c_int(1 if per_row else 0), _p(Q, _i8p))
    return Q


def quant_weight(W, s, gran: str):
    """Eq. 3 (W_hat = W diag(s)) then Eq. 1 per output channel or per tensor.

    Returns (W_bar int8 [N, K], w_scale fp32 [N] or [1])."""
    W = _f32(W)
    N, K = W.shape
    What = np.empty_like(W)
    sp = None if s is None else _f32(s)
    _lib.sqo_scale_weight_cols(_p(W, _f32p), _i64(N), _i64(K), _p(sp, _f32p), _p(What, _f32p))
    m = row_absmax(What)
    if gran == "per_channel":
        delta = np.array([step_size(v) for v in m], np.float32)
        return quantize(What, delta, True), delta
    if gran == "per_tensor":
        delta = np.array([step_size(m.max())], np.float32)
        return quantize(What, delta, False), delta
    raise ValueError(gran)


# --------------------------------------------------------------------------- #
# Runtime activation quantisation (Section 2, Table 2)
# --------------------------------------------------------------------------- #
def quant_act(X, gran: str, col_mul=None, static_scale=None):
    """Eq. 1 on an activation tensor [T, C_i].

    per_token: Delta_t from row t; per_tensor_dynamic: one Delta from the whole
    tensor of this call; per_tensor_static: Delta given (from calibration),
    values beyond it saturate.  Returns (X_bar, x_scale)."""
    X = _f32(X)
    if col_mul is not None:
        cm = _f32(col_mul)
        Y = np.empty_like(X)
        _lib.sqo_mul_cols(_p(X, _f32p), _i64(X.shape[0]), _i64(X.shape[1]), _i64(X.shape[1]),
                          _p(cm, _f32p), _p(Y, _f32p))
        X = Y
    if gran == "per_token":
        m = row_absmax(X)
        delta = np.array([step_size(v) for v in m], np.float32)
        return quantize(X, delta, True), delta
    if gran == "per_tensor_dynamic":
        m = row_absmax(X)
        delta = np.array([step_size(m.max() if m.size else 0.0)], np.float32)
        return quantize(X, delta, False), delta
    if gran == "per_tensor_static":
        delta = _f32(np.atleast_1d(static_scale))
        return quantize(X, delta, False), delta
    raise ValueError(gran)


def ln_stats(X, eps: float):
    """LayerNorm row statistics, fp64 two-pass, biased variance: (mu, rstd)."""
    X = _f32(X)
    M, C = X.shape
    mu, rstd = np.empty(M, np.float64), np.empty(M, np.float64)
    _lib.sqo_ln_stats_f64(_p(X, _f32p), _i64(M), _i64(C), _i64(C), ctypes.c_double(eps),
                          _p(mu, _f64p), _p(rstd, _f64p))
    return mu, rstd


def ln_apply(X, mu, rstd, gamma_hat, beta_hat):
    """Normative fp32 element-wise LayerNorm given fp32 statistics (not rounded to A)."""
    X = _f32(X)
    M, C = X.shape
    mu, rstd = _f32(mu), _f32(rstd)
    g = _f32(gamma_hat)
    b = None if beta_hat is None else _f32(beta_hat)
    Y = np.empty_like(X)
    _lib.sqo_ln_apply(_p(X, _f32p), _i64(M), _i64(C), _i64(C), _p(mu, _f32p), _p(rstd, _f32p),
                      _p(g, _f32p), _p(b, _f32p), _p(Y, _f32p))
    return Y


def ln_f64(X, gamma, beta, eps: float):
    X = _f32(X)
    M, C = X.shape
    g = np.ascontiguousarray(gamma, np.float64)
    b = None if beta is None else np.ascontiguousarray(beta, np.float64)
    Y = np.empty((M, C), np.float64)
    _lib.sqo_ln_f64(_p(X, _f32p), _i64(M), _i64(C), _i64(C), ctypes.c_double(eps), _p(g, _f64p),
                    _p(b, _f64p), _p(Y, _f64p))
    return Y


def ln_quant(X, gamma_hat, beta_hat, eps: float, gran: str, stats=None, static_scale=None):
    """LayerNorm with folded smoothing, then Eq. 1, with no rounding in between.

    `stats` = (mu, rstd) as fp32 arrays replaces the fp64 statistics (rounded to
    fp32) so that a kernel's own statistics can be fed back for a bit-exact
    comparison of the element-wise part.  Returns (X_bar, x_scale, y_fp32)."""
    if stats is None:
        mu, rstd = ln_stats(X, eps)
        stats = (mu.astype(np.float32), rstd.astype(np.float32))
    Y = ln_apply(X, stats[0], stats[1], gamma_hat, beta_hat)
    Q, d = quant_act(Y, gran, static_scale=static_scale)
    return Q, d, Y


# --------------------------------------------------------------------------- #
# INT8 GEMM + dequantisation (Eq. 2)
# --------------------------------------------------------------------------- #
def gemm_i32(Xq, Wq):
    """acc[t, o] = sum_j X_bar[t, j] W_bar[o, j]; brute force, int32-checked."""
    Xq, Wq = _i8(Xq), _i8(Wq)
    M, K = Xq.shape
    N, K2 = Wq.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    ov = _lib.sqo_gemm_i32(_p(Xq, _i8p), _p(Wq, _i8p), _i64(M), _i64(N), _i64(K), _i64(K), _i64(K),
                           _p(acc, _i32p))
    if ov:
        raise OverflowError("%d accumulators exceed int32" % ov)
    return acc


def gemm_i32_bt(Aq, Bq):
    """acc[t, o] = sum_j A[t, j] B[j, o] with B stored [K, N] (as V in P.V)."""
    Aq, Bq = _i8(Aq), _i8(Bq)
    M, K = Aq.shape
    K2, N = Bq.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    ov = _lib.sqo_gemm_i32_bt(_p(Aq, _i8p), _p(Bq, _i8p), _i64(M), _i64(N), _i64(K), _i64(K),
                              _i64(N), _p(acc, _i32p))
    if ov:
        raise OverflowError("%d accumulators exceed int32" % ov)
    return acc


def dequant(acc, x_scale, w_scale, bias=None, relu=False):
    """Eq. 2 plus bias/ReLU: fp32 y = fma(acc, Delta_x[t] * Delta_w[o], b_o), before output rounding."""
    acc = np.ascontiguousarray(acc, np.int32)
    M, N = acc.shape
    xs, ws = _f32(np.atleast_1d(x_scale)), _f32(np.atleast_1d(w_scale))
    assert xs.size in (1, M) and ws.size in (1, N)
    b = None if bias is None else _f32(bias)
    Y = np.empty((M, N), np.float32)
    _lib.sqo_dequant(_p(acc, _i32p), _i64(M), _i64(N), _p(xs, _f32p),
                     ctypes.c_int(1 if xs.size > 1 else 0), _p(ws, _f32p),
                     ctypes.c_int(1 if ws.size > 1 else 0), _p(b, _f32p),
                     ctypes.c_int(1 if relu else 0), _p(Y, _f32p))
    return Y


def requant(Y, r):
    """clamp(round(y * r)) with r a scalar or one multiplier per column."""
    Y = _f32(Y)
    r = _f32(np.atleast_1d(r))
    Q = np.empty(Y.shape, np.int8)
    _lib.sqo_requant(_p(Y, _f32p), _i64(Y.shape[0]), _i64(Y.shape[1]), _p(r, _f32p),
                     ctypes.c_int(1 if r.size > 1 else 0), _p(Q, _i8p))
    return Q


def w8a8_linear(Xq, x_scale, Wq, w_scale, bias=None, relu=False, out_dtype="f16",
                requant_mul=None):
    """The W8A8 linear layer after quantisation: Eq. 2 end to end.

    Returns (acc int32, out) where out is A-valued float32, or int8 when
    requant_mul is given."""
    acc = gemm_i32(Xq, Wq)
    y = dequant(acc, x_scale, w_scale, bias, relu)
    if requant_mul is not None:
        return acc, requant(y, requant_mul)
    return acc, round_to(y, out_dtype)


def scale_acc(acc, alpha: float):
    acc = np.ascontiguousarray(acc, np.int32)
    Y = np.empty(acc.shape, np.float32)
    _lib.sqo_scale_acc(_p(acc, _i32p), _i64(acc.size), ctypes.c_float(alpha), _p(Y, _f32p))
    return Y


def w8a8_bmm(A, B, alpha: float, b_is_kn: bool = False, out_dtype="f16", requant_mul=None):
    """Attention BMMs of Fig. 6 in INT8: for each leading index,
    out = (A B^T) * alpha (B stored [N, K]) or (A B) * alpha (B stored [K, N])."""
    A, B = _i8(A), _i8(B)
    lead = A.shape[:-2]
    A3 = A.reshape((-1,) + A.shape[-2:])
    B3 = B.reshape((-1,) + B.shape[-2:])
    accs, outs = [], []
    for a, b in zip(A3, B3):
        acc = gemm_i32_bt(a, b) if b_is_kn else gemm_i32(a, b)
        y = scale_acc(acc, alpha)
        accs.append(acc)
        outs.append(requant(y, requant_mul) if requant_mul is not None else round_to(y, out_dtype))
    shp = lead + accs[0].shape
    return np.stack(accs).reshape(shp), np.stack(outs).reshape(shp)


def softmax_causal(S):
    """fp32 causal softmax of one [S, S] (or [rows, cols]) score matrix."""
    S = _f32(S)
    P = np.empty_like(S)
    _lib.sqo_softmax_causal(_p(S, _f32p), _i64(S.shape[0]), _i64(S.shape[1]), _i64(S.shape[1]),
                            _p(P, _f32p))
    return P


def softmax_causal_f64(S):
    S = _f32(S)
    P = np.empty(S.shape, np.float64)
    _lib.sqo_softmax_causal_f64(_p(S, _f32p), _i64(S.shape[0]), _i64(S.shape[1]),
                                _i64(S.shape[1]), _p(P, _f64p))
    return P


def softmax_quant_p(S):
    """Softmax output lies in [0, 1], so its step size is fixed at 1/127: P_bar = round(127 p)."""
    P = softmax_causal(S)
    return requant(P, np.float32(127.0)), P


def softmax_prefix(S, first: int):
    """fp32 softmax where row i sees the first (first + i) keys; first=1 is softmax_causal."""
    S = _f32(S)
    P = np.empty_like(S)
    _lib.sqo_softmax_prefix(_p(S, _f32p), _i64(S.shape[0]), _i64(S.shape[1]), _i64(S.shape[1]),
                            _i64(first), _p(P, _f32p))
    return P


def kv_decode_attention(q, K, V, lens, alpha_qk: float, alpha_pv: float, out_dtype="f16",
                        requant_mul=None, score_dtype="f32"):
    """Generation-stage attention over an INT8 key/value cache (the Discussion's point that
    quantised activations also shrink the KV cache), in the precision mapping of Fig. 6:
    INT8 q.K^T -> floating-point softmax -> P_bar = round(127 p) -> INT8 P_bar.V.

    q [B, H, d] INT8: the newest token's query; K, V [B, H, L_max, d] INT8: the cache, of which
    sequence b holds lens[b] valid positions (the newest token's own k, v included).
    Returns (out [B, H, d], P_bar list per (b, h)), out = requant or rounded to out_dtype."""
    q, K, V = _i8(q), _i8(K), _i8(V)
    B, H, d = q.shape
    out = np.empty((B, H, d), np.int8 if requant_mul is not None else np.float32)
    Ps = []
    for b in range(B):
        L = int(lens[b])
        for h in range(H):
            acc = gemm_i32(q[b, h][None, :], K[b, h, :L])          # [1, L]
            s = round_to(scale_acc(acc, alpha_qk), score_dtype)
            p = softmax_prefix(s, L)
            Pq = requant(p, np.float32(127.0))
            acc2 = gemm_i32_bt(Pq, V[b, h, :L])                     # [1, d]
            y = scale_acc(acc2, alpha_pv)
            out[b, h] = (requant(y, requant_mul) if requant_mul is not None else round_to(y, out_dtype))[0]
            Ps.append(Pq[0])
    return out, Ps


def linear_f64(X, W, b=None):
    """fp64 truth: Y = X W^T + b with W stored [N, K]."""
    X = np.ascontiguousarray(X, np.float64)
    W = np.ascontiguousarray(W, np.float64)
    bb = None if b is None else np.ascontiguousarray(b, np.float64)
    M, K = X.shape
    N = W.shape[0]
    Y = np.empty((M, N), np.float64)
    _lib.sqo_linear_f64(_p(X, _f64p), _p(W, _f64p), _p(bb, _f64p), _i64(M), _i64(N), _i64(K),
                        _p(Y, _f64p))
    return Y


# --------------------------------------------------------------------------- #
# Whole decoder block (Fig. 6), static per-tensor activation steps (O3)
# --------------------------------------------------------------------------- #
def decoder_block_static(x, p, B, S, H, d, dtype="f16", eps=1e-5, score_dtype=None):
    """One pre-LayerNorm decoder block in the precision mapping of Fig. 6: INT8 for the four
    linear layers and the two attention BMMs, floating point for LayerNorm, softmax, ReLU and
    the residual adds.  `x` is [B*S, H*d] (A-valued float32); `p` holds, per linear
    ("qkv", "out_proj", "fc1", "fc2"), the INT8 weight `Wq`, `w_scale`, `bias`, and the static
    steps `d_ln1, d_q, d_k, d_v, d_attn, d_ln2, d_fc1` plus folded LayerNorm parameters
    `g1, b1, g2, b2`.  `score_dtype` is the type the attention scores are held in before the
    softmax (default: the activation dtype; "f32" when they never leave fp32).  Every intermediate
    is returned for stage-by-stage comparison."""
    f32 = np.float32
    hid = H * d
    out = {}
    # LN1 (smoothing folded) -> INT8, static step
    out["x1q"], _, _ = ln_quant(x, p["g1"], p["b1"], eps, "per_tensor_static", static_scale=p["d_ln1"])
    # QKV projection, re-quantised to INT8 with one static step per q / k / v
    acc = gemm_i32(out["x1q"], p["qkv"]["Wq"])
    y = dequant(acc, p["d_ln1"], p["qkv"]["w_scale"], p["qkv"]["bias"])
    r = np.concatenate([np.full(hid, f32(1) / f32(p["d_q"]), f32), np.full(hid, f32(1) / f32(p["d_k"]), f32),
                        np.full(hid, f32(1) / f32(p["d_v"]), f32)])
    out["qkv"] = requant(y, r)
    qkv = out["qkv"].reshape(B, S, 3, H, d)
    q = np.ascontiguousarray(qkv[:, :, 0].transpose(0, 2, 1, 3))
    k = np.ascontiguousarray(qkv[:, :, 1].transpose(0, 2, 1, 3))
    v = np.ascontiguousarray(qkv[:, :, 2].transpose(0, 2, 1, 3))
    # scores = Q K^T * (d_q d_k / sqrt(d)), rounded to the activation dtype
    alpha_qk = f32(f32(p["d_q"]) * f32(p["d_k"])) / f32(np.sqrt(f32(d)))
    _, out["scores"] = w8a8_bmm(q, k, float(alpha_qk), out_dtype=score_dtype or dtype)
    # causal softmax in floating point, P quantised with the fixed step 1/127
    Pq = np.empty((B, H, S, S), np.int8)
    for b in range(B):
        for h in range(H):
            Pq[b, h], _ = softmax_quant_p(out["scores"][b, h])
    out["P"] = Pq
    # attention output = P V * (d_v / 127), re-quantised with the out-projection's static input step
    alpha_pv = f32(p["d_v"]) / f32(127.0)
    _, o = w8a8_bmm(Pq, v, float(alpha_pv), b_is_kn=True, requant_mul=f32(1) / f32(p["d_attn"]))
    out["attn"] = np.ascontiguousarray(o.transpose(0, 2, 1, 3)).reshape(B * S, hid)
    # out-projection -> activation dtype, residual add
    _, out["proj"] = w8a8_linear(out["attn"], p["d_attn"], p["out_proj"]["Wq"], p["out_proj"]["w_scale"],
                                 bias=p["out_proj"]["bias"], out_dtype=dtype)
    out["h"] = round_to(_f32(x) + out["proj"], dtype)
    # LN2 (smoothing folded) -> INT8; FC1 + ReLU -> INT8; FC2 -> activation dtype; residual add
    out["x2q"], _, _ = ln_quant(out["h"], p["g2"], p["b2"], eps, "per_tensor_static", static_scale=p["d_ln2"])
    _, out["f1q"] = w8a8_linear(out["x2q"], p["d_ln2"], p["fc1"]["Wq"], p["fc1"]["w_scale"], bias=p["fc1"]["bias"],
                                relu=True, requant_mul=f32(1) / f32(p["d_fc1"]))
    _, out["fc2"] = w8a8_linear(out["f1q"], p["d_fc1"], p["fc2"]["Wq"], p["fc2"]["w_scale"], bias=p["fc2"]["bias"],
                                out_dtype=dtype)
    out["y"] = round_to(out["h"] + out["fc2"], dtype)
    return out


def decoder_block_static_decode(x, p, K_cache, V_cache, ctx, H, d, dtype="f16", eps=1e-5):
    """Generation stage of decoder_block_static: x [B, H*d] is the newest token of each sequence,
    K_cache / V_cache [B, H, L_max, d] INT8 hold the codes of the ctx[b] earlier positions.  The
    token's own k, v codes are stored at position ctx[b] (the caches are updated in place) and its
    attention runs over ctx[b] + 1 positions with fp32 scores (kv_decode_attention); everything
    else is the prompt block's arithmetic on one row per sequence."""
    f32 = np.float32
    B, hid = x.shape[0], H * d
    out = {}
    out["x1q"], _, _ = ln_quant(x, p["g1"], p["b1"], eps, "per_tensor_static", static_scale=p["d_ln1"])
    acc = gemm_i32(out["x1q"], p["qkv"]["Wq"])
    y = dequant(acc, p["d_ln1"], p["qkv"]["w_scale"], p["qkv"]["bias"])
    r = np.concatenate([np.full(hid, f32(1) / f32(p["d_q"]), f32), np.full(hid, f32(1) / f32(p["d_k"]), f32),
                        np.full(hid, f32(1) / f32(p["d_v"]), f32)])
    out["qkv"] = requant(y, r)
    qkv = out["qkv"].reshape(B, 3, H, d)
    lens = []
    for b in range(B):
        K_cache[b, :, int(ctx[b])] = qkv[b, 1]
        V_cache[b, :, int(ctx[b])] = qkv[b, 2]
        lens.append(int(ctx[b]) + 1)
    alpha_qk = f32(f32(p["d_q"]) * f32(p["d_k"])) / f32(np.sqrt(f32(d)))
    alpha_pv = f32(p["d_v"]) / f32(127.0)
    o, _ = kv_decode_attention(np.ascontiguousarray(qkv[:, 0]), K_cache, V_cache, lens, float(alpha_qk), float(alpha_pv),
                               requant_mul=f32(1) / f32(p["d_attn"]))
    out["attn"] = o.reshape(B, hid)
    _, out["proj"] = w8a8_linear(out["attn"], p["d_attn"], p["out_proj"]["Wq"], p["out_proj"]["w_scale"],
                                 bias=p["out_proj"]["bias"], out_dtype=dtype)
    out["h"] = round_to(_f32(x) + out["proj"], dtype)
    out["x2q"], _, _ = ln_quant(out["h"], p["g2"], p["b2"], eps, "per_tensor_static", static_scale=p["d_ln2"])
    _, out["f1q"] = w8a8_linear(out["x2q"], p["d_ln2"], p["fc1"]["Wq"], p["fc1"]["w_scale"], bias=p["fc1"]["bias"],
                                relu=True, requant_mul=f32(1) / f32(p["d_fc1"]))
    _, out["fc2"] = w8a8_linear(out["f1q"], p["d_fc1"], p["fc2"]["Wq"], p["fc2"]["w_scale"], bias=p["fc2"]["bias"],
                                out_dtype=dtype)
    out["y"] = round_to(out["h"] + out["fc2"], dtype)
    return out
