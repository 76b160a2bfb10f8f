"""ctypes binding of libsq: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors used purely as device memory; every step of the path runs in
the library's kernels.  There is no CPU or PyTorch fallback: if the shared library is
missing, or no CUDA device is present when a call is made, an exception is raised.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsq.so")

# enums of include/sq.h
SQ_OK = 0
(SQ_ERR_INVALID_ARG, SQ_ERR_SHAPE, SQ_ERR_ALIGN, SQ_ERR_UNSUPPORTED, SQ_ERR_CUDA, SQ_ERR_TIMEOUT,
 SQ_ERR_WORKSPACE) = range(1, 8)
SQ_F16, SQ_BF16, SQ_I8, SQ_I32 = 0, 1, 2, 3
SQ_PER_TENSOR_STATIC, SQ_PER_TENSOR_DYNAMIC, SQ_PER_TOKEN_DYNAMIC = 0, 1, 2
SQ_W_PER_TENSOR, SQ_W_PER_CHANNEL = 0, 1
SQ_EPI_NONE, SQ_EPI_RELU = 0, 1
SQ_OP_QUANT_ACT, SQ_OP_LN_QUANT, SQ_OP_QUANT_WEIGHT, SQ_OP_GEMM, SQ_OP_BMM, SQ_OP_GEMM_FUSED_QUANT = 0, 1, 2, 3, 4, 5
SQ_MAX_K = 133144
SQ_NOALLOC_MAX_ROWS = 16384

EXPORTS = ["sq_status_str", "sq_workspace_bytes", "sq_calib_absmax", "sq_smooth_scales",
           "sq_fold_ln_weight", "sq_quant_weight", "sq_quant_act", "sq_ln_quant", "sq_w8a8_gemm", "sq_w8a8_gemm_residual",
           "sq_w8a8_bmm", "sq_softmax_quant_p", "sq_residual_add", "sq_ln_quant_tensor_noalloc",
           "sq_selftest_bounded_wait", "sq_w8a8_attention", "sq_kv_cache_write", "sq_w8a8_decode_attention",
           "sq_token_absmax", "sq_clipped_absmax", "sq_selftest_row_wait", "sq_w8a8_gemm_fused_quant", "sq_quant_act_given_absmax", "sq_dequant_acc"]

_DT = {torch.float16: SQ_F16, torch.bfloat16: SQ_BF16, torch.int8: SQ_I8, torch.int32: SQ_I32}
GRAN = {"per_tensor_static": SQ_PER_TENSOR_STATIC, "per_tensor_dynamic": SQ_PER_TENSOR_DYNAMIC,
        "per_token": SQ_PER_TOKEN_DYNAMIC}
WGRAN = {"per_tensor": SQ_W_PER_TENSOR, "per_channel": SQ_W_PER_CHANNEL}

_lib = None


class SqError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__("%s failed: %s (%d)" % (where, status_str(code), code))


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libsq.so not built: run `python -m paper_2211_10438_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        c = ctypes
        vp, i64, i32, f32, sz = c.c_void_p, c.c_int64, c.c_int, c.c_float, c.c_size_t
        L.sq_status_str.restype = c.c_char_p
        L.sq_status_str.argtypes = [i32]
        L.sq_workspace_bytes.restype = sz
        L.sq_workspace_bytes.argtypes = [i32, i64, i64, i64]
        L.sq_calib_absmax.argtypes = [vp, i32, i64, i64, i64, vp, vp]
        L.sq_smooth_scales.argtypes = [vp, vp, i64, f32, vp, vp, vp]
        L.sq_fold_ln_weight.argtypes = [vp, vp, i32, vp, i64, vp, vp, vp]
        L.sq_quant_weight.argtypes = [vp, i32, i64, i64, vp, i32, vp, vp, vp, sz, vp]
        L.sq_quant_act.argtypes = [vp, i32, i64, i64, i32, vp, vp, vp, vp, sz, vp]
        L.sq_ln_quant.argtypes = [vp, i32, i64, i64, vp, vp, f32, i32, vp, vp, vp, vp, sz, vp]
        L.sq_w8a8_gemm.argtypes = [vp, vp, i64, i64, i64, vp, i32, vp, i32, vp, i32, i32, vp, i32, vp,
                                   vp, i32, i64, vp, sz, vp]
        L.sq_w8a8_gemm_residual.argtypes = [vp, vp, i64, i64, i64, vp, i32, vp, i32, vp, i32, vp, i64, vp, i32, i64,
                                            vp, sz, vp]
        L.sq_w8a8_gemm_fused_quant.argtypes = [vp, i32, i64, i64, i64, vp, vp, f32, i32, vp, vp, vp, vp, vp, i32, vp, i32, i32,
                                               vp, i32, vp, i64, vp, i32, i64, vp, sz, vp]
        L.sq_quant_act_given_absmax.argtypes = [vp, i32, i64, i64, vp, vp, vp, vp, sz, vp]
        L.sq_dequant_acc.argtypes = [vp, i64, i64, i64, vp, i32, vp, i32, vp, i32, i32, vp, i32, vp, i64, vp, i32, i64, vp]
        L.sq_w8a8_bmm.argtypes = [vp, vp, i64, i64, i64, i64, i64, c.POINTER(i64), c.POINTER(i64), i32, i32,
                                  f32, vp, vp, i32, c.POINTER(i64), vp, sz, vp]
        L.sq_softmax_quant_p.argtypes = [vp, i32, i64, i64, vp, vp]
        L.sq_residual_add.argtypes = [vp, vp, i32, i64, vp, vp]
        L.sq_ln_quant_tensor_noalloc.argtypes = [vp, i32, i64, i64, vp, vp, f32, vp, vp, vp]
        L.sq_selftest_bounded_wait.argtypes = [vp, c.c_uint32, vp]
        L.sq_selftest_row_wait.argtypes = [vp, c.c_uint32, vp]
        L.sq_w8a8_attention.argtypes = [vp, i64, i64, i64, i64, f32, f32, vp, vp, vp, sz, vp]
        L.sq_token_absmax.argtypes = [vp, i32, i64, i64, i64, vp, vp]
        L.sq_clipped_absmax.argtypes = [vp, i64, i64, vp, vp, vp]
        L.sq_kv_cache_write.argtypes = [vp, i64, i64, i64, i64, i64, vp, vp, vp, i64, vp, sz, vp]
        L.sq_w8a8_decode_attention.argtypes = [vp, i64, vp, vp, vp, vp, i64, vp, i64, i64, i64, i64, i64, f32, f32, vp,
                                               vp, i32, i64, vp, sz, vp]
        for name in EXPORTS[2:]:
            getattr(L, name).restype = i32
        _lib = L
    return _lib


def status_str(code: int) -> str:
    return lib().sq_status_str(int(code)).decode()


def _check(code, where):
    if code != SQ_OK:
        raise SqError(code, where)


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda:
        raise RuntimeError("libsq takes device memory only (got a CPU tensor); no CPU fallback exists")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    if not torch.cuda.is_available():
        raise RuntimeError("no CUDA device: libsq has no CPU fallback")
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def workspace_bytes(op: int, M: int = 0, N: int = 0, K: int = 0) -> int:
    return int(lib().sq_workspace_bytes(op, M, N, K))


def new_workspace(nbytes: int, device="cuda"):
    """Zero-filled, 256-byte aligned workspace (torch's allocator aligns to 512 bytes)."""
    return torch.zeros(max(256, (nbytes + 255) // 256 * 256), dtype=torch.uint8, device=device)


def device_status(workspace) -> int:
    """The sticky device status word at workspace[0] (synchronises)."""
    return int(workspace[:4].view(torch.int32).item())


def _ws(workspace):
    return (_ptr(workspace), 0 if workspace is None else workspace.numel())


def sq_calib_absmax(X, absmax_inout):
    rows, cols = X.shape
    _check(lib().sq_calib_absmax(_ptr(X), _DT[X.dtype], rows, cols, X.stride(0), _ptr(absmax_inout),
                                 _stream()), "sq_calib_absmax")
    return absmax_inout


def sq_smooth_scales(act_absmax, w_absmax, alpha, s_out=None, s_inv_out=None):
    C = act_absmax.numel()
    if s_out is None:
        s_out = torch.empty(C, dtype=torch.float32, device=act_absmax.device)
    _check(lib().sq_smooth_scales(_ptr(act_absmax), _ptr(w_absmax), C, float(alpha), _ptr(s_out),
                                  _ptr(s_inv_out), _stream()), "sq_smooth_scales")
    return s_out


def sq_fold_ln_weight(gamma, beta, s, gamma_out=None, beta_out=None):
    if gamma_out is None:
        gamma_out = torch.empty_like(gamma)
    if beta is not None and beta_out is None:
        beta_out = torch.empty_like(beta)
    _check(lib().sq_fold_ln_weight(_ptr(gamma), _ptr(beta), _DT[gamma.dtype], _ptr(s), gamma.numel(),
                                   _ptr(gamma_out), _ptr(beta_out), _stream()), "sq_fold_ln_weight")
    return gamma_out, beta_out


def sq_quant_weight(W, s, gran, Wq=None, w_scale=None, workspace=None):
    N, K = W.shape
    g = WGRAN[gran] if isinstance(gran, str) else gran
    if Wq is None:
        Wq = torch.empty((N, K), dtype=torch.int8, device=W.device)
    if w_scale is None:
        w_scale = torch.empty(N if g == SQ_W_PER_CHANNEL else 1, dtype=torch.float32, device=W.device)
    wp, wn = _ws(workspace)
    _check(lib().sq_quant_weight(_ptr(W), _DT[W.dtype], N, K, _ptr(s), g, _ptr(Wq), _ptr(w_scale), wp, wn,
                                 _stream()), "sq_quant_weight")
    return Wq, w_scale


def sq_quant_act(X, gran, col_mul=None, Xq=None, x_scale=None, workspace=None):
    M, C = X.shape
    g = GRAN[gran] if isinstance(gran, str) else gran
    if Xq is None:
        Xq = torch.empty((M, C), dtype=torch.int8, device=X.device)
    if x_scale is None:
        if g == SQ_PER_TENSOR_STATIC:
            raise ValueError("static quantisation needs x_scale as an input")
        x_scale = torch.empty(M if g == SQ_PER_TOKEN_DYNAMIC else 1, dtype=torch.float32, device=X.device)
    wp, wn = _ws(workspace)
    _check(lib().sq_quant_act(_ptr(X), _DT[X.dtype], M, C, g, _ptr(col_mul), _ptr(Xq), _ptr(x_scale), wp,
                              wn, _stream()), "sq_quant_act")
    return Xq, x_scale


def sq_quant_act_given_absmax(X, row_absmax, Xq=None, x_scale=None, workspace=None):
    """Per-token Eq. 1 with the token maxima given (agreed on across tensor-parallel ranks) -> (Xq, x_scale[M])."""
    M, C = X.shape
    if Xq is None:
        Xq = torch.empty((M, C), dtype=torch.int8, device=X.device)
    if x_scale is None:
        x_scale = torch.empty(M, dtype=torch.float32, device=X.device)
    wp, wn = _ws(workspace)
    _check(lib().sq_quant_act_given_absmax(_ptr(X), _DT[X.dtype], M, C, _ptr(row_absmax), _ptr(Xq), _ptr(x_scale), wp, wn,
                                           _stream()), "sq_quant_act_given_absmax")
    return Xq, x_scale


def sq_dequant_acc(acc, x_scale, w_scale, bias=None, relu=False, requant_mul=None, residual=None, out=None,
                   out_dtype=torch.float16):
    """Eq. 2 on an INT32 accumulator matrix [M, N] (the sum of tensor-parallel partial sums)."""
    M, N = acc.shape
    if out is None:
        odt = torch.int8 if requant_mul is not None else (residual.dtype if residual is not None else out_dtype)
        out = torch.empty((M, N), dtype=odt, device=acc.device)
    _check(lib().sq_dequant_acc(
        _ptr(acc), acc.stride(0), M, N, _ptr(x_scale), 1 if x_scale.numel() > 1 else 0, _ptr(w_scale),
        1 if w_scale.numel() > 1 else 0, _ptr(bias), _DT[bias.dtype] if bias is not None else SQ_F16,
        SQ_EPI_RELU if relu else SQ_EPI_NONE, _ptr(requant_mul),
        1 if (requant_mul is not None and requant_mul.numel() > 1) else 0, _ptr(residual),
        residual.stride(0) if residual is not None else 0, _ptr(out), _DT[out.dtype], out.stride(0), _stream()),
        "sq_dequant_acc")
    return out


def sq_ln_quant(X, gamma_hat, beta_hat, eps, gran, Xq=None, x_scale=None, dbg_mean_rstd=None,
                workspace=None):
    M, C = X.shape
    g = GRAN[gran] if isinstance(gran, str) else gran
    if Xq is None:
        Xq = torch.empty((M, C), dtype=torch.int8, device=X.device)
    if x_scale is None:
        if g == SQ_PER_TENSOR_STATIC:
            raise ValueError("static quantisation needs x_scale as an input")
        x_scale = torch.empty(M if g == SQ_PER_TOKEN_DYNAMIC else 1, dtype=torch.float32, device=X.device)
    wp, wn = _ws(workspace)
    _check(lib().sq_ln_quant(_ptr(X), _DT[X.dtype], M, C, _ptr(gamma_hat), _ptr(beta_hat), float(eps), g,
                             _ptr(Xq), _ptr(x_scale), _ptr(dbg_mean_rstd), wp, wn, _stream()),
           "sq_ln_quant")
    return Xq, x_scale


def sq_w8a8_gemm(Xq, Wq, x_scale, w_scale, workspace, bias=None, relu=False, requant_mul=None,
                 row_absmax_out=None, out=None, out_dtype=torch.float16):
    M, K = Xq.shape
    N = Wq.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=Xq.device)
    wp, wn = _ws(workspace)
    _check(lib().sq_w8a8_gemm(
        _ptr(Xq), _ptr(Wq), M, N, K, _ptr(x_scale), 1 if (x_scale is not None and x_scale.numel() > 1) else 0,
        _ptr(w_scale), 1 if (w_scale is not None and w_scale.numel() > 1) else 0, _ptr(bias),
        _DT[bias.dtype] if bias is not None else SQ_F16, SQ_EPI_RELU if relu else SQ_EPI_NONE,
        _ptr(requant_mul), 1 if (requant_mul is not None and requant_mul.numel() > 1) else 0,
        _ptr(row_absmax_out), _ptr(out), _DT[out.dtype], out.stride(0), wp, wn, _stream()), "sq_w8a8_gemm")
    return out


def sq_w8a8_gemm_residual(Xq, Wq, x_scale, w_scale, workspace, residual, bias=None, out=None):
    """The W8A8 linear plus the residual stream: out = round(round(y) + residual), out dtype = residual's."""
    M, K = Xq.shape
    N = Wq.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=residual.dtype, device=Xq.device)
    wp, wn = _ws(workspace)
    _check(lib().sq_w8a8_gemm_residual(
        _ptr(Xq), _ptr(Wq), M, N, K, _ptr(x_scale), 1 if (x_scale is not None and x_scale.numel() > 1) else 0,
        _ptr(w_scale), 1 if (w_scale is not None and w_scale.numel() > 1) else 0, _ptr(bias),
        _DT[bias.dtype] if bias is not None else SQ_F16, _ptr(residual), residual.stride(0),
        _ptr(out), _DT[out.dtype], out.stride(0), wp, wn, _stream()), "sq_w8a8_gemm_residual")
    return out


def sq_w8a8_gemm_fused_quant(X, Wq, w_scale, workspace, gran="per_token", x_scale=None, gamma_hat=None, beta_hat=None,
                             eps=1e-5, Xq_out=None, dbg_mean_rstd=None, bias=None, relu=False, requant_mul=None,
                             residual=None, out=None, out_dtype=None):
    """Decode-shaped W8A8 linear (M <= 32) on 16-bit activations: Eq. 1 (optionally behind the folded
    LayerNorm) runs in the GEMM kernel's prologue.  gran: "per_token" (x_scale: optional [M] output) or
    "per_tensor_static" (x_scale: [1] input)."""
    M, K = X.shape
    N = Wq.shape[0]
    g = GRAN[gran] if isinstance(gran, str) else gran
    if out is None:
        odt = out_dtype or (torch.int8 if requant_mul is not None else (residual.dtype if residual is not None else X.dtype))
        out = torch.empty((M, N), dtype=odt, device=X.device)
    wp, wn = _ws(workspace)
    _check(lib().sq_w8a8_gemm_fused_quant(
        _ptr(X), _DT[X.dtype], M, N, K, _ptr(gamma_hat), _ptr(beta_hat), float(eps), g, _ptr(x_scale), _ptr(Xq_out),
        _ptr(dbg_mean_rstd), _ptr(Wq), _ptr(w_scale), 1 if w_scale.numel() > 1 else 0, _ptr(bias),
        _DT[bias.dtype] if bias is not None else SQ_F16, SQ_EPI_RELU if relu else SQ_EPI_NONE, _ptr(requant_mul),
        1 if (requant_mul is not None and requant_mul.numel() > 1) else 0, _ptr(residual),
        residual.stride(0) if residual is not None else 0, _ptr(out), _DT[out.dtype], out.stride(0), wp, wn, _stream()),
        "sq_w8a8_gemm_fused_quant")
    return out


def sq_w8a8_bmm(A, B, batch, heads, M, N, K, strideA, strideB, b_is_kn, alpha, C, strideC, workspace,
                requant_mul=None, causal=False):
    """A, B, C are base tensors (any shape); strides are (batch, head, row) in elements."""
    arr = ctypes.c_int64 * 3
    wp, wn = _ws(workspace)
    _check(lib().sq_w8a8_bmm(_ptr(A), _ptr(B), batch, heads, M, N, K, arr(*strideA), arr(*strideB),
                             1 if b_is_kn else 0, 1 if causal else 0, float(alpha), _ptr(requant_mul), _ptr(C),
                             _DT[C.dtype],
                             arr(*strideC), wp, wn, _stream()), "sq_w8a8_bmm")
    return C


def sq_softmax_quant_p(scores, Pq=None):
    n_mat, S, S2 = scores.shape
    assert S == S2
    if Pq is None:
        Pq = torch.empty((n_mat, S, S), dtype=torch.int8, device=scores.device)
    _check(lib().sq_softmax_quant_p(_ptr(scores), _DT[scores.dtype], n_mat, S, _ptr(Pq), _stream()),
           "sq_softmax_quant_p")
    return Pq


def sq_residual_add(a, b, out=None):
    if out is None:
        out = torch.empty_like(a)
    _check(lib().sq_residual_add(_ptr(a), _ptr(b), _DT[a.dtype], a.numel(), _ptr(out), _stream()),
           "sq_residual_add")
    return out


def sq_ln_quant_tensor_noalloc(X, gamma_hat, beta_hat, eps, Xq=None, x_scale=None):
    """Per-tensor-dynamic fused LayerNorm+quantise for callers that cannot allocate a workspace:
    the library's built-in scratch array is used instead.  At most SQ_NOALLOC_MAX_ROWS rows; calls
    that overlap on the GPU race on that array.  Make the first call outside any stream capture."""
    M, C = X.shape
    if Xq is None:
        Xq = torch.empty((M, C), dtype=torch.int8, device=X.device)
    if x_scale is None:
        x_scale = torch.empty(1, dtype=torch.float32, device=X.device)
    _check(lib().sq_ln_quant_tensor_noalloc(_ptr(X), _DT[X.dtype], M, C, _ptr(gamma_hat), _ptr(beta_hat),
                                            float(eps), _ptr(Xq), _ptr(x_scale), _stream()),
           "sq_ln_quant_tensor_noalloc")
    return Xq, x_scale


def sq_selftest_bounded_wait(budget_cycles=200000):
    """Runs the library's bounded-wait self-test; returns the status word the kernel left
    (SQ_ERR_TIMEOUT | where << 8 when the wait gave up as designed)."""
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(lib().sq_selftest_bounded_wait(_ptr(word), int(budget_cycles), _stream()), "sq_selftest_bounded_wait")
    return int(word.item())


def sq_selftest_row_wait(budget_cycles=200000):
    """The same self-test for the row kernels' wait on a row's bulk copy (expected: SQ_ERR_TIMEOUT | 5 << 8)."""
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(lib().sq_selftest_row_wait(_ptr(word), int(budget_cycles), _stream()), "sq_selftest_row_wait")
    return int(word.item())


def sq_w8a8_attention(qkv, B, H, S, d, alpha_qk, alpha_pv, requant_mul, out, workspace):
    """Fused causal INT8 attention over the fused QKV code buffer [B*S, 3*H*d] -> out [B*S, H*d] int8."""
    wp, wn = _ws(workspace)
    _check(lib().sq_w8a8_attention(_ptr(qkv), B, H, S, d, float(alpha_qk), float(alpha_pv), _ptr(requant_mul),
                                   _ptr(out), wp, wn, _stream()), "sq_w8a8_attention")
    return out


def sq_kv_cache_write(qkv, B, T, H, d, pos0, k_cache, v_cache, L_max, workspace):
    """Copies K and V codes of T tokens per sequence from the QKV code buffer [B*T, 3*H*d] into the
    INT8 cache at positions pos0[b] .. (pos0: int32 device tensor or None = 0)."""
    wp, wn = _ws(workspace)
    _check(lib().sq_kv_cache_write(_ptr(qkv), qkv.stride(0), B, T, H, d, _ptr(pos0), _ptr(k_cache), _ptr(v_cache),
                                   L_max, wp, wn, _stream()), "sq_kv_cache_write")


def sq_w8a8_decode_attention(q, k_cache, v_cache, seq_lens, B, H, d, L_max, max_len, alpha_qk, alpha_pv, workspace,
                             requant_mul=None, out=None, out_dtype=None, k_new=None, v_new=None):
    """Attention of each sequence's newest token over the INT8 cache.  q: [B, >= H*d] int8 (row stride
    taken from the tensor); seq_lens: int32 device tensor [B]; out: [B, H*d] int8 / fp16 / bf16.
    k_new / v_new: [B, >= H*d] int8 rows of the newest token when it is not in the cache yet (same
    row stride for both); the kernel then appends them itself."""
    if k_new is not None and k_new.stride(0) != v_new.stride(0):
        raise ValueError("k_new and v_new must share one row stride")
    if out is None:
        out = torch.empty((B, H * d), dtype=out_dtype or (torch.int8 if requant_mul is not None else torch.float16),
                          device=q.device)
    wp, wn = _ws(workspace)
    _check(lib().sq_w8a8_decode_attention(_ptr(q), q.stride(0), _ptr(k_cache), _ptr(v_cache), _ptr(k_new), _ptr(v_new),
                                          k_new.stride(0) if k_new is not None else 0, _ptr(seq_lens), B, H, d,
                                          L_max, max_len, float(alpha_qk), float(alpha_pv), _ptr(requant_mul), _ptr(out),
                                          _DT[out.dtype], out.stride(0), wp, wn, _stream()), "sq_w8a8_decode_attention")
    return out


def sq_token_absmax(X, out=None):
    """Per-token absolute maximum of a calibration batch [M, C] -> fp32 [M]."""
    M, C = X.shape
    if out is None:
        out = torch.empty(M, dtype=torch.float32, device=X.device)
    _check(lib().sq_token_absmax(_ptr(X), _DT[X.dtype], M, C, X.stride(0), _ptr(out), _stream()), "sq_token_absmax")
    return out


def sq_clipped_absmax(token_absmax, n_clip):
    """Largest of the per-token maxima after the n_clip largest have been set aside -> (absmax[1], step[1])."""
    a = torch.empty(1, dtype=torch.float32, device=token_absmax.device)
    s = torch.empty(1, dtype=torch.float32, device=token_absmax.device)
    _check(lib().sq_clipped_absmax(_ptr(token_absmax), token_absmax.numel(), int(n_clip), _ptr(a), _ptr(s), _stream()),
           "sq_clipped_absmax")
    return a, s
