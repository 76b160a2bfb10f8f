"""GPU parity of the generation-stage linear with the activation quantiser in the GEMM's prologue
(sq_w8a8_gemm_fused_quant): 16-bit activations in, Eq. 1 (optionally behind the folded LayerNorm)
inside the weight-streaming kernel, Eq. 2 out.  Everything is compared with the oracle's unfused
definition on the same bytes: codes, step sizes and INT8 outputs byte for byte, 16-bit outputs
byte for byte as well (the epilogue arithmetic is fully specified)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import dev, host, assert_fp_close
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import synth

pytestmark = pytest.mark.gpu

TDT = {"f16": torch.float16, "bf16": torch.bfloat16}


def _acts(tid, M, K, dtype):
    n_out = max(1, K // 100)
    ch = synth.outlier_channels(4, K, count=n_out)
    fac = synth.outlier_factors(4, n_out, 20.0, 80.0)
    return synth.activations(4, tid, M, K, dtype, ch, fac)


def _ws(M, N, K):
    return sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_GEMM_FUSED_QUANT, M, N, K))


SHAPES = [(1, 384, 512), (3, 200, 272), (16, 1280, 4096), (17, 640, 1024), (32, 2048, 7168), (5, 256, 12288),
          (16, 512, 16384), (2, 128, 49152), (16, 4096, 12288)]


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_fused_per_token_quant_matches_quant_act_then_gemm(dtype, M, N, K):
    x = _acts(1, M, K, dtype)
    Wq = synth.int8_tensor(4, 2, (N, K))
    rng = synth.rng_for(4, 3)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(4, 4, N, dtype, std=0.5)
    want_q, want_s = oracle.quant_act(x, "per_token")
    _, want_y = oracle.w8a8_linear(want_q, want_s, Wq, wsc, bias=bias, out_dtype=dtype)
    ws = _ws(M, N, K)
    xs = torch.zeros(M, dtype=torch.float32, device="cuda")
    Xq = torch.zeros((M, K), dtype=torch.int8, device="cuda")
    y = sq.sq_w8a8_gemm_fused_quant(dev(x, dtype), dev(Wq), dev(wsc), ws, "per_token", x_scale=xs, Xq_out=Xq,
                                    bias=dev(bias, dtype))
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0
    assert np.array_equal(host(xs), want_s) and np.array_equal(host(Xq), want_q)
    assert_fp_close(host(y), want_y, dtype, "fused decode linear")
    assert np.array_equal(host(y), want_y)
    assert not ws[4:33024].any()  # header, meeting counters and arrival counters handed back zeroed
    # the same call with the codes and step sizes kept in the workspace gives the same bytes
    y2 = sq.sq_w8a8_gemm_fused_quant(dev(x, dtype), dev(Wq), dev(wsc), ws, "per_token", bias=dev(bias, dtype))
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    # and so does the two-launch path
    Xq2, xs2 = sq.sq_quant_act(dev(x, dtype), "per_token")
    y3 = sq.sq_w8a8_gemm(Xq2, dev(Wq), xs2, dev(wsc), ws, bias=dev(bias, dtype), out_dtype=TDT[dtype])
    assert torch.equal(y.view(torch.int16), y3.view(torch.int16))


@pytest.mark.parametrize("M,N,K", [(1, 384, 512), (16, 1280, 4096), (32, 640, 7168), (4, 256, 28672)])
def test_fused_static_quant_relu_requant(M, N, K):
    """The generation-stage FC1 of the static block: static input step (values beyond it saturate),
    ReLU, re-quantised INT8 output with a static step."""
    dtype = "f16"
    x = _acts(5, M, K, dtype)
    Wq = synth.int8_tensor(4, 6, (N, K))
    rng = synth.rng_for(4, 7)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(4, 8, N, dtype, std=0.5)
    delta = np.array([oracle.step_size(0.3 * float(np.abs(x).max()))], np.float32)  # the largest values saturate
    r = np.array([25.0], np.float32)
    want_q, _ = oracle.quant_act(x, "per_tensor_static", static_scale=delta)
    assert (np.abs(want_q) == 127).sum() >= 1
    _, want_y = oracle.w8a8_linear(want_q, delta, Wq, wsc, bias=bias, relu=True, requant_mul=r)
    ws = _ws(M, N, K)
    Xq = torch.zeros((M, K), dtype=torch.int8, device="cuda")
    y = sq.sq_w8a8_gemm_fused_quant(dev(x, dtype), dev(Wq), dev(wsc), ws, "per_tensor_static", x_scale=dev(delta), Xq_out=Xq,
                                    bias=dev(bias, dtype), relu=True, requant_mul=dev(r))
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0 and y.dtype == torch.int8
    assert np.array_equal(host(Xq), want_q)
    assert np.array_equal(host(y), want_y)
    assert np.abs(want_y).max() > 20
    assert not ws[4:33024].any()


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("gran", ["per_token", "per_tensor_static"])
@pytest.mark.parametrize("M,N,K", [(1, 384, 512), (16, 768, 7168), (32, 512, 12288), (7, 256, 20480)])
def test_fused_layernorm_quant(dtype, gran, M, N, K):
    """LayerNorm with folded parameters in the prologue.  The kernel's own row statistics, fed to the
    oracle's element-wise path, must reproduce codes, step sizes and outputs byte for byte; the
    statistics themselves are checked against the fp64 two-pass values."""
    x = _acts(9, M, K, dtype)
    g, b = synth.ln_params(4, 10, K, dtype)
    Wq = synth.int8_tensor(4, 11, (N, K))
    rng = synth.rng_for(4, 12)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    ws = _ws(M, N, K)
    stats = torch.zeros(2 * M, dtype=torch.float32, device="cuda")
    Xq = torch.zeros((M, K), dtype=torch.int8, device="cuda")
    kw, okw = {}, {}
    if gran == "per_tensor_static":
        delta = np.array([0.02], np.float32)
        kw["x_scale"], okw["static_scale"] = dev(delta), delta
    else:
        kw["x_scale"] = torch.zeros(M, dtype=torch.float32, device="cuda")
    y = sq.sq_w8a8_gemm_fused_quant(dev(x, dtype), dev(Wq), dev(wsc), ws, gran, gamma_hat=dev(g, dtype), beta_hat=dev(b, dtype),
                                    eps=1e-5, Xq_out=Xq, dbg_mean_rstd=stats, **kw)
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0
    st = host(stats).reshape(M, 2)
    mu, rstd = oracle.ln_stats(x, 1e-5)
    assert np.all(np.abs(st[:, 0] - mu) <= 1e-6 * np.maximum(np.abs(mu), np.sqrt(1.0 / rstd ** 2)))
    assert np.all(np.abs(st[:, 1] - rstd) <= 1e-6 * rstd)
    want_q, want_s, _ = oracle.ln_quant(x, g, b, 1e-5, gran, stats=(st[:, 0].copy(), st[:, 1].copy()), **okw)
    assert np.array_equal(host(Xq), want_q)
    if gran == "per_token":
        assert np.array_equal(host(kw["x_scale"]), want_s)
    _, want_y = oracle.w8a8_linear(want_q, want_s, Wq, wsc, out_dtype=dtype)
    assert np.array_equal(host(y), want_y)
    assert not ws[4:33024].any()


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_fused_quant_with_residual_epilogue(dtype):
    M, N, K = 16, 1024, 4096
    x = _acts(13, M, K, dtype)
    res = synth.activations(4, 14, M, N, dtype, [5], [30.0])
    Wq = synth.int8_tensor(4, 15, (N, K))
    wsc = synth.rng_for(4, 16).uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(4, 17, N, dtype, std=0.5)
    want_q, want_s = oracle.quant_act(x, "per_token")
    _, y = oracle.w8a8_linear(want_q, want_s, Wq, wsc, bias=bias, out_dtype=dtype)
    want = oracle.round_to(y + res, dtype)
    ws = _ws(M, N, K)
    got = sq.sq_w8a8_gemm_fused_quant(dev(x, dtype), dev(Wq), dev(wsc), ws, "per_token", bias=dev(bias, dtype),
                                      residual=dev(res, dtype))
    assert np.array_equal(host(got), want) and sq.device_status(ws) == 0


def test_fused_quant_calls_in_a_row_share_one_workspace():
    """Different token counts and shapes back to back on one stream and one workspace (the meeting
    counters must come back zeroed every time), behind a kernel that produces X on the same stream."""
    dtype = "bf16"
    N, K = 1536, 4096
    Wq = synth.int8_tensor(4, 20, (N, K))
    wsc = synth.rng_for(4, 21).uniform(1e-4, 1e-3, N).astype(np.float32)
    ws = _ws(32, N, K)
    Wd, wd = dev(Wq), dev(wsc)
    for it, M in enumerate([16, 1, 32, 5, 16, 16]):
        a = _acts(30 + it, M, K, dtype)
        b = _acts(40 + it, M, K, dtype)
        x = oracle.round_to(a + b, dtype)
        xd = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        sq.sq_residual_add(dev(a, dtype), dev(b, dtype), out=xd)  # X comes from the launch directly in front
        y = sq.sq_w8a8_gemm_fused_quant(xd, Wd, wd, ws, "per_token")
        want_q, want_s = oracle.quant_act(x, "per_token")
        _, want_y = oracle.w8a8_linear(want_q, want_s, Wq, wsc, out_dtype=dtype)
        assert np.array_equal(host(y), want_y), "call %d (M = %d)" % (it, M)
    assert sq.device_status(ws) == 0 and not ws[4:33024].any()


def test_fused_quant_argument_checks():
    M, N, K = 4, 256, 512
    x = torch.zeros((M, K), dtype=torch.float16, device="cuda")
    Wq = torch.zeros((N, K), dtype=torch.int8, device="cuda")
    wsc = torch.ones(N, device="cuda")
    ws = _ws(M, N, K)
    with pytest.raises(sq.SqError) as e:  # one step for the whole tensor is not offered fused
        sq.sq_w8a8_gemm_fused_quant(x, Wq, wsc, ws, "per_tensor_dynamic", x_scale=torch.ones(1, device="cuda"))
    assert e.value.code == sq.SQ_ERR_UNSUPPORTED
    with pytest.raises(sq.SqError) as e:  # more than 32 tokens
        sq.sq_w8a8_gemm_fused_quant(torch.zeros((33, K), dtype=torch.float16, device="cuda"), Wq, wsc, _ws(32, N, K), "per_token")
    assert e.value.code == sq.SQ_ERR_UNSUPPORTED
    with pytest.raises(sq.SqError) as e:  # static mode needs its step
        sq.sq_w8a8_gemm_fused_quant(x, Wq, wsc, ws, "per_tensor_static")
    assert e.value.code == sq.SQ_ERR_INVALID_ARG
    with pytest.raises(sq.SqError) as e:  # the plain GEMM's workspace is too small for the codes
        sq.sq_w8a8_gemm_fused_quant(x, Wq, wsc, sq.new_workspace(256), "per_token")
    assert e.value.code == sq.SQ_ERR_WORKSPACE
