"""GPU parity at the benchmark's full sizes, in the launch configurations bench.py times.
The oracle cannot brute-force 10^11..10^13 MACs, so each check is one of:
  * sampled token rows carried through the whole chain by the oracle (every stage of the
    per-token path is row-independent, so a sampled row has exactly one correct result);
  * a Freivalds check of the complete INT32 accumulator matrix in exact int64 arithmetic:
    Xq (Wq^T r) == ACC r for random integer vectors r (a wrong entry survives with p <= 1/255 per r);
  * full comparison where the stage is O(M*C) (quantisers, calibration absmax).
All inputs come from the seeded host generators; nothing produced by a CUDA kernel is fed to the oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import dev, host
from parity import attention_codes_valid, ln_codes_near_tie
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import pipeline as pl
from paper_2211_10438_b200 import synth

pytestmark = pytest.mark.gpu


def freivalds(Xq, Wq, acc, n_vec=3, seed=0):
    rng = np.random.default_rng(seed)
    X64, W64 = Xq.astype(np.int64), Wq.astype(np.int64)
    for _ in range(n_vec):
        r = rng.integers(-127, 128, size=Wq.shape[0]).astype(np.int64)
        lhs = X64 @ (W64.T @ r)
        rhs = acc.astype(np.int64) @ r
        if not np.array_equal(lhs, rhs):
            return False
    return True


def freivalds_big(Xq, Wq, acc, n_vec=2, seed=0, chunk=8192):
    """The same identity for operands of gigabytes: the products run in float64, weight rows a chunk at a
    time.  With |r| <= 63 every partial sum is an integer below 2^53 (127 * 127 * 63 * 81920 * ... stays
    under 9e15 for the shapes used), so float64 is exact."""
    rng = np.random.default_rng(seed)
    N, K = Wq.shape
    assert 127.0 * 127 * 63 * max(N, K) * 1.0 < 2.0 ** 53 / 127  # head-room for the second product
    for _ in range(n_vec):
        r = rng.integers(-63, 64, size=N).astype(np.float64)
        wr = np.zeros(K, np.float64)
        for n0 in range(0, N, chunk):
            wr += Wq[n0:n0 + chunk].astype(np.float64).T @ r[n0:n0 + chunk]
        lhs = np.concatenate([Xq[m0:m0 + chunk].astype(np.float64) @ wr for m0 in range(0, Xq.shape[0], chunk)])
        rhs = np.concatenate([acc[m0:m0 + chunk].astype(np.float64) @ r for m0 in range(0, acc.shape[0], chunk)])
        if not np.array_equal(lhs, rhs):
            return False
    return True


def test_opt13b_prefill_step_sampled_rows():
    """Config 2 exactly as bench.py runs it: LinearBlock.step at M=2048, hidden 5120, bf16,
    per-token dynamic / per-channel; 48 sampled tokens are carried through the oracle's chain."""
    wl = synth.WORKLOADS[2]
    M, hid = wl.tokens[0], wl.hidden
    ch, fac = wl.outliers()
    x_in = synth.activations(2, 1, M, hid, "bf16", ch, fac)
    attn = synth.activations(2, 2, M, hid, "bf16", ch, fac)
    g1, b1 = synth.ln_params(2, 3, hid, "bf16")
    g2, b2 = synth.ln_params(2, 4, hid, "bf16")
    rng = synth.rng_for(2, 5)
    lin, host_lin = {}, {}
    for i, l in enumerate(wl.linears):
        Wq = synth.int8_tensor(2, 10 + i, (l.N, l.K))
        w_scale = rng.uniform(1e-4, 1e-3, l.N).astype(np.float32)
        bias = synth.bias(2, 20 + i, l.N, "bf16")
        host_lin[l.name] = (Wq, w_scale, bias, l.relu)
        lin[l.name] = pl.PreparedLinear(l.name, dev(Wq), dev(w_scale), dev(bias, "bf16"), l.relu)
    lin["qkv"].gamma_hat, lin["qkv"].beta_hat = dev(g1, "bf16"), dev(b1, "bf16")
    lin["fc1"].gamma_hat, lin["fc1"].beta_hat = dev(g2, "bf16"), dev(b2, "bf16")
    blk = pl.LinearBlock(lin["qkv"], lin["out_proj"], lin["fc1"], lin["fc2"], M, torch.bfloat16)
    blk.step(dev(x_in, "bf16"), dev(attn, "bf16"))
    torch.cuda.synchronize()
    assert sq.device_status(blk.ws) == 0

    rows = np.sort(synth.rng_for(2, 6).choice(M, size=48, replace=False))
    # QKV branch: LayerNorm codes by the near-tie rule, step sizes to the statistics' tolerance, then the GEMM
    # exact on the GPU's own codes and step sizes (stage isolation)
    q1, s1, _ = oracle.ln_quant(x_in[rows], g1, b1, 1e-5, "per_token")
    got_q1, got_s1 = host(blk.buf["qkv"]["Xq"])[rows], host(blk.buf["qkv"]["xs"])[rows]
    assert np.all(np.abs(got_s1 - s1) <= 16 * np.spacing(s1))
    assert ln_codes_near_tie(got_q1, q1, x_in[rows], g1, b1, 1e-5, got_s1, "LN1 codes") <= 1e-3
    Wq, wsc, bias, relu = host_lin["qkv"]
    _, y_qkv = oracle.w8a8_linear(got_q1, got_s1, Wq, wsc, bias=bias, out_dtype="bf16")
    assert np.array_equal(host(blk.buf["qkv"]["Y"])[rows], y_qkv)
    # out-proj branch: the plain quantiser is bit-exact, and so is everything after it
    q2, s2 = oracle.quant_act(attn[rows], "per_token")
    assert np.array_equal(host(blk.buf["out_proj"]["Xq"])[rows], q2)
    assert np.array_equal(host(blk.buf["out_proj"]["xs"])[rows], s2)
    Wq, wsc, bias, relu = host_lin["out_proj"]
    _, h = oracle.w8a8_linear(q2, s2, Wq, wsc, bias=bias, out_dtype="bf16")
    assert np.array_equal(host(blk.buf["out_proj"]["Y"])[rows], h)
    # FC1: LayerNorm of h (the GPU's h equals the oracle's, just checked), GEMM exact on the GPU's codes
    q3, s3, _ = oracle.ln_quant(h, g2, b2, 1e-5, "per_token")
    got_q3, got_s3 = host(blk.buf["fc1"]["Xq"])[rows], host(blk.buf["fc1"]["xs"])[rows]
    assert np.all(np.abs(got_s3 - s3) <= 16 * np.spacing(s3))
    assert ln_codes_near_tie(got_q3, q3, h, g2, b2, 1e-5, got_s3, "LN2 codes") <= 1e-3
    Wq, wsc, bias, relu = host_lin["fc1"]
    _, a = oracle.w8a8_linear(got_q3, got_s3, Wq, wsc, bias=bias, relu=True, out_dtype="bf16")
    got_a = host(blk.buf["fc1"]["Y"])[rows]
    assert np.array_equal(got_a, a)
    # FC2: plain quantiser on the materialised FC1 output, then the GEMM: both exact
    q4, s4 = oracle.quant_act(got_a, "per_token")
    assert np.array_equal(host(blk.buf["fc2"]["Xq"])[rows], q4) and np.array_equal(host(blk.buf["fc2"]["xs"])[rows], s4)
    Wq, wsc, bias, relu = host_lin["fc2"]
    _, y = oracle.w8a8_linear(q4, s4, Wq, wsc, bias=bias, out_dtype="bf16")
    assert np.array_equal(host(blk.buf["fc2"]["Y"])[rows], y)


@pytest.mark.parametrize("name,M,N,K", [("opt13b-qkv", 2048, 15360, 5120), ("opt13b-fc2", 2048, 5120, 20480),
                                        ("mtnlg-outproj", 4096, 20480, 20480), ("opt30b-fc1-b4", 2048, 28672, 7168)])
def test_prefill_gemm_full_accumulator_matrix(name, M, N, K):
    Xq = synth.int8_tensor(30, 1, (M, K))
    Wq = synth.int8_tensor(30, 2, (N, K))
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K))
    acc = host(sq.sq_w8a8_gemm(dev(Xq), dev(Wq), None, None, ws, out_dtype=torch.int32))
    assert sq.device_status(ws) == 0
    assert freivalds(Xq, Wq, acc)
    rows = np.sort(synth.rng_for(30, 3).choice(M, size=24, replace=False))
    assert np.array_equal(acc[rows], oracle.gemm_i32(Xq[rows], Wq))
    cols = np.sort(synth.rng_for(30, 4).choice(N, size=24, replace=False))
    assert np.array_equal(acc[:, cols], oracle.gemm_i32(Xq, Wq[cols]))
    # dequantised output in the timed configuration (bf16, per-token x per-channel, bias) on the sampled rows
    rng = synth.rng_for(30, 5)
    xs = rng.uniform(0.01, 0.2, M).astype(np.float32)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(30, 6, N, "bf16", std=0.5)
    y = host(sq.sq_w8a8_gemm(dev(Xq), dev(Wq), dev(xs), dev(wsc), ws, bias=dev(bias, "bf16"), out_dtype=torch.bfloat16))
    want = oracle.round_to(oracle.dequant(acc[rows], xs[rows], wsc, bias), "bf16")
    assert np.array_equal(y[rows], want)


@pytest.mark.parametrize("name,N,K", [("gpt3-qkv", 36864, 12288), ("gpt3-fc2", 12288, 49152)])
@pytest.mark.parametrize("M", [1, 16])
def test_decode_gemm_full_size(name, N, K, M):
    Xq = synth.int8_tensor(31, 1, (M, K))
    Wq = synth.int8_tensor(31, 2, (N, K))
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K))
    rng = synth.rng_for(31, 3)
    xs = rng.uniform(0.01, 0.2, M).astype(np.float32)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    Wd = dev(Wq)
    acc = host(sq.sq_w8a8_gemm(dev(Xq), Wd, None, None, ws, out_dtype=torch.int32))
    want_acc = oracle.gemm_i32(Xq, Wq)  # M <= 16: the full product is affordable
    assert np.array_equal(acc, want_acc)
    y = host(sq.sq_w8a8_gemm(dev(Xq), Wd, dev(xs), dev(wsc), ws, out_dtype=torch.bfloat16))
    assert np.array_equal(y, oracle.round_to(oracle.dequant(want_acc, xs, wsc), "bf16"))
    assert sq.device_status(ws) == 0 and not ws[4:33024].any()


@pytest.mark.parametrize("gran", ["per_token", "per_tensor_dynamic", "per_tensor_static"])
def test_mtnlg_quantisers_full_tensor(gran):
    """Config 5 activation shape, M=4096 x 20480, outliers x100 in 0.5 % of channels: the plain
    quantiser is compared over the WHOLE tensor (bit-exact), the fused LayerNorm one on its statistics-fed codes."""
    wl = synth.WORKLOADS[5]
    M, C = 4096, wl.hidden
    ch, fac = wl.outliers()
    x = synth.activations(5, 1, M, C, "bf16", ch, fac)
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_LN_QUANT, M, 0, C))
    kw, okw = {}, {}
    if gran == "per_tensor_static":
        delta = np.array([oracle.step_size(0.8 * float(np.abs(x).max()))], np.float32)
        kw["x_scale"], okw["static_scale"] = dev(delta), delta
    Xq, xs = sq.sq_quant_act(dev(x, "bf16"), gran, workspace=ws, **kw)
    wq, wsx = oracle.quant_act(x, gran, **okw)
    assert np.array_equal(host(xs), wsx) and np.array_equal(host(Xq), wq)
    g, b = synth.ln_params(5, 2, C, "bf16")
    dbg = torch.zeros(2 * M, dtype=torch.float32, device="cuda")
    if gran == "per_tensor_static":
        kw["x_scale"] = dev(np.array([0.05], np.float32))
        okw["static_scale"] = np.array([0.05], np.float32)
    Xq, xs = sq.sq_ln_quant(dev(x, "bf16"), dev(g, "bf16"), dev(b, "bf16"), 1e-5, gran, dbg_mean_rstd=dbg, workspace=ws, **kw)
    st = host(dbg).reshape(M, 2)
    wq, wsx, _ = oracle.ln_quant(x, g, b, 1e-5, gran, stats=(st[:, 0].copy(), st[:, 1].copy()), **okw)
    assert np.array_equal(host(xs), wsx) and np.array_equal(host(Xq), wq)
    assert not ws.any()


def test_mtnlg_calibration_stream_and_alphas():
    """Config 5 calibration: running per-channel absmax over several [2048, 20480] batches with the
    same persistent outlier channels, then Eq. 4 for alpha in {0.5, 0.75, 0.85}."""
    wl = synth.WORKLOADS[5]
    C = wl.hidden
    ch, fac = wl.outliers()
    a = torch.zeros(C, dtype=torch.float32, device="cuda")
    want = None
    for j in range(4):
        xb = synth.activations(5, 10 + j, wl.extra["calib_tokens"], C, "bf16", ch, fac)
        sq.sq_calib_absmax(dev(xb, "bf16"), a)
        want = oracle.calib_absmax(xb, want)
    assert np.array_equal(host(a), want)
    assert set(np.argsort(want)[-len(ch):]) == set(ch)  # the outlier channels own the largest maxima
    W = synth.weights(5, 20, 1024, C, "bf16")
    aw = torch.zeros(C, dtype=torch.float32, device="cuda")
    sq.sq_calib_absmax(dev(W, "bf16"), aw)
    want_w = oracle.calib_absmax(W)
    assert np.array_equal(host(aw), want_w)
    for alpha in wl.extra["alphas"]:
        s = host(sq.sq_smooth_scales(a, aw, alpha))
        ref = oracle.smooth_scales(want, want_w, alpha)
        assert np.all(np.abs(s - ref) <= np.spacing(ref))
        Wq, wsc = sq.sq_quant_weight(dev(W, "bf16"), dev(s), "per_channel")
        oq, osc = oracle.quant_weight(W, s, "per_channel")  # same s on both sides
        assert np.array_equal(host(Wq), oq) and np.array_equal(host(wsc), osc)


def test_generation_attention_gpt3_shape_sampled_heads():
    """The KV-cache attention row exactly as bench.py launches it (96 heads x 128, batch 16, context
    lengths uniform in [1024, 2048], the kernel appending the newest token itself); 10 sampled
    (sequence, head) pairs go through the oracle, and the whole cache is checked for the append."""
    B, H, L, D = 16, 96, 2048, 128
    rng = synth.rng_for(40, 1)
    K = synth.int8_tensor(40, 2, (B, H, L, D), lo=-100, hi=100)
    V = synth.int8_tensor(40, 3, (B, H, L, D), lo=-100, hi=100)
    qkv = synth.int8_tensor(40, 4, (B, 3, H, D), lo=-100, hi=100)
    lens = rng.integers(L // 2, L + 1, B).astype(np.int32)
    for b in range(B):  # the newest token's true k, v; the cache holds junk at that position
        K[b, :, lens[b] - 1], V[b, :, lens[b] - 1] = qkv[b, 1], qkv[b, 2]
    Kj, Vj = K.copy(), V.copy()
    for b in range(B):
        Kj[b, :, lens[b] - 1], Vj[b, :, lens[b] - 1] = 99, -99
    kc = dev(Kj)
    vc = dev(np.ascontiguousarray(Vj.reshape(B, H, L // 4, 4, D).transpose(0, 1, 2, 4, 3)))
    qd = dev(qkv.reshape(B, 3 * H * D))
    a_qk, a_pv = np.float32(0.0009), np.float32(0.01 / 127)
    r = np.array([1000.0], np.float32)
    ws = sq.new_workspace(256)
    out = sq.sq_w8a8_decode_attention(qd, kc, vc, dev(lens), B, H, D, L, L, a_qk, a_pv, ws, requant_mul=dev(r),
                                      k_new=qd[:, H * D:], v_new=qd[:, 2 * H * D:])
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0
    got = host(out).reshape(B, H, D)
    pairs = {(int(b), int(h)) for b, h in zip(rng.integers(0, B, 10), rng.integers(0, H, 10))}
    for b, h in sorted(pairs):
        L_b = int(lens[b])
        sc = oracle.scale_acc(oracle.gemm_i32(qkv[b, 0, h][None, :], np.ascontiguousarray(K[b, h, :L_b])), float(a_qk))
        amb, multi, differ = attention_codes_valid(got[b, h][None, :], sc, [L_b], V[b, h, :L_b], a_pv, requant_mul=r)
        assert differ <= multi
        want, _ = oracle.kv_decode_attention(qkv[b:b + 1, 0, h:h + 1], K[b:b + 1, h:h + 1], V[b:b + 1, h:h + 1], [L_b],
                                             a_qk, a_pv, requant_mul=r)
        assert np.abs(want).max() > 5  # the comparison is not vacuous
    # the append: every sequence's newest position now holds its true k and v, nothing else moved
    gk = host(kc)
    gv = host(vc).transpose(0, 1, 2, 4, 3).reshape(B, H, L, D)
    assert np.array_equal(gk, K) and np.array_equal(gv, V)


def test_fused_attention_opt30b_shape_sampled_heads():
    """Fused prompt attention at the block benchmark's shape (56 heads x 128, S = 512, batch 16):
    8 sampled (sequence, head) pairs through the oracle's unfused chain with fp32 scores."""
    B, H, S, D = 16, 56, 512, 128
    qkv = synth.int8_tensor(41, 1, (B * S, 3 * H * D), lo=-100, hi=100)
    a_qk, a_pv = np.float32(0.0009), np.float32(0.01 / 127)
    r = np.array([1.0 / 0.004], np.float32)
    ws = sq.new_workspace(256)
    out = torch.empty((B * S, H * D), dtype=torch.int8, device="cuda")
    sq.sq_w8a8_attention(dev(qkv), B, H, S, D, a_qk, a_pv, dev(r), out, ws)
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0
    got = host(out).reshape(B, S, H, D)
    v5 = qkv.reshape(B, S, 3, H, D)
    rng = synth.rng_for(41, 2)
    for b, h in zip(rng.integers(0, B, 8), rng.integers(0, H, 8)):
        q, k, v = (np.ascontiguousarray(v5[b, :, i, h]) for i in range(3))
        _, scores = oracle.w8a8_bmm(q[None], k[None], float(a_qk), out_dtype="f32")
        P, _ = oracle.softmax_quant_p(scores[0])
        amb, multi, differ = attention_codes_valid(got[b, :, h], scores[0], np.arange(1, S + 1), v, a_pv, requant_mul=r,
                                                   P_oracle=P)
        assert amb <= 2e-3 and differ <= multi


# --------------------------------------------------------------------------------------------
# Config 5: the MT-NLG-530B layer shapes (hidden 20480, FFN 81920) at their own sizes
# --------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,M,N,K", [("mtnlg-fc1", 4096, 81920, 20480), ("mtnlg-fc2", 4096, 20480, 81920),
                                        ("mtnlg-qkv", 4096, 61440, 20480), ("mtnlg-fc2-16k", 16384, 20480, 81920)])
def test_mtnlg_prefill_gemm_full_accumulator_matrix(name, M, N, K):
    """The widest and the longest GEMMs of the configurations (K = 81920: 640 K blocks, the K split of a
    partly filled last wave active; N = 81920 / 61440), whole INT32 accumulator matrix by the Freivalds
    identity, 24 sampled rows and 24 sampled columns by brute force, the bf16 epilogue on the sampled rows."""
    Xq = synth.int8_tensor(32, 1, (M, K))
    Wq = synth.int8_tensor(32, 2, (N, K))
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K))
    Xd, Wd = dev(Xq), dev(Wq)
    acc_d = sq.sq_w8a8_gemm(Xd, Wd, None, None, ws, out_dtype=torch.int32)
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0
    acc = host(acc_d)
    del acc_d
    assert freivalds_big(Xq, Wq, acc)
    rows = np.sort(synth.rng_for(32, 3).choice(M, size=24, replace=False))
    assert np.array_equal(acc[rows], oracle.gemm_i32(Xq[rows], Wq))
    cols = np.sort(synth.rng_for(32, 4).choice(N, size=24, replace=False))
    assert np.array_equal(acc[:, cols], oracle.gemm_i32(Xq, np.ascontiguousarray(Wq[cols])))
    rng = synth.rng_for(32, 5)
    xs = rng.uniform(0.01, 0.2, M).astype(np.float32)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(32, 6, N, "bf16", std=0.5)
    y = sq.sq_w8a8_gemm(Xd, Wd, dev(xs), dev(wsc), ws, bias=dev(bias, "bf16"), out_dtype=torch.bfloat16)
    want = oracle.round_to(oracle.dequant(acc[rows], xs[rows], wsc, bias), "bf16")
    assert np.array_equal(host(y[torch.from_numpy(rows).cuda()]), want)
    assert sq.device_status(ws) == 0


@pytest.mark.parametrize("gran", ["per_token", "per_tensor_dynamic", "per_tensor_static"])
def test_mtnlg_ln_quant_16384_tokens(gran):
    """Fused LayerNorm + quantise at the largest token count of config 5 (16384 x 20480, outliers x100 in
    0.5 % of the channels), whole tensor: statistics against fp64, codes and step sizes exact given them."""
    wl = synth.WORKLOADS[5]
    M, C = 16384, wl.hidden
    ch, fac = wl.outliers()
    x = synth.activations(5, 3, M, C, "bf16", ch, fac)
    g, b = synth.ln_params(5, 2, C, "bf16")
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_LN_QUANT, M, 0, C))
    dbg = torch.zeros(2 * M, dtype=torch.float32, device="cuda")
    kw, okw = {}, {}
    if gran == "per_tensor_static":
        kw["x_scale"] = dev(np.array([0.05], np.float32))
        okw["static_scale"] = np.array([0.05], np.float32)
    Xq, xs = sq.sq_ln_quant(dev(x, "bf16"), dev(g, "bf16"), dev(b, "bf16"), 1e-5, gran, dbg_mean_rstd=dbg, workspace=ws, **kw)
    st = host(dbg).reshape(M, 2)
    mu, rstd = oracle.ln_stats(x, 1e-5)
    assert np.all(np.abs(st[:, 0] - mu) <= 1e-6 * np.maximum(np.abs(mu), 1.0 / rstd))
    assert np.all(np.abs(st[:, 1] - rstd) <= 1e-6 * rstd)
    wq, wsx, _ = oracle.ln_quant(x, g, b, 1e-5, gran, stats=(st[:, 0].copy(), st[:, 1].copy()), **okw)
    assert np.array_equal(host(xs), wsx) and np.array_equal(host(Xq), wq)
    assert sq.device_status(ws) == 0 and not ws[4:].any()


# --------------------------------------------------------------------------------------------
# Config 3: the OPT-30B-shaped block at its own size (hidden 7168, 56 heads x 128, FFN 28672, batch 4 x 512)
# --------------------------------------------------------------------------------------------
def test_opt30b_block_full_size_sampled_tokens_and_heads():
    """DecoderBlockStatic.forward as bench.py replays it, on 2048 tokens.  The oracle cannot walk 5 * 10^12
    MACs, so each stage is checked on a sample, fed the GPU's own upstream bytes: 16 tokens through
    LayerNorm codes (near-tie), QKV / out-proj+residual / FC1 / FC2+residual (exact); the fused attention
    on 2 (sequence, head) pairs over all 512 tokens (interval of valid codes)."""
    wl = synth.WORKLOADS[3]
    B, S, H, d, hid, ffn = 4, 512, wl.heads, wl.head_dim, wl.hidden, wl.ffn
    M, dtype, f32, eps = B * S, "f16", np.float32, 1e-5
    ch, fac = wl.outliers()
    x = synth.activations(3, 1, M, hid, dtype, ch, fac)
    g1, b1 = synth.ln_params(3, 30, hid, dtype)
    g2, b2 = synth.ln_params(3, 31, hid, dtype)
    rng = synth.rng_for(3, 40)
    P = {}
    lin = {}
    for i, l in enumerate(wl.linears):
        P[l.name] = dict(Wq=synth.int8_tensor(3, 50 + i, (l.N, l.K)), w_scale=rng.uniform(2e-4, 6e-4, l.N).astype(f32),
                         bias=synth.bias(3, 60 + i, l.N, dtype))
        lin[l.name] = pl.PreparedLinear(l.name, dev(P[l.name]["Wq"]), dev(P[l.name]["w_scale"]), dev(P[l.name]["bias"], dtype),
                                        l.relu)
    lin["qkv"].gamma_hat, lin["qkv"].beta_hat = dev(g1, dtype), dev(b1, dtype)
    lin["fc1"].gamma_hat, lin["fc1"].beta_hat = dev(g2, dtype), dev(b2, dtype)
    # static steps: given constants (what a calibration would hand over), picked so that every code range is used
    steps = dict(d_ln1=0.5, d_q=0.25, d_k=0.25, d_v=0.25, d_attn=0.06, d_ln2=0.5, d_fc1=0.4)
    blk = pl.DecoderBlockStatic(lin, steps, B, S, H, d, torch.float16)
    assert blk.fused_attention and blk.fuse_residual  # the configuration bench.py times
    y = blk.forward(dev(x, dtype))
    torch.cuda.synchronize()
    assert sq.device_status(blk.ws) == 0

    rows = np.sort(synth.rng_for(3, 41).choice(M, size=16, replace=False))
    ridx = torch.from_numpy(rows).cuda()
    take = lambda t: host(t[ridx])
    # LN1 -> QKV
    x1q = take(blk.x1q)
    q_or, _, _ = oracle.ln_quant(x[rows], g1, b1, eps, "per_tensor_static", static_scale=steps["d_ln1"])
    assert ln_codes_near_tie(x1q, q_or, x[rows], g1, b1, eps, steps["d_ln1"], "LN1 codes") <= 1e-3
    r = np.concatenate([np.full(hid, f32(1) / f32(steps[k]), f32) for k in ("d_q", "d_k", "d_v")])
    _, qkv_or = oracle.w8a8_linear(x1q, steps["d_ln1"], P["qkv"]["Wq"], P["qkv"]["w_scale"], bias=P["qkv"]["bias"], requant_mul=r)
    assert np.array_equal(take(blk.qkv), qkv_or)
    assert 20 < np.abs(qkv_or).max() and (np.abs(qkv_or) == 127).mean() < 0.05
    # attention: 2 (sequence, head) pairs, every token
    alpha_qk = float(f32(f32(steps["d_q"]) * f32(steps["d_k"])) / f32(np.sqrt(f32(d))))
    alpha_pv = float(f32(steps["d_v"]) / f32(127.0))
    r_attn = np.array([f32(1) / f32(steps["d_attn"])], f32)
    qkv_g = blk.qkv.view(B, S, 3, H, d)
    attn_g = blk.attn.view(B, S, H, d)
    for b, h in ((1, 7), (3, 50)):
        q, k, v = (np.ascontiguousarray(host(qkv_g[b, :, i, h])) for i in range(3))
        _, sc = oracle.w8a8_bmm(q[None], k[None], alpha_qk, out_dtype="f32")
        Por, _ = oracle.softmax_quant_p(sc[0])
        got = host(attn_g[b, :, h])
        amb, multi, differ = attention_codes_valid(got, sc[0], np.arange(1, S + 1), v, alpha_pv, requant_mul=r_attn, P_oracle=Por)
        assert amb <= 2e-3 and differ <= multi and np.abs(got).max() > 20
    # out-proj + residual, LN2, FC1, FC2 + residual on the sampled tokens
    attn_rows = take(blk.attn)
    _, proj = oracle.w8a8_linear(attn_rows, steps["d_attn"], P["out_proj"]["Wq"], P["out_proj"]["w_scale"],
                                 bias=P["out_proj"]["bias"], out_dtype=dtype)
    h_rows = take(blk.h)
    assert np.array_equal(h_rows, oracle.round_to(x[rows] + proj, dtype))
    x2q = take(blk.x2q)
    q_or, _, _ = oracle.ln_quant(h_rows, g2, b2, eps, "per_tensor_static", static_scale=steps["d_ln2"])
    assert ln_codes_near_tie(x2q, q_or, h_rows, g2, b2, eps, steps["d_ln2"], "LN2 codes") <= 1e-3
    _, f1q_or = oracle.w8a8_linear(x2q, steps["d_ln2"], P["fc1"]["Wq"], P["fc1"]["w_scale"], bias=P["fc1"]["bias"], relu=True,
                                   requant_mul=f32(1) / f32(steps["d_fc1"]))
    f1q = take(blk.f1q)
    assert np.array_equal(f1q, f1q_or) and np.abs(f1q).max() > 20
    _, fc2 = oracle.w8a8_linear(f1q, steps["d_fc1"], P["fc2"]["Wq"], P["fc2"]["w_scale"], bias=P["fc2"]["bias"], out_dtype=dtype)
    assert np.array_equal(take(y), oracle.round_to(h_rows + fc2, dtype))
