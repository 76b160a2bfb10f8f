"""GPU integration: the whole static-step W8A8 decoder block (Fig. 6 precision mapping) against the
oracle, stage by stage on the block's OWN intermediates (stage isolation): every stage is fed the
bytes the GPU produced upstream and must then match the oracle's stage byte for byte -- INT8 GEMM
outputs, residual adds, the final output -- except the two places where an order-dependent float
reduction decides a code: LayerNorm codes (near-tie rule against the fp64 LayerNorm) and the
attention output (the interval the admissible P matrices allow)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import dev, host
from parity import TAU_P, attention_codes_valid, ln_codes_near_tie, near_tie_codes
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import pipeline as pl
from paper_2211_10438_b200 import synth

pytestmark = pytest.mark.gpu


def _make_block(B, S, H, d, ffn, dtype):
    hid, M = H * d, B * S
    ch = synth.outlier_channels(3, hid, count=max(1, hid // 100))
    fac = synth.outlier_factors(3, len(ch), 20.0, 80.0)
    x = synth.activations(3, 1, M, hid, dtype, ch, fac)
    W = {"qkv": synth.weights(3, 10, 3 * hid, hid, dtype), "out_proj": synth.weights(3, 11, hid, hid, dtype),
         "fc1": synth.weights(3, 12, ffn, hid, dtype), "fc2": synth.weights(3, 13, hid, ffn, dtype)}
    bias = {n: synth.bias(3, 20 + i, W[n].shape[0], dtype) for i, n in enumerate(W)}
    g1, b1 = synth.ln_params(3, 30, hid, dtype)
    g2, b2 = synth.ln_params(3, 31, hid, dtype)
    return x, W, bias, (g1, b1, g2, b2)


def _oracle_prepare(x, W, bias, ln, B, S, H, d, dtype, alpha=0.5, eps=1e-5):
    """Offline transform + static-step calibration on the same batch, all with the oracle."""
    g1, b1, g2, b2 = ln
    hid = H * d
    p = {}
    mu, rstd = oracle.ln_stats(x, eps)
    ln1 = oracle.ln_apply(x, mu.astype(np.float32), rstd.astype(np.float32), g1, b1)  # unsmoothed LN1 output
    s1 = oracle.smooth_scales(oracle.calib_absmax(oracle.round_to(ln1, dtype)), oracle.calib_absmax(W["qkv"]), alpha)
    p["g1"], p["b1"] = oracle.fold_ln_weight(g1, b1, s1, dtype)
    p["s1"] = s1
    for n in W:
        p[n] = {"bias": bias[n]}
    p["qkv"]["Wq"], p["qkv"]["w_scale"] = oracle.quant_weight(W["qkv"], s1, "per_channel")
    p["out_proj"]["Wq"], p["out_proj"]["w_scale"] = oracle.quant_weight(W["out_proj"], None, "per_channel")
    p["fc2"]["Wq"], p["fc2"]["w_scale"] = oracle.quant_weight(W["fc2"], None, "per_channel")
    # static steps: maxima observed on this batch while walking the block with dynamic steps
    x1q, d1, _ = oracle.ln_quant(x, p["g1"], p["b1"], eps, "per_tensor_dynamic")
    p["d_ln1"] = float(d1[0])
    y = oracle.dequant(oracle.gemm_i32(x1q, p["qkv"]["Wq"]), d1, p["qkv"]["w_scale"], bias["qkv"])
    for i, k in enumerate(("d_q", "d_k", "d_v")):
        p[k] = oracle.step_size(float(np.abs(y[:, i * hid:(i + 1) * hid]).max()))
    p["d_attn"] = oracle.step_size(float(np.abs(y[:, 2 * hid:]).max()))  # attention output is a convex mix of V rows
    # second LayerNorm: smooth against FC1 using a provisional forward with these steps
    p["g2"], p["b2"], p["d_ln2"], p["d_fc1"] = g2, b2, 1.0, 1.0
    p["fc1"]["Wq"], p["fc1"]["w_scale"] = oracle.quant_weight(W["fc1"], None, "per_channel")
    tmp = oracle.decoder_block_static(x, p, B, S, H, d, dtype, eps)
    mu, rstd = oracle.ln_stats(tmp["h"], eps)
    ln2 = oracle.ln_apply(tmp["h"], mu.astype(np.float32), rstd.astype(np.float32), g2, b2)
    s2 = oracle.smooth_scales(oracle.calib_absmax(oracle.round_to(ln2, dtype)), oracle.calib_absmax(W["fc1"]), alpha)
    p["g2"], p["b2"] = oracle.fold_ln_weight(g2, b2, s2, dtype)
    p["s2"] = s2
    p["fc1"]["Wq"], p["fc1"]["w_scale"] = oracle.quant_weight(W["fc1"], s2, "per_channel")
    x2q, d2, _ = oracle.ln_quant(tmp["h"], p["g2"], p["b2"], eps, "per_tensor_dynamic")
    p["d_ln2"] = float(d2[0])
    f1 = oracle.dequant(oracle.gemm_i32(x2q, p["fc1"]["Wq"]), d2, p["fc1"]["w_scale"], bias["fc1"], relu=True)
    p["d_fc1"] = oracle.step_size(float(f1.max()))
    return p


@pytest.mark.parametrize("dtype,B,S,H,d,ffn", [("f16", 2, 128, 2, 128, 1024), ("bf16", 1, 256, 3, 64, 768)])
def test_decoder_block_static_against_oracle(dtype, B, S, H, d, ffn):
    x, W, bias, ln = _make_block(B, S, H, d, ffn, dtype)
    p = _oracle_prepare(x, W, bias, ln, B, S, H, d, dtype)
    fused = d == 128  # the pipeline then uses the fused attention kernel, whose scores stay in fp32
    want = oracle.decoder_block_static(x, p, B, S, H, d, dtype, score_dtype="f32" if fused else None)

    tdt = {"f16": torch.float16, "bf16": torch.bfloat16}[dtype]
    lin = {}
    for n in W:
        lin[n] = pl.PreparedLinear(n, dev(p[n]["Wq"]), dev(p[n]["w_scale"]), dev(bias[n], dtype), n == "fc1")
    lin["qkv"].gamma_hat, lin["qkv"].beta_hat = dev(p["g1"], dtype), dev(p["b1"], dtype)
    lin["fc1"].gamma_hat, lin["fc1"].beta_hat = dev(p["g2"], dtype), dev(p["b2"], dtype)
    steps = {k: p[k] for k in ("d_ln1", "d_q", "d_k", "d_v", "d_attn", "d_ln2", "d_fc1")}
    blk = pl.DecoderBlockStatic(lin, steps, B, S, H, d, tdt)
    y = blk.forward(dev(x, dtype))
    torch.cuda.synchronize()
    assert sq.device_status(blk.ws) == 0

    _check_block_stages(blk, y, x, p, B, S, H, d, dtype)
    # and the composed oracle block (its own intermediates all the way) stays within a few codes of it
    got, ref = host(y).astype(np.float64), want["y"].astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 5e-3


def _check_block_stages(blk, y, x, p, B, S, H, d, dtype, eps=1e-5):
    """Every stage of DecoderBlockStatic.forward against the oracle's stage on the GPU's own inputs."""
    f32 = np.float32
    hid = H * d
    # LN1 + static quantiser: codes near-tie against the oracle's
    x1q = host(blk.x1q)
    q_or, _, _ = oracle.ln_quant(x, p["g1"], p["b1"], eps, "per_tensor_static", static_scale=p["d_ln1"])
    assert ln_codes_near_tie(x1q, q_or, x, p["g1"], p["b1"], eps, p["d_ln1"], "LN1 codes") <= 1e-3
    # QKV GEMM with the re-quantising epilogue: exact on the GPU's LN1 codes
    r = np.concatenate([np.full(hid, f32(1) / f32(p[k]), f32) for k in ("d_q", "d_k", "d_v")])
    _, qkv_or = oracle.w8a8_linear(x1q, p["d_ln1"], p["qkv"]["Wq"], p["qkv"]["w_scale"], bias=p["qkv"]["bias"], requant_mul=r)
    qkv = host(blk.qkv)
    assert np.array_equal(qkv, qkv_or), "QKV codes"
    # attention on the GPU's QKV codes
    v5 = qkv.reshape(B, S, 3, H, d)
    alpha_qk = float(f32(f32(p["d_q"]) * f32(p["d_k"])) / f32(np.sqrt(f32(d))))
    alpha_pv = float(f32(p["d_v"]) / f32(127.0))
    r_attn = np.array([f32(1) / f32(p["d_attn"])], f32)
    attn = host(blk.attn).reshape(B, S, H, d)
    for b in range(B):
        for h in range(H):
            q, k, v = (np.ascontiguousarray(v5[b, :, i, h]) for i in range(3))
            if blk.fused_attention:  # fp32 scores, P never written: interval check
                _, sc = oracle.w8a8_bmm(q[None], k[None], alpha_qk, out_dtype="f32")
                amb, multi, differ = attention_codes_valid(attn[b, :, h], sc[0], np.arange(1, S + 1), v, alpha_pv,
                                                           requant_mul=r_attn)
                assert amb <= 2e-3 and differ <= multi
            else:  # three launches: scores exact, P near-tie on the GPU's scores, P.V exact on the GPU's P
                _, sc = oracle.w8a8_bmm(q[None], k[None], alpha_qk, out_dtype=dtype)
                sc_gpu = host(blk.scores)[b * H + h]
                tri = np.tril(np.ones((S, S), bool))  # tiles above the diagonal are never written
                assert np.array_equal(sc_gpu[tri], sc[0][tri]), "scores"
                P_gpu = host(blk.P)[b * H + h]
                P_or, _ = oracle.softmax_quant_p(np.where(tri, sc_gpu, 0.0).astype(np.float32))
                p64 = oracle.softmax_causal_f64(np.where(tri, sc_gpu, 0.0).astype(np.float32))
                assert near_tie_codes(P_gpu, P_or, 127.0 * p64, TAU_P, "P codes") <= 2e-3
                _, o = oracle.w8a8_bmm(P_gpu[None], v[None], alpha_pv, b_is_kn=True, requant_mul=r_attn)
                assert np.array_equal(attn[b, :, h], o[0]), "attention codes"
    # out-projection + residual: exact on the GPU's attention codes
    attn2 = attn.reshape(B * S, hid)
    _, proj = oracle.w8a8_linear(attn2, p["d_attn"], p["out_proj"]["Wq"], p["out_proj"]["w_scale"], bias=p["out_proj"]["bias"],
                                 out_dtype=dtype)
    h_gpu = host(blk.h)
    assert np.array_equal(h_gpu, oracle.round_to(np.asarray(x, f32) + proj, dtype)), "h = x + out_proj"
    # LN2 codes near-tie on the GPU's h; FC1 and FC2 exact on the GPU's codes
    x2q = host(blk.x2q)
    q_or, _, _ = oracle.ln_quant(h_gpu, p["g2"], p["b2"], eps, "per_tensor_static", static_scale=p["d_ln2"])
    assert ln_codes_near_tie(x2q, q_or, h_gpu, p["g2"], p["b2"], eps, p["d_ln2"], "LN2 codes") <= 1e-3
    _, f1q_or = oracle.w8a8_linear(x2q, p["d_ln2"], p["fc1"]["Wq"], p["fc1"]["w_scale"], bias=p["fc1"]["bias"], relu=True,
                                   requant_mul=f32(1) / f32(p["d_fc1"]))
    f1q = host(blk.f1q)
    assert np.array_equal(f1q, f1q_or), "FC1 codes"
    _, fc2 = oracle.w8a8_linear(f1q, p["d_fc1"], p["fc2"]["Wq"], p["fc2"]["w_scale"], bias=p["fc2"]["bias"], out_dtype=dtype)
    assert np.array_equal(host(y), oracle.round_to(h_gpu + fc2, dtype)), "y = h + FC2"
    assert np.abs(f1q).max() > 20 and np.abs(attn).max() > 20  # non-trivial codes


def test_decoder_block_is_deterministic():
    B, S, H, d, ffn = 1, 128, 2, 128, 512
    x, W, bias, ln = _make_block(B, S, H, d, ffn, "f16")
    p = _oracle_prepare(x, W, bias, ln, B, S, H, d, "f16")
    lin = {n: pl.PreparedLinear(n, dev(p[n]["Wq"]), dev(p[n]["w_scale"]), dev(bias[n], "f16"), n == "fc1") for n in W}
    lin["qkv"].gamma_hat, lin["qkv"].beta_hat = dev(p["g1"], "f16"), dev(p["b1"], "f16")
    lin["fc1"].gamma_hat, lin["fc1"].beta_hat = dev(p["g2"], "f16"), dev(p["b2"], "f16")
    steps = {k: p[k] for k in ("d_ln1", "d_q", "d_k", "d_v", "d_attn", "d_ln2", "d_fc1")}
    blk = pl.DecoderBlockStatic(lin, steps, B, S, H, d, torch.float16)
    xd = dev(x, "f16")
    a = blk.forward(xd).clone()
    b = blk.forward(xd).clone()
    assert torch.equal(a, b)


def test_host_streamed_block_matches_sequential_steps():
    """Five steps with different pinned host inputs through the overlapped copy/compute path give,
    byte for byte, what the same LinearBlock gives when stepped one input at a time."""
    M, hid, ffn = 384, 512, 2048
    rng = synth.rng_for(41, 1)
    shapes = {"qkv": (3 * hid, hid), "out_proj": (hid, hid), "fc1": (ffn, hid), "fc2": (hid, ffn)}
    lin = {}
    for i, (n, (N, K)) in enumerate(shapes.items()):
        lin[n] = pl.PreparedLinear(n, dev(synth.int8_tensor(41, 10 + i, (N, K))),
                                   dev(rng.uniform(1e-4, 1e-3, N).astype(np.float32)),
                                   dev(synth.bias(41, 20 + i, N, "bf16"), "bf16"), n == "fc1")
    for n, k in (("qkv", 3), ("fc1", 4)):
        g, b = synth.ln_params(41, k, hid, "bf16")
        lin[n].gamma_hat, lin[n].beta_hat = dev(g, "bf16"), dev(b, "bf16")
    blk = pl.LinearBlock(lin["qkv"], lin["out_proj"], lin["fc1"], lin["fc2"], M, torch.bfloat16)
    xs = [torch.from_numpy(synth.activations(41, 30 + i, M, hid, "bf16", [3, 77], [40.0, 25.0])).to(torch.bfloat16).pin_memory()
          for i in range(5)]
    ats = [torch.from_numpy(synth.activations(41, 40 + i, M, hid, "bf16", [3, 77], [40.0, 25.0])).to(torch.bfloat16).pin_memory()
           for i in range(5)]
    want = []
    for x, a in zip(xs, ats):
        want.append(blk.step(x.cuda(), a.cuda()).cpu().clone())
    outs = [torch.empty((M, hid), dtype=torch.bfloat16).pin_memory() for _ in range(5)]
    st = pl.HostStreamedBlock(blk, hid)
    for x, a, o in zip(xs, ats, outs):
        st.submit(x, a, o)
    st.drain()
    torch.cuda.synchronize()
    assert sq.device_status(blk.ws) == 0
    for o, w in zip(outs, want):
        assert torch.equal(o.view(torch.int16), w.view(torch.int16))


@pytest.mark.parametrize("fused,fuse_residual", [(True, True), (False, True), (False, False)])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_generation_stage_block_against_oracle(dtype, fused, fuse_residual):
    """Prompt pass of 128 tokens with the prompt block, cache filled from its QKV codes, then three
    generated tokens through the generation-stage block.  Every stage of every step is checked against
    the oracle's stage on the GPU's own upstream bytes; the composed oracle block, walking its own
    caches, must stay close."""
    B, S, H, d, ffn, L_max = 2, 128, 2, 128, 1024, 160
    hid = H * d
    f32 = np.float32
    eps = 1e-5
    x, W, bias, ln = _make_block(B, S, H, d, ffn, dtype)
    p = _oracle_prepare(x, W, bias, ln, B, S, H, d, dtype)
    prompt = oracle.decoder_block_static(x, p, B, S, H, d, dtype, score_dtype="f32")
    qkv = prompt["qkv"].reshape(B, S, 3, H, d)
    Kc, Vc = np.zeros((B, H, L_max, d), np.int8), np.zeros((B, H, L_max, d), np.int8)
    Kc[:, :, :S] = qkv[:, :, 1].transpose(0, 2, 1, 3)
    Vc[:, :, :S] = qkv[:, :, 2].transpose(0, 2, 1, 3)

    tdt = {"f16": torch.float16, "bf16": torch.bfloat16}[dtype]
    lin = {}
    for n in W:
        lin[n] = pl.PreparedLinear(n, dev(p[n]["Wq"]), dev(p[n]["w_scale"]), dev(bias[n], dtype), n == "fc1")
    lin["qkv"].gamma_hat, lin["qkv"].beta_hat = dev(p["g1"], dtype), dev(p["b1"], dtype)
    lin["fc1"].gamma_hat, lin["fc1"].beta_hat = dev(p["g2"], dtype), dev(p["b2"], dtype)
    steps = {k: p[k] for k in ("d_ln1", "d_q", "d_k", "d_v", "d_attn", "d_ln2", "d_fc1")}
    blk = pl.DecoderBlockStatic(lin, steps, B, S, H, d, tdt)
    blk.forward(dev(x, dtype))
    gen = pl.DecoderBlockDecode(lin, steps, B, H, d, L_max, tdt, fused=fused, fuse_residual=fuse_residual, keep_codes=True)
    assert gen.launches_per_step == 9 - 2 * fused - 2 * fuse_residual
    gen.load_prompt(blk.qkv, S)
    v_logical = lambda: host(gen.v_cache.permute(0, 1, 2, 4, 3).reshape(B, H, L_max, d))
    k_gpu, v_gpu = host(gen.k_cache), v_logical()  # what the GPU's own prompt pass cached

    r_qkv = np.concatenate([np.full(hid, f32(1) / f32(p[k]), f32) for k in ("d_q", "d_k", "d_v")])
    alpha_qk = float(f32(f32(p["d_q"]) * f32(p["d_k"])) / f32(np.sqrt(f32(d))))
    alpha_pv = float(f32(p["d_v"]) / f32(127.0))
    r_attn = np.array([f32(1) / f32(p["d_attn"])], f32)
    ch = synth.outlier_channels(3, hid, count=max(1, hid // 100))
    fac = synth.outlier_factors(3, len(ch), 20.0, 80.0)
    for t in range(3):
        xt = synth.activations(3, 100 + t, B, hid, dtype, ch, fac)
        want = oracle.decoder_block_static_decode(xt, p, Kc, Vc, [S + t] * B, H, d, dtype)
        y = gen.step(dev(xt, dtype), max_len=S + 3)
        torch.cuda.synchronize()
        assert sq.device_status(gen.ws) == 0
        # LN1 codes (near-tie), QKV codes (exact on the GPU's LN1 codes)
        x1q = host(gen.x1q)
        q_or, _, _ = oracle.ln_quant(xt, p["g1"], p["b1"], eps, "per_tensor_static", static_scale=p["d_ln1"])
        assert ln_codes_near_tie(x1q, q_or, xt, p["g1"], p["b1"], eps, p["d_ln1"], "LN1 codes") <= 2e-3
        _, qkv_or = oracle.w8a8_linear(x1q, p["d_ln1"], p["qkv"]["Wq"], p["qkv"]["w_scale"], bias=p["qkv"]["bias"], requant_mul=r_qkv)
        qkv_g = host(gen.qkv)
        assert np.array_equal(qkv_g, qkv_or), "QKV codes"
        # the append: position S + t of the cache now holds this token's k and v codes, nothing else moved
        q3 = qkv_g.reshape(B, 3, H, d)
        k_gpu[:, :, S + t], v_gpu[:, :, S + t] = q3[:, 1], q3[:, 2]
        assert np.array_equal(host(gen.k_cache), k_gpu) and np.array_equal(v_logical(), v_gpu)
        # attention of the new token over the GPU's cache: interval of valid codes
        attn = host(gen.attn).reshape(B, H, d)
        L = S + t + 1
        for b in range(B):
            for h in range(H):
                acc = oracle.gemm_i32(q3[b, 0, h][None, :], np.ascontiguousarray(k_gpu[b, h, :L]))
                sc = oracle.scale_acc(acc, alpha_qk)
                amb, multi, differ = attention_codes_valid(attn[b, h][None, :], sc, [L], v_gpu[b, h, :L], alpha_pv,
                                                           requant_mul=r_attn)
                assert differ <= multi
        # out-projection + residual, LN2, FC1, FC2 + residual on the GPU's own intermediates
        _, proj = oracle.w8a8_linear(attn.reshape(B, hid), p["d_attn"], p["out_proj"]["Wq"], p["out_proj"]["w_scale"],
                                     bias=p["out_proj"]["bias"], out_dtype=dtype)
        h_gpu = host(gen.h)
        assert np.array_equal(h_gpu, oracle.round_to(xt + proj, dtype)), "h"
        x2q = host(gen.x2q)
        q_or, _, _ = oracle.ln_quant(h_gpu, p["g2"], p["b2"], eps, "per_tensor_static", static_scale=p["d_ln2"])
        assert ln_codes_near_tie(x2q, q_or, h_gpu, p["g2"], p["b2"], eps, p["d_ln2"], "LN2 codes") <= 2e-3
        _, f1q_or = oracle.w8a8_linear(x2q, p["d_ln2"], p["fc1"]["Wq"], p["fc1"]["w_scale"], bias=p["fc1"]["bias"], relu=True,
                                       requant_mul=f32(1) / f32(p["d_fc1"]))
        f1q = host(gen.f1q)
        assert np.array_equal(f1q, f1q_or), "FC1 codes"
        _, fc2 = oracle.w8a8_linear(f1q, p["d_fc1"], p["fc2"]["Wq"], p["fc2"]["w_scale"], bias=p["fc2"]["bias"], out_dtype=dtype)
        assert np.array_equal(host(y), oracle.round_to(h_gpu + fc2, dtype)), "y"
        # the composed oracle block (own caches, own intermediates) stays close
        got, ref = host(y).astype(np.float64), want["y"].astype(np.float64)
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 5e-3, "step %d" % t
    assert host(gen.ctx).tolist() == [S + 3] * B
