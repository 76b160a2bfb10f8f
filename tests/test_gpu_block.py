"""GPU integration: the whole static-step W8A8 decoder block (Fig. 6 precision mapping) against the
oracle's composition of the same steps.  Strict, bit-exact parity is asserted stage by stage in the
other GPU test files; here upstream float reductions (LayerNorm statistics, softmax sums) may flip
codes that sit on a rounding tie, so integer tensors are compared by code distance and mismatch
fraction and the final output by relative error."""
import numpy as np
import pytest
import torch

import oracle
from helpers import dev, host
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

    def codes_close(name, got, ref, max_frac):
        diff = np.abs(host(got).astype(np.int32).reshape(ref.shape) - ref.astype(np.int32))
        assert diff.max() <= 2, "%s: codes differ by %d" % (name, diff.max())
        frac = (diff != 0).mean()
        assert frac <= max_frac, "%s: %.4f of codes differ" % (name, frac)

    codes_close("LN1 codes", blk.x1q, want["x1q"], 1e-3)
    codes_close("QKV codes", blk.qkv, want["qkv"], 5e-3)
    if not blk.fused_attention:  # the fused attention kernel never materialises P
        codes_close("P codes", blk.P, want["P"].reshape(B * H, S, S), 2e-2)
    codes_close("attention codes", blk.attn, want["attn"], 2e-2)
    codes_close("FC1 codes", blk.f1q, want["f1q"], 2e-2)
    got = host(y).astype(np.float64)
    ref = want["y"].astype(np.float64)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel <= 5e-3, "block output relative error %.3g" % rel
    # the quantised block stays close to the unquantised fp64 block on the linear part it shares:
    # out-proj input is what it is, so only sanity-check magnitudes here
    assert np.isfinite(got).all() and np.abs(got).max() < 1e4


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
    generated tokens through the generation-stage block; each step against the oracle's generation
    block, which walks its own caches (oracle prompt codes -> oracle cache)."""
    B, S, H, d, ffn, L_max = 2, 128, 2, 128, 1024, 160
    hid = H * d
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

    def codes_close(name, got, ref, max_frac):
        diff = np.abs(host(got).astype(np.int32).reshape(ref.shape) - ref.astype(np.int32))
        assert diff.max() <= 2, "%s: codes differ by %d" % (name, diff.max())
        assert (diff != 0).mean() <= max_frac, "%s: %.4f of codes differ" % (name, (diff != 0).mean())

    ch = synth.outlier_channels(3, hid, count=max(1, hid // 100))
    fac = synth.outlier_factors(3, len(ch), 20.0, 80.0)
    for t in range(3):
        xt = synth.activations(3, 100 + t, B, hid, dtype, ch, fac)
        want = oracle.decoder_block_static_decode(xt, p, Kc, Vc, [S + t] * B, H, d, dtype)
        y = gen.step(dev(xt, dtype), max_len=S + 3)
        torch.cuda.synchronize()
        assert sq.device_status(gen.ws) == 0
        codes_close("LN1 codes", gen.x1q, want["x1q"], 2e-3)
        codes_close("QKV codes", gen.qkv, want["qkv"], 1e-2)
        codes_close("attention codes", gen.attn, want["attn"], 3e-2)
        codes_close("FC1 codes", gen.f1q, want["f1q"], 3e-2)
        got, ref = host(y).astype(np.float64), want["y"].astype(np.float64)
        rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert rel <= 5e-3, "step %d: block output relative error %.3g" % (t, rel)
    # the cache now holds S + 3 positions per sequence, equal to the oracle's up to near-tie codes
    assert host(gen.ctx).tolist() == [S + 3] * B
    codes_close("K cache", gen.k_cache[:, :, :S + 3], Kc[:, :, :S + 3], 5e-3)
    v_logical = gen.v_cache.permute(0, 1, 2, 4, 3).reshape(B, H, L_max, d)
    codes_close("V cache", v_logical[:, :, :S + 3], Vc[:, :, :S + 3], 5e-3)
