"""GPU tests of the shipped offline walk: pipeline.prepare_linear (calibration absmax -> Eq. 4 -> fold
into LayerNorm and weight -> Eq. 1 on the weight) and pipeline.calibrate_static_steps (static
per-tensor steps of the O3 block), against the oracle's composition of the same steps."""
import numpy as np
import pytest
import torch

import oracle
from helpers import dev, host
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import pipeline as pl
from paper_2211_10438_b200 import synth

pytestmark = pytest.mark.gpu


def _block_inputs(B, S, H, d, ffn, dtype, n_batches):
    hid, M = H * d, B * S
    ch = synth.outlier_channels(3, hid, count=max(1, hid // 100))
    fac = synth.outlier_factors(3, len(ch), 20.0, 80.0)
    xs = [synth.activations(3, 200 + j, M, hid, dtype, ch, fac) for j in range(n_batches)]
    W = {"qkv": synth.weights(3, 10, 3 * hid, hid, dtype), "out_proj": synth.weights(3, 11, hid, hid, dtype),
         "fc1": synth.weights(3, 12, ffn, hid, dtype), "fc2": synth.weights(3, 13, hid, ffn, dtype)}
    bias = {n: synth.bias(3, 20 + i, W[n].shape[0], dtype) for i, n in enumerate(W)}
    return xs, W, bias, synth.ln_params(3, 30, hid, dtype), synth.ln_params(3, 31, hid, dtype)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("w_gran", ["per_channel", "per_tensor"])
def test_prepare_linear_against_oracle(dtype, w_gran):
    N, K, alpha = 768, 512, 0.5
    ch = synth.outlier_channels(3, K, count=5)
    calib = [synth.activations(3, 300 + j, 96, K, dtype, ch, np.full(5, 60.0)) for j in range(3)]
    W = synth.weights(3, 310, N, K, dtype)
    b = synth.bias(3, 311, N, dtype)
    gamma, beta = synth.ln_params(3, 312, K, dtype)
    ws = sq.new_workspace(4096)
    got = pl.prepare_linear("l", dev(W, dtype), dev(b, dtype), False, [dev(c, dtype) for c in calib], alpha, w_gran, ws,
                            dev(gamma, dtype), dev(beta, dtype))
    ax = None
    for c in calib:
        ax = oracle.calib_absmax(c, ax)
    assert np.array_equal(host(got.act_absmax), ax)  # running maximum over the batches, exact
    s_or = oracle.smooth_scales(ax, oracle.calib_absmax(W), alpha)
    s = host(got.s)
    assert np.all(np.abs(s - s_or) <= np.spacing(s_or))  # device pow against libm: one unit in the last place
    # everything downstream of s is exact given the same s
    gh, bh = oracle.fold_ln_weight(gamma, beta, s, dtype)
    assert np.array_equal(host(got.gamma_hat), gh) and np.array_equal(host(got.beta_hat), bh)
    Wq, wsc = oracle.quant_weight(W, s, w_gran)
    assert np.array_equal(host(got.Wq), Wq) and np.array_equal(host(got.w_scale), wsc)
    # a linear whose input is not smoothed (out-proj, FC2): no calibration batches, s = None
    got2 = pl.prepare_linear("l2", dev(W, dtype), dev(b, dtype), False, None, alpha, w_gran, ws)
    Wq2, wsc2 = oracle.quant_weight(W, None, w_gran)
    assert got2.s is None and np.array_equal(host(got2.Wq), Wq2) and np.array_equal(host(got2.w_scale), wsc2)


def _oracle_static_steps(xs, p, B, S, H, d, dtype, eps=1e-5):
    """The oracle's walk of one decoder block with dynamic steps, keeping the maxima that become the static steps."""
    f32 = np.float32
    hid = H * d
    mx = {k: 0.0 for k in ("d_ln1", "d_q", "d_k", "d_v", "d_attn", "d_ln2", "d_fc1")}
    for x in xs:
        x1q, d1, _ = oracle.ln_quant(x, p["g1"], p["b1"], eps, "per_tensor_dynamic")
        y = oracle.round_to(oracle.dequant(oracle.gemm_i32(x1q, p["qkv"]["Wq"]), d1, p["qkv"]["w_scale"], p["qkv"]["bias"]), dtype)
        dq, dk, dv = (oracle.step_size(float(np.abs(y[:, i * hid:(i + 1) * hid]).max())) for i in range(3))
        r = np.concatenate([np.full(hid, f32(1) / f32(v), f32) for v in (dq, dk, dv)])
        _, qkv = oracle.w8a8_linear(x1q, d1, p["qkv"]["Wq"], p["qkv"]["w_scale"], bias=p["qkv"]["bias"], requant_mul=r)
        v5 = qkv.reshape(B, S, 3, H, d)
        q, k, v = (np.ascontiguousarray(v5[:, :, i].transpose(0, 2, 1, 3)) for i in range(3))
        _, sc = oracle.w8a8_bmm(q, k, float(f32(f32(dq) * f32(dk)) / f32(np.sqrt(f32(d)))), out_dtype=dtype)
        Pq = np.stack([np.stack([oracle.softmax_quant_p(sc[b, h])[0] for h in range(H)]) for b in range(B)])
        alpha_pv = float(f32(dv) / f32(127.0))
        _, of = oracle.w8a8_bmm(Pq, v, alpha_pv, b_is_kn=True, out_dtype=dtype)
        d_attn = oracle.step_size(float(np.abs(of).max()))
        _, oq = oracle.w8a8_bmm(Pq, v, alpha_pv, b_is_kn=True, requant_mul=f32(1) / f32(d_attn))
        attn = np.ascontiguousarray(oq.transpose(0, 2, 1, 3)).reshape(B * S, hid)
        _, proj = oracle.w8a8_linear(attn, d_attn, p["out_proj"]["Wq"], p["out_proj"]["w_scale"], bias=p["out_proj"]["bias"],
                                     out_dtype=dtype)
        h = oracle.round_to(x + proj, dtype)
        x2q, d2, _ = oracle.ln_quant(h, p["g2"], p["b2"], eps, "per_tensor_dynamic")
        f1 = oracle.round_to(oracle.dequant(oracle.gemm_i32(x2q, p["fc1"]["Wq"]), d2, p["fc1"]["w_scale"], p["fc1"]["bias"], relu=True), dtype)
        for k_, v_ in (("d_ln1", float(d1[0])), ("d_q", dq), ("d_k", dk), ("d_v", dv), ("d_attn", d_attn),
                       ("d_ln2", float(d2[0])), ("d_fc1", oracle.step_size(float(np.abs(f1).max())))):
            mx[k_] = max(mx[k_], v_)
    return mx


@pytest.mark.parametrize("dtype,B,S,H,d,ffn", [("f16", 1, 128, 2, 128, 1024), ("bf16", 2, 64, 3, 64, 768)])
def test_calibrate_static_steps_against_oracle_walk(dtype, B, S, H, d, ffn):
    """The block is prepared by the library (prepare_linear on float weights), its parameters are read
    back and handed to the oracle, and both walk the same calibration batches.  The steps come out of a
    chain of quantised stages, so a LayerNorm code on a rounding boundary may move a downstream maximum
    by a part in 10^4: LN1's step (nothing upstream) must agree to the statistics' tolerance, the others
    to 1e-3 relative."""
    xs, W, bias, (g1, b1), (g2, b2) = _block_inputs(B, S, H, d, ffn, dtype, 3)
    hid = H * d
    ws = sq.new_workspace(4096)
    tdt = {"f16": torch.float16, "bf16": torch.bfloat16}[dtype]
    # the smoothed linears are calibrated on LayerNorm-output-like samples of their input
    ch = synth.outlier_channels(3, hid, count=max(1, hid // 100))
    ln_samples = [dev(synth.activations(3, 400 + j, 64, hid, dtype, ch, np.full(len(ch), 30.0)), dtype) for j in range(2)]
    lin = {}
    for n in W:
        smoothed = n in ("qkv", "fc1")
        g, b = ((g1, b1) if n == "qkv" else (g2, b2)) if smoothed else (None, None)
        lin[n] = pl.prepare_linear(n, dev(W[n], dtype), dev(bias[n], dtype), n == "fc1", ln_samples if smoothed else None, 0.5,
                                   "per_channel", ws, None if g is None else dev(g, dtype), None if b is None else dev(b, dtype))
    got = pl.calibrate_static_steps(lin, [dev(x, dtype) for x in xs], B, S, H, d, tdt)
    p = {n: dict(Wq=host(lin[n].Wq), w_scale=host(lin[n].w_scale), bias=bias[n]) for n in W}
    p["g1"], p["b1"] = host(lin["qkv"].gamma_hat), host(lin["qkv"].beta_hat)
    p["g2"], p["b2"] = host(lin["fc1"].gamma_hat), host(lin["fc1"].beta_hat)
    want = _oracle_static_steps(xs, p, B, S, H, d, dtype)
    assert set(got) == set(want)
    assert abs(got["d_ln1"] - want["d_ln1"]) <= 16 * np.spacing(np.float32(want["d_ln1"]))
    for k in want:
        assert abs(got[k] - want[k]) <= 1e-3 * want[k], (k, got[k], want[k])
    # the steps are usable: a block built from them runs and uses the code range
    blk = pl.DecoderBlockStatic(lin, got, B, S, H, d, tdt)
    blk.forward(dev(xs[0], dtype))
    torch.cuda.synchronize()
    assert sq.device_status(blk.ws) == 0
    for t in (blk.x1q, blk.qkv, blk.attn, blk.x2q, blk.f1q):
        assert int(t.abs().max()) >= 60  # calibrated on batches like this one: the codes use the range


def test_calibrate_static_steps_clips_the_largest_tokens():
    """clip_frac sets the largest tokens aside for the materialised tensors (Section 5.2): with one batch whose
    last token is scaled up, a clip of one token's worth brings the steps of q/k/v back to the unscaled batch's."""
    B, S, H, d, ffn, dtype = 1, 128, 2, 128, 512, "f16"
    xs, W, bias, (g1, b1), (g2, b2) = _block_inputs(B, S, H, d, ffn, dtype, 1)
    ws = sq.new_workspace(4096)
    lin = {}
    for n in W:
        lin[n] = pl.prepare_linear(n, dev(W[n], dtype), dev(bias[n], dtype), n == "fc1", None, 0.5, "per_channel", ws)
    for n, (g, b) in (("qkv", (g1, b1)), ("fc1", (g2, b2))):
        lin[n].gamma_hat, lin[n].beta_hat = dev(g, dtype), dev(b, dtype)
    base = pl.calibrate_static_steps(lin, [dev(xs[0], dtype)], B, S, H, d, torch.float16)
    clipped = pl.calibrate_static_steps(lin, [dev(xs[0], dtype)], B, S, H, d, torch.float16, clip_frac=0.02)
    for k in ("d_q", "d_k", "d_v", "d_attn", "d_fc1"):
        assert clipped[k] <= base[k]
    assert any(clipped[k] < base[k] for k in ("d_q", "d_k", "d_v", "d_fc1"))
    assert clipped["d_ln1"] == base["d_ln1"]
