"""GPU parity of the fused causal INT8 attention kernel against the oracle's unfused definition
(Q.K^T -> fp32 scores -> causal softmax -> P = round(127 p) -> P.V -> requant).
The kernel sums each softmax row in a different order (online, tile by tile) and never writes P, so
a P code whose exact value sits on a rounding boundary may be either neighbour.  Every output code
must lie in the interval that the admissible P matrices allow (parity.attention_codes_valid); where
no P code is ambiguous that interval is the oracle's single value."""
import numpy as np
import pytest
import torch

import oracle
from helpers import dev, host
from parity import attention_codes_valid
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import synth

pytestmark = pytest.mark.gpu


def _oracle_attention(qkv, B, H, S, d, alpha_qk, alpha_pv, r, dtype):
    v5 = qkv.reshape(B, S, 3, H, d)
    q, k, v = (np.ascontiguousarray(v5[:, :, i].transpose(0, 2, 1, 3)) for i in range(3))
    _, scores = oracle.w8a8_bmm(q, k, alpha_qk, out_dtype=dtype)
    P = np.empty((B, H, S, S), np.int8)
    for b in range(B):
        for h in range(H):
            P[b, h], _ = oracle.softmax_quant_p(scores[b, h])
    acc, o = oracle.w8a8_bmm(P, v, alpha_pv, b_is_kn=True, requant_mul=r)
    return np.ascontiguousarray(o.transpose(0, 2, 1, 3)).reshape(B * S, H * d), P


@pytest.mark.parametrize("B,H,S", [(1, 2, 128), (2, 3, 512), (1, 1, 384), (1, 2, 208), (2, 1, 16), (1, 1, 1024), (1, 2, 2048)])
def test_fused_attention_against_oracle_chain(B, H, S):
    dtype = "f32"  # the fused kernel never rounds the scores to a 16-bit type
    d = 128
    qkv = synth.int8_tensor(50, S, (B * S, 3 * H * d), lo=-100, hi=100)
    alpha_qk = np.float32(0.0009)   # scores of a few units: a softmax with real spread
    alpha_pv = np.float32(0.01 / 127)
    r = np.array([1.0 / 0.004], np.float32)
    want, P = _oracle_attention(qkv, B, H, S, d, alpha_qk, alpha_pv, r, dtype)
    tdt = torch.float16
    ws = sq.new_workspace(256)
    qd = dev(qkv)
    out = torch.full((B * S, H * d), 77, dtype=torch.int8, device="cuda")
    sq.sq_w8a8_attention(qd, B, H, S, d, alpha_qk, alpha_pv, dev(r), out, ws)
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0
    got = host(out).reshape(B, S, H, d)
    v5 = qkv.reshape(B, S, 3, H, d)
    for b in range(B):
        for h in range(H):
            q, k, v = (np.ascontiguousarray(v5[b, :, i, h]) for i in range(3))
            _, scores = oracle.w8a8_bmm(q[None], k[None], float(alpha_qk), out_dtype="f32")
            amb, multi, differ = attention_codes_valid(got[b, :, h], scores[0], np.arange(1, S + 1), v, alpha_pv,
                                                       requant_mul=r, P_oracle=P[b, h])
            # few P codes are ambiguous, and an output differs from the oracle's own only where the
            # ambiguity leaves more than one valid value
            assert amb <= 2e-3 and differ <= multi
    assert np.abs(want).max() > 20  # the comparison is not vacuous
    # the library's own unfused chain (fp16 scores) stays close: it differs by the score rounding only
    hid, row = H * d, 3 * H * d
    scores = torch.empty((B * H, S, S), dtype=tdt, device="cuda")
    flat = qd.view(-1)
    sq.sq_w8a8_bmm(flat, flat[hid:], B, H, S, S, d, (S * row, d, row), (S * row, d, row), False, alpha_qk, scores,
                   (H * S * S, S * S, S), ws, causal=True)
    Pq = sq.sq_softmax_quant_p(scores)
    out2 = torch.empty((B * S, hid), dtype=torch.int8, device="cuda")
    sq.sq_w8a8_bmm(Pq, flat[2 * hid:], B, H, S, d, S, (H * S * S, S * S, S), (S * row, d, row), True, alpha_pv, out2,
                   (S * hid, d, hid), ws, requant_mul=dev(r), causal=True)
    d2 = (out.int() - out2.int()).abs()
    assert int(d2.max()) <= 16 and float(d2.float().mean()) <= 0.5  # sanity only: different score precision


def test_fused_attention_first_token_and_determinism():
    B, H, S, d = 1, 2, 256, 128
    qkv = synth.int8_tensor(51, 1, (B * S, 3 * H * d), lo=-90, hi=90)
    ws = sq.new_workspace(256)
    r = dev(np.array([127.0], np.float32))
    outs = []
    for _ in range(2):
        out = torch.empty((B * S, H * d), dtype=torch.int8, device="cuda")
        sq.sq_w8a8_attention(dev(qkv), B, H, S, d, 0.001, 1.0 / 127, r, out, ws)
        outs.append(out)
    assert torch.equal(outs[0], outs[1])
    # query 0 sees only key 0: P = 127 exactly, so out[0] = clamp(round(127 * v[0] / 127 * 127)) saturates like v[0]'s sign
    v0 = qkv.reshape(S, 3, H, d)[0, 2]            # [H, d]
    want0 = np.clip(np.rint(v0.astype(np.float64) * 127.0), -127, 127).astype(np.int8).reshape(-1)
    assert np.array_equal(host(outs[0])[0], want0)


def test_fused_attention_rejects_other_head_dims():
    qkv = torch.zeros((64, 3 * 64), dtype=torch.int8, device="cuda")
    out = torch.zeros((64, 64), dtype=torch.int8, device="cuda")
    with pytest.raises(sq.SqError) as e:
        sq.sq_w8a8_attention(qkv, 1, 1, 64, 64, 1.0, 1.0, torch.ones(1, device="cuda"), out, sq.new_workspace(256))
    assert e.value.code == 4
