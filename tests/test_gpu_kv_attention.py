"""GPU parity of the INT8 KV cache path: the cache-filling kernel (byte-exact against the layout's
definition) and the generation-stage attention kernel against the oracle's step-by-step definition
(q.K^T -> fp32 scores -> softmax -> P = round(127 p) -> P.V -> requant / 16-bit float).
exp and the softmax sum are taken in a different order on the GPU, so a P code on a rounding
boundary may differ by one and move an output code: integer outputs are compared by code distance
and mismatch fraction, float outputs by a bound derived from one P code of slack."""
import numpy as np
import pytest
import torch

import oracle
from helpers import dev, host
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import synth

pytestmark = pytest.mark.gpu
D = 128


def _cache_layout(K, V, L_max):
    """Logical [B, H, L, d] keys / values -> the two cache layouts, written out from their definition."""
    B, H, L, d = K.shape
    kc = np.zeros((B, H, L_max, d), np.int8)
    kc[:, :, :L] = K
    vl = np.zeros((B, H, L_max, d), np.int8)
    vl[:, :, :L] = V
    vc = np.ascontiguousarray(vl.reshape(B, H, L_max // 4, 4, d).transpose(0, 1, 2, 4, 3))  # [.., L/4, d, 4]
    return kc, vc


def _split_qkv(qkv, B, T, H):
    v5 = qkv.reshape(B, T, 3, H, D)
    return tuple(np.ascontiguousarray(v5[:, :, i].transpose(0, 2, 1, 3)) for i in range(3))  # [B, H, T, d]


@pytest.mark.parametrize("B,T,H,L_max", [(2, 64, 3, 64), (1, 37, 2, 48), (3, 1, 2, 16), (2, 5, 1, 32)])
def test_kv_cache_write_prompt_fill_is_byte_exact(B, T, H, L_max):
    qkv = synth.int8_tensor(60, T, (B * T, 3 * H * D))
    _, K, V = _split_qkv(qkv, B, T, H)
    want_k, want_v = _cache_layout(K, V, L_max)
    ws = sq.new_workspace(256)
    kc = torch.zeros((B, H, L_max, D), dtype=torch.int8, device="cuda")
    vc = torch.zeros((B, H, L_max // 4, D, 4), dtype=torch.int8, device="cuda")
    sq.sq_kv_cache_write(dev(qkv), B, T, H, D, None, kc, vc, L_max, ws)
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0
    assert np.array_equal(host(kc), want_k)
    assert np.array_equal(host(vc), want_v)


def test_kv_cache_write_appends_at_ragged_positions():
    """Tokens appended one by one (and in a run of 5) at per-sequence positions that are not multiples
    of four land where a prompt-sized fill would have put them, and touch nothing else."""
    B, H, L_max = 3, 2, 40
    pos = np.array([0, 7, 30], np.int32)
    ws = sq.new_workspace(256)
    kc = torch.full((B, H, L_max, D), 55, dtype=torch.int8, device="cuda")
    vc = torch.full((B, H, L_max // 4, D, 4), 55, dtype=torch.int8, device="cuda")
    want_k = np.full((B, H, L_max, D), 55, np.int8)
    want_vl = np.full((B, H, L_max, D), 55, np.int8)
    for step, T in enumerate([1, 1, 5, 1]):
        qkv = synth.int8_tensor(61, step, (B * T, 3 * H * D))
        _, K, V = _split_qkv(qkv, B, T, H)
        sq.sq_kv_cache_write(dev(qkv), B, T, H, D, dev(pos), kc, vc, L_max, ws)
        for b in range(B):
            want_k[b, :, pos[b]:pos[b] + T] = K[b]
            want_vl[b, :, pos[b]:pos[b] + T] = V[b]
        pos = pos + T
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0
    want_v = np.ascontiguousarray(want_vl.reshape(B, H, L_max // 4, 4, D).transpose(0, 1, 2, 4, 3))
    assert np.array_equal(host(kc), want_k)
    assert np.array_equal(host(vc), want_v)


def test_kv_cache_write_refuses_to_run_off_the_cache():
    B, H, L_max = 2, 1, 16
    ws = sq.new_workspace(256)
    kc = torch.zeros((B, H, L_max, D), dtype=torch.int8, device="cuda")
    vc = torch.zeros((B, H, L_max // 4, D, 4), dtype=torch.int8, device="cuda")
    qkv = synth.int8_tensor(62, 1, (B * 2, 3 * H * D), lo=1, hi=100)
    sq.sq_kv_cache_write(dev(qkv), B, 2, H, D, dev(np.array([3, 15], np.int32)), kc, vc, L_max, ws)
    torch.cuda.synchronize()
    assert sq.device_status(ws) & 0xff == sq.SQ_ERR_SHAPE
    assert host(kc)[0, 0, 3:5].all() and not host(kc)[1].any() and not host(vc)[1].any()
    with pytest.raises(sq.SqError):
        sq.sq_kv_cache_write(dev(qkv), B, 2, H, D, None, kc, vc, 18, ws)  # L_max not a multiple of 4


def _run_decode(q, K, V, lens, L_max, max_len, alpha_qk, alpha_pv, r=None, out_dtype=None):
    B, H, _ = q.shape
    kc, vc = _cache_layout(K, V, L_max)
    ws = sq.new_workspace(256)
    out = sq.sq_w8a8_decode_attention(dev(q.reshape(B, H * D)), dev(kc), dev(vc), dev(np.asarray(lens, np.int32)), B, H, D,
                                      L_max, max_len, alpha_qk, alpha_pv, ws, requant_mul=None if r is None else dev(r),
                                      out_dtype=out_dtype)
    torch.cuda.synchronize()
    return out, sq.device_status(ws)


CASES = [  # B, H, lens, L_max: ragged tails, single positions, clusters of 1 .. 8, several tiles per warp
    (2, 3, [37, 5], 64),
    (1, 2, [1], 4),
    (3, 1, [2, 3, 4], 8),
    (1, 2, [2048], 2048),        # few heads: split over 8 CTAs
    (1, 3, [1999], 2048),        # ragged split
    (2, 2, [700, 31], 1024),     # one CTA of the cluster holds nothing for the short sequence
    (4, 40, [513, 512, 100, 260], 640),   # many heads: a narrow cluster
    (1, 1, [8200], 8224),
]


@pytest.mark.parametrize("B,H,lens,L_max", CASES)
def test_decode_attention_int8_out_against_oracle(B, H, lens, L_max):
    L = max(lens)
    q = synth.int8_tensor(63, L, (B, H, D), lo=-100, hi=100)
    K = synth.int8_tensor(63, L + 1, (B, H, L, D), lo=-100, hi=100)
    V = synth.int8_tensor(63, L + 2, (B, H, L, D), lo=-100, hi=100)
    alpha_qk, alpha_pv = np.float32(0.0009), np.float32(0.01 / 127)
    r = np.array([1.0 / 0.0008], np.float32)
    want, _ = oracle.kv_decode_attention(q, K, V, lens, alpha_qk, alpha_pv, requant_mul=r)
    out, status = _run_decode(q, K, V, lens, L_max, L, alpha_qk, alpha_pv, r=r)
    assert status == 0
    got = host(out).reshape(B, H, D).astype(np.int32)
    diff = np.abs(got - want.astype(np.int32))
    assert diff.max() <= 2, "output codes differ by %d" % diff.max()
    assert (diff != 0).mean() <= 1e-2, "%.4f of output codes differ" % (diff != 0).mean()
    assert np.abs(want).max() > 20  # the comparison is not vacuous


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_decode_attention_float_out_against_oracle(dtype):
    B, H, lens, L_max = 2, 5, [300, 1025], 1028
    L = max(lens)
    q = synth.int8_tensor(64, 1, (B, H, D), lo=-100, hi=100)
    K = synth.int8_tensor(64, 2, (B, H, L, D), lo=-100, hi=100)
    V = synth.int8_tensor(64, 3, (B, H, L, D), lo=-127, hi=127)
    alpha_qk, alpha_pv = np.float32(0.0011), np.float32(0.02 / 127)
    want, Ps = oracle.kv_decode_attention(q, K, V, lens, alpha_qk, alpha_pv, out_dtype=dtype)
    tdt = {"f16": torch.float16, "bf16": torch.bfloat16}[dtype]
    out, status = _run_decode(q, K, V, lens, L_max, L_max, alpha_qk, alpha_pv, out_dtype=tdt)
    assert status == 0
    got = host(out).reshape(B, H, D)
    # a handful of P codes may sit on a rounding boundary: each moves an output by at most 127 * alpha_pv
    eps = {"f16": 2.0 ** -10, "bf16": 2.0 ** -7}[dtype]
    tol = 3 * 127 * float(alpha_pv) + 2 * eps * np.abs(want)
    assert np.all(np.abs(got - want) <= tol)
    assert (got == want).mean() >= 0.9  # and most elements agree to the bit


def test_decode_attention_closed_forms_and_edges():
    B, H, L_max = 3, 2, 64
    q = synth.int8_tensor(65, 1, (B, H, D), lo=-100, hi=100)
    K = synth.int8_tensor(65, 2, (B, H, L_max, D), lo=-100, hi=100)
    V = synth.int8_tensor(65, 3, (B, H, L_max, D))
    alpha_pv = np.float32(0.25) / np.float32(127.0)
    # one cached position -> P = 127 exactly -> out = v * 127 * alpha_pv, to the bit;
    # no cached position -> zeros; identical keys -> uniform P = round(127 / L)
    K[2, :, :50] = K[2, :, :1]
    lens = [1, 0, 50]
    out, status = _run_decode(q, K, V, lens, L_max, 50, 0.001, alpha_pv, out_dtype=torch.float16)
    assert status == 0
    got = host(out).reshape(B, H, D)
    want0 = ((V[0, :, 0].astype(np.float32) * np.float32(127.0)) * alpha_pv).astype(np.float16).astype(np.float32)
    assert np.array_equal(got[0], want0)
    assert not got[1].any()
    pb = int(np.rint(127.0 / 50))
    want2 = ((pb * V[2, :, :50].astype(np.int64).sum(1)).astype(np.float32) * alpha_pv).astype(np.float16).astype(np.float32)
    assert np.array_equal(got[2], want2)
    # determinism: the same launch twice gives the same bytes
    out2, _ = _run_decode(q, K, V, lens, L_max, 50, 0.001, alpha_pv, out_dtype=torch.float16)
    assert torch.equal(out, out2)


def test_decode_attention_flags_a_length_beyond_the_stated_bound():
    B, H, L_max = 1, 1, 256
    q = synth.int8_tensor(66, 1, (B, H, D))
    K = synth.int8_tensor(66, 2, (B, H, L_max, D))
    V = synth.int8_tensor(66, 3, (B, H, L_max, D))
    out, status = _run_decode(q, K, V, [200], L_max, 128, 0.001, 0.001, out_dtype=torch.float16)
    assert status & 0xff == sq.SQ_ERR_SHAPE
    # what it computed is the attention over the first max_len positions
    want, _ = oracle.kv_decode_attention(q, K, V, [128], np.float32(0.001), np.float32(0.001), out_dtype="f16")
    assert np.abs(host(out).reshape(B, H, D) - want).max() <= 3 * 127 * 0.001 + 1e-2 * np.abs(want).max()
    # with the newest token's rows given, a truncated sequence appends nothing: the cache keeps its bytes
    kc, vc = _cache_layout(K, V, L_max)
    kd, vd = dev(kc), dev(vc)
    k_new = synth.int8_tensor(66, 4, (B, H * D))
    v_new = synth.int8_tensor(66, 5, (B, H * D))
    ws = sq.new_workspace(256)
    out2 = sq.sq_w8a8_decode_attention(dev(q.reshape(B, H * D)), kd, vd, dev(np.array([200], np.int32)), B, H, D, L_max, 128,
                                       0.001, 0.001, ws, out_dtype=torch.float16, k_new=dev(k_new), v_new=dev(v_new))
    torch.cuda.synchronize()
    assert sq.device_status(ws) & 0xff == sq.SQ_ERR_SHAPE
    assert np.array_equal(host(kd), kc) and np.array_equal(host(vd), vc)
    assert torch.equal(out2, out)  # the attention over the first max_len cached positions, as without the new rows
    ws = sq.new_workspace(256)
    with pytest.raises(sq.SqError):  # host-side validation
        sq.sq_w8a8_decode_attention(dev(q.reshape(1, D)), dev(K), dev(V), dev(np.array([5], np.int32)), 1, 1, D, L_max, 512,
                                    0.001, 0.001, ws, out_dtype=torch.float16)
    with pytest.raises(sq.SqError):
        sq.sq_w8a8_decode_attention(dev(q.reshape(1, D)), dev(K), dev(V), dev(np.array([5], np.int32)), 1, 1, D, L_max, 256,
                                    -1.0, 0.001, ws, out_dtype=torch.float16)


def test_decode_attention_continues_the_prompt_kernel():
    """Prompt pass with the fused attention kernel, cache filled from the same QKV codes, then the last
    prompt token re-computed by the decode kernel from the cache: the two kernels agree on that row."""
    B, H, S = 2, 3, 256
    qkv = synth.int8_tensor(67, 1, (B * S, 3 * H * D), lo=-100, hi=100)
    alpha_qk, alpha_pv = 0.0009, 0.01 / 127
    r = dev(np.array([1.0 / 0.0008], np.float32))
    ws = sq.new_workspace(256)
    qd = dev(qkv)
    out_prompt = torch.empty((B * S, H * D), dtype=torch.int8, device="cuda")
    sq.sq_w8a8_attention(qd, B, H, S, D, alpha_qk, alpha_pv, r, out_prompt, ws)
    kc = torch.zeros((B, H, S, D), dtype=torch.int8, device="cuda")
    vc = torch.zeros((B, H, S // 4, D, 4), dtype=torch.int8, device="cuda")
    sq.sq_kv_cache_write(qd, B, S, H, D, None, kc, vc, S, ws)
    q_last = qd.view(B, S, 3 * H * D)[:, -1]           # strided rows of the QKV buffer, read in place
    lens = torch.full((B,), S, dtype=torch.int32, device="cuda")
    out_dec = sq.sq_w8a8_decode_attention(q_last, kc, vc, lens, B, H, D, S, S, alpha_qk, alpha_pv, ws, requant_mul=r)
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0
    last = out_prompt.view(B, S, H * D)[:, -1].int()
    d = (last - out_dec.int()).abs()
    assert int(d.max()) <= 2 and float((d != 0).float().mean()) <= 2e-2


@pytest.mark.parametrize("B,H,lens,L_max", [(2, 3, [37, 5], 64), (3, 1, [1, 2, 4], 8), (1, 2, [2048], 2048),
                                            (1, 3, [1997], 2048), (2, 2, [700, 33], 1024), (4, 40, [513, 512, 100, 261], 640)])
def test_decode_attention_appends_the_newest_token_itself(B, H, lens, L_max):
    """With k_new / v_new the newest position is NOT in the cache: it holds junk there.  The kernel
    must give the result of the pre-appended path and leave the cache as a separate append would."""
    L = max(lens)
    q = synth.int8_tensor(68, L, (B, H, D), lo=-100, hi=100)
    K = synth.int8_tensor(68, L + 1, (B, H, L, D), lo=-100, hi=100)
    V = synth.int8_tensor(68, L + 2, (B, H, L, D), lo=-100, hi=100)
    alpha_qk, alpha_pv = np.float32(0.0009), np.float32(0.01 / 127)
    r = np.array([1.0 / 0.0008], np.float32)
    want, _ = oracle.kv_decode_attention(q, K, V, lens, alpha_qk, alpha_pv, requant_mul=r)
    # the newest token's rows, laid out like a QKV code buffer [B, 3*H*d]; junk at its cache position
    qkv = np.zeros((B, 3, H, D), np.int8)
    Kj, Vj = K.copy(), V.copy()
    for b in range(B):
        qkv[b, 0], qkv[b, 1], qkv[b, 2] = q[b], K[b, :, lens[b] - 1], V[b, :, lens[b] - 1]
        Kj[b, :, lens[b] - 1] = 113
        Vj[b, :, lens[b] - 1] = -113
    kc_np, vc_np = _cache_layout(Kj, Vj, L_max)
    kc, vc = dev(kc_np), dev(vc_np)
    qd = dev(qkv.reshape(B, 3 * H * D))
    ws = sq.new_workspace(256)
    hid = H * D
    out = sq.sq_w8a8_decode_attention(qd, kc, vc, dev(np.asarray(lens, np.int32)), B, H, D, L_max, L, alpha_qk, alpha_pv, ws,
                                      requant_mul=dev(r), k_new=qd[:, hid:], v_new=qd[:, 2 * hid:])
    torch.cuda.synchronize()
    assert sq.device_status(ws) == 0
    diff = np.abs(host(out).reshape(B, H, D).astype(np.int32) - want.astype(np.int32))
    assert diff.max() <= 2 and (diff != 0).mean() <= 1e-2
    # and byte for byte what the pre-appended path gives on the true cache
    kt, vt = _cache_layout(K, V, L_max)
    ref = sq.sq_w8a8_decode_attention(qd, dev(kt), dev(vt), dev(np.asarray(lens, np.int32)), B, H, D, L_max, L, alpha_qk,
                                      alpha_pv, ws, requant_mul=dev(r))
    assert torch.equal(out, ref)
    # the cache now holds the true rows at the newest positions, everything else untouched
    want_k, want_v = _cache_layout(K, V, L_max)
    got_k, got_v = host(kc), host(vc)
    for b in range(B):
        n = lens[b]
        assert np.array_equal(got_k[b, :, :n], want_k[b, :, :n])
        g = (n + 3) // 4
        logical = got_v[b].transpose(0, 1, 3, 2).reshape(H, L_max, D)   # [H, L_max/4, 4, d] -> positions
        assert np.array_equal(logical[:, :n], V[b, :, :n])
        assert np.array_equal(got_k[b, :, n:], kc_np[b, :, n:]) and g >= 1
