"""GPU parity, streaming stages: calibration absmax, smoothing factor, LayerNorm fold, weight and
activation quantisation, fused LayerNorm+quantise, softmax+P quantisation.  Every stage is fed
the same bytes as the oracle (stage isolation); integer outputs and step sizes must be
bit-exact, except where an order-dependent float reduction sits upstream (LayerNorm statistics,
softmax sum), which is compared through the near-tie rule."""
import numpy as np
import pytest
import torch

import oracle
from helpers import TDT, dev, host
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import synth

pytestmark = pytest.mark.gpu


def _acts(cfg, tid, M, C, dtype, n_out=4, fac=50.0):
    ch = synth.outlier_channels(cfg, C, count=n_out)
    return synth.activations(cfg, tid, M, C, dtype, ch, np.full(n_out, fac))


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("rows,cols,ld", [(300, 1000, 1000), (2048, 5120, 5120), (77, 264, 512),
                                          (129, 1003, 1003), (1, 8, 8), (64, 7168, 7168),
                                          # the streaming kernel: several column slabs, ragged last slab,
                                          # strided rows, fewer rows than row groups, many rows per group
                                          (6600, 20480, 20480), (11000, 12296, 12360), (66000, 2048, 2048),
                                          (13200, 10240, 10304)])
def test_calib_absmax_exact(dtype, rows, cols, ld):
    x = _acts(7, 1, rows, ld, dtype)
    xd = dev(x, dtype)
    a = torch.zeros(cols, dtype=torch.float32, device="cuda")
    view = xd[:, :cols]
    sq.sq_calib_absmax(view, a)
    want = oracle.calib_absmax(x[:, :cols])
    assert np.array_equal(host(a), want)
    # running maximum over a second batch
    x2 = _acts(7, 2, rows, ld, dtype, fac=70.0)
    sq.sq_calib_absmax(dev(x2, dtype)[:, :cols], a)
    assert np.array_equal(host(a), oracle.calib_absmax(x2[:, :cols], want))


@pytest.mark.parametrize("alpha", [0.0, 0.5, 0.75, 0.85, 1.0])
def test_smooth_scales_and_fold(alpha):
    C = 5120
    rng = synth.rng_for(8, 1)
    ax = np.abs(rng.standard_normal(C)).astype(np.float32) * 30
    aw = np.abs(rng.standard_normal(C)).astype(np.float32) * 0.1
    ax[3] = 0.0  # exercises the floor
    aw[5] = 0.0
    s_inv = torch.empty(C, dtype=torch.float32, device="cuda")
    s = sq.sq_smooth_scales(dev(ax), dev(aw), alpha, s_inv_out=s_inv)
    want = oracle.smooth_scales(ax, aw, alpha)
    got = host(s)
    # device pow may differ from libm in the last place of the double; allow 1 ulp of fp32
    assert np.all(np.abs(got - want) <= np.spacing(np.abs(want)))
    assert np.array_equal(host(s_inv), oracle.smooth_scales_inv(got))
    for dtype in ("f16", "bf16"):
        gamma, beta = synth.ln_params(8, 2, C, dtype)
        gh, bh = sq.sq_fold_ln_weight(dev(gamma, dtype), dev(beta, dtype), s)
        wg, wb = oracle.fold_ln_weight(gamma, beta, got, dtype)  # same s on both sides
        assert np.array_equal(host(gh), wg) and np.array_equal(host(bh), wb)
        gh2, none = sq.sq_fold_ln_weight(dev(gamma, dtype), None, s)
        assert none is None and np.array_equal(host(gh2), wg)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("gran", ["per_channel", "per_tensor"])
@pytest.mark.parametrize("N,K,smooth", [(512, 512, True), (300, 5120, True), (64, 20480, False),
                                        (5, 81920, True)])
def test_quant_weight_exact(dtype, gran, N, K, smooth):
    w = synth.weights(9, 1, N, K, dtype)
    s = None
    if smooth:
        s = (np.abs(synth.rng_for(9, 2).standard_normal(K)) * 5 + 0.05).astype(np.float32)
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_QUANT_WEIGHT, N, N, K))
    Wq, w_scale = sq.sq_quant_weight(dev(w, dtype), None if s is None else dev(s), gran, workspace=ws)
    want_q, want_s = oracle.quant_weight(w, s, gran)
    assert np.array_equal(host(w_scale), want_s)
    assert np.array_equal(host(Wq), want_q)
    assert not ws.any()  # workspace handed back zero-filled


SHAPES_ACT = [(16, 512), (37, 5120), (5, 20480), (3, 28672), (2, 49152), (2, 81920), (3, 131072),
              (1, 8), (130, 7168), (9, 4104), (1, 262144), (3, 40968), (2, 57352), (2, 73736), (3, 32776)]


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("gran", ["per_token", "per_tensor_dynamic", "per_tensor_static"])
@pytest.mark.parametrize("M,C", SHAPES_ACT)
def test_quant_act_exact(dtype, gran, M, C):
    x = _acts(10, 1, M, C, dtype, n_out=min(4, C))
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_QUANT_ACT, M, 0, C))
    if gran == "per_tensor_static":
        # a calibrated step smaller than this batch's maximum: the excess must saturate
        delta = np.array([oracle.step_size(0.5 * np.abs(x).max())], np.float32)
        Xq, xs = sq.sq_quant_act(dev(x, dtype), gran, x_scale=dev(delta), workspace=ws)
        want_q, want_s = oracle.quant_act(x, gran, static_scale=delta)
        assert np.abs(want_q).max() == 127
    else:
        Xq, xs = sq.sq_quant_act(dev(x, dtype), gran, workspace=ws)
        want_q, want_s = oracle.quant_act(x, gran)
    assert np.array_equal(host(xs), want_s)
    assert np.array_equal(host(Xq), want_q)
    assert not ws.any()


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("gran", ["per_token", "per_tensor_dynamic"])
def test_quant_act_col_mul_exact(dtype, gran):
    M, C = 33, 5120
    x = _acts(10, 2, M, C, dtype)
    cm = oracle.smooth_scales_inv((np.abs(synth.rng_for(10, 3).standard_normal(C)) * 4 + 0.1).astype(np.float32))
    ws = sq.new_workspace(256)
    Xq, xs = sq.sq_quant_act(dev(x, dtype), gran, col_mul=dev(cm), workspace=ws)
    want_q, want_s = oracle.quant_act(x, gran, col_mul=cm)
    assert np.array_equal(host(xs), want_s) and np.array_equal(host(Xq), want_q)


def test_quant_act_all_zero_rows():
    x = np.zeros((4, 512), np.float32)
    x[2, 7] = 3.0
    Xq, xs = sq.sq_quant_act(dev(x, "f16"), "per_token")
    want_q, want_s = oracle.quant_act(x, "per_token")
    assert np.array_equal(host(Xq), want_q) and np.array_equal(host(xs), want_s)
    assert host(xs)[0] == np.float32(1e-5) / np.float32(127)


def _near_tie_ok(q_gpu, q_or, y64, delta, tau):
    """Codes may differ by one, and only where the exact pre-rounding value sits within tau
    of a rounding boundary (a half-integer)."""
    q_gpu = q_gpu.astype(np.int32)
    q_or = q_or.astype(np.int32)
    diff = q_gpu != q_or
    if not diff.any():
        return 0.0
    assert np.abs(q_gpu - q_or).max() <= 1
    v = (y64 / delta)[diff]
    dist = np.abs(np.abs(v - np.floor(v)) - 0.5)
    assert np.all(dist <= tau), "code differs away from a tie: %g" % dist.max()
    return diff.mean()


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("gran", ["per_token", "per_tensor_dynamic", "per_tensor_static"])
@pytest.mark.parametrize("M,C", [(16, 512), (37, 5120), (130, 7168), (6, 20480), (3000, 7168), (1500, 12288), (40, 4096),
                                 (21, 8192), (33, 9216), (19, 14336), (9, 12296), (4, 28672),
                                 # every group of every CTA busy at the sizes whose parameters sit in tensor memory
                                 (700, 20480), (1300, 14336), (1900, 4096), (1200, 9216)])
def test_ln_quant(dtype, gran, M, C):
    eps = 1e-5
    x = _acts(11, 1, M, C, dtype)
    gamma, beta = synth.ln_params(11, 2, C, dtype)
    s = oracle.smooth_scales(np.abs(x).max(0) / 5 + 0.1, np.full(C, 0.08, np.float32), 0.5)
    gh, bh = oracle.fold_ln_weight(gamma, beta, s, dtype)
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_LN_QUANT, M, 0, C))
    dbg = torch.zeros(2 * M, dtype=torch.float32, device="cuda")
    static = None
    kw = {}
    if gran == "per_tensor_static":
        mu64, rstd64 = oracle.ln_stats(x, eps)
        y = oracle.ln_apply(x, mu64.astype(np.float32), rstd64.astype(np.float32), gh, bh)
        static = np.array([oracle.step_size(0.7 * np.abs(y).max())], np.float32)
        kw["x_scale"] = dev(static)
    Xq, xs = sq.sq_ln_quant(dev(x, dtype), dev(gh, dtype), dev(bh, dtype), eps, gran, dbg_mean_rstd=dbg,
                            workspace=ws, **kw)
    st = host(dbg).reshape(M, 2)
    mu64, rstd64 = oracle.ln_stats(x, eps)
    # the kernel's fp32 statistics against the fp64 two-pass definition
    assert np.all(np.abs(st[:, 0] - mu64) <= 1e-6 * np.maximum(np.abs(mu64), np.sqrt(1.0 / rstd64 ** 2)))
    assert np.all(np.abs(st[:, 1] - rstd64) <= 1e-6 * rstd64)
    # bit-exact element-wise part once the oracle is given the kernel's own statistics
    want_q, want_s, _ = oracle.ln_quant(x, gh, bh, eps, gran, stats=(st[:, 0].copy(), st[:, 1].copy()),
                                        static_scale=static)
    assert np.array_equal(host(xs), want_s)
    assert np.array_equal(host(Xq), want_q)
    # without feeding statistics back: near-tie rule against the fp64 LayerNorm
    q0, s0, _ = oracle.ln_quant(x, gh, bh, eps, gran, static_scale=static)
    y64 = oracle.ln_f64(x, gh.astype(np.float64), bh.astype(np.float64), eps)
    d = s0[:, None].astype(np.float64) if s0.size > 1 else float(s0[0])
    assert np.all(np.abs(host(xs) - s0) <= 16 * np.spacing(s0))
    frac = _near_tie_ok(host(Xq), q0, y64, d, tau=127 * 2.0 ** -16)
    assert frac <= 1e-3
    # second call without the debug output gives the same bytes (workspace was restored)
    Xq2, xs2 = sq.sq_ln_quant(dev(x, dtype), dev(gh, dtype), dev(bh, dtype), eps, gran, workspace=ws, **kw)
    assert torch.equal(Xq, Xq2) and torch.equal(xs, xs2)
    assert not ws.any()


def test_ln_quant_without_beta():
    M, C = 12, 1024
    x = _acts(11, 5, M, C, "bf16")
    gamma, _ = synth.ln_params(11, 6, C, "bf16")
    dbg = torch.zeros(2 * M, dtype=torch.float32, device="cuda")
    Xq, xs = sq.sq_ln_quant(dev(x, "bf16"), dev(gamma, "bf16"), None, 1e-5, "per_token", dbg_mean_rstd=dbg)
    st = host(dbg).reshape(M, 2)
    want_q, want_s, _ = oracle.ln_quant(x, gamma, None, 1e-5, "per_token", stats=(st[:, 0].copy(), st[:, 1].copy()))
    assert np.array_equal(host(Xq), want_q) and np.array_equal(host(xs), want_s)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("n_mat,S", [(3, 64), (2, 512), (1, 8), (2, 1024)])
def test_softmax_quant_p(dtype, n_mat, S):
    rng = synth.rng_for(12, S)
    sc = synth.to_dtype_f32(rng.standard_normal((n_mat, S, S)).astype(np.float32) * 2.5, dtype)
    Pq = host(sq.sq_softmax_quant_p(dev(sc, dtype)))
    for m in range(n_mat):
        want, _ = oracle.softmax_quant_p(sc[m])
        p64 = oracle.softmax_causal_f64(sc[m])
        assert not np.triu(Pq[m], 1).any()
        frac = _near_tie_ok(Pq[m], want, p64, 1.0 / 127.0, tau=127 * 2.0 ** -18)
        assert frac <= 1e-3
        assert Pq[m][0, 0] == 127


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_residual_add(dtype):
    rng = synth.rng_for(13, 1)
    a = synth.to_dtype_f32(rng.standard_normal(4096 * 3).astype(np.float32) * 3, dtype)
    b = synth.to_dtype_f32(rng.standard_normal(4096 * 3).astype(np.float32), dtype)
    out = sq.sq_residual_add(dev(a, dtype), dev(b, dtype))
    assert np.array_equal(host(out), oracle.round_to(a + b, dtype))


# --------------------------------------------------------------------------- #
# Static-step calibration with the largest tokens set aside (Section 5.2)
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M,C", [(1, 8), (37, 520), (512, 7168), (4099, 64)])
def test_token_absmax_exact(dtype, M, C):
    ch = synth.outlier_channels(7, C, count=max(1, C // 100))
    x = synth.activations(7, M, M, C, dtype, ch, synth.outlier_factors(7, len(ch), 20.0, 80.0))
    got = sq.sq_token_absmax(dev(x, dtype))
    assert np.array_equal(host(got), oracle.row_absmax(x))


@pytest.mark.parametrize("T,n_clip", [(1, 0), (1, 5), (100, 2), (4099, 0), (4099, 82), (65536, 1311), (65536, 65535),
                                      (300000, 6000)])
def test_clipped_absmax_exact(T, n_clip):
    rng = synth.rng_for(7, T + n_clip)
    v = np.abs(rng.standard_normal(T)).astype(np.float32) * 9
    v[rng.integers(0, T, max(1, T // 50))] *= 40.0       # a few huge tokens
    if T > 10:
        v[3], v[7] = v[5], v[5]                           # ties
        v[1] = 0.0
    a, s = sq.sq_clipped_absmax(dev(v), n_clip)
    want = oracle.clipped_absmax(v, n_clip)
    assert host(a)[0] == want
    assert host(s)[0] == oracle.step_size(float(want))


def test_clipped_static_step_end_to_end():
    """Four calibration batches -> per-token maxima side by side -> the top 2 % set aside -> static step;
    quantising with that step saturates exactly the tokens that were set aside (and no others)."""
    C, Mb = 512, 256
    batches = [synth.activations(7, 50 + i, Mb, C, "f16", [5], [1.0]) for i in range(4)]
    for b in batches:
        b[::64] *= 30.0                                    # 1.6 % of the tokens are huge
    ta = torch.empty(4 * Mb, dtype=torch.float32, device="cuda")
    for i, b in enumerate(batches):
        sq.sq_token_absmax(dev(b, "f16"), out=ta[i * Mb:(i + 1) * Mb])
    n_clip = oracle.clip_count(4 * Mb, 0.02)
    a, step = sq.sq_clipped_absmax(ta, n_clip)
    allx = np.concatenate(batches)
    want = oracle.clipped_absmax(oracle.row_absmax(allx), n_clip)
    assert host(a)[0] == want
    q, _ = oracle.quant_act(allx, "per_tensor_static", static_scale=float(host(step)[0]))
    saturated_rows = (np.abs(q) == 127).any(1) & (oracle.row_absmax(allx) > want)
    assert saturated_rows.sum() == (oracle.row_absmax(allx) > want).sum() <= n_clip
    assert want < 0.2 * oracle.row_absmax(allx).max()
