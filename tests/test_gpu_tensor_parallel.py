"""GPU tests of the two kernels tensor-parallel serving adds (per-token quantiser with agreed-on token
maxima; Eq. 2 on INT32 sums already in memory) and of a row-parallel layer emulated on one GPU: the
ranks' shards are processed one after the other and the two collectives are stood in for by an
element-wise maximum and an integer add of the ranks' buffers (no rank ever waits for another)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import dev, host
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import synth
from paper_2211_10438_b200 import tensor_parallel as tp

pytestmark = pytest.mark.gpu
TDT = {"f16": torch.float16, "bf16": torch.bfloat16}


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M,C", [(1, 8), (37, 5120), (300, 20480), (5, 40960), (3, 81920)])
def test_quant_act_given_absmax_exact(dtype, M, C):
    ch = synth.outlier_channels(70, C, count=max(1, C // 200))
    x = synth.activations(70, 1, M, C, dtype, ch, np.full(len(ch), 50.0))
    own = oracle.row_absmax(x)
    # (a) with the rows' own maxima: the per-token dynamic quantiser, bit for bit
    q, s = sq.sq_quant_act_given_absmax(dev(x, dtype), dev(own))
    wq, wsx = oracle.quant_act(x, "per_token")
    assert np.array_equal(host(q), wq) and np.array_equal(host(s), wsx)
    # (b) with larger maxima (another rank's slice held the row's maximum) and, for one row, a smaller one (saturates)
    given = (own * synth.rng_for(70, 2).uniform(1.0, 3.0, M)).astype(np.float32)
    given[0] = own[0] * np.float32(0.5)
    q, s = sq.sq_quant_act_given_absmax(dev(x, dtype), dev(given))
    delta = np.array([oracle.step_size(float(v)) for v in given], np.float32)
    assert np.array_equal(host(s), delta) and np.array_equal(host(q), oracle.quantize(x, delta, True))
    assert np.abs(host(q)[0]).max() == 127


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M,N", [(1, 8), (16, 512), (300, 5128), (2048, 5120)])
@pytest.mark.parametrize("variant", ["plain", "relu", "requant", "residual", "per_tensor"])
def test_dequant_acc_matches_the_gemm_epilogue(dtype, M, N, variant):
    rng = synth.rng_for(71, 1)
    acc = rng.integers(-2 ** 27, 2 ** 27, (M, N)).astype(np.int32)
    per_tensor = variant == "per_tensor"
    xs = rng.uniform(0.01, 0.2, 1 if per_tensor else M).astype(np.float32)
    wsc = rng.uniform(1e-9, 1e-8, 1 if per_tensor else N).astype(np.float32)
    bias = synth.bias(71, 2, N, dtype, std=0.5)
    kw = {}
    y = oracle.dequant(acc, xs, wsc, bias, relu=variant == "relu")
    if variant == "requant":
        r = rng.uniform(20.0, 60.0, N).astype(np.float32)
        want = oracle.requant(y, r)
        kw["requant_mul"] = dev(r)
    elif variant == "residual":
        res = synth.activations(71, 3, M, N, dtype, [], [])
        want = oracle.round_to(oracle.round_to(y, dtype) + res, dtype)
        kw["residual"] = dev(res, dtype)
    else:
        want = oracle.round_to(y, dtype)
    got = sq.sq_dequant_acc(dev(acc), dev(xs), dev(wsc), bias=dev(bias, dtype), relu=variant == "relu", out_dtype=TDT[dtype], **kw)
    assert np.array_equal(host(got), want)
    assert np.abs(want.astype(np.float64)).max() > 0.5


def test_dequant_acc_equals_fused_epilogue_on_a_real_gemm():
    M, N, K = 200, 1024, 2048
    Xq, Wq = synth.int8_tensor(72, 1, (M, K)), synth.int8_tensor(72, 2, (N, K))
    rng = synth.rng_for(72, 3)
    xs, wsc = rng.uniform(0.01, 0.2, M).astype(np.float32), rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(72, 4, N, "bf16", std=0.5)
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K))
    fused = sq.sq_w8a8_gemm(dev(Xq), dev(Wq), dev(xs), dev(wsc), ws, bias=dev(bias, "bf16"), relu=True, out_dtype=torch.bfloat16)
    acc = sq.sq_w8a8_gemm(dev(Xq), dev(Wq), None, None, ws, out_dtype=torch.int32)
    two = sq.sq_dequant_acc(acc, dev(xs), dev(wsc), bias=dev(bias, "bf16"), relu=True, out_dtype=torch.bfloat16)
    assert torch.equal(fused.view(torch.int16), two.view(torch.int16))


@pytest.mark.parametrize("world", [2, 4, 8])
def test_row_parallel_layer_emulated_on_one_gpu_is_bit_exact(world):
    """FC2 of an OPT-13B-shaped block (20480 -> 5120) on 384 tokens, cut over `world` ranks along its input
    channels.  Unsharded library call, emulated tensor-parallel path and the oracle give the same bytes."""
    M, N, K, dtype = 384, 5120, 20480, "bf16"
    ch = synth.outlier_channels(73, K, count=40)
    a = synth.activations(73, 1, M, K, dtype, ch, np.full(40, 40.0))
    Wq = synth.int8_tensor(73, 2, (N, K))
    wsc = synth.rng_for(73, 3).uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(73, 4, N, dtype)
    ad, Wd, wd, bd = dev(a, dtype), dev(Wq), dev(wsc), dev(bias, dtype)
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K))
    # unsharded
    Xq_full, xs_full = sq.sq_quant_act(ad, "per_token")
    y_full = sq.sq_w8a8_gemm(Xq_full, Wd, xs_full, wd, ws, bias=bd, out_dtype=torch.bfloat16)
    # emulated ranks
    shards = [tp.shard_row_parallel(Wd, wd, bd, world, r) for r in range(world)]
    slices = [ad[:, s.lo:s.hi].contiguous() for s in shards]
    amax = [sq.sq_token_absmax(x) for x in slices]
    agreed = torch.stack(amax).max(dim=0).values            # stands in for the max-all-reduce
    acc_sum = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    for s, x in zip(shards, slices):
        q, xs = sq.sq_quant_act_given_absmax(x, agreed)
        assert torch.equal(q, Xq_full[:, s.lo:s.hi]) and torch.equal(xs, xs_full)
        acc_sum += sq.sq_w8a8_gemm(q, s.Wq, None, None, ws, out_dtype=torch.int32)   # stands in for the INT32 sum-all-reduce
    y_tp = sq.sq_dequant_acc(acc_sum, xs_full, wd, bias=bd, out_dtype=torch.bfloat16)
    assert torch.equal(y_tp.view(torch.int16), y_full.view(torch.int16))
    # and against the oracle on sampled rows
    rows = np.sort(synth.rng_for(73, 5).choice(M, size=12, replace=False))
    oq, os_ = oracle.quant_act(a[rows], "per_token")
    _, oy = oracle.w8a8_linear(oq, os_, Wq, wsc, bias=bias, out_dtype=dtype)
    assert np.array_equal(host(y_tp)[rows], oy)
    assert sq.device_status(ws) == 0


def test_tensor_parallel_block_world_one_equals_linear_block():
    """TensorParallelLinears with a single rank (no process group) is the unsharded LinearBlock, byte for byte."""
    from paper_2211_10438_b200 import pipeline as pl
    M, hid, ffn, hd = 256, 512, 2048, 128
    rng = synth.rng_for(74, 1)
    shapes = {"qkv": (3 * hid, hid), "out_proj": (hid, hid), "fc1": (ffn, hid), "fc2": (hid, ffn)}
    lin = {}
    for i, (n, (N, K)) in enumerate(shapes.items()):
        lin[n] = pl.PreparedLinear(n, dev(synth.int8_tensor(74, 10 + i, (N, K))), dev(rng.uniform(1e-4, 1e-3, N).astype(np.float32)),
                                   dev(synth.bias(74, 20 + i, N, "bf16"), "bf16"), n == "fc1")
    for n, k in (("qkv", 3), ("fc1", 4)):
        g, b = synth.ln_params(74, k, hid, "bf16")
        lin[n].gamma_hat, lin[n].beta_hat = dev(g, "bf16"), dev(b, "bf16")
    x = dev(synth.activations(74, 30, M, hid, "bf16", [3, 77], [40.0, 25.0]), "bf16")
    attn = dev(synth.activations(74, 31, M, hid, "bf16", [5], [30.0]), "bf16")
    ref = pl.LinearBlock(lin["qkv"], lin["out_proj"], lin["fc1"], lin["fc2"], M, torch.bfloat16).step(x, attn)
    blk = tp.TensorParallelLinears(lin, M, hid, hd, torch.bfloat16, world=1, rank=0)
    got = blk.step(x, attn)
    assert torch.equal(got.view(torch.int16), ref.view(torch.int16))
    assert sq.device_status(blk.ws) == 0
