"""GPU parity, tensor-core stages: INT8 GEMM accumulators (bit-exact), the dequantisation epilogue
(tolerance stated by the benchmark spec: 1e-3 relative or 2 ULP; the arithmetic is fully specified, so exact
equality is also checked), re-quantised INT8 outputs (bit-exact) and the attention BMMs."""
import numpy as np
import pytest
import torch

import oracle
from helpers import assert_fp_close, dev, host
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ws():
    # the largest scratch any shape below asks for: the weight-streaming kernel's at 32 tokens, the K split's above
    w = sq.new_workspace(max(sq.workspace_bytes(sq.SQ_OP_GEMM, 32, 65536, 32768), 64 << 20))
    yield w
    assert sq.device_status(w) == 0, "a device-side wait timed out"


# (M, N, K): one tile, several tiles, ragged M / N / K tails, single row, N < 128, wide K
SHAPES = [(16, 512, 512), (128, 256, 128), (128, 128, 128), (129, 257, 144), (300, 520, 272),
          (1, 64, 16), (200, 72, 2048), (256, 1024, 5120), (77, 2000, 1040), (515, 384, 640),
          # CTA-pair kernel: many tiles per pair, each of the three tile widths, odd tile counts
          (2048, 768, 512), (1000, 5120, 1024), (384, 640, 256), (640, 1344, 384), (2048, 5120, 256)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_gemm_accumulators_exact(ws, M, N, K):
    Xq = synth.int8_tensor(20, 1, (M, K))
    Wq = synth.int8_tensor(20, 2, (N, K))
    acc = sq.sq_w8a8_gemm(dev(Xq), dev(Wq), None, None, ws, out_dtype=torch.int32)
    assert np.array_equal(host(acc), oracle.gemm_i32(Xq, Wq))
    assert sq.device_status(ws) == 0


def test_gemm_all_127_and_identity(ws):
    M, N, K = 130, 260, 1024
    ones = np.full((M, K), 127, np.int8)
    acc = sq.sq_w8a8_gemm(dev(ones), dev(np.full((N, K), -127, np.int8)), None, None, ws, out_dtype=torch.int32)
    assert np.all(host(acc) == -16129 * K)
    Xq = synth.int8_tensor(20, 3, (M, 256))
    eye = (127 * np.eye(256)).astype(np.int8)
    acc = sq.sq_w8a8_gemm(dev(Xq), dev(eye), None, None, ws, out_dtype=torch.int32)
    assert np.array_equal(host(acc), 127 * Xq.astype(np.int32))


@pytest.mark.parametrize("M", [130, 16])
def test_gemm_longest_supported_reduction_hits_the_int32_edge(ws, M):
    # K = 133120 (the largest multiple of 128 below the 133144 bound), every product = 127 * 127 or -(127 * 127)
    N, K = 128, 133120
    X = np.full((M, K), 127, np.int8)
    W = np.full((N, K), 127, np.int8)
    W[1::2] = -127
    acc = host(sq.sq_w8a8_gemm(dev(X), dev(W), None, None, ws, out_dtype=torch.int32))
    want = np.where(np.arange(N) % 2 == 0, 16129 * K, -16129 * K).astype(np.int64)
    assert want.max() < 2 ** 31 and np.array_equal(acc.astype(np.int64), np.broadcast_to(want, (M, N)))


def test_gemm_run_to_run_identical(ws):
    Xq, Wq = synth.int8_tensor(20, 4, (384, 2048)), synth.int8_tensor(20, 5, (1536, 2048))
    a = sq.sq_w8a8_gemm(dev(Xq), dev(Wq), None, None, ws, out_dtype=torch.int32)
    b = sq.sq_w8a8_gemm(dev(Xq), dev(Wq), None, None, ws, out_dtype=torch.int32)
    assert torch.equal(a, b)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M,N,K", [(16, 512, 512), (129, 257, 144), (300, 520, 272), (256, 1024, 5120)])
@pytest.mark.parametrize("per_token,per_channel,use_bias,relu", [(True, True, True, False), (False, False, False, False),
                                                                 (True, False, True, True), (False, True, True, True)])
def test_gemm_dequant_epilogue(ws, dtype, M, N, K, per_token, per_channel, use_bias, relu):
    Xq = synth.int8_tensor(21, 1, (M, K))
    Wq = synth.int8_tensor(21, 2, (N, K))
    rng = synth.rng_for(21, 3)
    xs = (rng.uniform(0.01, 0.2, M if per_token else 1)).astype(np.float32)
    wsc = (rng.uniform(1e-4, 1e-3, N if per_channel else 1)).astype(np.float32)
    bias = synth.bias(21, 4, N, dtype, std=0.5) if use_bias else None
    tdt = {"f16": torch.float16, "bf16": torch.bfloat16}[dtype]
    y = sq.sq_w8a8_gemm(dev(Xq), dev(Wq), dev(xs), dev(wsc), ws, bias=None if bias is None else dev(bias, dtype),
                        relu=relu, out_dtype=tdt)
    _, want = oracle.w8a8_linear(Xq, xs, Wq, wsc, bias=bias, relu=relu, out_dtype=dtype)
    got = host(y)
    assert_fp_close(got, want, dtype, "dequant epilogue")
    assert np.array_equal(got, want), "epilogue arithmetic is fully specified: expected identical values"


@pytest.mark.parametrize("per_col", [False, True])
@pytest.mark.parametrize("M,N,K", [(200, 328, 1024), (2048, 5120, 256), (1024, 640, 384)])
def test_gemm_requant_and_row_absmax(ws, per_col, M, N, K):
    Xq = synth.int8_tensor(22, 1, (M, K))
    Wq = synth.int8_tensor(22, 2, (N, K))
    rng = synth.rng_for(22, 3)
    xs = rng.uniform(0.01, 0.2, M).astype(np.float32)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(22, 4, N, "f16", std=0.5)
    r = rng.uniform(0.5, 2.0, N if per_col else 1).astype(np.float32)
    rmax = torch.zeros(M, dtype=torch.float32, device="cuda")
    q = sq.sq_w8a8_gemm(dev(Xq), dev(Wq), dev(xs), dev(wsc), ws, bias=dev(bias, "f16"), relu=True,
                        requant_mul=dev(r), row_absmax_out=rmax, out_dtype=torch.int8)
    acc = oracle.gemm_i32(Xq, Wq)
    y = oracle.dequant(acc, xs, wsc, bias, relu=True)
    assert np.array_equal(host(q), oracle.requant(y, r))
    assert np.array_equal(host(rmax), np.abs(y).max(1))


def test_gemm_strided_output(ws):
    M, N, K, ldy = 64, 200, 256, 264
    Xq, Wq = synth.int8_tensor(23, 1, (M, K)), synth.int8_tensor(23, 2, (N, K))
    xs = np.full(1, 0.05, np.float32)
    wsc = np.full(1, 0.002, np.float32)
    buf = torch.full((M, ldy), -7.0, dtype=torch.float16, device="cuda")
    sq.sq_w8a8_gemm(dev(Xq), dev(Wq), dev(xs), dev(wsc), ws, out=buf[:, :N])
    _, want = oracle.w8a8_linear(Xq, xs, Wq, wsc, out_dtype="f16")
    got = host(buf)
    assert np.array_equal(got[:, :N], want)
    assert np.all(got[:, N:] == -7.0)  # nothing written beyond the N columns


# long reductions whose tile count leaves a partly filled last wave: with the recommended workspace
# the tiles of that wave are cut along K (2 .. 4 pieces) and meet in the workspace; without it they are not
SPLIT_SHAPES = [(512, 4096, 12288), (2048, 5120, 20480), (300, 2304, 16400), (2048, 7168, 28672), (520, 1000, 12304),
                (256, 20480, 12288),
                # a single wave filling at most half of the machine: every tile cut into up to 8 pieces
                # (one row of 128 x 128 tiles up to 128 tokens, CTA pairs above)
                (96, 2048, 12288), (128, 3000, 13008), (70, 7168, 14336), (128, 20480, 12288), (256, 7168, 14336),
                (65, 4096, 12288)]


@pytest.mark.parametrize("M,N,K", SPLIT_SHAPES)
def test_gemm_last_wave_k_split_is_exact(M, N, K):
    Xq, Wq = synth.int8_tensor(27, 1, (M, K)), synth.int8_tensor(27, 2, (N, K))
    rng = synth.rng_for(27, 3)
    xs = rng.uniform(0.01, 0.2, M).astype(np.float32)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(27, 4, N, "f16", std=0.5)
    need = sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K)
    big, small = sq.new_workspace(need), sq.new_workspace(256)
    want_acc = oracle.gemm_i32(Xq, Wq)
    want = oracle.round_to(oracle.dequant(want_acc, xs, wsc, bias, relu=True), "f16")
    Xd, Wd = dev(Xq), dev(Wq)
    for ws in (big, small, big):  # the second use of `big` must find its counters zeroed by the first
        acc = sq.sq_w8a8_gemm(Xd, Wd, None, None, ws, out_dtype=torch.int32)
        assert np.array_equal(host(acc), want_acc)
        y = sq.sq_w8a8_gemm(Xd, Wd, dev(xs), dev(wsc), ws, bias=dev(bias, "f16"), relu=True, out_dtype=torch.float16)
        assert np.array_equal(host(y), want)
        assert sq.device_status(ws) == 0
    assert not big[4:33024].any(), "header and counters not handed back zero-filled"


# Reductions too short for the K split whose tile count leaves a partly filled last wave: the tiles of that wave
# are cut into 2 or 4 COLUMN parts (74 CTA pairs; 256 x 256 tiles).  100 tiles -> 26 left over -> halves;
# 80 tiles -> 6 left over -> quarters (halves for INT8 output), here with ragged M and an N tail that leaves
# the last tile's third quarter with 8 columns and its fourth with none.  Every epilogue, element by element.
N_SPLIT_SHAPES = [(1200, 5120, 1152), (1000, 5000, 1152)]


@pytest.mark.parametrize("epilogue", ["i32", "bf16", "f16_relu", "i8_requant_absmax", "bf16_residual"])
@pytest.mark.parametrize("M,N,K", N_SPLIT_SHAPES)
def test_gemm_last_wave_n_split_every_epilogue(ws, M, N, K, epilogue):
    Xq, Wq = synth.int8_tensor(31, 1, (M, K)), synth.int8_tensor(31, 2, (N, K))
    rng = synth.rng_for(31, 3)
    xs = rng.uniform(0.01, 0.2, M).astype(np.float32)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    acc = oracle.gemm_i32(Xq, Wq)
    Xd, Wd = dev(Xq), dev(Wq)
    if epilogue == "i32":
        got = sq.sq_w8a8_gemm(Xd, Wd, None, None, ws, out_dtype=torch.int32)
        assert np.array_equal(host(got), acc)
    elif epilogue in ("bf16", "f16_relu"):
        dtype, relu = ("bf16", False) if epilogue == "bf16" else ("f16", True)
        bias = synth.bias(31, 4, N, dtype, std=0.5)
        got = sq.sq_w8a8_gemm(Xd, Wd, dev(xs), dev(wsc), ws, bias=dev(bias, dtype), relu=relu,
                              out_dtype=torch.bfloat16 if dtype == "bf16" else torch.float16)
        assert np.array_equal(host(got), oracle.round_to(oracle.dequant(acc, xs, wsc, bias, relu=relu), dtype))
    elif epilogue == "i8_requant_absmax":
        bias = synth.bias(31, 4, N, "f16", std=0.5)
        r = rng.uniform(0.5, 2.0, N).astype(np.float32)
        rmax = torch.zeros(M, dtype=torch.float32, device="cuda")
        got = sq.sq_w8a8_gemm(Xd, Wd, dev(xs), dev(wsc), ws, bias=dev(bias, "f16"), relu=True, requant_mul=dev(r),
                              row_absmax_out=rmax, out_dtype=torch.int8)
        y = oracle.dequant(acc, xs, wsc, bias, relu=True)
        assert np.array_equal(host(got), oracle.requant(y, r))
        assert np.array_equal(host(rmax), np.abs(y).max(1))
    else:
        bias = synth.bias(31, 4, N, "bf16", std=0.5)
        res = synth.to_dtype_f32(rng.standard_normal((M, N)).astype(np.float32) * 4, "bf16")
        y = oracle.round_to(oracle.dequant(acc, xs, wsc, bias), "bf16")
        got = sq.sq_w8a8_gemm_residual(Xd, Wd, dev(xs), dev(wsc), ws, dev(res, "bf16"), bias=dev(bias, "bf16"),
                                       out=torch.zeros((M, N), dtype=torch.bfloat16, device="cuda"))
        assert np.array_equal(host(got), oracle.round_to(y + res, "bf16"))
    assert sq.device_status(ws) == 0


# the residual connection folded into the epilogue: bit for bit the unfused pair of calls.  Shapes: one
# CTA pair tile with ragged M, single-CTA narrow and wide tiles, the weight-streaming kernel (shared
# tiles), a K-split last wave (fix-up path), a strided residual and output
RESIDUAL_SHAPES = [(300, 520, 272), (2048, 1024, 512), (128, 3000, 13008), (100, 40960, 256), (1, 128, 128),
                   (16, 1280, 4096), (32, 12288, 6144), (512, 4096, 12288), (2, 4096, 49152)]


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M,N,K", RESIDUAL_SHAPES)
def test_gemm_residual_epilogue(ws, dtype, M, N, K):
    Xq, Wq = synth.int8_tensor(29, 1, (M, K)), synth.int8_tensor(29, 2, (N, K))
    rng = synth.rng_for(29, 3)
    xs = rng.uniform(0.01, 0.2, M).astype(np.float32)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(29, 4, N, dtype, std=0.5)
    ld = N + 24  # residual and output rows are strided views
    res = synth.to_dtype_f32(rng.standard_normal((M, ld)).astype(np.float32) * 4, dtype)
    y = oracle.round_to(oracle.dequant(oracle.gemm_i32(Xq, Wq), xs, wsc, bias), dtype)
    want = oracle.round_to(y + res[:, :N], dtype)
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    res_d = dev(res, dtype)
    out = torch.zeros((M, ld), dtype=tdt, device="cuda")
    sq.sq_w8a8_gemm_residual(dev(Xq), dev(Wq), dev(xs), dev(wsc), ws, res_d[:, :N], bias=dev(bias, dtype), out=out[:, :N])
    assert np.array_equal(host(out)[:, :N], want)
    assert not host(out)[:, N:].any(), "wrote outside the N columns"
    # and it equals the two separate calls
    y_d = sq.sq_w8a8_gemm(dev(Xq), dev(Wq), dev(xs), dev(wsc), ws, bias=dev(bias, dtype), out_dtype=tdt)
    two = sq.sq_residual_add(y_d, res_d[:, :N].contiguous())
    assert torch.equal(out[:, :N], two)


def test_gemm_residual_argument_checks(ws):
    X, W = torch.zeros((4, 64), dtype=torch.int8, device="cuda"), torch.zeros((12, 64), dtype=torch.int8, device="cuda")
    one = torch.ones(1, device="cuda")
    r = torch.zeros((4, 16), dtype=torch.float16, device="cuda")
    with pytest.raises(sq.SqError) as e:  # N = 12 is not a multiple of 8
        sq.sq_w8a8_gemm_residual(X, W, one, one, ws, r[:, :12], out=torch.empty((4, 12), dtype=torch.float16, device="cuda"))
    assert e.value.code == sq.SQ_ERR_ALIGN


# decode-shaped calls: swapped operands and K splits with INT32 scratch in the workspace up to 32 tokens
DECODE_SHAPES = [(1, 128, 128), (16, 512, 512), (3, 200, 272), (16, 1280, 4096), (8, 12288, 6144), (5, 136, 12288),
                 (16, 36864, 1024), (2, 4096, 49152),
                 (17, 512, 512), (32, 1280, 4096), (33, 200, 272), (64, 12288, 6144), (48, 136, 12288), (64, 36864, 1024),
                 (64, 1024, 8192), (40, 520, 4096), (64, 1536, 6144)]  # above 32 tokens: the prefill kernel, narrow tiles


@pytest.mark.parametrize("M,N,K", DECODE_SHAPES)
def test_decode_gemm_exact_and_workspace_restored(ws, M, N, K):
    Xq = synth.int8_tensor(25, 1, (M, K))
    Wq = synth.int8_tensor(25, 2, (N, K))
    rng = synth.rng_for(25, 3)
    xs = rng.uniform(0.01, 0.2, M).astype(np.float32)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(25, 4, N, "bf16", std=0.5)
    want_acc = oracle.gemm_i32(Xq, Wq)
    Xd, Wd = dev(Xq), dev(Wq)
    for _ in range(2):  # the second call must find the scratch zeroed by the first
        acc = sq.sq_w8a8_gemm(Xd, Wd, None, None, ws, out_dtype=torch.int32)
        assert np.array_equal(host(acc), want_acc)
        y = sq.sq_w8a8_gemm(Xd, Wd, dev(xs), dev(wsc), ws, bias=dev(bias, "bf16"), relu=True, out_dtype=torch.bfloat16)
        want = oracle.round_to(oracle.dequant(want_acc, xs, wsc, bias, relu=True), "bf16")
        assert np.array_equal(host(y), want)
    assert sq.device_status(ws) == 0
    assert not ws[4:33024].any(), "header and counters not handed back zero-filled"


@pytest.mark.parametrize("M,N,K,per_col", [(1, 384, 512, True), (16, 1280, 4096, True), (7, 200, 272, False),
                                           (16, 36864, 1024, True), (40, 1280, 4096, True), (64, 200, 272, False)])
def test_decode_gemm_requant_int8_out(ws, M, N, K, per_col):
    """Decode-shaped GEMM with the requantising epilogue (INT8 codes out, as the QKV and FC1
    projections of a static-step block emit them): byte-exact, the epilogue is fully specified fp32."""
    Xq, Wq = synth.int8_tensor(26, 1, (M, K)), synth.int8_tensor(26, 2, (N, K))
    rng = synth.rng_for(26, 3)
    xs = np.array([0.03], np.float32)
    wsc = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = synth.bias(26, 4, N, "f16", std=0.5)
    r = rng.uniform(5.0, 40.0, N if per_col else 1).astype(np.float32)
    acc = oracle.gemm_i32(Xq, Wq)
    want = oracle.requant(oracle.dequant(acc, xs, wsc, bias, relu=True), r)
    got = sq.sq_w8a8_gemm(dev(Xq), dev(Wq), dev(xs), dev(wsc), ws, bias=dev(bias, "f16"), relu=True, requant_mul=dev(r),
                          out_dtype=torch.int8)
    assert got.dtype == torch.int8
    assert np.array_equal(host(got), want)
    assert np.abs(want).max() > 20 and (np.abs(want) < 127).mean() > 0.5  # non-trivial codes
    assert sq.device_status(ws) == 0
    assert not ws[4:33024].any()


def test_decode_gemm_without_scratch_falls_back_to_single_split():
    M, N, K = 4, 256, 8192
    Xq, Wq = synth.int8_tensor(25, 5, (M, K)), synth.int8_tensor(25, 6, (N, K))
    small = sq.new_workspace(256)
    with pytest.raises(sq.SqError):  # the documented size is required
        sq.sq_w8a8_gemm(dev(Xq), dev(Wq), None, None, small, out_dtype=torch.int32)


@pytest.mark.parametrize("M", [1, 16, 32])
def test_single_matrix_bmm_with_few_rows_applies_alpha(M):
    """A one-matrix BMM with contiguous operands and M <= 32 takes the weight-streaming kernel:
    its scalar factor alpha (there are no step-size arrays in a BMM call) must reach the epilogue."""
    N, K = 384, 512
    A, B = synth.int8_tensor(27, 1, (M, K)), synth.int8_tensor(27, 2, (N, K))
    alpha = np.float32(0.00731)
    r = np.array([3.7], np.float32)
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K))
    want_acc, want16 = oracle.w8a8_bmm(A[None], B[None], float(alpha), out_dtype="f16")
    _, want8 = oracle.w8a8_bmm(A[None], B[None], float(alpha), requant_mul=r)
    Ad, Bd = dev(A), dev(B)
    for tdt, want in ((torch.int32, want_acc[0]), (torch.float16, want16[0]), (torch.int8, want8[0])):
        C = torch.empty((M, N), dtype=tdt, device="cuda")
        sq.sq_w8a8_bmm(Ad, Bd, 1, 1, M, N, K, (M * K, M * K, K), (N * K, N * K, K), False, alpha, C, (M * N, M * N, N), ws,
                       requant_mul=dev(r) if tdt == torch.int8 else None)
        assert np.array_equal(host(C), want), str(tdt)
    assert np.abs(want8).max() > 20 and sq.device_status(ws) == 0


@pytest.mark.parametrize("gran", ["per_channel", "per_tensor"])
def test_quant_weight_then_decode_gemm_back_to_back(gran):
    """sq_quant_weight followed directly, on the same stream, by a decode-shaped sq_w8a8_gemm that
    consumes its output: the GEMM starts fetching weights before it waits for its predecessor, so
    the weight writer must be complete by then -- repeated to give an overlap the chance to show."""
    M, N, K = 16, 4096, 4096
    W = synth.weights(28, 1, N, K, "bf16")
    s = synth.rng_for(28, 2).uniform(0.5, 2.0, K).astype(np.float32)
    Xq = synth.int8_tensor(28, 3, (M, K))
    want_Wq, want_ws = oracle.quant_weight(W, s, gran)
    want = oracle.gemm_i32(Xq, want_Wq)
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K))
    Wd, sd, Xd = dev(W, "bf16"), dev(s), dev(Xq)
    Wq = torch.empty((N, K), dtype=torch.int8, device="cuda")
    wsc = torch.empty(N if gran == "per_channel" else 1, dtype=torch.float32, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    for it in range(5):
        Wq.fill_(it + 1)  # stale codes a too-early fetch would pick up
        sq.sq_quant_weight(Wd, sd, gran, Wq=Wq, w_scale=wsc, workspace=ws)
        sq.sq_w8a8_gemm(Xd, Wq, None, None, ws, out=acc)
        assert np.array_equal(host(acc), want), "iteration %d" % it
    assert np.array_equal(host(Wq), want_Wq) and np.array_equal(host(wsc), want_ws)
    assert sq.device_status(ws) == 0


@pytest.mark.parametrize("out", ["f16", "i8", "i32"])
def test_gemm_unaligned_output_rows(ws, out):
    # row stride that is not a multiple of 16 bytes: the epilogue writes rows directly instead of by TMA
    M, N, K, ldy = 150, 201, 256, 203
    Xq, Wq = synth.int8_tensor(23, 3, (M, K)), synth.int8_tensor(23, 4, (N, K))
    xs = np.full(1, 0.05, np.float32)
    wsc = np.full(1, 0.002, np.float32)
    tdt = {"f16": torch.float16, "i8": torch.int8, "i32": torch.int32}[out]
    buf = torch.full((M, ldy), 5, dtype=tdt, device="cuda")
    r = np.array([0.9], np.float32)
    sq.sq_w8a8_gemm(dev(Xq), dev(Wq), dev(xs), dev(wsc), ws, out=buf[:, :N],
                    requant_mul=dev(r) if out == "i8" else None)
    acc = oracle.gemm_i32(Xq, Wq)
    y = oracle.dequant(acc, xs, wsc)
    want = {"f16": oracle.round_to(y, "f16"), "i8": oracle.requant(y, r), "i32": acc}[out]
    got = host(buf)
    assert np.array_equal(got[:, :N], want)
    assert np.all(got[:, N:] == 5)


def _qkv_views(B, H, S, d, seed):
    T = B * S
    qkv = synth.int8_tensor(24, seed, (T, 3 * H * d))
    return qkv


@pytest.mark.parametrize("B,H,S,d", [(1, 2, 128, 128), (2, 3, 512, 128), (1, 1, 200, 64), (2, 2, 136, 128)])
def test_bmm_qk_from_fused_qkv_buffer(ws, B, H, S, d):
    qkv = _qkv_views(B, H, S, d, 1)
    row = 3 * H * d
    qkv_d = dev(qkv)
    alpha = np.float32(0.0123)
    out = torch.empty((B, H, S, S), dtype=torch.float16, device="cuda")
    acc = torch.empty((B, H, S, S), dtype=torch.int32, device="cuda")
    q_view = qkv_d.view(-1)  # Q at column 0, K at column H*d
    k_view = qkv_d.view(-1)[H * d:]
    for o in (out, acc):
        sq.sq_w8a8_bmm(q_view, k_view, B, H, S, S, d, (S * row, d, row), (S * row, d, row), False, alpha, o,
                       (H * S * S, S * S, S), ws)
    q = qkv.reshape(B, S, 3, H, d)[:, :, 0].transpose(0, 2, 1, 3)
    k = qkv.reshape(B, S, 3, H, d)[:, :, 1].transpose(0, 2, 1, 3)
    want_acc, want = oracle.w8a8_bmm(np.ascontiguousarray(q), np.ascontiguousarray(k), alpha, out_dtype="f16")
    assert np.array_equal(host(acc), want_acc)
    assert_fp_close(host(out), want, "f16", "QK^T")
    assert np.array_equal(host(out), want)


@pytest.mark.parametrize("B,H,S,d", [(1, 2, 128, 128), (2, 3, 512, 128), (1, 2, 144, 64), (1, 1, 256, 16)])
def test_bmm_pv_with_kn_operand(ws, B, H, S, d):
    qkv = _qkv_views(B, H, S, d, 2)
    row = 3 * H * d
    P = synth.int8_tensor(24, 3, (B, H, S, S), lo=0, hi=127)
    alpha = np.float32(3.1e-4)
    r = np.array([1.7], np.float32)
    qkv_d = dev(qkv)
    v_view = qkv_d.view(-1)[2 * H * d:]
    acc = torch.empty((B * S, H * d), dtype=torch.int32, device="cuda")
    o8 = torch.empty((B * S, H * d), dtype=torch.int8, device="cuda")
    of = torch.empty((B * S, H * d), dtype=torch.float16, device="cuda")
    Pd = dev(P)
    for o, rq in ((acc, None), (o8, dev(r)), (of, None)):
        sq.sq_w8a8_bmm(Pd, v_view, B, H, S, d, S, (H * S * S, S * S, S), (S * row, d, row), True, alpha, o,
                       (S * H * d, d, H * d), ws, requant_mul=rq)
    v = np.ascontiguousarray(qkv.reshape(B, S, 3, H, d)[:, :, 2].transpose(0, 2, 1, 3))  # [B,H,S,d]
    want_acc, want_q = oracle.w8a8_bmm(P, v, alpha, b_is_kn=True, requant_mul=r)
    _, want_f = oracle.w8a8_bmm(P, v, alpha, b_is_kn=True, out_dtype="f16")
    to_rows = lambda a: a.transpose(0, 2, 1, 3).reshape(B * S, H * d)  # [B,H,S,d] -> [B*S, H*d]
    assert np.array_equal(host(acc), to_rows(want_acc))
    assert np.array_equal(host(o8), to_rows(want_q))
    assert np.array_equal(host(of), to_rows(want_f))


@pytest.mark.parametrize("B,H,S,d", [(1, 2, 512, 128), (2, 1, 384, 64), (1, 1, 208, 128)])
def test_bmm_causal_skips_only_what_attention_never_reads(ws, B, H, S, d):
    qkv = _qkv_views(B, H, S, d, 7)
    row = 3 * H * d
    qkv_d = dev(qkv)
    flat = qkv_d.view(-1)
    alpha = np.float32(0.004)
    sentinel = -777.0
    scores = torch.full((B, H, S, S), sentinel, dtype=torch.float16, device="cuda")
    sq.sq_w8a8_bmm(flat, flat[H * d:], B, H, S, S, d, (S * row, d, row), (S * row, d, row), False, alpha, scores,
                   (H * S * S, S * S, S), ws, causal=True)
    q = np.ascontiguousarray(qkv.reshape(B, S, 3, H, d)[:, :, 0].transpose(0, 2, 1, 3))
    k = np.ascontiguousarray(qkv.reshape(B, S, 3, H, d)[:, :, 1].transpose(0, 2, 1, 3))
    v = np.ascontiguousarray(qkv.reshape(B, S, 3, H, d)[:, :, 2].transpose(0, 2, 1, 3))
    _, want = oracle.w8a8_bmm(q, k, alpha, out_dtype="f16")
    got = host(scores)
    tril = np.tril(np.ones((S, S), bool))
    assert np.array_equal(got[..., tril], want[..., tril])  # every score a causal softmax reads
    upper = got[..., ~tril]
    assert np.all((upper == sentinel) | (upper == want[..., ~tril]))  # the rest: computed or left alone
    # P.V with a lower-triangular P: causal K-slice skipping leaves the result unchanged
    P = np.tril(synth.int8_tensor(24, 8, (B, H, S, S), lo=0, hi=127))
    a2 = np.float32(2.5e-4)
    acc = torch.empty((B * S, H * d), dtype=torch.int32, device="cuda")
    sq.sq_w8a8_bmm(dev(P), flat[2 * H * d:], B, H, S, d, S, (H * S * S, S * S, S), (S * row, d, row), True, a2, acc,
                   (S * H * d, d, H * d), ws, causal=True)
    want_acc, _ = oracle.w8a8_bmm(P, v, a2, b_is_kn=True, out_dtype="f16")
    assert np.array_equal(host(acc), want_acc.transpose(0, 2, 1, 3).reshape(B * S, H * d))
