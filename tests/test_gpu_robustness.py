"""GPU robustness checks that are not about arithmetic: the bounded waits really give up and report,
and kernels write nothing outside their output tensors (guard bands around every output)."""
import numpy as np
import pytest
import torch

from helpers import dev
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import synth

pytestmark = pytest.mark.gpu

GUARD = 64 * 1024  # bytes of canary before and after each output


def test_bounded_wait_gives_up_and_reports():
    word = sq.sq_selftest_bounded_wait(budget_cycles=200000)  # ~0.1 ms
    assert word & 0xFF == 6, "expected SQ_ERR_TIMEOUT in the status word, got %d" % word
    assert (word >> 8) == 15
    # the context is still usable afterwards
    x = torch.ones(8, device="cuda")
    assert float(x.sum()) == 8.0


def test_row_kernel_wait_gives_up_and_reports():
    """The wait of the row kernels (quantisers, fused LayerNorm) for a row's bulk copy: on a barrier
    nothing completes it expires, leaves SQ_ERR_TIMEOUT | 5 << 8 in the status word and returns."""
    word = sq.sq_selftest_row_wait(budget_cycles=200000)
    assert word == (sq.SQ_ERR_TIMEOUT | (5 << 8)), "status word %d" % word
    assert float(torch.ones(8, device="cuda").sum()) == 8.0  # the context is still usable


def test_row_kernels_leave_a_given_status_word_alone_when_nothing_expires():
    """Per-token and static calls now take the workspace as their status word: a clean run leaves it zero."""
    x = dev(synth.activations(1, 2, 40, 5120, "bf16", [3], [50.0]), "bf16")
    g = torch.ones(5120, dtype=torch.bfloat16, device="cuda")
    ws = sq.new_workspace(256)
    sq.sq_quant_act(x, "per_token", workspace=ws)
    sq.sq_ln_quant(x, g, None, 1e-5, "per_token", workspace=ws)
    sq.sq_quant_act(x, "per_tensor_static", x_scale=torch.full((1,), 0.1, device="cuda"), workspace=ws)
    torch.cuda.synchronize()
    assert not ws.any()


def _guarded(nbytes, dtype):
    """A uint8 arena with canaries; returns (arena, view of the payload as `dtype`)."""
    arena = torch.full((GUARD + nbytes + GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
    return arena, arena[GUARD:GUARD + nbytes].view(dtype)


def _guards_intact(arena, nbytes):
    return bool((arena[:GUARD] == 0xA5).all()) and bool((arena[GUARD + nbytes:] == 0xA5).all())


@pytest.mark.parametrize("M,N,K,out", [(300, 520, 272, torch.bfloat16), (2048, 5120, 256, torch.int8),
                                        (16, 1280, 4096, torch.bfloat16), (129, 257, 144, torch.int32)])
def test_gemm_writes_only_its_output(M, N, K, out):
    Xq, Wq = dev(synth.int8_tensor(40, 1, (M, K))), dev(synth.int8_tensor(40, 2, (N, K)))
    xs = torch.full((M,), 0.05, device="cuda")
    wsc = torch.full((N,), 0.002, device="cuda")
    r = torch.full((1,), 0.9, device="cuda")
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K))
    esz = torch.empty(0, dtype=out).element_size()
    arena, Y = _guarded(M * N * esz, out)
    sq.sq_w8a8_gemm(Xq, Wq, xs, wsc, ws, out=Y.view(M, N), requant_mul=r if out == torch.int8 else None)
    torch.cuda.synchronize()
    assert _guards_intact(arena, M * N * esz)
    assert sq.device_status(ws) == 0


@pytest.mark.parametrize("M,C,ln", [(37, 5120, True), (130, 7168, False), (5, 20480, True), (3, 81920, False)])
def test_quantisers_write_only_their_outputs(M, C, ln):
    x = dev(synth.activations(40, 3, M, C, "bf16", [1, 5], [50.0, 60.0]), "bf16")
    g, b = (dev(a, "bf16") for a in synth.ln_params(40, 4, C, "bf16"))
    a_q, Xq = _guarded(M * C, torch.int8)
    a_s, xs = _guarded(M * 4, torch.float32)
    if ln:
        sq.sq_ln_quant(x, g, b, 1e-5, "per_token", Xq=Xq.view(M, C), x_scale=xs)
    else:
        sq.sq_quant_act(x, "per_token", Xq=Xq.view(M, C), x_scale=xs)
    torch.cuda.synchronize()
    assert _guards_intact(a_q, M * C) and _guards_intact(a_s, M * 4)
    assert int(Xq.abs().max()) == 127
