"""sq_ln_quant_tensor_noalloc: the per-tensor-dynamic LayerNorm+quantise for callers that cannot
allocate device memory (plug-ins handed only input/output buffers, engines with a pre-sized arena,
loops where cudaMalloc's implicit synchronisation is not allowed).  Its scratch is a fixed array
inside the library, so the check is simply: same bytes as sq_ln_quant with a caller workspace,
on two calls in a row (the second call sees the array as the first one left it).

Collected last on purpose: a failure here cannot hide another test's result under `-x`."""
import numpy as np
import pytest
import torch

from helpers import dev
from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import synth

pytestmark = pytest.mark.gpu


def _case(M, C, dtype, tid):
    ch = synth.outlier_channels(14, C, count=4)
    x = synth.activations(14, tid, M, C, dtype, ch, np.full(4, 60.0))
    gamma, beta = synth.ln_params(14, tid + 1, C, dtype)
    return dev(x, dtype), dev(gamma, dtype), dev(beta, dtype)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_noalloc_matches_workspace_entry_point_twice(dtype):
    eps = 1e-5
    # two different problems back to back: the second call's maximum is SMALLER than the first's,
    # so a scratch word that was not re-zeroed would give a wrong step size
    cases = [_case(96, 5120, dtype, 1), _case(33, 1024, dtype, 5)]
    cases[1] = (cases[1][0] * 0.25, cases[1][1], cases[1][2])
    for x, g, b in cases:
        M, C = x.shape
        ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_LN_QUANT, M, 0, C))
        want_q, want_s = sq.sq_ln_quant(x, g, b, eps, "per_tensor_dynamic", workspace=ws)
        got_q, got_s = sq.sq_ln_quant_tensor_noalloc(x, g, b, eps)
        torch.cuda.synchronize()
        assert torch.equal(got_s, want_s)
        assert torch.equal(got_q, want_q)
        assert int(got_q.abs().max()) == 127


def test_noalloc_without_beta_and_repeat():
    x, g, _ = _case(64, 7168, "bf16", 9)
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_LN_QUANT, 64, 0, 7168))
    want_q, want_s = sq.sq_ln_quant(x, g, None, 1e-5, "per_tensor_dynamic", workspace=ws)
    for _ in range(2):
        got_q, got_s = sq.sq_ln_quant_tensor_noalloc(x, g, None, 1e-5)
        assert torch.equal(got_q, want_q) and torch.equal(got_s, want_s)


def test_noalloc_rejects_more_rows_than_its_scratch_holds():
    M, C = sq.SQ_NOALLOC_MAX_ROWS + 1, 64
    x = torch.zeros((M, C), dtype=torch.float16, device="cuda")
    g = torch.ones(C, dtype=torch.float16, device="cuda")
    with pytest.raises(sq.SqError) as e:
        sq.sq_ln_quant_tensor_noalloc(x, g, None, 1e-5)
    assert e.value.code == 4 and "SQ_ERR_UNSUPPORTED" in str(e.value)
    # the limit itself is accepted
    xq, xs = sq.sq_ln_quant_tensor_noalloc(x[:sq.SQ_NOALLOC_MAX_ROWS], g, None, 1e-5)
    torch.cuda.synchronize()
    assert not xq.any()
