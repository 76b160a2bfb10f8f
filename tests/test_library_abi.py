"""Host-side checks that need no GPU: the C-ABI library builds, loads and exports every symbol the
header declares, and argument validation answers before any CUDA work."""
import ctypes
import os
import re

import pytest

from paper_2211_10438_b200 import binding as sq
from paper_2211_10438_b200 import build as sq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    sq_build.build()
    return sq.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "sq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert set(names) == set(sq.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    assert sq.status_str(0) == "SQ_OK"
    assert sq.status_str(6) == "SQ_ERR_TIMEOUT"
    assert sq.status_str(99) == "SQ_ERR_UNKNOWN"


def test_workspace_sizes(lib):
    assert sq.workspace_bytes(sq.SQ_OP_GEMM, 2048, 15360, 5120) >= 256
    assert sq.workspace_bytes(sq.SQ_OP_LN_QUANT, 100, 0, 512) >= 256 + 800


def test_validation_without_cuda(lib):
    p = ctypes.c_void_p(0x1000)  # never dereferenced: validation fails first
    i8 = ctypes.c_void_p(0x2000)
    # alpha outside [0, 1]
    assert lib.sq_smooth_scales(p, p, 8, 1.5, p, None, None) == 1
    assert lib.sq_smooth_scales(p, p, 8, -0.1, p, None, None) == 1
    # zero-sized problems are no-ops
    assert lib.sq_smooth_scales(p, p, 0, 0.5, p, None, None) == 0
    assert lib.sq_calib_absmax(p, sq.SQ_BF16, 0, 64, 64, p, None) == 0
    assert lib.sq_quant_act(p, sq.SQ_BF16, 0, 64, 2, None, i8, p, None, 0, None) == 0
    # bad dtype / shape / alignment
    assert lib.sq_calib_absmax(p, sq.SQ_I8, 4, 64, 64, p, None) == 1
    assert lib.sq_calib_absmax(p, sq.SQ_F16, 4, 64, 32, p, None) == 2
    assert lib.sq_quant_act(p, sq.SQ_F16, 4, 60, 2, None, i8, p, None, 0, None) == 3
    assert lib.sq_quant_act(ctypes.c_void_p(0x1002), sq.SQ_F16, 4, 64, 2, None, i8, p, None, 0, None) == 3
    assert lib.sq_quant_act(p, sq.SQ_F16, 4, 64, 1, None, i8, p, None, 0, None) == 7  # needs workspace
    # GEMM: K beyond the INT32-safe bound, misaligned K, missing workspace, missing requant
    ws = ctypes.c_void_p(0x10000)
    args = lambda K, out_dt=sq.SQ_F16, rq=None, wsp=ws, wsn=256: lib.sq_w8a8_gemm(
        i8, i8, 16, 16, K, p, 1, p, 1, None, 0, 0, rq, 0, None, p, out_dt, 16, wsp, wsn, None)
    assert args(sq.SQ_MAX_K + 8) == 4
    assert args(24) == 3
    assert args(64, wsp=None, wsn=0) == 7
    assert args(64, out_dt=sq.SQ_I8) == 1
    assert args(64, rq=p) == 1
    # GEMM with the residual add: residual required, 16-bit output only, whole 8-element vectors
    big = sq.workspace_bytes(sq.SQ_OP_GEMM, 16, 16, 64)
    res = lambda r=p, out_dt=sq.SQ_F16, N=16, ldr=16, M=16: lib.sq_w8a8_gemm_residual(
        i8, i8, M, N, 64, p, 1, p, 1, None, 0, r, ldr, p, out_dt, 16, ws, big, None)
    assert res(r=None) == 1
    assert res(out_dt=sq.SQ_I32) == 1
    assert res(ldr=8) == 2
    assert res(ldr=20) == 3
    assert res(N=12, ldr=16) == 3
    assert res(r=ctypes.c_void_p(0x1008)) == 3
    assert res(M=0) == 0
    arr = ctypes.c_int64 * 3
    assert lib.sq_w8a8_bmm(i8, i8, 1, 1, 16, 256, 64, arr(0, 0, 64), arr(0, 0, 256), 1, 0, 1.0, None, p,
                           sq.SQ_F16, arr(0, 0, 256), ws, 256, None) == 4  # [K,N] B limited to N <= 128
    assert lib.sq_w8a8_bmm(i8, i8, 1, 1, 16, 64, 64, arr(0, 0, 72), arr(0, 0, 64), 0, 0, 1.0, None, p,
                           sq.SQ_F16, arr(0, 0, 64), ws, 256, None) == 3  # stride not a multiple of 16


def test_binding_refuses_cpu_tensors(lib):
    import torch
    with pytest.raises(RuntimeError):
        sq.sq_calib_absmax(torch.zeros(4, 8, dtype=torch.float16), torch.zeros(8))
