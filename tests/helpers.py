"""Shared helpers for the parity tests (no method arithmetic here)."""
import numpy as np
import torch

TDT = {"f16": torch.float16, "bf16": torch.bfloat16}


def dev(a, dtype=None):
    """numpy (A-valued float32 / int8 / float32) -> CUDA tensor of the given dtype."""
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(TDT.get(dtype, dtype))
    return t.cuda()


def host(t):
    """CUDA tensor -> numpy; fp16/bf16 are widened to float32 exactly."""
    if t.dtype in (torch.float16, torch.bfloat16):
        t = t.float()
    return t.cpu().numpy()


def ulp(y, dtype):
    """Spacing of `dtype` at |y| (normal range)."""
    mant = {"f16": 10, "bf16": 7}[dtype]
    e = np.floor(np.log2(np.maximum(np.abs(y), 1e-30)))
    emin = {"f16": -14, "bf16": -126}[dtype]
    return np.exp2(np.maximum(e, emin) - mant)


def assert_fp_close(got, want, dtype, what=""):
    """The stated tolerance for dequantised outputs: 1e-3 relative or 2 ULP of the output type."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    tol = np.maximum(1e-3 * np.abs(want), 2 * ulp(want, dtype))
    bad = np.abs(got - want) > tol
    assert not bad.any(), "%s: %d of %d outside tolerance, worst |diff| %.3g" % (
        what, bad.sum(), bad.size, np.abs(got - want).max())
