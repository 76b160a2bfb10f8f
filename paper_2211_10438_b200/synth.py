"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no part of the method's arithmetic: it only draws tensors.
Both the CUDA tests/benchmark and the CPU oracle's tests read the bytes made
here, so the two sides always see identical inputs.

Activation model (Section 3 of the paper, observations 2 and 3): values are
N(0, 1) except in a small seeded set of OUTLIER CHANNELS that is fixed across
all tokens and all calibration batches; every value of such a channel is
multiplied by a per-channel factor of 20-100.  Weights are flat: N(0, 0.02).
These tensors stand in for the Pile calibration sentences and for real
OPT / GPT-3 / MT-NLG activations, none of which are available offline.
"""
from dataclasses import dataclass, field

import numpy as np

SEED_BASE = 0x5EED0000
OUTLIER_SALT = 0xC4A77E15


def rng_for(config: int, tensor_id: int, salt: int = 0) -> np.random.Generator:
    """Counter-based generator keyed by (config, tensor id)."""
    seed = (SEED_BASE + 256 * config + tensor_id) ^ salt
    return np.random.Generator(np.random.Philox(key=seed))


def to_dtype_f32(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round fp64/fp32 draws once to fp16/bf16 and widen back to float32."""
    x = np.asarray(x, np.float32)
    if dtype == "f16":
        return x.astype(np.float16).astype(np.float32)
    if dtype == "bf16":
        import torch
        return torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    raise ValueError(dtype)


def outlier_channels(config: int, C: int, count: int = None, frac: float = None):
    """The persistent outlier-channel set of one activation stream."""
    g = rng_for(config, 0, OUTLIER_SALT)
    n = count if count is not None else max(1, int(np.ceil(frac * C)))
    return np.sort(g.choice(C, size=n, replace=False))


def outlier_factors(config: int, n: int, lo: float, hi: float):
    g = rng_for(config, 1, OUTLIER_SALT)
    if lo == hi:
        return np.full(n, lo, np.float64)
    return g.uniform(lo, hi, size=n)


def activations(config: int, tensor_id: int, M: int, C: int, dtype: str, channels, factors):
    """[M, C] activations: N(0,1) with the given outlier channels scaled."""
    g = rng_for(config, tensor_id)
    x = g.standard_normal((M, C), dtype=np.float32)
    if len(channels):
        x[:, channels] *= np.asarray(factors, np.float32)[None, :]
    return to_dtype_f32(x, dtype)


def weights(config: int, tensor_id: int, N: int, K: int, dtype: str, std: float = 0.02):
    g = rng_for(config, tensor_id)
    return to_dtype_f32(g.standard_normal((N, K), dtype=np.float32) * np.float32(std), dtype)


def bias(config: int, tensor_id: int, N: int, dtype: str, std: float = 0.01):
    g = rng_for(config, tensor_id)
    return to_dtype_f32(g.standard_normal(N, dtype=np.float32) * np.float32(std), dtype)


def ln_params(config: int, tensor_id: int, C: int, dtype: str):
    """gamma = 1 + 0.1 N(0,1), beta = 0.1 N(0,1)."""
    g = rng_for(config, tensor_id)
    gamma = 1.0 + 0.1 * g.standard_normal(C, dtype=np.float32)
    beta = 0.1 * g.standard_normal(C, dtype=np.float32)
    return to_dtype_f32(gamma, dtype), to_dtype_f32(beta, dtype)


def int8_tensor(config: int, tensor_id: int, shape, lo: int = -127, hi: int = 127):
    """Uniform INT8 codes, for tests that feed the integer stages directly."""
    g = rng_for(config, tensor_id)
    return g.integers(lo, hi + 1, size=shape, dtype=np.int8)


# --------------------------------------------------------------------------- #
# Workload shapes
# --------------------------------------------------------------------------- #
@dataclass
class LinearShape:
    name: str
    N: int
    K: int
    relu: bool = False
    ln_input: bool = False  # input comes from a LayerNorm with folded smoothing


@dataclass
class Workload:
    config: int
    name: str
    dtype: str
    hidden: int
    tokens: tuple
    linears: tuple
    outlier_count: int = None
    outlier_frac: float = None
    outlier_lo: float = 50.0
    outlier_hi: float = 50.0
    alpha: float = 0.5
    heads: int = 0
    head_dim: int = 0
    ffn: int = 0
    extra: dict = field(default_factory=dict)

    def outliers(self, C=None):
        C = C or self.hidden
        ch = outlier_channels(self.config, C, self.outlier_count, self.outlier_frac)
        return ch, outlier_factors(self.config, len(ch), self.outlier_lo, self.outlier_hi)


def _block_linears(h, ffn):
    return (LinearShape("qkv", 3 * h, h, ln_input=True), LinearShape("out_proj", h, h),
            LinearShape("fc1", ffn, h, relu=True, ln_input=True), LinearShape("fc2", h, ffn))


WORKLOADS = {
    # tiny single linear; calibration = the same X
    1: Workload(1, "tiny-linear", "f16", 512, (16,), (LinearShape("linear", 512, 512),),
                outlier_count=4, outlier_lo=50.0, outlier_hi=50.0),
    # OPT-13B-shaped linears, prefill, M = 4 x 512
    2: Workload(2, "opt13b-prefill", "bf16", 5120, (2048,), _block_linears(5120, 20480),
                outlier_frac=0.01, outlier_lo=20.0, outlier_hi=80.0, heads=40, head_dim=128,
                ffn=20480),
    # OPT-30B-shaped full decoder block, static scales
    3: Workload(3, "opt30b-block", "f16", 7168, (512, 2048, 8192), _block_linears(7168, 28672),
                outlier_frac=0.01, outlier_lo=20.0, outlier_hi=80.0, heads=56, head_dim=128,
                ffn=28672, extra={"seq": 512, "calib_samples": 128}),
    # decode-shaped small-M GEMMs at GPT-3 / OPT-175B shape
    4: Workload(4, "gpt3-decode", "bf16", 12288, (1, 2, 4, 8, 16),
                (LinearShape("qkv", 36864, 12288), LinearShape("fc1", 49152, 12288),
                 LinearShape("fc2", 12288, 49152)),
                outlier_frac=0.01, outlier_lo=20.0, outlier_hi=80.0),
    # MT-NLG-530B-shaped prefill sweep
    5: Workload(5, "mtnlg-prefill", "bf16", 20480, (4096, 8192, 16384),
                _block_linears(20480, 81920), outlier_frac=0.005, outlier_lo=100.0,
                outlier_hi=100.0, extra={"alphas": (0.5, 0.75, 0.85), "calib_batches": 512,
                                         "calib_tokens": 2048}),
}
