"""Call sequences of the hot path (orchestration only: every step is a libsq call).

`prepare_linear` is the offline transform of Section 4 (calibrate -> Eq. 4 -> fold -> quantise
weights); `LinearBlock.step` is the runtime path of one decoder block's four linear layers
(fused LayerNorm+quantise / quantise -> INT8 GEMM with dequant epilogue).
"""
from dataclasses import dataclass

import torch

from . import binding as sq


@dataclass
class PreparedLinear:
    name: str
    Wq: torch.Tensor        # [N, K] int8
    w_scale: torch.Tensor   # [N] or [1] fp32
    bias: torch.Tensor      # [N] A or None
    relu: bool
    s: torch.Tensor = None          # smoothing factor [K] (None: input not smoothed)
    gamma_hat: torch.Tensor = None  # folded LayerNorm parameters when the input is a LayerNorm
    beta_hat: torch.Tensor = None
    act_absmax: torch.Tensor = None


def prepare_linear(name, W, bias, relu, calib_batches, alpha, w_gran, workspace, gamma=None, beta=None):
    """Offline: per-channel absmax over the calibration batches, Eq. 4, fold into the LayerNorm
    (when gamma is given), fold into W and quantise it.  With calib_batches=None the input is
    left unsmoothed (out-proj / FC2)."""
    dev = W.device
    K = W.shape[1]
    s = gh = bh = ax = None
    if calib_batches is not None:
        ax = torch.zeros(K, dtype=torch.float32, device=dev)
        for xb in calib_batches:
            sq.sq_calib_absmax(xb, ax)
        aw = torch.zeros(K, dtype=torch.float32, device=dev)
        sq.sq_calib_absmax(W, aw)
        s = sq.sq_smooth_scales(ax, aw, alpha)
        if gamma is not None:
            gh, bh = sq.sq_fold_ln_weight(gamma, beta, s)
    Wq, w_scale = sq.sq_quant_weight(W, s, w_gran, workspace=workspace)
    return PreparedLinear(name, Wq, w_scale, bias, relu, s, gh, bh, ax)


class LinearBlock:
    """The four W8A8 linears of one decoder block at a fixed token count, dynamic per-token (or
    per-tensor) activation quantisation: LN1->QKV, attn_out->out_proj, LN2->FC1(+ReLU), ->FC2."""

    def __init__(self, qkv, out_proj, fc1, fc2, M, act_dtype, gran="per_token", eps=1e-5):
        self.lin = {"qkv": qkv, "out_proj": out_proj, "fc1": fc1, "fc2": fc2}
        self.M, self.dt, self.gran, self.eps = M, act_dtype, gran, eps
        dev = qkv.Wq.device
        ns = M if gran == "per_token" else 1
        self.buf = {}
        for n, l in self.lin.items():
            N, K = l.Wq.shape
            self.buf[n] = dict(Xq=torch.empty((M, K), dtype=torch.int8, device=dev),
                               xs=torch.empty(ns, dtype=torch.float32, device=dev),
                               Y=torch.empty((M, N), dtype=act_dtype, device=dev))
        need = max(sq.workspace_bytes(sq.SQ_OP_GEMM, M, max(l.Wq.shape[0] for l in self.lin.values()),
                                      max(l.Wq.shape[1] for l in self.lin.values())),
                   sq.workspace_bytes(sq.SQ_OP_LN_QUANT, M, 0, 0))
        self.ws = sq.new_workspace(need, dev)
        self.launches_per_step = 8 if gran != "per_tensor_dynamic" else 12
        self.gemm_events = None  # optional list collecting (start, stop) CUDA events per GEMM

    def _gemm(self, name):
        l, b = self.lin[name], self.buf[name]
        ev = None
        if self.gemm_events is not None:
            ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
            ev[0].record()
        sq.sq_w8a8_gemm(b["Xq"], l.Wq, b["xs"], l.w_scale, self.ws, bias=l.bias, relu=l.relu, out=b["Y"])
        if ev is not None:
            ev[1].record()
            self.gemm_events.append((name, ev))
        return b["Y"]

    def step(self, x_in, attn_out):
        """x_in: block input [M, hidden]; attn_out: attention output [M, hidden] (the attention
        itself is a separate path).  Returns the FC2 output."""
        q, o, f1, f2 = (self.lin[n] for n in ("qkv", "out_proj", "fc1", "fc2"))
        b = self.buf
        sq.sq_ln_quant(x_in, q.gamma_hat, q.beta_hat, self.eps, self.gran, Xq=b["qkv"]["Xq"],
                       x_scale=b["qkv"]["xs"], workspace=self.ws)
        self._gemm("qkv")
        sq.sq_quant_act(attn_out, self.gran, Xq=b["out_proj"]["Xq"], x_scale=b["out_proj"]["xs"],
                        workspace=self.ws)
        h = self._gemm("out_proj")
        sq.sq_ln_quant(h, f1.gamma_hat, f1.beta_hat, self.eps, self.gran, Xq=b["fc1"]["Xq"],
                       x_scale=b["fc1"]["xs"], workspace=self.ws)
        a = self._gemm("fc1")
        sq.sq_quant_act(a, self.gran, Xq=b["fc2"]["Xq"], x_scale=b["fc2"]["xs"], workspace=self.ws)
        return self._gemm("fc2")

    def gemm_ops(self):
        return sum(2 * self.M * l.Wq.shape[0] * l.Wq.shape[1] for l in self.lin.values())


def synth_device_activations(M, C, dtype, channels, factors, seed, device="cuda"):
    """Device-side draw of the outlier-channel activation model (inputs only, no method math)."""
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    x = torch.randn((M, C), generator=g, device=device, dtype=torch.float32)
    if len(channels):
        idx = torch.as_tensor(channels, device=device, dtype=torch.long)
        x[:, idx] *= torch.as_tensor(factors, device=device, dtype=torch.float32)[None, :]
    return x.to(dtype)


def synth_device_weights(N, K, dtype, seed, std=0.02, device="cuda"):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return (torch.randn((N, K), generator=g, device=device, dtype=torch.float32) * std).to(dtype)
