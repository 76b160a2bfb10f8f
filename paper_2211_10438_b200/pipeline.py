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
        need = max([sq.workspace_bytes(sq.SQ_OP_GEMM, M, l.Wq.shape[0], l.Wq.shape[1]) for l in self.lin.values()] +
                   [sq.workspace_bytes(sq.SQ_OP_LN_QUANT, M, 0, 0)])
        self.ws = sq.new_workspace(need, dev)
        self.launches_per_step = 8 if gran != "per_tensor_dynamic" else 12
        self.gemm_events = None  # optional list collecting (start, stop) CUDA events per GEMM

    def _gemm(self, name, out=None):
        l, b = self.lin[name], self.buf[name]
        Y = b["Y"] if out is None else out
        ev = None
        if self.gemm_events is not None:
            ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
            ev[0].record()
        sq.sq_w8a8_gemm(b["Xq"], l.Wq, b["xs"], l.w_scale, self.ws, bias=l.bias, relu=l.relu, out=Y)
        if ev is not None:
            ev[1].record()
            self.gemm_events.append((name, ev))
        return Y

    def step(self, x_in, attn_out, out=None):
        """x_in: block input [M, hidden]; attn_out: attention output [M, hidden] (the attention
        itself is a separate path).  Returns the FC2 output (written to `out` when given)."""
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
        return self._gemm("fc2", out=out)

    def gemm_ops(self):
        return sum(2 * self.M * l.Wq.shape[0] * l.Wq.shape[1] for l in self.lin.values())

    def gemm_bytes(self):
        """Algorithmic bytes of the four GEMMs: M*K + N*K (INT8) + M*N outputs in the activation dtype."""
        return sum(self.M * l.Wq.shape[1] + l.Wq.shape[0] * l.Wq.shape[1] + 2 * self.M * l.Wq.shape[0]
                   for l in self.lin.values())


class HostStreamedBlock:
    """Runs LinearBlock steps on inputs that live in pinned HOST memory and returns results to
    pinned host memory, with the copies of neighbouring steps overlapped with the kernels: step
    i+1's inputs go up on one stream and step i-1's result comes down on another while step i
    computes.  Two device slots per buffer; events order slot reuse.  All copies of every step
    are issued and waited for inside whatever region the caller times."""

    def __init__(self, block, hidden):
        self.block = block
        dev = block.ws.device
        M, dt = block.M, block.dt
        e = lambda: torch.empty((M, hidden), dtype=dt, device=dev)
        self.dx, self.da, self.dy = [e(), e()], [e(), e()], [e(), e()]
        self.s_in, self.s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        ev = lambda: [torch.cuda.Event(), torch.cuda.Event()]
        self.in_done, self.comp_done, self.out_done = ev(), ev(), ev()
        self.i = 0

    def submit(self, hx, ha, hy):
        """Queue one step: hx, ha pinned host inputs, hy pinned host output.  Returns at once; hy
        is valid after drain() (or after the out_done event of its slot)."""
        k, first = self.i & 1, self.i < 2
        comp = torch.cuda.current_stream()
        with torch.cuda.stream(self.s_in):
            if not first:
                self.s_in.wait_event(self.comp_done[k])  # step i-2 has finished reading this slot
            self.dx[k].copy_(hx, non_blocking=True)
            self.da[k].copy_(ha, non_blocking=True)
            self.in_done[k].record(self.s_in)
        comp.wait_event(self.in_done[k])
        if not first:
            comp.wait_event(self.out_done[k])  # step i-2's result has left this slot
        self.block.step(self.dx[k], self.da[k], out=self.dy[k])
        self.comp_done[k].record(comp)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.comp_done[k])
            hy.copy_(self.dy[k], non_blocking=True)
            self.out_done[k].record(self.s_out)
        self.i += 1

    def drain(self):
        """Make the compute stream wait for every queued copy-out."""
        comp = torch.cuda.current_stream()
        for k in range(min(self.i, 2)):
            comp.wait_event(self.out_done[k])


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


class DecoderBlockStatic:
    """A full W8A8 decoder block with per-tensor STATIC activation steps (level O3), as seven libsq
    launches from 1024 tokens up (nine below; two more without the fused attention kernel):
    LN1+quantise -> QKV GEMM (INT8 out) -> fused attention (or Q.K^T BMM -> softmax+quantise P ->
    P.V BMM; INT8 out) -> out-proj GEMM with the residual add in its epilogue (or GEMM -> residual
    add) -> LN2+quantise -> FC1 GEMM (+ReLU, INT8 out) -> FC2 GEMM with the residual add in its
    epilogue.  Q, K, V are read in place from the fused QKV buffer.

    `lin` maps "qkv" / "out_proj" / "fc1" / "fc2" to PreparedLinear; `steps` holds the calibrated
    static steps d_ln1, d_q, d_k, d_v, d_attn, d_ln2, d_fc1 (python floats)."""

    def __init__(self, lin, steps, B, S, H, d, act_dtype, eps=1e-5, fused_attention=None):
        self.lin, self.B, self.S, self.H, self.d, self.dt, self.eps = lin, B, S, H, d, act_dtype, eps
        # the fused attention kernel covers head dimension 128; otherwise BMM -> softmax -> BMM
        self.fused_attention = (d == 128) if fused_attention is None else fused_attention
        dev = lin["qkv"].Wq.device
        M, hid, ffn = B * S, H * d, lin["fc1"].Wq.shape[0]
        self.M, self.hid = M, hid
        f32 = lambda v: torch.tensor([v], dtype=torch.float32, device=dev)
        self.steps = dict(steps)
        self.s = {k: f32(v) for k, v in steps.items()}
        one = torch.tensor(1.0, dtype=torch.float32)
        inv = lambda v: float(one / torch.tensor(v, dtype=torch.float32))  # fp32 reciprocal, as the oracle takes it
        self.r_qkv = torch.cat([torch.full((hid,), inv(steps["d_q"])), torch.full((hid,), inv(steps["d_k"])),
                                torch.full((hid,), inv(steps["d_v"]))]).to(torch.float32).to(dev)
        self.r_attn = f32(inv(steps["d_attn"]))
        self.r_fc1 = f32(inv(steps["d_fc1"]))
        t32 = lambda v: torch.tensor(v, dtype=torch.float32)
        self.alpha_qk = float((t32(steps["d_q"]) * t32(steps["d_k"])) / torch.sqrt(t32(float(d))))
        self.alpha_pv = float(t32(steps["d_v"]) / t32(127.0))
        e = lambda shape, dt: torch.empty(shape, dtype=dt, device=dev)
        self.x1q, self.qkv = e((M, hid), torch.int8), e((M, 3 * hid), torch.int8)
        self.scores, self.P = e((B * H, S, S), act_dtype), e((B * H, S, S), torch.int8)
        self.attn, self.h = e((M, hid), torch.int8), e((M, hid), act_dtype)
        self.x2q, self.f1q = e((M, hid), torch.int8), e((M, ffn), torch.int8)
        self.y = e((M, hid), act_dtype)
        need = max([sq.workspace_bytes(sq.SQ_OP_GEMM, M, l.Wq.shape[0], l.Wq.shape[1]) for l in lin.values()] +
                   [sq.workspace_bytes(sq.SQ_OP_LN_QUANT, M, 0, hid)])
        self.ws = sq.new_workspace(need, dev)
        self.fuse_residual = M >= 1024
        self.tmp = None if self.fuse_residual else e((M, hid), act_dtype)
        self.launches_per_step = (7 if self.fused_attention else 9) + (0 if self.fuse_residual else 2)

    def forward(self, x):
        L, s, B, S, H, d, hid = self.lin, self.s, self.B, self.S, self.H, self.d, self.hid
        row = 3 * hid
        sq.sq_ln_quant(x, L["qkv"].gamma_hat, L["qkv"].beta_hat, self.eps, "per_tensor_static", Xq=self.x1q,
                       x_scale=s["d_ln1"], workspace=self.ws)
        sq.sq_w8a8_gemm(self.x1q, L["qkv"].Wq, s["d_ln1"], L["qkv"].w_scale, self.ws, bias=L["qkv"].bias,
                        requant_mul=self.r_qkv, out=self.qkv)
        if self.fused_attention:
            sq.sq_w8a8_attention(self.qkv, B, H, S, d, self.alpha_qk, self.alpha_pv, self.r_attn, self.attn, self.ws)
        else:
            flat = self.qkv.view(-1)
            sq.sq_w8a8_bmm(flat, flat[hid:], B, H, S, S, d, (S * row, d, row), (S * row, d, row), False,
                           self.alpha_qk, self.scores, (H * S * S, S * S, S), self.ws, causal=True)
            sq.sq_softmax_quant_p(self.scores, self.P)
            sq.sq_w8a8_bmm(self.P, flat[2 * hid:], B, H, S, d, S, (H * S * S, S * S, S), (S * row, d, row), True,
                           self.alpha_pv, self.attn, (S * hid, d, hid), self.ws, requant_mul=self.r_attn, causal=True)
        self._linear_residual(self.attn, L["out_proj"], s["d_attn"], x, self.h)
        sq.sq_ln_quant(self.h, L["fc1"].gamma_hat, L["fc1"].beta_hat, self.eps, "per_tensor_static", Xq=self.x2q,
                       x_scale=s["d_ln2"], workspace=self.ws)
        sq.sq_w8a8_gemm(self.x2q, L["fc1"].Wq, s["d_ln2"], L["fc1"].w_scale, self.ws, bias=L["fc1"].bias, relu=True,
                        requant_mul=self.r_fc1, out=self.f1q)
        self._linear_residual(self.f1q, L["fc2"], s["d_fc1"], self.h, self.y)
        return self.y

    def _linear_residual(self, xq, l, d_x, residual, out):
        """out = residual + W8A8 linear(xq): one launch with the add in the GEMM epilogue from 1024 tokens
        up (measured on B200: 3312 -> 3262 us per layer at 8192 tokens), two launches below, where the
        single tile per CTA leaves the longer epilogue exposed (512 tokens: 291 against 296 us)."""
        if self.fuse_residual:
            sq.sq_w8a8_gemm_residual(xq, l.Wq, d_x, l.w_scale, self.ws, residual, bias=l.bias, out=out)
        else:
            sq.sq_w8a8_gemm(xq, l.Wq, d_x, l.w_scale, self.ws, bias=l.bias, out=self.tmp)
            sq.sq_residual_add(residual, self.tmp, out=out)

    def ops(self):
        """Integer ops of the four GEMMs and two BMMs of one forward."""
        M, hid, S, d = self.M, self.hid, self.S, self.d
        lin = sum(2 * M * l.Wq.shape[0] * l.Wq.shape[1] for l in self.lin.values())
        return lin + 2 * (2 * self.B * self.H * S * S * d)


class DecoderBlockDecode:
    """Generation stage of DecoderBlockStatic: one new token per sequence against an INT8 KV cache,
    as seven libsq launches: LN1 + static quantiser -> QKV GEMM (INT8 out) -> attention of the new
    token over the cache, which also appends its k, v (INT8 out) -> out-proj GEMM with the residual
    add in its epilogue -> LN2 + static quantiser -> FC1 GEMM (+ReLU, INT8 out) -> FC2 GEMM with the
    residual add in its epilogue.
    `fused=True` moves both LayerNorm+quantise steps into the prologues of the GEMMs that consume
    them (five launches).  Measured on B200 (OPT-30B shapes, batch 16, one CUDA graph per step): inside
    a chain of dependent launches the separate quantiser kernel overlaps the GEMM's own start-up and
    the seven-launch form is the faster one (152 against 158 us per layer); for a GEMM called on its
    own the fused form wins.  `fuse_residual=False` keeps the residual adds as kernels of their own
    (nine launches with `fused=False`: about 3 us more).  Same `lin` / `steps` as the prompt block.  `ctx`
    (int32 device tensor [B]) counts the positions each sequence has cached.  `keep_codes` also
    writes the LayerNorm codes of the fused form to x1q / x2q so that a checker can look at them."""

    def __init__(self, lin, steps, B, H, d, L_max, act_dtype, eps=1e-5, fused=False, keep_codes=False,
                 fuse_residual=True):
        self.lin, self.B, self.H, self.d, self.L_max, self.dt, self.eps = lin, B, H, d, L_max, act_dtype, eps
        self.fused = fused and B <= 32
        self.fuse_residual = fuse_residual
        self.keep_codes = keep_codes
        dev = lin["qkv"].Wq.device
        hid, ffn = H * d, lin["fc1"].Wq.shape[0]
        self.hid = hid
        f32 = lambda v: torch.tensor([v], dtype=torch.float32, device=dev)
        self.s = {k: f32(v) for k, v in steps.items()}
        one = torch.tensor(1.0, dtype=torch.float32)
        inv = lambda v: float(one / torch.tensor(v, dtype=torch.float32))
        self.r_qkv = torch.cat([torch.full((hid,), inv(steps["d_q"])), torch.full((hid,), inv(steps["d_k"])),
                                torch.full((hid,), inv(steps["d_v"]))]).to(torch.float32).to(dev)
        self.r_attn, self.r_fc1 = f32(inv(steps["d_attn"])), f32(inv(steps["d_fc1"]))
        t32 = lambda v: torch.tensor(v, dtype=torch.float32)
        self.alpha_qk = float((t32(steps["d_q"]) * t32(steps["d_k"])) / torch.sqrt(t32(float(d))))
        self.alpha_pv = float(t32(steps["d_v"]) / t32(127.0))
        e = lambda shape, dt: torch.empty(shape, dtype=dt, device=dev)
        self.x1q, self.qkv, self.attn = e((B, hid), torch.int8), e((B, 3 * hid), torch.int8), e((B, hid), torch.int8)
        self.proj, self.h = e((B, hid), act_dtype), e((B, hid), act_dtype)
        self.x2q, self.f1q = e((B, hid), torch.int8), e((B, ffn), torch.int8)
        self.fc2, self.y = e((B, hid), act_dtype), e((B, hid), act_dtype)
        self.k_cache = torch.zeros((B, H, L_max, d), dtype=torch.int8, device=dev)
        self.v_cache = torch.zeros((B, H, L_max // 4, d, 4), dtype=torch.int8, device=dev)
        self.ctx = torch.zeros(B, dtype=torch.int32, device=dev)
        self.lens = torch.ones(B, dtype=torch.int32, device=dev)  # ctx + 1: what the new token attends over
        op = sq.SQ_OP_GEMM_FUSED_QUANT if self.fused else sq.SQ_OP_GEMM
        need = max([sq.workspace_bytes(op, B, l.Wq.shape[0], l.Wq.shape[1]) for l in lin.values()] +
                   [sq.workspace_bytes(sq.SQ_OP_LN_QUANT, B, 0, hid)])
        self.ws = sq.new_workspace(need, dev)
        self.launches_per_step = 9 - (2 if self.fused else 0) - (2 if self.fuse_residual else 0)

    def load_prompt(self, qkv_codes, S):
        """Fill the cache from a prompt pass's QKV code buffer [B*S, 3*H*d]; every sequence then holds S positions."""
        sq.sq_kv_cache_write(qkv_codes, self.B, S, self.H, self.d, None, self.k_cache, self.v_cache, self.L_max, self.ws)
        self.ctx.fill_(S)
        self.lens.fill_(S + 1)

    def step(self, x, max_len=None, advance=True):
        """x [B, H*d]: the newest token of each sequence.  max_len: host-side bound of ctx + 1
        (default: the cache capacity).  Returns the block output [B, H*d]."""
        L, s, B, H, d = self.lin, self.s, self.B, self.H, self.d
        max_len = self.L_max if max_len is None else max_len
        hid = self.hid
        if self.fused:
            sq.sq_w8a8_gemm_fused_quant(x, L["qkv"].Wq, L["qkv"].w_scale, self.ws, "per_tensor_static", x_scale=s["d_ln1"],
                                        gamma_hat=L["qkv"].gamma_hat, beta_hat=L["qkv"].beta_hat, eps=self.eps,
                                        Xq_out=self.x1q if self.keep_codes else None, bias=L["qkv"].bias,
                                        requant_mul=self.r_qkv, out=self.qkv)
        else:
            sq.sq_ln_quant(x, L["qkv"].gamma_hat, L["qkv"].beta_hat, self.eps, "per_tensor_static", Xq=self.x1q,
                           x_scale=s["d_ln1"], workspace=self.ws)
            sq.sq_w8a8_gemm(self.x1q, L["qkv"].Wq, s["d_ln1"], L["qkv"].w_scale, self.ws, bias=L["qkv"].bias,
                            requant_mul=self.r_qkv, out=self.qkv)
        # the attention kernel takes the new k, v rows from the QKV buffer and caches them
        sq.sq_w8a8_decode_attention(self.qkv, self.k_cache, self.v_cache, self.lens, B, H, d, self.L_max, max_len,
                                    self.alpha_qk, self.alpha_pv, self.ws, requant_mul=self.r_attn, out=self.attn,
                                    k_new=self.qkv[:, hid:], v_new=self.qkv[:, 2 * hid:])
        if self.fuse_residual:
            sq.sq_w8a8_gemm_residual(self.attn, L["out_proj"].Wq, s["d_attn"], L["out_proj"].w_scale, self.ws, x,
                                     bias=L["out_proj"].bias, out=self.h)
        else:
            sq.sq_w8a8_gemm(self.attn, L["out_proj"].Wq, s["d_attn"], L["out_proj"].w_scale, self.ws,
                            bias=L["out_proj"].bias, out=self.proj)
            sq.sq_residual_add(x, self.proj, out=self.h)
        if self.fused:
            sq.sq_w8a8_gemm_fused_quant(self.h, L["fc1"].Wq, L["fc1"].w_scale, self.ws, "per_tensor_static", x_scale=s["d_ln2"],
                                        gamma_hat=L["fc1"].gamma_hat, beta_hat=L["fc1"].beta_hat, eps=self.eps,
                                        Xq_out=self.x2q if self.keep_codes else None, bias=L["fc1"].bias, relu=True,
                                        requant_mul=self.r_fc1, out=self.f1q)
        else:
            sq.sq_ln_quant(self.h, L["fc1"].gamma_hat, L["fc1"].beta_hat, self.eps, "per_tensor_static", Xq=self.x2q,
                           x_scale=s["d_ln2"], workspace=self.ws)
            sq.sq_w8a8_gemm(self.x2q, L["fc1"].Wq, s["d_ln2"], L["fc1"].w_scale, self.ws, bias=L["fc1"].bias, relu=True,
                            requant_mul=self.r_fc1, out=self.f1q)
        if self.fuse_residual:
            sq.sq_w8a8_gemm_residual(self.f1q, L["fc2"].Wq, s["d_fc1"], L["fc2"].w_scale, self.ws, self.h,
                                     bias=L["fc2"].bias, out=self.y)
        else:
            sq.sq_w8a8_gemm(self.f1q, L["fc2"].Wq, s["d_fc1"], L["fc2"].w_scale, self.ws, bias=L["fc2"].bias,
                            out=self.fc2)
            sq.sq_residual_add(self.h, self.fc2, out=self.y)
        if advance:  # bookkeeping of the sequence lengths, not part of the arithmetic
            torch._foreach_add_([self.ctx, self.lens], 1)
        return self.y

    def bytes_per_step(self, ctx_sum):
        """Algorithmic HBM bytes of one step: INT8 weights once + the cache positions attended over."""
        w = sum(l.Wq.numel() for l in self.lin.values())
        return w + 2 * self.H * self.d * (ctx_sum + self.B)


def calibrate_static_steps(lin, calib_batches, B, S, H, d, act_dtype, eps=1e-5, clip_frac=0.0):
    """Static per-tensor steps for DecoderBlockStatic from calibration batches (each [B*S, H*d]):
    the block is walked with DYNAMIC steps and floating-point intermediates, and for every tensor
    that will later be quantised statically the absolute maximum of each calibration token is kept
    (Section 5.1: smoothing factors and static steps are calibrated once, offline).  At the end the
    static step of a tensor is Eq. 1's step of the largest token maximum over all batches, the
    `clip_frac` largest tokens set aside first (Section 5.2; 0 = none).  Every tensor operation and
    every step size is a libsq call (sq_token_absmax, sq_clipped_absmax); the host only moves the
    resulting scalars.  LN1 / LN2 outputs are never materialised in floating point: their static step
    is the largest of the per-batch steps the dynamic per-tensor quantiser found (no clipping there)."""
    dev = lin["qkv"].Wq.device
    M, hid, ffn = B * S, H * d, lin["fc1"].Wq.shape[0]
    row = 3 * hid
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_LN_QUANT, M, 0, hid), dev)
    e = lambda shape, dt: torch.empty(shape, dtype=dt, device=dev)
    x1q, xs = e((M, hid), torch.int8), e(1, torch.float32)
    qkv_f, qkv_q = e((M, row), act_dtype), e((M, row), torch.int8)
    scores, P = e((B * H, S, S), act_dtype), e((B * H, S, S), torch.int8)
    attn_f, attn_q = e((M, hid), act_dtype), e((M, hid), torch.int8)
    proj, h = e((M, hid), act_dtype), e((M, hid), act_dtype)
    x2q, xs2 = e((M, hid), torch.int8), e(1, torch.float32)
    f1 = e((M, ffn), act_dtype)
    names = ("d_ln1", "d_q", "d_k", "d_v", "d_attn", "d_ln2", "d_fc1")
    token_max = {k: [] for k in names}   # per tensor: the token maxima of every batch (device tensors)
    t32 = lambda v: torch.tensor(v, dtype=torch.float32)

    def step_of(token_absmax):
        """Eq. 1's step of the largest token maximum (libsq; one device scalar read back)."""
        _, st = sq.sq_clipped_absmax(token_absmax, 0)
        return float(st.item())

    for x in calib_batches:
        sq.sq_ln_quant(x, lin["qkv"].gamma_hat, lin["qkv"].beta_hat, eps, "per_tensor_dynamic", Xq=x1q, x_scale=xs,
                       workspace=ws)
        sq.sq_w8a8_gemm(x1q, lin["qkv"].Wq, xs, lin["qkv"].w_scale, ws, bias=lin["qkv"].bias, out=qkv_f)
        token_max["d_ln1"].append(xs.clone())  # the batch's own step (LN1's output is never materialised)
        tm = [sq.sq_token_absmax(qkv_f[:, i * hid:(i + 1) * hid]) for i in range(3)]
        for k, v in zip(("d_q", "d_k", "d_v"), tm):
            token_max[k].append(v)
        dq, dk, dv = (step_of(v) for v in tm)
        one = t32(1.0)
        r = torch.cat([torch.full((hid,), float(one / t32(v))) for v in (dq, dk, dv)]).to(torch.float32).to(dev)
        sq.sq_w8a8_gemm(x1q, lin["qkv"].Wq, xs, lin["qkv"].w_scale, ws, bias=lin["qkv"].bias, requant_mul=r, out=qkv_q)
        flat = qkv_q.view(-1)
        sq.sq_w8a8_bmm(flat, flat[hid:], B, H, S, S, d, (S * row, d, row), (S * row, d, row), False,
                       float(t32(dq) * t32(dk) / torch.sqrt(t32(float(d)))), scores, (H * S * S, S * S, S), ws)
        sq.sq_softmax_quant_p(scores, P)
        sq.sq_w8a8_bmm(P, flat[2 * hid:], B, H, S, d, S, (H * S * S, S * S, S), (S * row, d, row), True,
                       float(t32(dv) / t32(127.0)), attn_f, (S * hid, d, hid), ws)
        ta = sq.sq_token_absmax(attn_f)
        token_max["d_attn"].append(ta)
        d_attn = step_of(ta)
        ra = torch.tensor([float(one / t32(d_attn))], dtype=torch.float32, device=dev)
        sq.sq_w8a8_bmm(P, flat[2 * hid:], B, H, S, d, S, (H * S * S, S * S, S), (S * row, d, row), True,
                       float(t32(dv) / t32(127.0)), attn_q, (S * hid, d, hid), ws, requant_mul=ra)
        da = torch.tensor([d_attn], dtype=torch.float32, device=dev)
        sq.sq_w8a8_gemm(attn_q, lin["out_proj"].Wq, da, lin["out_proj"].w_scale, ws, bias=lin["out_proj"].bias, out=proj)
        sq.sq_residual_add(x, proj, out=h)
        sq.sq_ln_quant(h, lin["fc1"].gamma_hat, lin["fc1"].beta_hat, eps, "per_tensor_dynamic", Xq=x2q, x_scale=xs2,
                       workspace=ws)
        token_max["d_ln2"].append(xs2.clone())
        sq.sq_w8a8_gemm(x2q, lin["fc1"].Wq, xs2, lin["fc1"].w_scale, ws, bias=lin["fc1"].bias, relu=True, out=f1)
        token_max["d_fc1"].append(sq.sq_token_absmax(f1))
    out = {}
    for k in names:
        allmax = torch.cat(token_max[k])
        if k in ("d_ln1", "d_ln2"):  # per-batch steps: the static step is the largest of them (a selection, no arithmetic)
            largest, _ = sq.sq_clipped_absmax(allmax, 0)
            out[k] = float(largest.item())
        else:
            n_clip = int(clip_frac * allmax.numel() + 0.5)
            _, st = sq.sq_clipped_absmax(allmax, n_clip)
            out[k] = float(st.item())
    return out
