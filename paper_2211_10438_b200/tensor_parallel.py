"""Tensor-parallel sharding of the W8A8 linears (Section 5.3: the larger models are served with
FasterTransformer's tensor parallelism; the decoding-stage table has 8-GPU rows).

Megatron-style split of one decoder block over `world` ranks, one process per GPU:

  * QKV and FC1 are COLUMN-parallel: rank r keeps a slice of the output channels (whole heads for
    QKV) with their step sizes and bias.  No exchange: the output stays sharded along N.
  * out-proj and FC2 are ROW-parallel: rank r keeps a slice of the INPUT channels.  The weight is
    quantised BEFORE it is cut (Eq. 1's step of an output channel is taken over the whole row), so
    all ranks share one w_scale and every rank's GEMM leaves raw INT32 partial sums that add
    exactly: an INT32 sum-all-reduce followed by ONE dequantisation (sq_dequant_acc) gives, bit for
    bit, the result of the unsharded layer.
  * A row-parallel layer's input is spread over the ranks along its channels.  Per-token dynamic
    quantisation then needs the token maxima over ALL slices: sq_token_absmax of the local slice,
    a max-all-reduce of the [M] values, sq_quant_act_given_absmax.  Static steps need no exchange.

This file holds the partition logic and the two exchanges (torch.distributed; NCCL on GPUs, gloo
in the CPU tests).  All arithmetic is libsq calls; nothing here computes on tensors itself.
"""
from dataclasses import dataclass

import torch
import torch.distributed as dist


def shard_bounds(n: int, world: int, rank: int, multiple: int = 1):
    """[lo, hi) of rank's share of n items cut into `world` contiguous shares of whole `multiple`s
    (the first n/multiple mod world ranks get one unit more)."""
    if n % multiple != 0:
        raise ValueError("%d is not a multiple of %d" % (n, multiple))
    units = n // multiple
    base, extra = divmod(units, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return lo * multiple, hi * multiple


def qkv_row_index(hidden: int, head_dim: int, world: int, rank: int):
    """Rows of the fused QKV weight [3*hidden, K] (Q | K | V blocks) that rank keeps: its heads of each block,
    laid out again as Q_r | K_r | V_r so that the local output is a fused QKV buffer of the local heads."""
    lo, hi = shard_bounds(hidden, world, rank, head_dim)
    return torch.cat([torch.arange(b * hidden + lo, b * hidden + hi) for b in range(3)])


@dataclass
class ShardedLinear:
    Wq: torch.Tensor        # local INT8 weight
    w_scale: torch.Tensor   # [N_local] (column-parallel) or the full [N] (row-parallel)
    bias: torch.Tensor      # local slice (column-parallel) or the full bias, added once after the reduce
    parallel: str           # "column" | "row"
    lo: int                 # first output (column) / input (row) channel kept
    hi: int


def shard_column_parallel(Wq, w_scale, bias, world, rank, rows=None, multiple=16):
    """Split by OUTPUT channels.  Wq [N, K], w_scale [N] (or [1]), bias [N] or None.  `rows`: explicit row index
    (qkv_row_index) instead of a contiguous share."""
    N = Wq.shape[0]
    if rows is None:
        lo, hi = shard_bounds(N, world, rank, multiple)
        rows = torch.arange(lo, hi)
    else:
        lo, hi = int(rows[0]), int(rows[-1]) + 1
    rows = rows.to(Wq.device)
    ws = w_scale if w_scale.numel() == 1 else w_scale[rows].contiguous()
    return ShardedLinear(Wq[rows].contiguous(), ws, None if bias is None else bias[rows].contiguous(), "column", lo, hi)


def shard_row_parallel(Wq, w_scale, bias, world, rank, multiple=16, lo_hi=None):
    """Split by INPUT channels a weight that was quantised whole: every rank keeps the full w_scale and bias."""
    K = Wq.shape[1]
    lo, hi = lo_hi if lo_hi is not None else shard_bounds(K, world, rank, multiple)
    return ShardedLinear(Wq[:, lo:hi].contiguous(), w_scale, bias, "row", lo, hi)


# ------------------------------------------------------------------------------------------
# The two exchanges of a row-parallel layer (collectives only: no arithmetic of the method here)
# ------------------------------------------------------------------------------------------
def allreduce_token_absmax(local_absmax, group=None):
    """[M] fp32 token maxima of the local slice -> maxima over all ranks' slices, in place."""
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(local_absmax, op=dist.ReduceOp.MAX, group=group)
    return local_absmax


def allreduce_partial_sums(acc, group=None):
    """[M, N] INT32 partial sums of the local K slice -> exact sums over all ranks, in place."""
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(acc, op=dist.ReduceOp.SUM, group=group)
    return acc


class TensorParallelLinears:
    """The four W8A8 linears of one decoder block (per-token dynamic activations, per-channel weights, as
    pipeline.LinearBlock) on rank `rank` of `world`: LN1 -> QKV (column-parallel), attention output slice
    -> out-proj (row-parallel), LN2 -> FC1 (column-parallel, ReLU), FC1 slice -> FC2 (row-parallel).
    `lin` maps names to pipeline.PreparedLinear of the WHOLE layer (weights quantised unsharded); the
    constructor keeps this rank's slices.  Every rank returns the same, full FC2 output."""

    def __init__(self, lin, M, hidden, head_dim, act_dtype, world, rank, eps=1e-5, group=None):
        from . import binding as sq
        self.sq, self.M, self.dt, self.eps, self.group = sq, M, act_dtype, eps, group
        self.world, self.rank = world, rank
        self.src = lin
        qrows = qkv_row_index(hidden, head_dim, world, rank)
        self.qkv = shard_column_parallel(lin["qkv"].Wq, lin["qkv"].w_scale, lin["qkv"].bias, world, rank, rows=qrows)
        self.fc1 = shard_column_parallel(lin["fc1"].Wq, lin["fc1"].w_scale, lin["fc1"].bias, world, rank)
        # the row-parallel layers consume exactly what the column-parallel ones in front produce locally
        self.head_lo, self.head_hi = shard_bounds(hidden, world, rank, head_dim)
        self.out_proj = shard_row_parallel(lin["out_proj"].Wq, lin["out_proj"].w_scale, lin["out_proj"].bias, world, rank,
                                           lo_hi=(self.head_lo, self.head_hi))
        self.fc2 = shard_row_parallel(lin["fc2"].Wq, lin["fc2"].w_scale, lin["fc2"].bias, world, rank,
                                      lo_hi=(self.fc1.lo, self.fc1.hi))
        dev = lin["qkv"].Wq.device
        e = lambda shape, dt: torch.empty(shape, dtype=dt, device=dev)
        self.buf = {}
        for name, sh in (("qkv", self.qkv), ("out_proj", self.out_proj), ("fc1", self.fc1), ("fc2", self.fc2)):
            N, K = sh.Wq.shape
            self.buf[name] = dict(Xq=e((M, K), torch.int8), xs=e(M, torch.float32), amax=e(M, torch.float32),
                                  Y=e((M, N), act_dtype), acc=e((M, N), torch.int32) if sh.parallel == "row" else None)
        need = max(sq.workspace_bytes(sq.SQ_OP_GEMM, M, s.Wq.shape[0], s.Wq.shape[1])
                   for s in (self.qkv, self.out_proj, self.fc1, self.fc2))
        self.ws = sq.new_workspace(need, dev)

    def _row_parallel(self, name, x_slice, sh, out=None):
        """x_slice [M, K_local] (16-bit): token maxima agreed on across ranks -> codes -> local INT32 partial
        sums -> exact sum over ranks -> Eq. 2 once."""
        sq, b = self.sq, self.buf[name]
        sq.sq_token_absmax(x_slice, out=b["amax"])
        allreduce_token_absmax(b["amax"], self.group)
        sq.sq_quant_act_given_absmax(x_slice, b["amax"], Xq=b["Xq"], x_scale=b["xs"], workspace=self.ws)
        sq.sq_w8a8_gemm(b["Xq"], sh.Wq, None, None, self.ws, out=b["acc"])
        allreduce_partial_sums(b["acc"], self.group)
        return sq.sq_dequant_acc(b["acc"], b["xs"], sh.w_scale, bias=sh.bias, out=b["Y"] if out is None else out)

    def step(self, x_in, attn_out_slice, out=None):
        """x_in [M, hidden] (replicated); attn_out_slice [M, local heads * head_dim]: this rank's heads of the
        attention output.  Returns the FC2 output [M, hidden], identical on every rank."""
        sq, b = self.sq, self.buf
        q, f1 = self.src["qkv"], self.src["fc1"]
        sq.sq_ln_quant(x_in, q.gamma_hat, q.beta_hat, self.eps, "per_token", Xq=b["qkv"]["Xq"], x_scale=b["qkv"]["xs"],
                       workspace=self.ws)
        sq.sq_w8a8_gemm(b["qkv"]["Xq"], self.qkv.Wq, b["qkv"]["xs"], self.qkv.w_scale, self.ws, bias=self.qkv.bias,
                        out=b["qkv"]["Y"])
        h = self._row_parallel("out_proj", attn_out_slice, self.out_proj)
        sq.sq_ln_quant(h, f1.gamma_hat, f1.beta_hat, self.eps, "per_token", Xq=b["fc1"]["Xq"], x_scale=b["fc1"]["xs"],
                       workspace=self.ws)
        a = sq.sq_w8a8_gemm(b["fc1"]["Xq"], self.fc1.Wq, b["fc1"]["xs"], self.fc1.w_scale, self.ws, bias=self.fc1.bias,
                            relu=True, out=b["fc1"]["Y"])
        return self._row_parallel("fc2", a, self.fc2, out=out)

    def gemm_ops(self):
        """Integer ops of this rank's four GEMMs."""
        return sum(2 * self.M * s.Wq.shape[0] * s.Wq.shape[1] for s in (self.qkv, self.out_proj, self.fc1, self.fc2))

    def exchanged_bytes(self):
        """Bytes each rank contributes to the collectives of one step (two [M] fp32 + two [M, hidden] int32)."""
        return sum(4 * self.M + 4 * self.M * s.Wq.shape[0] for s in (self.out_proj, self.fc2))
