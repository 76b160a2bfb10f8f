"""Single-kernel workloads on synthetic data: a few calls of one libsq entry point at a named shape.

    python -m paper_2211_10438_b200.workloads <name> [--calls N] [shape options]

Meant for profilers and quick timing: every workload allocates its operands with a seeded
generator, calls the entry point `--calls` times on the current CUDA device, synchronises, checks
the device status word and prints the mean time per call (CUDA events, after one untimed call).
Names: decode_gemm, attention, kv_attention, ln_quant, quant_act.
"""
import argparse

import torch

from . import binding as sq


def _time(fn, calls):
    fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(calls):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / calls * 1e3


def _gen(seed=0x5EED):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return g


def decode_gemm(args):
    """Decode-shaped W8A8 GEMM: M tokens against an [N, K] INT8 weight (default: GPT-3 FC1)."""
    g = _gen()
    N, K = args.N, args.K
    Wq = torch.randint(-127, 128, (N, K), dtype=torch.int8, device="cuda", generator=g)
    w_scale = torch.rand(N, device="cuda", generator=g) * 1e-3
    ws = sq.new_workspace(max(sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K) for M in args.M))
    for M in args.M:
        X = torch.randint(-127, 128, (M, K), dtype=torch.int8, device="cuda", generator=g)
        xs = torch.rand(M, device="cuda", generator=g)
        Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        us = _time(lambda: sq.sq_w8a8_gemm(X, Wq, xs, w_scale, ws, out=Y), args.calls)
        print("decode_gemm M=%d N=%d K=%d: %.1f us, %.0f GB/s of weights" % (M, N, K, us, N * K / us / 1e3))
    return ws


def attention(args):
    """Fused causal INT8 attention over a QKV code buffer (default: OPT-30B heads, S = 512, batch 4)."""
    g = _gen()
    B, H, S, d = args.B, args.H, args.S, 128
    qkv = torch.randint(-100, 101, (B * S, 3 * H * d), dtype=torch.int8, device="cuda", generator=g)
    out = torch.empty((B * S, H * d), dtype=torch.int8, device="cuda")
    r = torch.tensor([100.0], device="cuda")
    ws = sq.new_workspace(4096)
    us = _time(lambda: sq.sq_w8a8_attention(qkv, B, H, S, d, 0.0009, 0.0001, r, out, ws), args.calls)
    print("attention B=%d H=%d S=%d: %.1f us" % (B, H, S, us))
    return ws


def kv_attention(args):
    """Generation-stage attention over an INT8 KV cache (default: GPT-3 heads, batch 16, context
    lengths uniform in [L/2, L], L = 2048); the kernel appends the newest token itself."""
    g = _gen()
    B, H, L, d = args.B, args.H, args.L, 128
    kc = torch.randint(-100, 101, (B, H, L, d), dtype=torch.int8, device="cuda", generator=g)
    vc = torch.randint(-100, 101, (B, H, L // 4, d, 4), dtype=torch.int8, device="cuda", generator=g)
    qkv = torch.randint(-100, 101, (B, 3 * H * d), dtype=torch.int8, device="cuda", generator=g)
    lens = torch.randint(L // 2, L + 1, (B,), dtype=torch.int32, device="cuda", generator=g)
    out = torch.empty((B, H * d), dtype=torch.int8, device="cuda")
    r = torch.tensor([1000.0], device="cuda")
    ws = sq.new_workspace(256)
    us = _time(lambda: sq.sq_w8a8_decode_attention(qkv, kc, vc, lens, B, H, d, L, L, 0.0009, 0.01 / 127, ws, requant_mul=r,
                                                   out=out, k_new=qkv[:, H * d:], v_new=qkv[:, 2 * H * d:]), args.calls)
    byts = 2 * H * d * int(lens.sum().item())
    print("kv_attention B=%d H=%d L<=%d: %.1f us, %.0f GB/s of cache (%d bytes)" % (B, H, L, us, byts / us / 1e3, byts))
    return ws


def _rows(args, ln):
    g = _gen()
    M, C = args.rows, args.C
    dt = torch.float16 if args.dtype == "f16" else torch.bfloat16
    x = torch.randn((M, C), device="cuda", dtype=dt, generator=g)
    x[:, ::200] *= 100
    Xq = torch.empty((M, C), dtype=torch.int8, device="cuda")
    xs = torch.empty(M, dtype=torch.float32, device="cuda")
    gamma = torch.ones(C, dtype=dt, device="cuda")
    beta = torch.zeros(C, dtype=dt, device="cuda")
    ws = sq.new_workspace(sq.workspace_bytes(sq.SQ_OP_LN_QUANT, M, 0, C))
    if ln:
        us = _time(lambda: sq.sq_ln_quant(x, gamma, beta, 1e-5, "per_token", Xq=Xq, x_scale=xs, workspace=ws), args.calls)
    else:
        us = _time(lambda: sq.sq_quant_act(x, "per_token", Xq=Xq, x_scale=xs, workspace=ws), args.calls)
    print("%s %dx%d: %.1f us, %.0f GB/s (3 B/element)" % ("ln_quant" if ln else "quant_act", M, C, us, 3 * M * C / us / 1e3))
    return ws


def ln_quant(args):
    """Fused LayerNorm + per-token quantise of a bf16 / fp16 [rows, C] tensor (default 8192 x 20480)."""
    return _rows(args, True)


def quant_act(args):
    """Per-token quantise of a bf16 / fp16 [rows, C] tensor (default 8192 x 20480)."""
    return _rows(args, False)


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("name", choices=["decode_gemm", "attention", "kv_attention", "ln_quant", "quant_act"])
    ap.add_argument("--calls", type=int, default=20)
    ap.add_argument("--M", type=lambda s: [int(v) for v in s.split(",")], default=[1, 16], help="decode_gemm: token counts")
    ap.add_argument("--N", type=int, default=49152)
    ap.add_argument("--K", type=int, default=12288)
    ap.add_argument("--B", type=int, default=None, help="batch (attention: 4, kv_attention: 16)")
    ap.add_argument("--H", type=int, default=None, help="heads (attention: 56, kv_attention: 96)")
    ap.add_argument("--S", type=int, default=512)
    ap.add_argument("--L", type=int, default=2048)
    ap.add_argument("--rows", type=int, default=8192)
    ap.add_argument("--C", type=int, default=20480)
    ap.add_argument("--dtype", choices=["bf16", "f16"], default="bf16", help="ln_quant / quant_act: activation type")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: the library has no CPU fallback")
    if args.B is None:
        args.B = 4 if args.name == "attention" else 16
    if args.H is None:
        args.H = 56 if args.name == "attention" else 96
    sq.lib()
    ws = globals()[args.name](args)
    status = sq.device_status(ws)
    if status != 0:
        raise SystemExit("device status word = %d" % status)


if __name__ == "__main__":
    main()
