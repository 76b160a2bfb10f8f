"""Single-kernel workloads on synthetic data: a few calls of one libsq entry point at a named shape.

    python -m paper_2211_10438_b200.workloads <name> [--calls N] [shape options]

Meant for profilers and quick timing: every workload allocates its operands with a seeded
generator, calls the entry point `--calls` times on the current CUDA device, synchronises, checks
the device status word and prints the mean time per call (CUDA events, after one untimed call).
Names: gemm, decode_gemm, generation_block, attention, kv_attention, ln_quant, quant_act.
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


def _codes(shape, values, g):
    """INT8 operand codes of a given value class: what the tensor cores draw depends on the data."""
    if values == "zeros":
        return torch.zeros(shape, dtype=torch.int8, device="cuda")
    if values == "ones":
        return torch.ones(shape, dtype=torch.int8, device="cuda")
    if values == "tri":  # small codes, triangular around zero: what a smoothed LLM activation quantises to, mostly
        a = torch.randint(-8, 9, shape, dtype=torch.int8, device="cuda", generator=g)
        return a + torch.randint(-8, 9, shape, dtype=torch.int8, device="cuda", generator=g)
    return torch.randint(-127, 128, shape, dtype=torch.int8, device="cuda", generator=g)  # "full"


def gemm(args):
    """Prefill-shaped W8A8 GEMM (default: the OPT-13B FC1 of config 2), bf16 output, per-token x
    per-channel step sizes.  --values picks the operand value class (the power the tensor cores draw,
    and with it the sustained clock, depends on the data), --no-split withholds the scratch the
    K split of a partly filled last wave needs, --int-mm times torch._int_mm (cuBLASLt, INT32
    output, no epilogue) on the same operands for context."""
    g = _gen()
    for M in args.M:
        N, K = args.N, args.K
        X = _codes((M, K), args.values, g)
        Wq = _codes((N, K), args.values, g)
        xs = torch.rand(M, device="cuda", generator=g) * 0.1
        wsc = torch.rand(N, device="cuda", generator=g) * 1e-3
        Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        ws = sq.new_workspace(256 if args.no_split else sq.workspace_bytes(sq.SQ_OP_GEMM, M, N, K))
        us = _time(lambda: sq.sq_w8a8_gemm(X, Wq, xs, wsc, ws, out=Y), args.calls)
        line = "gemm M=%d N=%d K=%d values=%s%s: %.1f us, %.0f TOPS" % (
            M, N, K, args.values, " no-split" if args.no_split else "", us, 2.0 * M * N * K / us / 1e6)
        if args.int_mm:
            Wt = Wq.t()
            us2 = _time(lambda: torch._int_mm(X, Wt), args.calls)
            line += "; torch._int_mm %.1f us, %.0f TOPS" % (us2, 2.0 * M * N * K / us2 / 1e6)
        print(line)
        if sq.device_status(ws) != 0:
            raise SystemExit("device status word = %d" % sq.device_status(ws))
        if args.trace:
            _print_gemm_trace()
        del X, Wq, Y
    return sq.new_workspace(256)


def _print_gemm_trace():
    """The MMA warps' cycle counts of the last launch (needs --lib .../libsq_trace.so)."""
    import ctypes

    import numpy as np
    tiles = 16
    buf = (ctypes.c_ulonglong * (160 * (tiles + 1) * 4))()
    fn = getattr(sq.lib(), "sq_debug_gemm_trace", None)
    if fn is None:
        raise SystemExit("--trace needs the trace build: python -m paper_2211_10438_b200.build --trace, then --lib .../libsq_trace.so")
    if fn(buf) != 0:
        raise SystemExit("sq_debug_gemm_trace failed")
    t = np.frombuffer(buf, dtype=np.uint64).reshape(160, tiles + 1, 4).astype(np.float64)
    t = t[t[:, tiles, 1] > 0]                       # CTAs whose MMA warp ran (the even CTA of every pair)
    n_tiles = (t[:, :tiles, 3] > 0).sum(axis=1)
    later = np.concatenate([t[i, 1:int(n_tiles[i]), :] for i in range(len(t)) if n_tiles[i] > 1] or [np.zeros((0, 4))])
    span_cyc, span_ns, epi = t[:, tiles, 0], t[:, tiles, 1], t[:, tiles, 2]
    print("  MMA warp, %d CTA pairs, %d-%d tiles each; per tile after the first (mean, SM cycles): index arithmetic %.0f, "
          "wait for the accumulator slot %.0f, K loop %.0f = %.1f per K block of 4 MMAs (128 cycles each at full rate)"
          % (len(t), n_tiles.min(), n_tiles.max(), later[:, 0].mean(), later[:, 1].mean(), later[:, 2].mean(),
             (later[:, 2] / later[:, 3]).mean()))
    print("  first MMA -> last commit: median %.1f us, %.0f cycles: SM clock during the launch %.0f MHz; "
          "epilogue warp 0 drains the fourth tile's slot in %.0f cycles"
          % (np.median(span_ns) / 1e3, np.median(span_cyc), np.median(span_cyc / span_ns * 1e3), np.median(epi[epi > 0]) if (epi > 0).any() else 0))


def decode_gemm(args):
    """Decode-shaped W8A8 GEMM: M tokens against an [N, K] INT8 weight (default: GPT-3 FC1).
    --fused: bf16 activations in, per-token quantisation in the kernel's prologue."""
    g = _gen()
    N, K = args.N, args.K
    Wq = torch.randint(-127, 128, (N, K), dtype=torch.int8, device="cuda", generator=g)
    w_scale = torch.rand(N, device="cuda", generator=g) * 1e-3
    ws = sq.new_workspace(max(sq.workspace_bytes(sq.SQ_OP_GEMM_FUSED_QUANT, M, N, K) for M in args.M))
    for M in args.M:
        Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        if args.fused:
            x = torch.randn((M, K), dtype=torch.bfloat16, device="cuda", generator=g)
            us = _time(lambda: sq.sq_w8a8_gemm_fused_quant(x, Wq, w_scale, ws, "per_token", out=Y), args.calls)
        else:
            X = torch.randint(-127, 128, (M, K), dtype=torch.int8, device="cuda", generator=g)
            xs = torch.rand(M, device="cuda", generator=g)
            us = _time(lambda: sq.sq_w8a8_gemm(X, Wq, xs, w_scale, ws, out=Y), args.calls)
        print("decode_gemm%s M=%d N=%d K=%d: %.1f us, %.0f GB/s of weights" % (
            " (quantiser in the prologue)" if args.fused else "", M, N, K, us, N * K / us / 1e3))
    return ws


def generation_block(args):
    """One generation-stage step of the OPT-30B-shaped static W8A8 block (hidden 7168, 56 heads,
    FFN 28672; batch --B, context --S cached positions): random INT8 weights and cache, fixed
    static steps.  Seven launches per step; --fused: five (the LayerNorm+quantise steps run in the
    prologues of the GEMMs that consume them)."""
    from . import pipeline as pl
    g = _gen()
    H, d, hid, ffn, B = 56, 128, 7168, 28672, args.B
    dt = torch.float16
    lin = {}
    for name, (N, K) in (("qkv", (3 * hid, hid)), ("out_proj", (hid, hid)), ("fc1", (ffn, hid)), ("fc2", (hid, ffn))):
        lin[name] = pl.PreparedLinear(name, torch.randint(-127, 128, (N, K), dtype=torch.int8, device="cuda", generator=g),
                                      torch.rand(N, device="cuda", generator=g) * 1e-3,
                                      (torch.randn(N, device="cuda", generator=g) * 0.01).to(dt), name == "fc1")
    for name in ("qkv", "fc1"):
        lin[name].gamma_hat = (1 + 0.1 * torch.randn(hid, device="cuda", generator=g)).to(dt)
        lin[name].beta_hat = (0.1 * torch.randn(hid, device="cuda", generator=g)).to(dt)
    steps = dict(d_ln1=0.05, d_q=0.02, d_k=0.02, d_v=0.02, d_attn=0.01, d_ln2=0.05, d_fc1=0.02)
    L_max = 2048
    blk = pl.DecoderBlockDecode(lin, steps, B, H, d, L_max, dt, fused=args.fused)
    blk.k_cache.random_(-100, 100, generator=g)
    blk.v_cache.random_(-100, 100, generator=g)
    blk.ctx.fill_(args.S)
    blk.lens.fill_(args.S + 1)
    x = torch.randn((B, hid), device="cuda", dtype=dt, generator=g)
    us = _time(lambda: blk.step(x, max_len=args.S + 1, advance=False), args.calls)
    byts = blk.bytes_per_step(args.S * B)
    print("generation_block B=%d ctx=%d, %d launches per step: %.1f us per step (stream, no graph), %.0f GB/s of weights + cache"
          % (B, args.S, blk.launches_per_step, us, byts / us / 1e3))
    return blk.ws


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
    ap.add_argument("name", choices=["gemm", "decode_gemm", "generation_block", "attention", "kv_attention", "ln_quant",
                                     "quant_act"])
    ap.add_argument("--calls", type=int, default=20)
    ap.add_argument("--lib", default=None, help="path of another build of the library (libsq_issue_only.so, libsq_trace.so)")
    ap.add_argument("--M", type=lambda s: [int(v) for v in s.split(",")], default=None,
                    help="token counts (decode_gemm: 1,16; gemm: 2048)")
    ap.add_argument("--N", type=int, default=None, help="output channels (decode_gemm: 49152; gemm: 20480)")
    ap.add_argument("--K", type=int, default=None, help="input channels (decode_gemm: 12288; gemm: 5120)")
    ap.add_argument("--values", choices=["full", "tri", "ones", "zeros"], default="full", help="gemm: operand value class")
    ap.add_argument("--no-split", action="store_true", help="gemm: no scratch for the K split of the last wave")
    ap.add_argument("--int-mm", action="store_true", help="gemm: also time torch._int_mm (cuBLASLt) for context")
    ap.add_argument("--trace", action="store_true", help="gemm: print the MMA warps' cycle counts (trace build given with --lib)")
    ap.add_argument("--fused", action="store_true", help="decode_gemm / generation_block: quantiser inside the GEMM")
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
    if args.M is None:
        args.M = [2048] if args.name == "gemm" else [1, 16]
    if args.N is None:
        args.N = 20480 if args.name == "gemm" else 49152
    if args.K is None:
        args.K = 5120 if args.name == "gemm" else 12288
    if args.B is None:
        args.B = 4 if args.name == "attention" else 16
    if args.H is None:
        args.H = 56 if args.name == "attention" else 96
    if args.lib:
        sq.LIB_PATH = args.lib
    sq.lib()
    ws = globals()[args.name](args)
    status = sq.device_status(ws)
    if status != 0:
        raise SystemExit("device status word = %d" % status)


if __name__ == "__main__":
    main()
