"""Tensor-parallel sharding of the W8A8 linears, host-side logic on two gloo ranks (CPU): the partition
(which rows / columns a rank keeps), the two exchanges of a row-parallel layer, and the claims the
design rests on.  The arithmetic of each rank is done by the oracle here (no GPU in this test):
  * sum over ranks of the K-sliced INT32 partial sums == the unsharded oracle GEMM, exactly;
  * a K-sharded activation needs the max-all-reduce of the token maxima: with it every rank's codes
    are the slices of the unsharded quantiser's codes, without it they are not;
  * column-parallel outputs, laid side by side, are the unsharded output;
  * Eq. 2 applied once to the reduced sums is the unsharded layer's output bit for bit."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2211_10438_b200 import synth
    from paper_2211_10438_b200 import tensor_parallel as tp

    M, hidden, head_dim, ffn = 12, 256, 64, 768
    ch = synth.outlier_channels(6, ffn, count=6)
    a = synth.activations(6, 1, M, ffn, "bf16", ch, np.full(6, 40.0))          # FC1 output: FC2's input, sharded over ranks
    W2 = synth.weights(6, 2, hidden, ffn, "bf16")
    b2 = synth.bias(6, 3, hidden, "bf16")
    Wq2, ws2 = oracle.quant_weight(W2, None, "per_channel")                       # quantised WHOLE, then cut
    res = {}

    # ---- row-parallel FC2 ----
    sh = tp.shard_row_parallel(torch.from_numpy(Wq2), torch.from_numpy(ws2), torch.from_numpy(b2), world, rank)
    lo, hi = sh.lo, sh.hi
    res["k_bounds"] = (lo, hi)
    a_loc = np.ascontiguousarray(a[:, lo:hi])
    amax = torch.from_numpy(oracle.row_absmax(a_loc))
    local_amax = amax.clone()
    tp.allreduce_token_absmax(amax)                                               # gloo MAX
    res["amax_is_global"] = bool(np.array_equal(amax.numpy(), oracle.row_absmax(a)))
    delta = np.array([oracle.step_size(float(v)) for v in amax.numpy()], np.float32)
    q_loc = oracle.quantize(a_loc, delta, True)
    q_full, d_full = oracle.quant_act(a, "per_token")
    res["codes_are_slices"] = bool(np.array_equal(q_loc, q_full[:, lo:hi]) and np.array_equal(delta, d_full))
    d_local_only = np.array([oracle.step_size(float(v)) for v in local_amax.numpy()], np.float32)
    res["local_maxima_would_differ"] = bool(not np.array_equal(oracle.quantize(a_loc, d_local_only, True), q_full[:, lo:hi]))
    acc = torch.from_numpy(oracle.gemm_i32(q_loc, np.ascontiguousarray(sh.Wq.numpy())))
    part = acc.clone()
    tp.allreduce_partial_sums(acc)                                                # gloo INT32 SUM
    acc_full = oracle.gemm_i32(q_full, Wq2)
    res["partial_sums_add_exactly"] = bool(np.array_equal(acc.numpy(), acc_full))
    res["partial_is_not_the_sum"] = bool(not np.array_equal(part.numpy(), acc_full))
    y = oracle.round_to(oracle.dequant(acc.numpy(), delta, sh.w_scale.numpy(), sh.bias.numpy()), "bf16")
    _, y_full = oracle.w8a8_linear(q_full, d_full, Wq2, ws2, bias=b2, out_dtype="bf16")
    res["output_bit_exact"] = bool(np.array_equal(y, y_full))

    # ---- column-parallel QKV (whole heads per rank, Q_r | K_r | V_r) and FC1 ----
    x = synth.activations(6, 4, M, hidden, "bf16", [3], [30.0])
    Wqkv = synth.weights(6, 5, 3 * hidden, hidden, "bf16")
    bq = synth.bias(6, 6, 3 * hidden, "bf16")
    Wq1, ws1 = oracle.quant_weight(Wqkv, None, "per_channel")
    rows = tp.qkv_row_index(hidden, head_dim, world, rank)
    shq = tp.shard_column_parallel(torch.from_numpy(Wq1), torch.from_numpy(ws1), torch.from_numpy(bq), world, rank, rows=rows)
    xq, xs = oracle.quant_act(x, "per_token")
    _, y_loc = oracle.w8a8_linear(xq, xs, shq.Wq.numpy(), shq.w_scale.numpy(), bias=shq.bias.numpy(), out_dtype="bf16")
    _, y_all = oracle.w8a8_linear(xq, xs, Wq1, ws1, bias=bq, out_dtype="bf16")
    res["qkv_slice_matches"] = bool(np.array_equal(y_loc, y_all[:, rows.numpy()]))
    hl, hh = tp.shard_bounds(hidden, world, rank, head_dim)
    res["qkv_rows_are_whole_heads"] = bool(len(rows) == 3 * (hh - hl) and (hh - hl) % head_dim == 0
                                           and np.array_equal(rows.numpy()[:hh - hl], np.arange(hl, hh)))
    # every column is owned by exactly one rank: gather the index sets
    owned = torch.zeros(3 * hidden, dtype=torch.int32)
    owned[rows] = 1
    dist.all_reduce(owned)
    res["qkv_partition_is_exact"] = bool((owned == 1).all())
    kown = torch.zeros(ffn, dtype=torch.int32)
    kown[lo:hi] = 1
    dist.all_reduce(kown)
    res["k_partition_is_exact"] = bool((kown == 1).all())
    dist.barrier()
    out[rank] = res
    dist.destroy_process_group()


def test_row_and_column_parallel_on_two_ranks():
    world, port = 2, 29621
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        for k, v in res[rank].items():
            if k != "k_bounds":
                assert v is True, "rank %d: %s" % (rank, k)
    assert res[0]["k_bounds"] == (0, 384) and res[1]["k_bounds"] == (384, 768)


def test_shard_bounds_cover_everything_once():
    sys.path.insert(0, ROOT)
    from paper_2211_10438_b200 import tensor_parallel as tp
    for n, world, mult in ((7168, 8, 128), (28672, 8, 16), (5120, 3, 128), (20480, 7, 16), (128, 4, 128)):
        edges = [tp.shard_bounds(n, world, r, mult) for r in range(world)]
        assert edges[0][0] == 0 and edges[-1][1] == n
        for (a, b), (c, d) in zip(edges, edges[1:]):
            assert b == c and (b - a) % mult == 0 and b >= a
        sizes = [b - a for a, b in edges]
        assert max(sizes) - min(sizes) <= mult  # balanced to within one unit
