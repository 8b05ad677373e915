"""Tensor-parallel sharding (host-side slicing and the collectives around the matmul), without a GPU: the oracle stands
in for the local matmul, and two CPU processes with the gloo backend run the row-parallel sum and the column-parallel
concatenation."""
import os
import socket
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

import oracle
from paper_2511_19438_b200 import tp
from paper_2511_19438_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def make_case(act):
    K, N, M = 1024, 512, 3
    L = wl.make_linear(K, N, seed=wl.seed_for("tp", act), act_order=act)
    x = wl.make_x(M, K, wl.seed_for("tp-x", act))
    return L, x, oracle.gemm_f64(x, L.qweight, L.qzeros, L.scales, L.g_idx, 128)


@pytest.mark.parametrize("act", [False, True])
@pytest.mark.parametrize("world", [2, 4])
def test_shards_reproduce_the_layer(act, world):
    L, x, want = make_case(act)
    w_full = oracle.dequant_f32(L.qweight, L.qzeros, L.scales, L.g_idx, 128)
    # column-parallel: each shard is a column slab of the layer, bit for bit
    cols = []
    for r in range(world):
        S = tp.shard_columns(L, r, world)
        n0 = r * L.N // world
        assert np.array_equal(oracle.dequant_f32(S.qweight, S.qzeros, S.scales, S.g_idx, 128), w_full[:, n0:n0 + S.N])
        cols.append(oracle.gemm_f64(x, S.qweight, S.qzeros, S.scales, S.g_idx, 128))
    assert np.array_equal(np.concatenate(cols, axis=1), want)
    # row-parallel: the shards' rows partition the layer's rows, each shard dequantises to its rows of the layer,
    # and the partial products add up
    seen = np.zeros(L.K, dtype=int)
    acc = np.zeros_like(want)
    for r in range(world):
        rows = tp.row_shard_rows(L, r, world)
        seen[rows] += 1
        S = tp.shard_rows(L, r, world)
        assert S.K == L.K // world and (S.g_idx is None) == (L.g_idx is None)
        assert np.array_equal(oracle.dequant_f32(S.qweight, S.qzeros, S.scales, S.g_idx, 128), w_full[rows])
        acc += oracle.gemm_f64(np.ascontiguousarray(x[:, rows]), S.qweight, S.qzeros, S.scales, S.g_idx, 128)
    assert np.all(seen == 1)
    assert np.allclose(acc, want, rtol=1e-12, atol=1e-10)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    L, x, want = make_case(True)
    # row-parallel: this rank's partial product as the fp16 tensor its matmul would return
    S = tp.shard_rows(L, rank, world)
    rows = tp.row_shard_rows(L, rank, world)
    part = oracle.gemm_f64(np.ascontiguousarray(x[:, rows]), S.qweight, S.qzeros, S.scales, S.g_idx, 128)
    y = tp.all_reduce_partials(torch.from_numpy(part.astype(np.float16)))
    # column-parallel: this rank's column shard
    C = tp.shard_columns(L, rank, world)
    ycol = torch.from_numpy(oracle.gemm_f64(x, C.qweight, C.qzeros, C.scales, C.g_idx, 128).astype(np.float16))
    ycat = tp.all_gather_columns(ycol)
    dist.barrier()
    out.put((rank, y.numpy().astype(np.float64), ycat.numpy().astype(np.float64)))
    dist.destroy_process_group()


def test_two_ranks_sum_row_shards_and_gather_column_shards():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get() for _ in procs]
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    _L, _x, want = make_case(True)
    for rank, y, ycat in results:
        # two roundings to fp16 (each partial, then the sum)
        assert np.all(np.abs(y - want) <= 3 * 2.0 ** -11 * np.abs(want) + 2.0 ** -9)
        assert np.array_equal(ycat, want.astype(np.float16).astype(np.float64))
    assert np.array_equal(results[0][1], results[1][1])
