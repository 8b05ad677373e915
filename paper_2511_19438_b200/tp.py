"""Tensor-parallel sharding of a GPTQ layer (host-side slicing of the checkpoint arrays) and the two matmul forms.

Not in the paper, which runs one GPU (Section 4.1).  A layer is cut before the repack, so every rank repacks and
multiplies an ordinary, smaller layer:

* column-parallel (qkv, gate_up): rank r owns output columns [r N/R, (r+1) N/R); no exchange, the outputs are
  concatenated (or stay sharded for the next, row-parallel layer);
* row-parallel (o, down): rank r owns a slab of quantisation groups, multiplies its slice of x and the partial results are
  summed over the ranks.  Here the sum is one ``torch.distributed.all_reduce`` on fp32 copies of the partial outputs (two
  roundings to fp16: each partial, then the sum); the form with the reduction fused into the matmul's epilogue over peer
  memory is not built.

Only array slicing and the collective live here; the matmul is :func:`harness.gemm`.
"""
from __future__ import annotations

import numpy as np

from .workloads import QuantLinear


def shard_columns(L: QuantLinear, rank: int, world: int) -> QuantLinear:
    """Columns [rank N / world, (rank + 1) N / world) of the layer; N / world must be a multiple of 128."""
    assert 0 <= rank < world and L.N % world == 0 and (L.N // world) % 128 == 0
    n0, n1 = rank * L.N // world, (rank + 1) * L.N // world
    return QuantLinear(L.K, n1 - n0, L.group_size, np.ascontiguousarray(L.qweight[:, n0:n1]),
                       np.ascontiguousarray(L.qzeros[:, n0 // 8:n1 // 8]), np.ascontiguousarray(L.scales[:, n0:n1]),
                       L.g_idx, L.seed, L.zeros_minus_one)


def row_shard_rows(L: QuantLinear, rank: int, world: int) -> np.ndarray:
    """The rows of x (columns of the activation matrix) rank `rank` multiplies: the rows of its slab of groups, in
    checkpoint order.  Without act-order that is a contiguous range; with act-order it is wherever g_idx points into
    the slab."""
    G = L.K // L.group_size
    assert 0 <= rank < world and G % world == 0 and (L.K // world) % 128 == 0
    g0, g1 = rank * G // world, (rank + 1) * G // world
    if L.g_idx is None:
        return np.arange(g0 * L.group_size, g1 * L.group_size)
    return np.nonzero((L.g_idx >= g0) & (L.g_idx < g1))[0]


def shard_rows(L: QuantLinear, rank: int, world: int) -> QuantLinear:
    """The slab of quantisation groups [rank G / world, (rank + 1) G / world) as a layer of K / world rows.  Its row i
    is checkpoint row ``row_shard_rows(L, rank, world)[i]``; rows are packed eight to a word, so the slab's words are
    rebuilt from the nibbles when act-order scatters its rows."""
    rows = row_shard_rows(L, rank, world)
    G = L.K // L.group_size
    g0, g1 = rank * G // world, (rank + 1) * G // world
    if L.g_idx is None:
        qweight = np.ascontiguousarray(L.qweight[rows[0] // 8:(rows[-1] + 1) // 8])
        g_idx = None
    else:
        w = L.qweight.view(np.uint32)
        nib = (w[rows // 8, :] >> (4 * (rows % 8)).astype(np.uint32)[:, None]) & np.uint32(15)      # [K / world, N]
        nib = nib.reshape(len(rows) // 8, 8, L.N)
        packed = np.zeros((len(rows) // 8, L.N), dtype=np.uint32)
        for i in range(8):
            packed |= nib[:, i, :] << np.uint32(4 * i)
        qweight = packed.view(np.int32)
        g_idx = (L.g_idx[rows] - g0).astype(np.int32)
    return QuantLinear(len(rows), L.N, L.group_size, qweight, np.ascontiguousarray(L.qzeros[g0:g1]),
                       np.ascontiguousarray(L.scales[g0:g1]), g_idx, L.seed, L.zeros_minus_one)


def all_reduce_partials(y_partial, group=None):
    """Sum of the ranks' partial outputs (a torch tensor on any device the process group supports): all-reduce in fp32,
    one rounding back to the input dtype."""
    import torch
    import torch.distributed as dist
    acc = y_partial.to(torch.float32)
    dist.all_reduce(acc, op=dist.ReduceOp.SUM, group=group)
    return acc.to(y_partial.dtype)


def all_gather_columns(y_shard, group=None):
    """Concatenates the ranks' column shards of a column-parallel layer along the last dimension."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    parts = [torch.empty_like(y_shard) for _ in range(world)]
    dist.all_gather(parts, y_shard.contiguous(), group=group)
    return torch.cat(parts, dim=-1)
