"""Partition of one round over several GPUs (one process per GPU).

Every ciphertext index is an independent unit through all steps of the path
(pack, encode, encrypt, weighted sum with rescale, decrypt, decode), and so is
every entry of the plaintext remainder: rank r of a job of `world` ranks takes
the contiguous range [count * r / world, count * (r + 1) / world) of each, with
context, keys and mask replicated.  No step exchanges data; only when one
place needs the whole decoded model are the ranks' pieces gathered.

A second layout serves a server whose clients' ciphertexts arrive on different
GPUs: rank r holds the ciphertexts of the clients [C * r / world, C * (r + 1) /
world), forms their weighted sum on all limbs without the rescale, and the
sum over clients then crosses the ranks once -- `scatter_sum`, a
reduce-scatter of 64-bit words after which rank r owns the ciphertext
indices of its shard_range and rescales and decrypts those.  That is the one
layout of the path with a real exchange step.

This module is host-side index arithmetic plus those two collectives; it
launches nothing else and imports neither the CUDA library nor the oracle, so
the same functions serve the benchmark (NCCL, CUDA tensors) and its CPU tests
(gloo).
"""
from __future__ import annotations

from typing import List, Tuple

import torch


def shard_range(count: int, rank: int, world: int) -> Tuple[int, int]:
    """[begin, end) of rank `rank`: contiguous, disjoint, covering [0, count), sizes differing by at most one."""
    if world < 1 or not 0 <= rank < world or count < 0:
        raise ValueError("shard_range(%d, %d, %d)" % (count, rank, world))
    return count * rank // world, count * (rank + 1) // world


def slot_range(T: int, n: int, k: int, rank: int, world: int) -> Tuple[int, int, int, int]:
    """(t_begin, t_end, slot_begin, slot_end) of a rank: its ciphertext indices and the packed
    slots they hold; slot_end stops at k, the number of encrypted parameters (ragged last ciphertext)."""
    tb, te = shard_range(T, rank, world)
    return tb, te, min(k, tb * n), min(k, te * n)


def slot_edges(T: int, n: int, k: int, world: int) -> List[Tuple[int, int]]:
    """The packed-slot range of every rank (cut at ciphertext boundaries)."""
    return [slot_range(T, n, k, r, world)[2:] for r in range(world)]


def even_edges(count: int, world: int) -> List[Tuple[int, int]]:
    return [shard_range(count, r, world) for r in range(world)]


def gather_pieces(local: torch.Tensor, edges: List[Tuple[int, int]], rank: int) -> torch.Tensor:
    """All ranks' pieces of a vector, in order, on every rank.  edges[r] = [begin, end) of rank r's
    piece (contiguous, covering the vector).  One all_gather of equal-size padded buffers: the
    only collective of the partitioned path, needed only where one place wants the whole model."""
    world = len(edges)
    b, e = edges[rank]
    if local.numel() != e - b:
        raise ValueError("piece of rank %d has %d entries, %d expected" % (rank, local.numel(), e - b))
    if world == 1:
        return local
    import torch.distributed as dist
    width = max(re - rb for rb, re in edges)
    mine = torch.zeros(width, dtype=local.dtype, device=local.device)
    mine[: e - b] = local
    parts: List[torch.Tensor] = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine)
    out = torch.empty(edges[-1][1], dtype=local.dtype, device=local.device)
    for r, (rb, re) in enumerate(edges):
        out[rb:re] = parts[r][: re - rb]
    return out


def scatter_sum(partial: torch.Tensor, rank: int, world: int) -> torch.Tensor:
    """Sum over all ranks of `partial` (int64 [T][...]: the weighted sums of each rank's clients,
    canonical residues), of which rank r keeps the rows of shard_range(T, r, world).  The words
    are added as 64-bit integers with wrap-around, i.e. as unsigned integers: exact while
    world * q < 2^64 (he_rescale_partial_sum checks that bound).  One reduce-scatter under NCCL
    (rows padded to equal shares when T is not a multiple of world); gloo has no reduce-scatter,
    so there the sum is an all-reduce and the rank slices its rows."""
    T = partial.shape[0]
    b, e = shard_range(T, rank, world)
    if world == 1:
        return partial
    import torch.distributed as dist
    if dist.get_backend() != "nccl":
        total = partial.clone()
        dist.all_reduce(total, op=dist.ReduceOp.SUM)
        return total[b:e].contiguous()
    width = -(-T // world)
    row = partial[0].numel() if T else 0
    flat = partial.reshape(T, row)
    if T == width * world:
        send = flat
    else:                                            # unequal shares: every rank's rows at r * width, zero padding
        send = torch.zeros((world * width, row), dtype=partial.dtype, device=partial.device)
        for r in range(world):
            rb, re = shard_range(T, r, world)
            send[r * width: r * width + (re - rb)] = flat[rb:re]
    recv = torch.empty((width, row), dtype=partial.dtype, device=partial.device)
    dist.reduce_scatter_tensor(recv, send, op=dist.ReduceOp.SUM)
    return recv[: e - b].reshape((e - b,) + tuple(partial.shape[1:]))
