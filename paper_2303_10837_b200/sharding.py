"""Partition of one round over several GPUs (one process per GPU).

Every ciphertext index is an independent unit through all steps of the path
(pack, encode, encrypt, weighted sum with rescale, decrypt, decode), and so is
every entry of the plaintext remainder: rank r of a job of `world` ranks takes
the contiguous range [count * r / world, count * (r + 1) / world) of each, with
context, keys and mask replicated.  No step exchanges data; only when one
place needs the whole decoded model are the ranks' pieces gathered.

This module is host-side index arithmetic plus that gather; it launches
nothing and imports neither the CUDA library nor the oracle, so the same
functions serve the benchmark (NCCL, CUDA tensors) and its CPU tests (gloo).
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
