"""Column-parallel (N-sharded) use of the W4A16 GEMM on several GPUs, one process per GPU.

The product C[M, N] = A[M, K] . Dequant(W)[K, N] has no exchange step when W is cut along N: every rank
holds the packed weights of its own columns (whole 64-column tiles), computes its slice of C with the same
``w4a16_gemm`` call, and nothing crosses NVLink unless the consumer wants the whole C, in which case one
all-gather of M x N 16-bit values (NCCL, or gloo on CPU) assembles it.  This module is plumbing only:
index arithmetic, slicing of the raw arrays and the optional gather.
"""
from __future__ import annotations

from typing import List, Tuple

TILE = 64   # columns per packed tile: shard boundaries are multiples of it


def column_shard(N: int, world: int, rank: int) -> Tuple[int, int]:
    """Columns [n0, n1) of rank ``rank``: whole tiles, sizes differ by at most one tile, the first
    ``tiles % world`` ranks get the extra one."""
    if N <= 0 or N % TILE or world < 1 or not 0 <= rank < world:
        raise ValueError("N must be a positive multiple of %d and 0 <= rank < world" % TILE)
    tiles = N // TILE
    base, rem = divmod(tiles, world)
    t0 = rank * base + min(rank, rem)
    t1 = t0 + base + (1 if rank < rem else 0)
    return t0 * TILE, t1 * TILE


def column_shards(N: int, world: int) -> List[Tuple[int, int]]:
    return [column_shard(N, world, r) for r in range(world)]


def shard_raw_weights(Wq_raw, S_raw, Z_raw, n0: int, n1: int):
    """Slices of the raw arrays (columns are the last axis of all three); Z_raw may be None."""
    cut = lambda a: None if a is None else a[..., n0:n1].contiguous() if hasattr(a, "contiguous") else a[..., n0:n1].copy()
    return cut(Wq_raw), cut(S_raw), cut(Z_raw)


def gather_columns(C_local, N: int, dist, world: int, rank: int):
    """All-gather the ranks' column slices [M, n1 - n0] into the whole C [M, N] on every rank.  Shards may
    differ by one tile, so every rank sends a slice padded to the widest shard."""
    import torch
    shards = column_shards(N, world)
    widest = max(b - a for a, b in shards)
    M = C_local.shape[0]
    send = torch.zeros((M, widest), dtype=C_local.dtype, device=C_local.device)
    send[:, : C_local.shape[1]] = C_local
    recv = [torch.empty_like(send) for _ in range(world)]
    dist.all_gather(recv, send)
    out = torch.empty((M, N), dtype=C_local.dtype, device=C_local.device)
    for (a, b), piece in zip(shards, recv):
        out[:, a:b] = piece[:, : b - a]
    return out
