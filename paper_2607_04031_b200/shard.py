"""Sharding one GEMM of the path over several GPUs (one process per GPU, torch.distributed for the exchange).

Blocks of the tile-major layout (Section 3) never straddle a shard boundary when the boundary is a multiple of the
block extent, so every rank re-lays-out and reads its own slice with the single-GPU calls unchanged:

  "n"       column-parallel: rank r owns whole block columns n in [n0, n1).  No exchange; outputs concatenate.
  "k"       row-parallel: rank r owns whole block rows k in [k0, k1) and the matching columns of A.  The fp32
            partial results are summed over ranks (one all-reduce).
  "expert"  grouped problems: rank r owns experts [e0, e1) and computes the token rows routed to them.  Rows of
            other ranks' experts are filled in by the exchange.

The arithmetic stays in the CUDA library; this module only slices, launches and combines.  The combine_* functions
take already computed local results, so the exchange logic runs on any backend (NCCL on GPUs, gloo in CPU tests).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch
import torch.distributed as dist

MODES = ("n", "k", "expert")


@dataclass(frozen=True)
class Shard:
    """What one rank owns: weight columns [n0, n1), weight rows [k0, k1), experts [e0, e1)."""
    mode: str
    rank: int
    world: int
    n0: int
    n1: int
    k0: int
    k1: int
    e0: int = 0
    e1: int = 1


def _even_cut(units: int, world: int, rank: int):
    """Contiguous ranges whose sizes differ by at most one unit."""
    return (units * rank) // world, (units * (rank + 1)) // world


def plan(mode: str, N: int, K: int, block_rows: int, block_cols: int, world: int, E: int = 1):
    """One Shard per rank.  Boundaries are multiples of the memory tile's extent along the cut dimension
    (block_cols for "n"; block_rows, rounded up to 8 rows so that A's slice keeps a 16-byte pitch, for "k");
    row-major weights (block_rows == 0) cut "n" at 64 columns, the granularity the GEMM accepts, and "k" at 8
    rows.  Raises when a rank would own nothing."""
    if mode not in MODES:
        raise ValueError(f"mode must be one of {MODES}")
    if world < 1:
        raise ValueError("world must be positive")
    unit_n = block_cols if block_rows else 64
    unit_k = math.lcm(block_rows, 8) if block_rows else 8         # the K slice of A keeps a 16-byte row pitch
    if N % unit_n or K % unit_k:
        raise ValueError("N and K must be whole numbers of blocks")
    units = {"n": N // unit_n, "k": K // unit_k, "expert": E}[mode]
    if units < world:
        raise ValueError(f"{units} units cannot be cut over {world} ranks")
    shards = []
    for r in range(world):
        lo, hi = _even_cut(units, world, r)
        if mode == "n":
            shards.append(Shard(mode, r, world, lo * unit_n, hi * unit_n, 0, K, 0, E))
        elif mode == "k":
            shards.append(Shard(mode, r, world, 0, N, lo * unit_k, hi * unit_k, 0, E))
        else:
            shards.append(Shard(mode, r, world, 0, N, 0, K, lo, hi))
    return shards


def local_weight(W_rowmajor: torch.Tensor, s: Shard) -> torch.Tensor:
    """The rank's slice of a row-major [K, N] weight (or [E, K, N] stack), contiguous."""
    if W_rowmajor.dim() == 3:
        return W_rowmajor[s.e0:s.e1, s.k0:s.k1, s.n0:s.n1].contiguous()
    return W_rowmajor[s.k0:s.k1, s.n0:s.n1].contiguous()


def local_activations(A: torch.Tensor, s: Shard, offsets_host=None) -> torch.Tensor:
    """The part of A [rows, K] the rank multiplies: all of it ("n"), its K columns ("k"), its experts' rows."""
    if s.mode == "k":
        return A[:, s.k0:s.k1].contiguous()
    if s.mode == "expert":
        return A[int(offsets_host[s.e0]):int(offsets_host[s.e1])].contiguous()
    return A


def local_offsets(offsets_host, s: Shard):
    """Row offsets of the rank's experts, rebased to its first row (host list of e1 - e0 + 1 ints)."""
    base = int(offsets_host[s.e0])
    return [int(offsets_host[e]) - base for e in range(s.e0, s.e1 + 1)]


# ------------------------------------------------------------------------------------------------- exchange

def combine_n(C_local: torch.Tensor, shards, group=None) -> torch.Tensor:
    """Concatenate the ranks' column slices [M, n1 - n0] into [M, N].  Slices may differ in width by one block,
    so each rank's slice travels as its own broadcast-free all_gather entry after padding to the widest."""
    world = len(shards)
    if world == 1:
        return C_local
    M = C_local.shape[0]
    widest = max(s.n1 - s.n0 for s in shards)
    mine = C_local
    if C_local.shape[1] != widest:
        mine = torch.zeros((M, widest), dtype=C_local.dtype, device=C_local.device)
        mine[:, :C_local.shape[1]] = C_local
    parts = [torch.empty((M, widest), dtype=C_local.dtype, device=C_local.device) for _ in range(world)]
    dist.all_gather(parts, mine.contiguous(), group=group)
    return torch.cat([parts[s.rank][:, :s.n1 - s.n0] for s in shards], dim=1)


def combine_k(C_partial: torch.Tensor, group=None) -> torch.Tensor:
    """Sum the ranks' fp32 partial results in place (all-reduce) and return the tensor."""
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(C_partial, op=dist.ReduceOp.SUM, group=group)
    return C_partial


def combine_expert(C_rows_local: torch.Tensor, s: Shard, offsets_host, total_rows: int, group=None) -> torch.Tensor:
    """Place the rank's rows at their global position in a zeroed [total_rows, N] tensor and sum over ranks: every
    row is non-zero on exactly one rank, so the sum is an exact gather of rows of unequal counts."""
    N = C_rows_local.shape[1]
    full = torch.zeros((total_rows, N), dtype=C_rows_local.dtype, device=C_rows_local.device)
    full[int(offsets_host[s.e0]):int(offsets_host[s.e1])] = C_rows_local
    if s.world > 1:
        dist.all_reduce(full, op=dist.ReduceOp.SUM, group=group)
    return full


# ------------------------------------------------------------------------------------------- sharded calls

class ShardedWeight:
    """A rank's slice of one weight, re-laid-out tile-major on its GPU by the library's own relayout call."""

    def __init__(self, W_rowmajor_local: torch.Tensor, s: Shard, G: int, block_rows: int, block_cols: int):
        from . import binding as tl
        self.shard, self.G, self.block_rows, self.block_cols = s, G, block_rows, block_cols
        self.K, self.N = s.k1 - s.k0, s.n1 - s.n0
        self.experts = s.e1 - s.e0 if W_rowmajor_local.dim() == 3 else 0
        if tuple(W_rowmajor_local.shape[-2:]) != (self.K, self.N):
            raise ValueError("the local weight does not have the shard's shape")
        if block_rows == 0:
            self.W = W_rowmajor_local.contiguous()
        else:
            self.W = torch.empty_like(W_rowmajor_local)
            for e in range(max(self.experts, 1)):
                src = W_rowmajor_local[e] if self.experts else W_rowmajor_local
                dst = self.W[e] if self.experts else self.W
                tl.relayout(src, dst, self.K, self.N, W_rowmajor_local.element_size(), G, block_rows, block_cols,
                            tl.TO_TILE_MAJOR)


def gemm_local(A_local: torch.Tensor, W: ShardedWeight, cta=(0, 0, 0)) -> torch.Tensor:
    """The rank's own launch: [M, n1 - n0] columns ("n") or the fp32 partial sum over its K rows ("k")."""
    from . import binding as tl
    M = A_local.shape[0]
    C = torch.empty((M, W.N), dtype=torch.float32, device=A_local.device)
    tl.gemm(A_local, W.W, C, M, W.N, W.K, W.G, W.block_rows, W.block_cols, cta)
    return C


def gemm(A_local: torch.Tensor, W: ShardedWeight, shards, group=None, cta=(0, 0, 0), gather: bool = True):
    """C = A x B with B cut by `shards` ("n" or "k"); A_local is what local_activations() returns.  Returns the full
    [M, N] fp32 result on every rank ("n" with gather=False: the rank's own columns only)."""
    s = W.shard
    if s.mode not in ("n", "k"):
        raise ValueError("use gemm_grouped for expert shards")
    C = gemm_local(A_local, W, cta)
    if s.mode == "n":
        return combine_n(C, shards, group) if gather else C
    return combine_k(C, group)


def gemm_grouped_local(A_rows_local: torch.Tensor, W: ShardedWeight, offsets_host, cta=(0, 0, 0)) -> torch.Tensor:
    """The rank's own grouped launch over its experts' token rows: [rows of experts e0..e1, N] fp32."""
    from . import binding as tl
    s = W.shard
    if s.mode != "expert":
        raise ValueError("gemm_grouped takes an expert shard")
    offs = local_offsets(offsets_host, s)
    rows = offs[-1]
    C = torch.empty((rows, W.N), dtype=torch.float32, device=A_rows_local.device)
    if rows:
        d_offs = torch.tensor(offs, dtype=torch.int32, device=A_rows_local.device)
        tl.gemm_grouped(A_rows_local, W.W, C, d_offs, s.e1 - s.e0, rows, W.N, W.K, W.G, W.block_rows, W.block_cols,
                        cta)
    return C


def gemm_grouped(A_rows_local: torch.Tensor, W: ShardedWeight, offsets_host, total_rows: int, group=None,
                 cta=(0, 0, 0)):
    """Grouped GEMM with the experts cut over ranks; returns the full [total_rows, N] fp32 result on every rank."""
    C = gemm_grouped_local(A_rows_local, W, offsets_host, cta)
    return combine_expert(C, W.shard, offsets_host, total_rows, group)
