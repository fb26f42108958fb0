"""1-D row distribution of the local product over several GPUs (one process per GPU).

Output rows are independent, so a rank that holds all of A computes any contiguous range of rows of
C_L with no exchange afterwards.  The plumbing here is torch.distributed only (NCCL on GPUs, gloo in
the CPU tests): each rank starts with a contiguous slice of A's rows, the slices are all-gathered so
that every rank holds A in its own memory before any kernel reads it, and the rows of C_L are then
cut into ranges of near-equal work by spsyrk_plan_partition.  No arithmetic of the method lives in
this module.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def row_slice_bounds(m: int, world: int) -> list[int]:
    """Rows [b[r], b[r + 1]) of A start on rank r."""
    return [m * r // world for r in range(world + 1)]


def _allgather_ragged(local: torch.Tensor, counts: list[int], group=None) -> torch.Tensor:
    """Concatenation over ranks of 1-D tensors of different lengths (counts[r] on rank r)."""
    world = len(counts)
    width = max(max(counts), 1)
    padded = torch.zeros(width, dtype=local.dtype, device=local.device)
    padded[: local.numel()] = local
    pieces = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(pieces, padded, group=group)
    return torch.cat([pieces[r][: counts[r]] for r in range(world)])


def allgather_csr(m: int, rowptr_local: torch.Tensor, colidx_local: torch.Tensor, vals_local: torch.Tensor, group=None):
    """Every rank passes its slice of A (slice-local row pointers starting at 0, rows as cut by
    row_slice_bounds) and receives the whole matrix: (rowptr int64 [m + 1], colidx, vals)."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    b = row_slice_bounds(m, world)
    assert rowptr_local.numel() == b[rank + 1] - b[rank] + 1 and int(rowptr_local[0]) == 0
    nnz_local = torch.tensor([colidx_local.numel()], dtype=torch.int64, device=rowptr_local.device)
    nnz_all = [torch.empty_like(nnz_local) for _ in range(world)]
    dist.all_gather(nnz_all, nnz_local, group=group)
    nnz = [int(t.item()) for t in nnz_all]
    lengths = _allgather_ragged(rowptr_local[1:] - rowptr_local[:-1], [b[r + 1] - b[r] for r in range(world)], group)
    rowptr = torch.zeros(m + 1, dtype=torch.int64, device=rowptr_local.device)
    torch.cumsum(lengths, 0, out=rowptr[1:])
    colidx = _allgather_ragged(colidx_local, nnz, group)
    vals = _allgather_ragged(vals_local, nnz, group)
    return rowptr, colidx, vals


def rank_rows(bounds: list[int], rank: int) -> tuple[int, int]:
    """The output rows of `rank` from the bounds of spsyrk_plan_partition (parts == world size)."""
    return int(bounds[rank]), int(bounds[rank + 1])
