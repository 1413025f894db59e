"""Splitting one SpMM over several GPUs without any collective (host arithmetic only).

Two splits need no exchange of data between ranks:

* columns of the dense operands: every rank holds all of A and the columns [c0, c0 + n) of B and C.
  Through the C ABI this is the ordinary call on offset base pointers with the full leading
  dimensions (`ldb`, `ldc` stay those of the whole matrices); the plan is made for n columns.
* rows of A and C, with B replicated: every rank plans the contiguous row range [r0, r1) with
  its row pointers rebased to zero and writes rows r0..r1-1 of C.  Ranges are balanced by
  rows + nonzeros, the merge-path split of the nnz-balanced family one level up.

Nothing here touches a GPU; the functions return index ranges.
"""
from __future__ import annotations

import numpy as np


def column_shard(N: int, world: int, rank: int, align: int = 1) -> tuple[int, int]:
    """Columns [c0, c0 + n) of rank `rank`: `align`-column groups dealt out as evenly as possible,
    earlier ranks take the extra groups, the last group may be ragged.  A rank can get n == 0."""
    if world < 1 or not 0 <= rank < world or N < 0 or align < 1:
        raise ValueError("bad shard request")
    groups = (N + align - 1) // align
    base, extra = divmod(groups, world)
    g0 = rank * base + min(rank, extra)
    g1 = g0 + base + (1 if rank < extra else 0)
    c0, c1 = min(g0 * align, N), min(g1 * align, N)
    return c0, c1 - c0


def row_shard_bounds(rowptr, world: int) -> np.ndarray:
    """Row boundaries b[0..world] (b[0] = 0, b[world] = M): rank k owns rows b[k]..b[k+1]-1.
    The merged list of M row ends and nnz nonzeros is cut into `world` equal parts; a boundary is
    the first row whose position in that list (row index + nonzeros before it) reaches the cut."""
    rowptr = np.asarray(rowptr, dtype=np.int64)
    M = rowptr.size - 1
    if world < 1 or M < 0:
        raise ValueError("bad shard request")
    total = M + int(rowptr[-1])
    pos = np.arange(M + 1, dtype=np.int64) + rowptr          # non-decreasing (strictly increasing, in fact)
    cuts = (np.arange(world + 1, dtype=np.int64) * total + world - 1) // world
    b = np.searchsorted(pos, cuts, side="left").astype(np.int64)
    b[0], b[-1] = 0, M
    return b


def row_shard_csr(rowptr, colind, vals, r0: int, r1: int):
    """CSR arrays of rows [r0, r1): rebased row pointers (a copy) and views of colind / vals."""
    rowptr = np.asarray(rowptr)
    p0, p1 = int(rowptr[r0]), int(rowptr[r1])
    return (rowptr[r0:r1 + 1] - rowptr[r0]).astype(np.int32), colind[p0:p1], vals[p0:p1]
