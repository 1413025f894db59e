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


# ---- row split with a row-sharded dense operand: one all-gather into local memory, then the ordinary call ----
def b_row_shard(K: int, world: int, rank: int) -> tuple[int, int, int]:
    """Rows of B held by `rank` when B is dealt out in `world` equal contiguous pieces: returns
    (k0, k1, rows_per_rank) with rows_per_rank = ceil(K / world); the last pieces may be short or empty
    (k1 - k0 < rows_per_rank) and are padded to rows_per_rank rows in the exchange buffers."""
    if world < 1 or not 0 <= rank < world or K < 0:
        raise ValueError("bad shard request")
    per = -(-K // world) if K else 0
    k0 = min(rank * per, K)
    k1 = min(k0 + per, K)
    return k0, k1, per


def gather_b(b_local, K: int, out=None, group=None):
    """All ranks' pieces of B (b_row_shard) gathered into THIS rank's own memory with one
    all_gather_into_tensor (NCCL over NVLink on GPUs, gloo on CPU); returns the [K, N] view of the gathered
    buffer.  `b_local` is [rows_per_rank, N] (pad rows beyond this rank's share are ignored by the result
    view only if they fall beyond K, so pad with anything).  The SpMM kernels then read B from local memory
    only: no kernel is ever handed a peer's pointer."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    per, N = b_local.shape
    if out is None:
        out = torch.empty((world * per, N), dtype=b_local.dtype, device=b_local.device)
    if world == 1:
        out[:per].copy_(b_local)
    else:
        dist.all_gather_into_tensor(out, b_local.contiguous(), group=group)
    return out[:K]


class RowSplitSpmm:
    """One product C = alpha*A*B + beta*C over the ranks of a process group: rank k owns the rows
    row_shard_bounds()[k] .. [k+1]-1 of A and C (balanced by rows + nonzeros) and the b_row_shard piece of B.
    Every call gathers B into a rank-local buffer (one collective), then runs the rank's own plan on it."""

    def __init__(self, rowptr_h, colind_h, vals_h, M: int, K: int, N: int, dtype: int, device, group=None, **plan_kw):
        import torch
        import torch.distributed as dist
        from . import binding as sd
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.group, self.K, self.N = group, K, N
        b = row_shard_bounds(rowptr_h, self.world)
        self.r0, self.r1 = int(b[self.rank]), int(b[self.rank + 1])
        rp, cj, v = row_shard_csr(rowptr_h, colind_h, vals_h, self.r0, self.r1)
        as_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a.view(np.int16) if a.dtype == np.uint16 else a)).to(device)
        self.rowptr, self.colind, self.vals = as_dev(rp), as_dev(cj if cj.size else np.zeros(1, cj.dtype)), \
            as_dev(v if v.size else np.zeros(1, v.dtype))
        self.plan = sd.Plan(self.rowptr, self.colind, self.vals, self.r1 - self.r0, K, N, dtype=dtype, **plan_kw)
        self.k0, self.k1, self.per = b_row_shard(K, self.world, self.rank)
        bdt = torch.float32 if dtype == sd.SD_F32 else torch.int16
        self.b_full = torch.empty((self.world * self.per, N), dtype=bdt, device=device)

    def run(self, b_local, c_local, alpha: float = 1.0, beta: float = 0.0, stream=None):
        """b_local: [rows_per_rank, N] piece of B; c_local: [r1 - r0, N] rows of C of this rank."""
        bf = gather_b(b_local, self.K, out=self.b_full, group=self.group)
        if self.r1 > self.r0:
            self.plan.spmm(bf, c_local, alpha, beta, stream)
        return c_local

    def close(self):
        self.plan.close()
