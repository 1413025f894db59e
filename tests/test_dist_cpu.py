"""Host-side logic of the multi-rank bench path on CPU: two gloo ranks reduce their local step
time (max) and work (sum) exactly as bench.py does under torchrun."""
import os
import socket
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    assert bench.dist_env() == (rank, rank, world)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 3.0 + rank            # rank 1 is the slow one
    local_flops = 10.0 * (rank + 1)
    ms = bench.max_over_ranks(local_ms)
    fl = bench.sum_over_ranks(local_flops)
    bench.barrier()
    out.put((rank, ms, fl))
    dist.destroy_process_group()


def test_two_rank_reduction_max_time_sum_work():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, 4.0, 30.0), (1, 4.0, 30.0)]


def test_single_process_reductions_are_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.5) == 1.5 and bench.sum_over_ranks(2.5) == 2.5
    bench.barrier()


# ---- splitting one product over ranks without a collective (host arithmetic + oracle, CPU only) ----
def test_column_shards_partition_the_width():
    sys.path.insert(0, ROOT)
    from paper_2608_05033_b200.shard import column_shard
    for N, world, align in ((256, 8, 4), (100, 3, 4), (7, 4, 1), (3, 8, 4), (0, 2, 4), (128, 1, 8)):
        got = [column_shard(N, world, r, align) for r in range(world)]
        assert got[0][0] == 0 and sum(n for _, n in got) == N
        for (c0, n), (c1, _) in zip(got, got[1:]):
            assert c0 + n == c1
        assert all(c0 % align == 0 for c0, n in got if n)
        sizes = [(-(-n // align)) for _, n in got]
        assert max(sizes) - min(sizes) <= 1


def test_row_shards_balance_rows_plus_nonzeros():
    import numpy as np
    sys.path.insert(0, ROOT)
    import workloads as W
    from paper_2608_05033_b200.shard import row_shard_bounds
    w = W.g5_skewed(M=1 << 13, N=4, scale_c=2.4e7 / 512, cap=2000)
    for world in (1, 2, 3, 8):
        b = row_shard_bounds(w.rowptr, world)
        assert b[0] == 0 and b[-1] == w.M and np.all(np.diff(b) >= 0)
        work = np.array([(b[k + 1] - b[k]) + (w.rowptr[b[k + 1]] - w.rowptr[b[k]]) for k in range(world)])
        ideal = (w.M + w.nnz) / world
        longest = int(np.diff(w.rowptr).max()) + 1
        assert np.all(np.abs(work - ideal) <= longest + 1)      # off by at most one row's weight
    assert list(row_shard_bounds(np.zeros(6, np.int32), 5)) == [0, 1, 2, 3, 4, 5]


def _shard_worker(rank, world, port, out):
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import oracle
    import workloads as W
    from paper_2608_05033_b200.shard import column_shard, row_shard_bounds, row_shard_csr
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    w = W.g3_gcn_rmat(scale=10, N=12)
    # rows: this rank's range with rebased pointers, all of B
    b = row_shard_bounds(w.rowptr, world)
    r0, r1 = int(b[rank]), int(b[rank + 1])
    rp, cj, v = row_shard_csr(w.rowptr, w.colind, w.vals, r0, r1)
    mine, _ = oracle.spmm(rp, cj, v, w.B, w.N)
    rows_full = torch.zeros((w.M, w.N), dtype=torch.float64)
    rows_full[r0:r1] = torch.from_numpy(mine)
    dist.all_reduce(rows_full)                      # test-side assembly only: disjoint rows, zeros elsewhere
    # columns: all of A, this rank's columns of B
    c0, n = column_shard(w.N, world, rank, 4)
    cols_full = torch.zeros((w.M, w.N), dtype=torch.float64)
    if n:
        part, _ = oracle.spmm(w.rowptr, w.colind, w.vals, np.ascontiguousarray(w.B[:, c0:c0 + n]), n)
        cols_full[:, c0:c0 + n] = torch.from_numpy(part)
    dist.all_reduce(cols_full)
    if rank == 0:
        ref, _ = oracle.spmm(w.rowptr, w.colind, w.vals, w.B, w.N)
        out.put((bool(np.array_equal(rows_full.numpy(), ref)), bool(np.array_equal(cols_full.numpy(), ref))))
    dist.destroy_process_group()


def test_two_ranks_row_and_column_shards_reassemble_the_product():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == (True, True)


# ---- row split with a row-sharded B: one all-gather into local memory, then the rank's own rows ----
def test_b_row_shards_cover_every_row_once():
    sys.path.insert(0, ROOT)
    from paper_2608_05033_b200.shard import b_row_shard
    for K, world in ((1000, 2), (1001, 4), (5, 8), (0, 3), (64, 1)):
        pieces = [b_row_shard(K, world, r) for r in range(world)]
        assert pieces[0][0] == 0 and pieces[-1][1] == K
        for (a0, a1, per), (b0, b1, _) in zip(pieces, pieces[1:]):
            assert a1 == b0 and a1 - a0 <= per
        assert len({p[2] for p in pieces}) == 1 and pieces[0][2] * world >= K


def _gather_worker(rank, world, port, out):
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import oracle
    import workloads as W
    from paper_2608_05033_b200.shard import b_row_shard, gather_b, row_shard_bounds, row_shard_csr
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    w = W.g3_gcn_rmat(scale=10, N=12)                       # K = 1024 + an odd split below
    K = w.K - 3                                             # make the last piece short: drop three rows / columns
    keep = w.colind < K
    lengths = np.add.reduceat(keep.astype(np.int64), w.rowptr[:-1]) * (np.diff(w.rowptr) > 0)
    rowptr = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    colind, vals, B = w.colind[keep], w.vals[keep], np.ascontiguousarray(w.B[:K])
    k0, k1, per = b_row_shard(K, world, rank)
    piece = np.zeros((per, w.N), dtype=np.float32)          # this rank only ever sees its own rows of B
    piece[:k1 - k0] = B[k0:k1]
    piece[k1 - k0:] = np.nan                                # pad rows lie beyond K: they must never be read
    b_full = gather_b(torch.from_numpy(piece), K).numpy()   # one collective, lands in this rank's memory
    same_b = bool(np.array_equal(b_full, B))
    bounds = row_shard_bounds(rowptr, world)
    r0, r1 = int(bounds[rank]), int(bounds[rank + 1])
    rp, cj, v = row_shard_csr(rowptr, colind, vals, r0, r1)
    mine, _ = oracle.spmm(rp, cj, v, np.ascontiguousarray(b_full), w.N)
    full = torch.zeros((w.M, w.N), dtype=torch.float64)
    full[r0:r1] = torch.from_numpy(mine)
    dist.all_reduce(full)                                   # test-side assembly only
    flags = torch.tensor([1.0 if same_b else 0.0])
    dist.all_reduce(flags, op=dist.ReduceOp.MIN)
    if rank == 0:
        ref, _ = oracle.spmm(rowptr, colind, vals, B, w.N)
        out.put((bool(flags.item() == 1.0), bool(np.array_equal(full.numpy(), ref))))
    dist.destroy_process_group()


def test_two_ranks_gather_row_sharded_b_then_compute_their_rows():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gather_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == (True, True)
