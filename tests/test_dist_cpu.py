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
