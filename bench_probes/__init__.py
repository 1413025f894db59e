"""Gather-path probes used by bench.py (--probe, --probe-paths): a small CUDA library of its own
(libgather_paths.so, built from gather_paths.cu), separate from the SpMM library and never
loaded by it.  It replays an index stream as bare row gathers through several fetch paths."""
from __future__ import annotations

import ctypes as C
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "gather_paths.cu")
LIB = os.path.join(HERE, "libgather_paths.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")

PATHS = {0: "plain loads, 4 in flight per lane", 1: "plain loads, 8 in flight", 2: "plain loads, 16 in flight",
         3: "L2 evict-last hint, 4 in flight", 4: "L1 no-allocate, 4 in flight",
         5: "tile order, indices staged in shared memory, evict-last", 6: "half warp per row, two vectors per lane",
         7: "bulk-copy ring (cp.async.bulk, 512 B per copy) + shared loads",
         8: "hub rows in distributed shared memory, cluster of 4", 9: "hub rows in distributed shared memory, cluster of 8",
         10: "hub rows in distributed shared memory, cluster of 16",
         11: "cp.async 16-byte copies into a per-warp shared-memory ring, 16 rows in flight per warp, L1 bypassed",
         12: "cp.async ring, 16 rows in flight per warp, through L1",
         13: "cp.async ring, 32 rows in flight per warp, L1 bypassed"}
HUB_CLUSTER = {8: 4, 9: 8, 10: 16}
HUB_ROWS_PER_CTA = 256

_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(SRC):
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call([NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
                               "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-o", tmp, SRC])
        os.replace(tmp, LIB)
    return LIB


def load():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB):
            raise RuntimeError(f"{LIB} is missing: run `python -c 'import bench_probes; bench_probes.build()'`")
        lib = C.CDLL(LIB)
        lib.gp_sink_floats.restype = C.c_long
        lib.gp_gather.restype = C.c_int
        lib.gp_gather.argtypes = [C.c_int, C.c_void_p, C.c_long, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.POINTER(C.c_int), C.c_void_p]
        _lib = lib
    return _lib


def sink_floats() -> int:
    return int(load().gp_sink_floats())


def gather(path: int, idx, count: int, table, row_bytes: int, sink, err=None, hubrows=None, stream=None) -> int:
    """Launch one replay; torch tensors in, returns the resident CTAs per SM (clusters for the hub paths)."""
    info = C.c_int(0)
    rc = load().gp_gather(path, idx.data_ptr(), count, table.data_ptr(), row_bytes, sink.data_ptr(),
                          err.data_ptr() if err is not None else None,
                          hubrows.data_ptr() if hubrows is not None else None, C.byref(info),
                          stream.cuda_stream if stream is not None else None)
    if rc != 0:
        raise RuntimeError(f"gp_gather(path={path}) failed: {rc}")
    return info.value
