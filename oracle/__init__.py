"""ctypes front end of the CPU oracle (oracle/sd_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the bench's CPU-baseline leg import this
package.  It shares nothing with the CUDA library: it compiles its own C file
with gcc and never loads the library's shared object.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sd_oracle.c")
_SO = os.path.join(_HERE, "libsd_oracle.so")

F32, BF16 = 0, 1
ROWSPLIT, MERGE, BSR_TC, HYBRID = 1, 2, 3, 4
FAMILY_NAMES = {ROWSPLIT: "rowsplit", MERGE: "merge", BSR_TC: "bsr_tc", HYBRID: "hybrid"}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc -O2 -fopenmp (no fast-math: plain IEEE double)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


class Info(C.Structure):
    _fields_ = [
        ("M", C.c_int64), ("K", C.c_int64), ("N", C.c_int64), ("nnz", C.c_int64),
        ("row_hist", C.c_int64 * 32),
        ("sum_r2", C.c_uint64),
        ("max_r", C.c_int64),
        ("empty_rows", C.c_int64),
        ("sum_span", C.c_uint64),
        ("max_span", C.c_int64),
        ("sum_gap", C.c_uint64),
        ("diag", C.c_int64),
        ("unsorted_rows", C.c_int64),
        ("long_rows", C.c_int64),
        ("nnz_long_rows", C.c_int64),
        ("nnzb16", C.c_int64),
        ("blk_hist", C.c_int64 * 9),
        ("nnz_dense_blocks", C.c_int64),
    ]

    def as_dict(self) -> dict:
        d = {}
        for name, _ in self._fields_:
            v = getattr(self, name)
            d[name] = list(v) if hasattr(v, "__len__") else int(v)
        return d


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.sdo_bsr16_count.restype = C.c_int64
        _lib.sdo_window_segments.restype = C.c_int64
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _csr(rowptr, colind, vals):
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    colind = np.ascontiguousarray(colind, dtype=np.int32)
    vals = np.ascontiguousarray(vals)
    if vals.dtype == np.float32:
        dt = F32
    elif vals.dtype == np.uint16:
        dt = BF16
    else:
        raise TypeError("vals must be float32 or uint16 (bf16 bits)")
    return rowptr, colind, vals, dt


def _dense(B, dt):
    B = np.asarray(B)
    want = np.float32 if dt == F32 else np.uint16
    if B.dtype != want or B.ndim != 2 or B.strides[1] != B.itemsize:
        raise TypeError("dense operand must be a row-major 2-D array of the value dtype")
    return B, B.strides[0] // B.itemsize


def num_threads() -> int:
    return int(lib().sdo_num_threads())


def spmm(rowptr, colind, vals, B, N, Cin=None, alpha=1.0, beta=0.0, want_abs=True):
    """O1: returns (Cref, S) as float64 [M, N]; S is None unless want_abs."""
    rowptr, colind, vals, dt = _csr(rowptr, colind, vals)
    M = rowptr.size - 1
    B, ldb = _dense(B, dt)
    ldcin = 0
    if beta != 0.0:
        Cin = np.asarray(Cin)
        assert Cin.dtype == np.float32 and Cin.strides[1] == 4
        ldcin = Cin.strides[0] // 4
    Cref = np.empty((M, N), dtype=np.float64)
    S = np.empty((M, N), dtype=np.float64) if want_abs else None
    rc = lib().sdo_spmm(C.c_int64(M), C.c_int64(N), _p(rowptr), _p(colind), _p(vals), C.c_int(dt),
                        _p(B), C.c_int64(ldb), _p(Cin) if beta != 0.0 else None, C.c_int64(ldcin),
                        C.c_float(alpha), C.c_float(beta), _p(Cref), _p(S), C.c_int64(N))
    assert rc == 0
    return Cref, S


def spmm_rows(rows, rowptr, colind, vals, B, N, Cin=None, alpha=1.0, beta=0.0, want_abs=True):
    """O1 on selected rows: returns (Cref, S) as float64 [len(rows), N]; S is None unless want_abs."""
    rowptr, colind, vals, dt = _csr(rowptr, colind, vals)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    B, ldb = _dense(B, dt)
    ldcin = 0
    if beta != 0.0:
        Cin = np.asarray(Cin)
        assert Cin.dtype == np.float32 and Cin.strides[1] == 4
        ldcin = Cin.strides[0] // 4
    Cref = np.empty((rows.size, N), dtype=np.float64)
    S = np.empty((rows.size, N), dtype=np.float64) if want_abs else None
    rc = lib().sdo_spmm_rows(C.c_int64(rows.size), _p(rows), C.c_int64(N), _p(rowptr), _p(colind),
                             _p(vals), C.c_int(dt), _p(B), C.c_int64(ldb),
                             _p(Cin) if beta != 0.0 else None, C.c_int64(ldcin),
                             C.c_float(alpha), C.c_float(beta), _p(Cref), _p(S))
    assert rc == 0
    return Cref, S


def check(rowptr, colind, vals, B, N, Cgot, Cin=None, alpha=1.0, beta=0.0, rel=None, abs_tol=1e-6):
    """Compare a float32 result with O1 entry by entry under
    |C - Cref| <= rel*(|alpha| S + |beta||Cin|) + abs_tol  (rel: 1e-5 fp32, 1e-2 bf16)."""
    rowptr, colind, vals, dt = _csr(rowptr, colind, vals)
    M = rowptr.size - 1
    if rel is None:
        rel = 1e-5 if dt == F32 else 1e-2
    B, ldb = _dense(B, dt)
    Cgot = np.asarray(Cgot)
    assert Cgot.dtype == np.float32 and Cgot.shape[0] == M and (M == 0 or Cgot.strides[1] == 4)
    ldc = Cgot.strides[0] // 4 if M else max(N, 1)
    ldcin = 0
    if beta != 0.0:
        Cin = np.asarray(Cin)
        assert Cin.dtype == np.float32 and Cin.strides[1] == 4
        ldcin = Cin.strides[0] // 4
    out = np.zeros(7, dtype=np.float64)
    rc = lib().sdo_check(C.c_int64(M), C.c_int64(N), _p(rowptr), _p(colind), _p(vals), C.c_int(dt),
                         _p(B), C.c_int64(ldb), _p(Cin) if beta != 0.0 else None, C.c_int64(ldcin),
                         C.c_float(alpha), C.c_float(beta), _p(Cgot), C.c_int64(ldc),
                         C.c_double(rel), C.c_double(abs_tol), _p(out))
    assert rc == 0
    return {"violations": int(out[0]), "nonfinite": int(out[1]), "max_ratio": float(out[2]),
            "worst": (int(out[3]), int(out[4])), "max_abs_err": float(out[5]),
            "paper_rule_violations": int(out[6]), "rel": rel,
            "ok": int(out[0]) == 0 and int(out[1]) == 0}


def bsr16(rowptr, colind, vals, M, K):
    """O2: returns (browptr int32[Mb+1], bcol int32[nnzb], bval [nnzb,16,16] in the value dtype)."""
    rowptr, colind, vals, dt = _csr(rowptr, colind, vals)
    Mb = (M + 15) // 16
    browptr = np.zeros(Mb + 1, dtype=np.int32)
    nnzb = int(lib().sdo_bsr16_count(C.c_int64(M), C.c_int64(K), _p(rowptr), _p(colind), _p(browptr)))
    bcol = np.zeros(nnzb, dtype=np.int32)
    bval = np.zeros((nnzb, 16, 16), dtype=vals.dtype)
    rc = lib().sdo_bsr16_fill(C.c_int64(M), C.c_int64(K), _p(rowptr), _p(colind), _p(vals), C.c_int(dt),
                              _p(browptr), _p(bcol), _p(bval))
    assert rc == 0
    return browptr, bcol, bval


def summary(rowptr, colind, M, K, N) -> Info:
    """O3: integer structure summary."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    colind = np.ascontiguousarray(colind, dtype=np.int32)
    info = Info()
    rc = lib().sdo_summary(C.c_int64(M), C.c_int64(K), C.c_int64(N), _p(rowptr), _p(colind), C.byref(info))
    assert rc == 0
    return info


def decide(info: Info, dtype: int = F32) -> int:
    """O4: family rule on the integers of O3 (parity unpinned: thresholds are not in the paper)."""
    return int(lib().sdo_decide(C.byref(info), C.c_int(dtype)))


def decide_windows(info: Info, dtype: int, l2_bytes: int) -> int:
    """O4: number of column windows of the merge family (parity unpinned: this build's rule)."""
    return int(lib().sdo_decide_windows(C.byref(info), C.c_int(dtype), C.c_int64(l2_bytes)))


def decide_class_split(info: Info, dtype: int) -> bool:
    """O4: class split of the window-major schedule at one window (parity unpinned: this build's rule)."""
    return bool(lib().sdo_decide_class_split(C.byref(info), C.c_int(dtype)))


def window_segments(rowptr, colind, M, K, W, short_len=32):
    """O4: window-major segment list ordered by (window, class, row).
    Returns (seg_ptr, seg_row, perm, bounds[3W+1])."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    colind = np.ascontiguousarray(colind, dtype=np.int32)
    nnz = int(rowptr[-1])
    seg_ptr = np.zeros(nnz + M + 1, np.int32)
    seg_row = np.zeros(nnz + M, np.int32)
    perm = np.zeros(max(nnz, 1), np.int32)
    bounds = np.zeros(3 * W + 1, np.int64)
    S = int(lib().sdo_window_segments(C.c_int64(M), C.c_int64(K), _p(rowptr), _p(colind), C.c_int32(W),
                                      C.c_int32(short_len), _p(seg_ptr), _p(seg_row), _p(perm), _p(bounds)))
    return seg_ptr[:S + 1].copy(), seg_row[:S].copy(), perm[:nnz].copy(), bounds


def decide_hybrid(info: Info, dtype: int, windows: int) -> bool:
    """O4: hybrid family in place of the windowed class split (parity unpinned: this build's rule)."""
    return bool(lib().sdo_decide_hybrid(C.byref(info), C.c_int(dtype), C.c_int(windows)))


def decide_family(info: Info, dtype: int, l2_bytes: int) -> int:
    """O4: the family a plan is built with (decide, then the hybrid family where decide_hybrid says so)."""
    return int(lib().sdo_decide_family(C.byref(info), C.c_int(dtype), C.c_int64(l2_bytes)))


def hybrid_schedule(rowptr, colind, M, K, W, heavy_len, chunk_nnz=128):
    """O4: schedule of the hybrid family by its sequential definition.
    Returns (heavy_rows, chunk_ptr, ranges [nc, 2], order, light_rows)."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    colind = np.ascontiguousarray(colind, dtype=np.int32)
    nnz = int(rowptr[-1])
    heavy = np.zeros(max(M, 1), np.int32)
    chunk_ptr = np.zeros(M + 1, np.int32)
    ranges = np.zeros(2 * max(nnz, 1), np.int32)
    order = np.zeros(max(nnz, 1), np.int32)
    light = np.zeros(max(M, 1), np.int32)
    counts = np.zeros(3, np.int64)
    rc = lib().sdo_hybrid_schedule(C.c_int64(M), C.c_int64(K), _p(rowptr), _p(colind), C.c_int32(W),
                                   C.c_int32(heavy_len), C.c_int32(chunk_nnz), _p(heavy), _p(chunk_ptr), _p(ranges),
                                   _p(order), _p(light), _p(counts))
    assert rc == 0
    nl, nc, nlight = (int(x) for x in counts)
    return (heavy[:nl].copy(), chunk_ptr[:nl + 1].copy(), ranges[:2 * nc].reshape(nc, 2).copy(), order[:nc].copy(),
            light[:nlight].copy())


def hist_bin(v: int) -> int:
    return int(lib().sdo_hist_bin(C.c_int64(v)))


def merge_coords(ptr, items: int):
    """O4: merge-path tile start coordinates by the sequential two-pointer merge."""
    ptr = np.ascontiguousarray(ptr, dtype=np.int32)
    S = ptr.size - 1
    total = S + int(ptr[-1] - ptr[0])
    ntiles = (total + items - 1) // items
    out = np.zeros(ntiles + 1, dtype=np.int32)
    rc = lib().sdo_merge_coords(C.c_int64(S), _p(ptr), C.c_int64(items), C.c_int64(ntiles), _p(out))
    assert rc == 0
    return out


# ---- closed-form footprint indicators (Sec. 3.1 Eq. 4, Sec. 3.3 Eq. 10-13) ----
def rho_ell(info: Info) -> float:
    """Value-slot expansion of ELL: m * max_i r_i / nnz (Eq. 4)."""
    return info.M * info.max_r / info.nnz


def rho_bsr16(info: Info) -> float:
    """Value-slot expansion of BSR with b = 16: b^2 nnzb_b / nnz (Eq. 4)."""
    return 256 * info.nnzb16 / info.nnz


def tile_coverage16(info: Info) -> float:
    """Occupied 16x16 tiles over all tiles, ceil(M/16) * ceil(K/16)."""
    return info.nnzb16 / (((info.M + 15) // 16) * ((info.K + 15) // 16))


def csr_bytes(info: Info, value_bytes: int = 4) -> int:
    """Representation footprint of CSR with 32-bit indices (Eq. 10):
    values + column indices + row pointers."""
    return (value_bytes + 4) * info.nnz + 4 * (info.M + 1)


def bsr16_bytes(info: Info, value_bytes: int = 4) -> int:
    """Representation footprint of BSR-16: 256 value slots and one block-column
    index per occupied block, plus block-row pointers."""
    return (256 * value_bytes + 4) * info.nnzb16 + 4 * ((info.M + 15) // 16 + 1)


def working_set_bytes(rep_bytes: int, info: Info, value_bytes: int = 4, workspace: int = 0):
    """(M_R, M_T) of Eq. 11-12 for SpMM: read side = representation + workspace +
    dense B; total adds dense C (fp32)."""
    m_r = rep_bytes + workspace + info.K * info.N * value_bytes
    return m_r, m_r + info.M * info.N * 4


# ---- O5: extended structure analysis (Sec. 3.1, Eq. 4, Eq. 10) ----
SHAPE_NAMES = {0: "uniform", 1: "moderate", 2: "skewed", 3: "power-law", 4: "bimodal"}


class Features(C.Structure):
    _fields_ = [("row_q", C.c_int64 * 3), ("col_q", C.c_int64 * 3), ("col_max", C.c_int64), ("col_empty", C.c_int64),
                ("sum_d2", C.c_uint64), ("ell_slots", C.c_int64), ("sell_slots", C.c_int64 * 3),
                ("nnzb", C.c_int64 * 3), ("rep_bytes", C.c_int64 * 8), ("shape_class", C.c_int32),
                ("value_bytes", C.c_int32)]

    def as_dict(self) -> dict:
        d = {}
        for name, _ in self._fields_:
            v = getattr(self, name)
            d[name] = list(v) if hasattr(v, "__len__") else int(v)
        return d


def quartile(values, q: int) -> int:
    """Nearest-rank quartile: the ceil(q n / 4)-th smallest (0 for no values)."""
    v = np.ascontiguousarray(values, dtype=np.int32)
    lib().sdo_quartile.restype = C.c_int64
    return int(lib().sdo_quartile(_p(v), C.c_int64(v.size), C.c_int(q)))


def sell_slots(rowptr, c: int) -> int:
    """Numerator of rho_SELL(c) (Eq. 4), slices of c consecutive rows in storage order."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    lib().sdo_sell_slots.restype = C.c_int64
    return int(lib().sdo_sell_slots(C.c_int64(rowptr.size - 1), _p(rowptr), C.c_int64(c)))


def block_count(rowptr, colind, b: int) -> int:
    """nnzb_b of Eq. 4: occupied b x b blocks."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    colind = np.ascontiguousarray(colind, dtype=np.int32)
    lib().sdo_block_count.restype = C.c_int64
    return int(lib().sdo_block_count(C.c_int64(rowptr.size - 1), _p(rowptr), _p(colind), C.c_int64(b)))


def shape_class(info: Info) -> int:
    """Row-length shape class (parity unpinned: the paper names the classes, not the cut-offs)."""
    return int(lib().sdo_shape_class(C.byref(info)))


def features(rowptr, colind, M, K, info: Info, value_bytes: int = 4) -> Features:
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    colind = np.ascontiguousarray(colind, dtype=np.int32)
    f = Features()
    rc = lib().sdo_features(C.c_int64(M), C.c_int64(K), _p(rowptr), _p(colind), C.c_int(value_bytes),
                            C.byref(info), C.byref(f))
    assert rc == 0
    return f
