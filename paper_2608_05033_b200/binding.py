"""Thin ctypes binding of libsd.so: argument marshalling only.

The functions carry the C names (sd_plan_create, sd_plan_create_ex, sd_spmm,
sd_spmm_host, sd_plan_destroy, sd_plan_get_info, sd_plan_get_bsr,
sd_plan_get_tiles, sd_last_error); `Plan` is a small convenience wrapper over
them.  torch is used for device memory and streams only.  There is no
fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(PKG, "libsd.so")

SD_OK, SD_ERR_INVALID_ARG, SD_ERR_UNSUPPORTED, SD_ERR_ALLOC, SD_ERR_CUDA, SD_ERR_INTERNAL = range(6)
SD_F32, SD_BF16 = 0, 1
SD_AUTO, SD_ROWSPLIT, SD_MERGE, SD_BSR_TC, SD_HYBRID = 0, 1, 2, 3, 4
FAMILY_NAMES = {SD_ROWSPLIT: "rowsplit", SD_MERGE: "merge", SD_BSR_TC: "bsr_tc", SD_HYBRID: "hybrid"}

EXPORTS = ["sd_plan_create", "sd_plan_create_ex", "sd_spmm", "sd_spmm_host", "sd_spmm_host_async", "sd_plan_sync", "sd_plan_update_values", "sd_plan_save", "sd_plan_load", "sd_plan_destroy",
           "sd_plan_get_info", "sd_plan_get_features", "sd_plan_get_bsr", "sd_plan_get_tiles", "sd_plan_get_segments", "sd_plan_get_hybrid", "sd_plan_device_status", "sd_spmm_merge_static", "sd_last_error",
           "sd_version"]


class sd_plan_desc_t(C.Structure):
    _fields_ = [("rowptr", C.c_void_p), ("colind", C.c_void_p), ("vals", C.c_void_p),
                ("M", C.c_int64), ("K", C.c_int64), ("N", C.c_int64),
                ("dtype", C.c_int32), ("family", C.c_int32), ("windows", C.c_int32),
                ("validate", C.c_int32), ("stream", C.c_void_p), ("test_wait_expiry", C.c_int32),
                ("heavy_len", C.c_int32)]


class sd_plan_info_t(C.Structure):
    _fields_ = [("M", C.c_int64), ("K", C.c_int64), ("N", C.c_int64), ("nnz", C.c_int64),
                ("row_hist", C.c_int64 * 32), ("sum_r2", C.c_uint64), ("max_r", C.c_int64),
                ("empty_rows", C.c_int64), ("sum_span", C.c_uint64), ("max_span", C.c_int64),
                ("sum_gap", C.c_uint64), ("diag", C.c_int64), ("unsorted_rows", C.c_int64),
                ("long_rows", C.c_int64), ("nnz_long_rows", C.c_int64), ("nnzb16", C.c_int64),
                ("blk_hist", C.c_int64 * 9), ("nnz_dense_blocks", C.c_int64),
                ("family", C.c_int32), ("dtype", C.c_int32), ("windows", C.c_int32),
                ("tile_items", C.c_int32), ("num_tiles", C.c_int64), ("num_segments", C.c_int64),
                ("plan_bytes", C.c_int64), ("sm_count", C.c_int32), ("launches", C.c_int32),
                ("l2_bytes", C.c_int64), ("class_split", C.c_int32), ("heavy_len", C.c_int32)]

    def as_dict(self) -> dict:
        d = {}
        for name, _ in self._fields_:
            v = getattr(self, name)
            d[name] = list(v) if hasattr(v, "__len__") else int(v)
        return d


SHAPE_NAMES = {0: "uniform", 1: "moderate", 2: "skewed", 3: "power-law", 4: "bimodal"}


class sd_features_t(C.Structure):
    _fields_ = [("row_q", C.c_int64 * 3), ("col_q", C.c_int64 * 3), ("col_max", C.c_int64), ("col_empty", C.c_int64),
                ("sum_d2", C.c_uint64), ("ell_slots", C.c_int64), ("sell_slots", C.c_int64 * 3), ("nnzb", C.c_int64 * 3),
                ("rep_bytes", C.c_int64 * 8), ("shape_class", C.c_int32), ("value_bytes", C.c_int32),
                ("borrowed_bytes", C.c_int64), ("plan_bytes", C.c_int64), ("d_r", C.c_int64), ("d_s", C.c_int64),
                ("m_r", C.c_int64), ("m_t", C.c_int64), ("work_units", C.c_int64), ("sm_count", C.c_int32),
                ("reserved", C.c_int32), ("l2_bytes", C.c_int64)]


_lib = None


def load():
    """Load libsd.so.  Raises if it has not been built (there is no other code path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2608_05033_b200.build` "
                           "(nvcc, sm_100a). The library has no CPU or PyTorch fallback.")
    lib = C.CDLL(LIB_PATH)
    lib.sd_plan_create.restype = C.c_void_p
    lib.sd_plan_create.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64]
    lib.sd_plan_create_ex.restype = C.c_int
    lib.sd_plan_create_ex.argtypes = [C.POINTER(sd_plan_desc_t), C.POINTER(C.c_void_p)]
    lib.sd_spmm.restype = C.c_int
    lib.sd_spmm.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_float, C.c_float,
                            C.c_void_p]
    lib.sd_spmm_host.restype = C.c_int
    lib.sd_spmm_host.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_float, C.c_float]
    lib.sd_spmm_host_async.restype = C.c_int
    lib.sd_spmm_host_async.argtypes = lib.sd_spmm_host.argtypes
    lib.sd_plan_update_values.restype = C.c_int
    lib.sd_plan_update_values.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    lib.sd_plan_sync.restype = C.c_int
    lib.sd_plan_sync.argtypes = [C.c_void_p]
    lib.sd_plan_save.restype = C.c_int
    lib.sd_plan_save.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]
    lib.sd_plan_load.restype = C.c_int
    lib.sd_plan_load.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_void_p)]
    lib.sd_plan_destroy.restype = None
    lib.sd_plan_destroy.argtypes = [C.c_void_p]
    lib.sd_plan_get_info.restype = C.c_int
    lib.sd_plan_get_info.argtypes = [C.c_void_p, C.POINTER(sd_plan_info_t)]
    lib.sd_plan_get_features.restype = C.c_int
    lib.sd_plan_get_features.argtypes = [C.c_void_p, C.POINTER(sd_features_t)]
    lib.sd_plan_get_bsr.restype = C.c_int
    lib.sd_plan_get_bsr.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.sd_plan_get_tiles.restype = C.c_int
    lib.sd_plan_get_tiles.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.POINTER(C.c_int64)]
    lib.sd_plan_get_segments.restype = C.c_int
    lib.sd_plan_get_segments.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.sd_plan_get_hybrid.restype = C.c_int
    lib.sd_plan_get_hybrid.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.sd_plan_device_status.restype = C.c_int
    lib.sd_plan_device_status.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
    lib.sd_spmm_merge_static.restype = C.c_int
    lib.sd_spmm_merge_static.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int64,
                                         C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_float, C.c_float, C.c_void_p]
    lib.sd_last_error.restype = C.c_int
    lib.sd_last_error.argtypes = [C.c_char_p, C.c_size_t]
    lib.sd_version.restype = C.c_char_p
    _lib = lib
    return lib


class SdError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"sd status {code}: {text}")
        self.code = code


def sd_last_error() -> tuple[int, str]:
    buf = C.create_string_buffer(512)
    code = load().sd_last_error(buf, 512)
    return code, buf.value.decode(errors="replace")


def _raise(code: int):
    raise SdError(code, sd_last_error()[1])


def _ptr(t):
    """Address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream_handle(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


# ---- the C calls, by name ------------------------------------------------------------
def sd_plan_create(rowptr, colind, vals, M: int, K: int, N: int):
    h = load().sd_plan_create(_ptr(rowptr), _ptr(colind), _ptr(vals), M, K, N)
    if not h:
        _raise(sd_last_error()[0])
    return h


def sd_plan_create_ex(rowptr, colind, vals, M: int, K: int, N: int, dtype: int = SD_F32,
                      family: int = SD_AUTO, windows: int = 0, validate: bool = False, stream=None,
                      test_wait_expiry: int = 0, heavy_len: int = 0):
    d = sd_plan_desc_t(_ptr(rowptr), _ptr(colind), _ptr(vals), M, K, N, dtype, family, windows,
                       int(validate), _stream_handle(stream) if stream is not None else None, test_wait_expiry,
                       heavy_len)
    out = C.c_void_p()
    rc = load().sd_plan_create_ex(C.byref(d), C.byref(out))
    if rc != SD_OK:
        _raise(rc)
    return out.value


def sd_spmm(plan, B, ldb: int, Cmat, ldc: int, alpha: float, beta: float, stream=None):
    rc = load().sd_spmm(plan, _ptr(B), ldb, _ptr(Cmat), ldc, alpha, beta, _stream_handle(stream))
    if rc != SD_OK:
        _raise(rc)


def sd_spmm_host_async(plan, B_host, ldb: int, C_host, ldc: int, alpha: float, beta: float):
    rc = load().sd_spmm_host_async(plan, _ptr(B_host), ldb, _ptr(C_host), ldc, alpha, beta)
    if rc != SD_OK:
        _raise(rc)


def sd_plan_update_values(plan, vals, stream=None):
    rc = load().sd_plan_update_values(plan, _ptr(vals), _stream_handle(stream))
    if rc != SD_OK:
        _raise(rc)


def sd_plan_sync(plan):
    rc = load().sd_plan_sync(plan)
    if rc != SD_OK:
        _raise(rc)


def sd_spmm_host(plan, B_host, ldb: int, C_host, ldc: int, alpha: float, beta: float):
    rc = load().sd_spmm_host(plan, _ptr(B_host), ldb, _ptr(C_host), ldc, alpha, beta)
    if rc != SD_OK:
        _raise(rc)


def sd_spmm_merge_static(rowptr, colind, vals, M: int, K: int, N: int, nnz: int, B, ldb: int, Cmat, ldc: int,
                         alpha: float, beta: float, stream=None):
    """Merge-path SpMM without a plan and without any allocation (fixed 4 MiB scratch inside the
    library; see include/sd.h for the size limit and the sharing rules)."""
    rc = load().sd_spmm_merge_static(_ptr(rowptr), _ptr(colind), _ptr(vals), M, K, N, nnz, _ptr(B), ldb, _ptr(Cmat),
                                     ldc, alpha, beta, _stream_handle(stream))
    if rc != SD_OK:
        _raise(rc)


def sd_plan_save(plan) -> bytes:
    """The plan's key and structure-only representation as a host blob (see include/sd.h)."""
    need = C.c_size_t(0)
    rc = load().sd_plan_save(plan, None, 0, C.byref(need))
    if rc != SD_OK:
        _raise(rc)
    buf = (C.c_ubyte * need.value)()
    rc = load().sd_plan_save(plan, buf, need.value, C.byref(need))
    if rc != SD_OK:
        _raise(rc)
    return bytes(buf)


def sd_plan_load(blob: bytes, rowptr, colind, vals):
    out = C.c_void_p()
    rc = load().sd_plan_load(blob, len(blob), _ptr(rowptr), _ptr(colind), _ptr(vals), C.byref(out))
    if rc != SD_OK:
        _raise(rc)
    return out.value


def sd_plan_destroy(plan):
    load().sd_plan_destroy(plan)


def sd_plan_get_info(plan) -> sd_plan_info_t:
    info = sd_plan_info_t()
    rc = load().sd_plan_get_info(plan, C.byref(info))
    if rc != SD_OK:
        _raise(rc)
    return info


def sd_plan_get_features(plan) -> sd_features_t:
    f = sd_features_t()
    rc = load().sd_plan_get_features(plan, C.byref(f))
    if rc != SD_OK:
        _raise(rc)
    return f


def sd_plan_get_bsr(plan):
    info = sd_plan_get_info(plan)
    Mb = (info.M + 15) // 16
    browptr = np.zeros(Mb + 1, np.int32)
    bcol = np.zeros(info.nnzb16, np.int32)
    bval = np.zeros((info.nnzb16, 16, 16), np.float32 if info.dtype == SD_F32 else np.uint16)
    rc = load().sd_plan_get_bsr(plan, browptr.ctypes.data, bcol.ctypes.data, bval.ctypes.data)
    if rc != SD_OK:
        _raise(rc)
    return browptr, bcol, bval


def sd_plan_get_segments(plan):
    """Returns (seg_ptr, seg_row, colind, vals, win_seg) of a plan with column windows."""
    info = sd_plan_get_info(plan)
    S, nnz, W = info.num_segments, info.nnz, info.windows
    seg_ptr = np.zeros(S + 1, np.int32)
    seg_row = np.zeros(S, np.int32)
    colind = np.zeros(nnz, np.int32)
    vals = np.zeros(nnz, np.float32 if info.dtype == SD_F32 else np.uint16)
    win_seg = np.zeros(3 * W + 1, np.int64)
    rc = load().sd_plan_get_segments(plan, seg_ptr.ctypes.data, seg_row.ctypes.data, colind.ctypes.data,
                                     vals.ctypes.data, win_seg.ctypes.data)
    if rc != SD_OK:
        _raise(rc)
    return seg_ptr, seg_row, colind, vals, win_seg


def sd_plan_get_hybrid(plan):
    """Returns (heavy_rows, chunk_ptr, ranges [nc, 2], order, light_rows) of a plan of the hybrid family."""
    info = sd_plan_get_info(plan)
    nl, nc = info.num_tiles, info.num_segments
    heavy = np.zeros(nl, np.int32)
    chunk_ptr = np.zeros(nl + 1, np.int32)
    ranges = np.zeros((nc, 2), np.int32)
    order = np.zeros(nc, np.int32)
    light = np.zeros(info.M - nl, np.int32)
    rc = load().sd_plan_get_hybrid(plan, heavy.ctypes.data, chunk_ptr.ctypes.data, ranges.ctypes.data, order.ctypes.data,
                                   light.ctypes.data)
    if rc != SD_OK:
        _raise(rc)
    return heavy, chunk_ptr, ranges, order, light


def sd_plan_device_status(plan) -> int:
    st = C.c_int32(0)
    rc = load().sd_plan_device_status(plan, C.byref(st))
    if rc != SD_OK:
        _raise(rc)
    return st.value


def sd_plan_get_tiles(plan) -> np.ndarray:
    n = C.c_int64(0)
    rc = load().sd_plan_get_tiles(plan, None, 0, C.byref(n))
    if rc != SD_OK:
        _raise(rc)
    out = np.zeros(n.value, np.int32)
    rc = load().sd_plan_get_tiles(plan, out.ctypes.data, n.value, C.byref(n))
    if rc != SD_OK:
        _raise(rc)
    return out


# ---- convenience wrapper ----------------------------------------------------------------
class Plan:
    """Owns an sd_plan_t and keeps the borrowed CSR tensors alive."""

    def __init__(self, rowptr, colind, vals, M: int, K: int, N: int, dtype: int | None = None,
                 family: int = SD_AUTO, windows: int = 0, validate: bool = False, test_wait_expiry: int = 0,
                 heavy_len: int = 0):
        import torch
        if dtype is None:
            dtype = SD_F32 if vals.dtype == torch.float32 else SD_BF16
        self._keep = (rowptr, colind, vals)
        self.M, self.K, self.N, self.dtype = M, K, N, dtype
        self.handle = sd_plan_create_ex(rowptr, colind, vals, M, K, N, dtype, family, windows, validate,
                                        test_wait_expiry=test_wait_expiry, heavy_len=heavy_len)

    def spmm(self, B, Cmat, alpha: float = 1.0, beta: float = 0.0, stream=None):
        sd_spmm(self.handle, B, B.stride(0), Cmat, Cmat.stride(0), alpha, beta, stream)
        return Cmat

    def spmm_host(self, B_host, C_host, alpha: float = 1.0, beta: float = 0.0):
        ldb = B_host.strides[0] // B_host.itemsize if isinstance(B_host, np.ndarray) else B_host.stride(0)
        ldc = C_host.strides[0] // C_host.itemsize if isinstance(C_host, np.ndarray) else C_host.stride(0)
        sd_spmm_host(self.handle, B_host, ldb, C_host, ldc, alpha, beta)
        return C_host

    def spmm_host_async(self, B_host, C_host, alpha: float = 1.0, beta: float = 0.0):
        """Queues the copies and the kernels on the plan's own stream; `sync()` waits for them."""
        ldb = B_host.strides[0] // B_host.itemsize if isinstance(B_host, np.ndarray) else B_host.stride(0)
        ldc = C_host.strides[0] // C_host.itemsize if isinstance(C_host, np.ndarray) else C_host.stride(0)
        sd_spmm_host_async(self.handle, B_host, ldb, C_host, ldc, alpha, beta)
        return C_host

    def sync(self):
        sd_plan_sync(self.handle)

    def update_values(self, vals, stream=None):
        """New values for the same pattern; `vals` is borrowed from now on."""
        sd_plan_update_values(self.handle, vals, stream)
        self._keep = (self._keep[0], self._keep[1], vals)

    def save(self) -> bytes:
        return sd_plan_save(self.handle)

    @classmethod
    def load(cls, blob: bytes, rowptr, colind, vals):
        """A plan from a blob made by save(); the CSR arrays are borrowed like at creation."""
        self = cls.__new__(cls)
        self._keep = (rowptr, colind, vals)
        self.handle = sd_plan_load(blob, rowptr, colind, vals)
        info = sd_plan_get_info(self.handle)
        self.M, self.K, self.N, self.dtype = int(info.M), int(info.K), int(info.N), int(info.dtype)
        return self

    def device_status(self) -> int:
        return sd_plan_device_status(self.handle)

    def info(self) -> sd_plan_info_t:
        return sd_plan_get_info(self.handle)

    def features(self) -> sd_features_t:
        return sd_plan_get_features(self.handle)

    def close(self):
        if self.handle:
            sd_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
