"""ctypes binding of libspws.so: the same entry points as include/spws.h, argument marshalling
only.  PyTorch supplies device memory and the stream; every step of the path runs in the
library's kernels.  Importing this module fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspws.so")

# status codes
SPWS_OK = 0
SPWS_INVALID_ARGUMENT = 1
SPWS_UNSUPPORTED_EXPRESSION = 2
SPWS_DIM_MISMATCH = 3
SPWS_NONCANONICAL_INPUT = 4
SPWS_SCRATCH_TOO_SMALL = 5
SPWS_WORKSPACE_TOO_LARGE = 6
SPWS_CUDA_ERROR = 7
SPWS_INTERNAL_OVERFLOW = 8
SPWS_OUTPUT_TOO_SMALL = 9
SPWS_BAD_SEQUENCE = 10
# enums
SPWS_CSR, SPWS_CSF3, SPWS_COO = 0, 1, 2
SPWS_F32, SPWS_F64 = 0, 1
SPWS_DENSE, SPWS_SPARSE_ISM, SPWS_AUTO, SPWS_HASH = 0, 1, 2, 3
POLICIES = {"dense": SPWS_DENSE, "ism": SPWS_SPARSE_ISM, "sparse_ism": SPWS_SPARSE_ISM, "auto": SPWS_AUTO, "hash": SPWS_HASH}

EXPORTS = ("spws_create", "spws_destroy", "spws_set_stream", "spws_plan_create", "spws_plan_destroy",
           "spws_check_expression", "spws_workspace_size", "spws_workspace_size_exact", "spws_symbolic", "spws_numeric",
           "spws_get_stats", "spws_set_profiling", "spws_get_timings", "spws_execute_host", "spws_gather_ceiling",
           "spws_row_pointer_static", "spws_status_string", "spws_plan_create3", "spws_workspace_size3", "spws_symbolic3",
           "spws_numeric3")
STATIC_MAX_ROWS = 16777216
TIMING_GROUPS = ("sym_bounds", "sym_bin", "sym_ism_reg", "sym_ism_smem_s", "sym_ism_smem", "sym_dense_warp",
                 "sym_dense_cta", "sym_ism_global", "sym_hash", "sym_scan", "num_ism_reg", "num_ism_smem_s", "num_ism_smem",
                 "num_dense_warp", "num_dense_emit", "num_dense_cta", "num_ism_global", "num_hash", "ceil_dense_warp",
                 "ceil_dense_cta")
# class index of each per-class kernel group (rows_per_class / products_per_class / nnz_per_class)
CLASS_NAMES = ("empty", "ism_reg", "ism_smem_s", "ism_smem", "dense_warp", "dense_hub", "dense_cta", "ism_global", "hash_s", "hash")


class spws_tensor_t(ctypes.Structure):
    _fields_ = [("order", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("dims", ctypes.c_int64 * 3), ("n", ctypes.c_int64 * 3),
                ("pos", ctypes.c_void_p * 3), ("crd", ctypes.c_void_p * 3), ("val", ctypes.c_void_p)]


class spws_options_t(ctypes.Structure):
    _fields_ = [("validate", ctypes.c_int32), ("ism_warp_cap", ctypes.c_int32), ("ism_cta_cap", ctypes.c_int32),
                ("dense_unit_outputs", ctypes.c_int32), ("dense_max_span", ctypes.c_int32),
                ("fallback_cap", ctypes.c_int32), ("dense_span_words_per_product", ctypes.c_float),
                ("outer_cap", ctypes.c_int32), ("reserved", ctypes.c_int32 * 4)]


class spws_stats_t(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int64), ("products", ctypes.c_int64), ("nnz", ctypes.c_int64),
                ("max_row_products", ctypes.c_int64), ("rows_per_class", ctypes.c_int64 * 10),
                ("dense_units", ctypes.c_int64), ("device_status", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("products_per_class", ctypes.c_int64 * 10), ("nnz_per_class", ctypes.c_int64 * 10),
                ("launches_symbolic", ctypes.c_int32), ("launches_numeric", ctypes.c_int32),
                ("dense_warp_rows", ctypes.c_int64), ("dense_warp_products", ctypes.c_int64),
                ("dense_warp_nnz", ctypes.c_int64), ("bitmap_bytes", ctypes.c_int64)]


class SpwsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib():
    """The loaded library; raises if libspws.so is missing (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2404_04541_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        T = ctypes.POINTER(spws_tensor_t)
        L.spws_create.argtypes = [ctypes.POINTER(vp)]
        L.spws_destroy.argtypes = [vp]
        L.spws_set_stream.argtypes = [vp, vp]
        L.spws_plan_create.argtypes = [vp, ctypes.c_char_p, ctypes.POINTER(i32), i32, i32,
                                       ctypes.POINTER(spws_options_t), ctypes.POINTER(vp)]
        L.spws_plan_create3.argtypes = L.spws_plan_create.argtypes
        L.spws_workspace_size3.argtypes = [vp, T, T, T, ctypes.POINTER(sz)]
        L.spws_symbolic3.argtypes = [vp, T, T, T, T, vp, sz, ctypes.POINTER(ctypes.c_int64)]
        L.spws_numeric3.argtypes = [vp, T, T, T, T, vp, sz]
        L.spws_plan_destroy.argtypes = [vp]
        L.spws_check_expression.argtypes = [ctypes.c_char_p, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.spws_workspace_size.argtypes = [vp, T, T, ctypes.POINTER(sz)]
        L.spws_workspace_size_exact.argtypes = [vp, T, T, vp, sz, ctypes.POINTER(sz), vp]
        L.spws_symbolic.argtypes = [vp, T, T, T, vp, sz, ctypes.POINTER(ctypes.c_int64)]
        L.spws_numeric.argtypes = [vp, T, T, T, vp, sz]
        L.spws_gather_ceiling.argtypes = [vp, T, T, T, vp, sz, vp, vp]
        L.spws_get_stats.argtypes = [vp, ctypes.POINTER(spws_stats_t)]
        L.spws_set_profiling.argtypes = [vp, i32]
        L.spws_get_timings.argtypes = [vp, ctypes.POINTER(ctypes.c_float), i32]
        L.spws_execute_host.argtypes = [vp, T, T, T, vp, sz, ctypes.POINTER(sz)]
        L.spws_row_pointer_static.argtypes = [vp, ctypes.c_int64, vp, vp]
        L.spws_status_string.argtypes = [i32]
        L.spws_status_string.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name != "spws_status_string":
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().spws_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != SPWS_OK:
        raise SpwsError(status, where)


def check_expression(expr: str, fmts) -> int:
    """Host-only classification; returns the status and does not raise."""
    arr = (ctypes.c_int * 3)(*fmts)
    kind = ctypes.c_int(-1)
    return lib().spws_check_expression(expr.encode(), arr, ctypes.byref(kind))


def row_pointer_static(counts_ptr: int, n: int, pos_ptr: int, stream_ptr: int | None = None) -> int:
    """spws_row_pointer_static: device pointers in, status out (does not raise).  The scan's
    scratch is a fixed array inside the library, so this call allocates nothing."""
    return lib().spws_row_pointer_static(ctypes.c_void_p(counts_ptr), int(n), ctypes.c_void_p(pos_ptr),
                                         ctypes.c_void_p(stream_ptr))


# ---------------------------------------------------------------------------- tensors
def _ptr(t):
    """Address of a torch tensor's (or numpy array's) storage, or None."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data if t.size else None
    return t.data_ptr() if t.numel() else None


@dataclass
class TensorArrays:
    """Level arrays of a CSR matrix (order 2) or CSF 3-tensor (order 3); torch tensors on the
    device, or numpy arrays for the host entry point."""
    order: int
    dims: tuple
    pos: list
    crd: list
    val: object
    n: list = field(default_factory=lambda: [0, 0, 0])

    def c_struct(self) -> spws_tensor_t:
        t = spws_tensor_t()
        t.order = self.order
        for a in range(3):
            t.dims[a] = int(self.dims[a]) if a < len(self.dims) else 0
            t.n[a] = int(self.n[a])
            t.pos[a] = _ptr(self.pos[a]) if a < len(self.pos) else None
            t.crd[a] = _ptr(self.crd[a]) if a < len(self.crd) else None
        t.val = _ptr(self.val)
        return t


def csr_arrays(nrows, ncols, pos, crd, val) -> TensorArrays:
    nnz = int(crd.shape[0]) if crd is not None else 0
    return TensorArrays(2, (nrows, ncols, 0), [None, pos, None], [None, crd, None], val, [nrows, nnz, 0])


def csf3_arrays(dims, pos0, crd0, pos1, crd1, pos2, crd2, val) -> TensorArrays:
    n = [int(crd0.shape[0]), int(crd1.shape[0]), int(crd2.shape[0]) if crd2 is not None else 0]
    return TensorArrays(3, tuple(dims), [pos0, pos1, pos2], [crd0, crd1, crd2], val, n)


# ---------------------------------------------------------------------------- handle / plan
class Handle:
    def __init__(self, stream_ptr: int | None = None):
        self._h = ctypes.c_void_p()
        _check(lib().spws_create(ctypes.byref(self._h)), "spws_create")
        if stream_ptr is not None:
            self.set_stream(stream_ptr)

    def set_stream(self, stream_ptr: int):
        _check(lib().spws_set_stream(self._h, ctypes.c_void_p(stream_ptr)), "spws_set_stream")

    def close(self):
        if self._h:
            lib().spws_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Plan:
    def __init__(self, handle: Handle, expr: str, fmts, dtype, policy="auto", **options):
        self.handle = handle
        self._p = ctypes.c_void_p()
        self.np_dtype = np.dtype(dtype)
        vt = SPWS_F64 if self.np_dtype == np.float64 else SPWS_F32
        if self.np_dtype not in (np.dtype(np.float32), np.dtype(np.float64)):
            raise SpwsError(SPWS_INVALID_ARGUMENT, "Plan: value type")
        opt = spws_options_t()
        for k, v in options.items():
            if not hasattr(opt, k):
                raise SpwsError(SPWS_INVALID_ARGUMENT, f"Plan: unknown option {k}")
            setattr(opt, k, v)
        arr = (ctypes.c_int * len(fmts))(*fmts)
        pol = POLICIES[policy] if isinstance(policy, str) else int(policy)
        create = lib().spws_plan_create3 if len(fmts) == 4 else lib().spws_plan_create
        _check(create(handle._h, expr.encode(), arr, vt, pol, ctypes.byref(opt), ctypes.byref(self._p)), "spws_plan_create")

    def workspace_size(self, A: TensorArrays, B: TensorArrays, D: TensorArrays | None = None) -> int:
        out = ctypes.c_size_t(0)
        a, b = A.c_struct(), B.c_struct()
        if D is None:
            _check(lib().spws_workspace_size(self._p, ctypes.byref(a), ctypes.byref(b), ctypes.byref(out)),
                   "spws_workspace_size")
        else:
            d = D.c_struct()
            _check(lib().spws_workspace_size3(self._p, ctypes.byref(a), ctypes.byref(b), ctypes.byref(d), ctypes.byref(out)),
                   "spws_workspace_size3")
        return int(out.value)

    def workspace_size_exact(self, A: TensorArrays, B: TensorArrays, scratch_ptr: int | None = None, scratch_bytes: int = 0,
                             row_products_ptr: int | None = None) -> int:
        """spws_workspace_size_exact: without a scratch pointer, the bytes the sizing call itself
        needs; with one, the bytes both passes really use (runs two kernels, synchronises)."""
        out = ctypes.c_size_t(0)
        a, b = A.c_struct(), B.c_struct()
        _check(lib().spws_workspace_size_exact(self._p, ctypes.byref(a), ctypes.byref(b), ctypes.c_void_p(scratch_ptr), scratch_bytes,
                                               ctypes.byref(out), ctypes.c_void_p(row_products_ptr)), "spws_workspace_size_exact")
        return int(out.value)

    def symbolic(self, A, B, C, scratch_ptr: int, scratch_bytes: int, D=None):
        a, b, c = A.c_struct(), B.c_struct(), C.c_struct()
        sizes = (ctypes.c_int64 * 3)()
        if D is None:
            _check(lib().spws_symbolic(self._p, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c),
                                       ctypes.c_void_p(scratch_ptr), scratch_bytes, sizes), "spws_symbolic")
        else:
            d = D.c_struct()
            _check(lib().spws_symbolic3(self._p, ctypes.byref(a), ctypes.byref(b), ctypes.byref(d), ctypes.byref(c),
                                        ctypes.c_void_p(scratch_ptr), scratch_bytes, sizes), "spws_symbolic3")
        C.n = [int(sizes[0]), int(sizes[1]), int(sizes[2])]
        return C.n

    def numeric(self, A, B, C, scratch_ptr: int, scratch_bytes: int, D=None):
        a, b, c = A.c_struct(), B.c_struct(), C.c_struct()
        if D is None:
            _check(lib().spws_numeric(self._p, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c),
                                      ctypes.c_void_p(scratch_ptr), scratch_bytes), "spws_numeric")
        else:
            d = D.c_struct()
            _check(lib().spws_numeric3(self._p, ctypes.byref(a), ctypes.byref(b), ctypes.byref(d), ctypes.byref(c),
                                       ctypes.c_void_p(scratch_ptr), scratch_bytes), "spws_numeric3")

    def gather_ceiling(self, A, B, C, scratch_ptr: int, scratch_bytes: int, index_sum_ptr: int, value_sum_ptr: int):
        """spws_gather_ceiling: the dense numeric kernels' traversal with the workspace stripped;
        the two device words receive the sum of the gathered column indices and of the products."""
        a, b, c = A.c_struct(), B.c_struct(), C.c_struct()
        _check(lib().spws_gather_ceiling(self._p, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c),
                                         ctypes.c_void_p(scratch_ptr), scratch_bytes, ctypes.c_void_p(index_sum_ptr),
                                         ctypes.c_void_p(value_sum_ptr)), "spws_gather_ceiling")

    def get_stats(self) -> dict:
        s = spws_stats_t()
        st = lib().spws_get_stats(self._p, ctypes.byref(s))
        d = dict(rows=s.rows, products=s.products, nnz=s.nnz, max_row_products=s.max_row_products,
                 rows_per_class=list(s.rows_per_class), dense_units=s.dense_units, device_status=s.device_status,
                 products_per_class=list(s.products_per_class), nnz_per_class=list(s.nnz_per_class),
                 launches_symbolic=s.launches_symbolic, launches_numeric=s.launches_numeric,
                 dense_warp_rows=s.dense_warp_rows, dense_warp_products=s.dense_warp_products,
                 dense_warp_nnz=s.dense_warp_nnz, bitmap_bytes=s.bitmap_bytes)
        _check(st, "spws_get_stats")
        return d

    def set_profiling(self, enabled: bool):
        _check(lib().spws_set_profiling(self._p, int(bool(enabled))), "spws_set_profiling")

    def get_timings(self) -> dict:
        ms = (ctypes.c_float * len(TIMING_GROUPS))()
        _check(lib().spws_get_timings(self._p, ms, len(TIMING_GROUPS)), "spws_get_timings")
        return {name: float(ms[g]) for g, name in enumerate(TIMING_GROUPS)}

    def execute_host(self, A: TensorArrays, B: TensorArrays, C: TensorArrays, arena_ptr: int, arena_bytes: int):
        """A, B, C hold numpy (ideally pinned) host arrays; returns (status, sizes, arena_needed)."""
        a, b, c = A.c_struct(), B.c_struct(), C.c_struct()
        need = ctypes.c_size_t(0)
        st = lib().spws_execute_host(self._p, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c),
                                     ctypes.c_void_p(arena_ptr), arena_bytes, ctypes.byref(need))
        return st, [int(c.n[0]), int(c.n[1]), int(c.n[2])], int(need.value)

    def close(self):
        if self._p:
            lib().spws_plan_destroy(self._p)
            self._p = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
