"""ctypes front end of the CPU oracle (test infrastructure only; never on the product path).

Operands are the host containers of `workloads.formats`; values of any float type are widened
to float64 before the call (exact), the oracle computes in double / long double.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile oracle.cpp into liboracle.so (g++, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
               _SRC, "-o", _LIB]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        lib.oracle_spgemm.restype = vp
        lib.oracle_spgemm.argtypes = [i64, vp, vp, vp, vp, vp, vp, vp, i64, i32]
        lib.oracle_ttm.restype = vp
        lib.oracle_ttm.argtypes = [i64, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_ism_rowwise.restype = vp
        lib.oracle_ism_rowwise.argtypes = [i64, vp, vp, vp, vp, vp, vp, i64]
        lib.oracle_ism_outer.restype = vp
        lib.oracle_ism_outer.argtypes = [i64, i64, vp, vp, vp, vp, vp, vp, i64]
        lib.oracle_size.restype = i64
        lib.oracle_size.argtypes = [vp, i32]
        lib.oracle_copy.restype = None
        lib.oracle_copy.argtypes = [vp, i32, vp]
        lib.oracle_free.restype = None
        lib.oracle_free.argtypes = [vp]
        lib.oracle_hardware_threads.restype = i32
        _lib = lib
    return _lib


def hardware_threads() -> int:
    return int(_load().oracle_hardware_threads())


def _p(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _csr_args(M):
    pos = np.ascontiguousarray(M.pos, dtype=np.int64)
    crd = np.ascontiguousarray(M.crd, dtype=np.int32)
    val = np.ascontiguousarray(M.val, dtype=np.float64)
    return pos, crd, val


def _fetch(lib, h, what, n, dtype):
    out = np.empty(int(n), dtype=dtype)
    if n:
        lib.oracle_copy(h, what, _p(out))
    return out


@dataclass
class SpgemmResult:
    pos: np.ndarray        # int64 [rows+1]
    crd: np.ndarray        # int32 [nnz], sorted and unique inside each row
    val: np.ndarray        # float64: sum in loop order
    val_ref: np.ndarray    # float64: long-double accumulation rounded once
    abs: np.ndarray        # float64: sum |a*b| per entry
    products: np.ndarray   # int64 [rows]: intermediate products per row

    @property
    def nnz(self) -> int:
        return int(self.pos[-1])


@dataclass
class TtmResult:
    pos0: np.ndarray
    crd0: np.ndarray
    pos1: np.ndarray
    crd1: np.ndarray
    pos2: np.ndarray
    crd2: np.ndarray
    val: np.ndarray
    val_ref: np.ndarray
    abs: np.ndarray
    products: np.ndarray   # per input (i,j) fibre

    @property
    def nnz(self) -> int:
        return int(self.pos2[-1])


def _collect_csr(lib, h) -> SpgemmResult:
    try:
        nnz = lib.oracle_size(h, 1)
        return SpgemmResult(
            pos=_fetch(lib, h, 0, lib.oracle_size(h, 0), np.int64),
            crd=_fetch(lib, h, 1, nnz, np.int32),
            val=_fetch(lib, h, 2, nnz, np.float64),
            val_ref=_fetch(lib, h, 3, nnz, np.float64),
            abs=_fetch(lib, h, 4, lib.oracle_size(h, 6), np.float64),
            products=_fetch(lib, h, 5, lib.oracle_size(h, 2), np.int64),
        )
    finally:
        lib.oracle_free(h)


def spgemm(A, B, rows=None, threads: int = 1) -> SpgemmResult:
    """C = A*B row by row with an ordered-map workspace; `rows` selects output rows."""
    lib = _load()
    assert A.ncols == B.nrows
    a, b = _csr_args(A), _csr_args(B)
    if rows is None:
        rp, n_sel = None, 0
    else:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        rp, n_sel = _p(rows), rows.shape[0]
    h = lib.oracle_spgemm(A.nrows, _p(a[0]), _p(a[1]), _p(a[2]), _p(b[0]), _p(b[1]), _p(b[2]),
                          rp, n_sel, int(threads))
    return _collect_csr(lib, h)


def ttm(A, B) -> TtmResult:
    """C(i,j,l) = sum_k A(i,j,k) B(k,l); A, C in CSF, B in CSR."""
    lib = _load()
    assert A.dims[2] == B.nrows
    crd0 = np.ascontiguousarray(A.crd0, dtype=np.int32)
    pos1 = np.ascontiguousarray(A.pos1, dtype=np.int64)
    crd1 = np.ascontiguousarray(A.crd1, dtype=np.int32)
    pos2 = np.ascontiguousarray(A.pos2, dtype=np.int64)
    crd2 = np.ascontiguousarray(A.crd2, dtype=np.int32)
    val = np.ascontiguousarray(A.val, dtype=np.float64)
    b = _csr_args(B)
    h = lib.oracle_ttm(A.n_i, _p(crd0), _p(pos1), _p(crd1), _p(pos2), _p(crd2), _p(val),
                       _p(b[0]), _p(b[1]), _p(b[2]))
    try:
        nnz = lib.oracle_size(h, 1)
        return TtmResult(
            pos0=_fetch(lib, h, 6, 2, np.int64),
            crd0=_fetch(lib, h, 7, lib.oracle_size(h, 3), np.int32),
            pos1=_fetch(lib, h, 8, lib.oracle_size(h, 5), np.int64),
            crd1=_fetch(lib, h, 9, lib.oracle_size(h, 4), np.int32),
            pos2=_fetch(lib, h, 0, lib.oracle_size(h, 0), np.int64),
            crd2=_fetch(lib, h, 1, nnz, np.int32),
            val=_fetch(lib, h, 2, nnz, np.float64),
            val_ref=_fetch(lib, h, 3, nnz, np.float64),
            abs=_fetch(lib, h, 4, nnz, np.float64),
            products=_fetch(lib, h, 5, lib.oracle_size(h, 2), np.int64),
        )
    finally:
        lib.oracle_free(h)


def ism_rowwise(A, B, cap: int) -> SpgemmResult:
    """Algorithm 1 with a first-order Coord workspace of capacity `cap` per output row."""
    lib = _load()
    a, b = _csr_args(A), _csr_args(B)
    h = lib.oracle_ism_rowwise(A.nrows, _p(a[0]), _p(a[1]), _p(a[2]), _p(b[0]), _p(b[1]), _p(b[2]), int(cap))
    return _collect_csr(lib, h)


def ism_outer(A, B, cap: int) -> SpgemmResult:
    """Algorithm 1 with a second-order Coord workspace, loop order k -> i -> j (A by columns)."""
    lib = _load()
    At = A.transpose()
    a, b = _csr_args(At), _csr_args(B)
    h = lib.oracle_ism_outer(A.nrows, A.ncols, _p(a[0]), _p(a[1]), _p(a[2]), _p(b[0]), _p(b[1]), _p(b[2]), int(cap))
    return _collect_csr(lib, h)
