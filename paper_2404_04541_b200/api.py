"""Convenience layer over the binding: PyTorch allocates device memory and owns the stream, the
library does all the work.  There is no CPU or eager fallback: without the built library and a
CUDA device these calls raise.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from . import binding as B_

EXPR_SPGEMM = "C(i,j) = A(i,k) * B(k,j)"
EXPR_TTM = "C(i,j,l) = A(i,j,k) * B(k,l)"
EXPR_OUTER = "C(i,j) = A(k,i) * B(k,j)"
EXPR_SPTTM = "A(i,j,l) = B(k,i,j) * C(k,l)"
EXPR_SPTTM_I = "A(k,j,l) = B(k,i,j) * C(i,l)"
EXPR_SPMTTKRP = "A(i,j) = B(k,l,i) * C(k,j) * D(l,j)"


def _dev(a, dtype, device):
    if isinstance(a, torch.Tensor):
        return a.to(device=device, dtype=dtype).contiguous()
    return torch.from_numpy(np.ascontiguousarray(a)).to(device=device, dtype=dtype)


@dataclass
class DeviceCSR:
    nrows: int
    ncols: int
    pos: torch.Tensor
    crd: torch.Tensor
    val: torch.Tensor

    @property
    def nnz(self):
        return int(self.crd.shape[0])

    def arrays(self) -> B_.TensorArrays:
        return B_.csr_arrays(self.nrows, self.ncols, self.pos, self.crd, self.val)

    @staticmethod
    def from_host(M, device="cuda", dtype=None) -> "DeviceCSR":
        vt = torch.float64 if np.dtype(dtype or M.val.dtype) == np.float64 else torch.float32
        return DeviceCSR(M.nrows, M.ncols, _dev(M.pos, torch.int64, device), _dev(M.crd, torch.int32, device),
                         _dev(M.val, vt, device))


@dataclass
class DeviceCSF3:
    dims: tuple
    pos0: torch.Tensor
    crd0: torch.Tensor
    pos1: torch.Tensor
    crd1: torch.Tensor
    pos2: torch.Tensor
    crd2: torch.Tensor
    val: torch.Tensor

    def arrays(self) -> B_.TensorArrays:
        return B_.csf3_arrays(self.dims, self.pos0, self.crd0, self.pos1, self.crd1, self.pos2, self.crd2, self.val)

    @staticmethod
    def from_host(T, device="cuda") -> "DeviceCSF3":
        vt = torch.float64 if np.dtype(T.val.dtype) == np.float64 else torch.float32
        i64, i32 = torch.int64, torch.int32
        return DeviceCSF3(tuple(T.dims), _dev(T.pos0, i64, device), _dev(T.crd0, i32, device), _dev(T.pos1, i64, device),
                          _dev(T.crd1, i32, device), _dev(T.pos2, i64, device), _dev(T.crd2, i32, device),
                          _dev(T.val, vt, device))


class Context:
    """A library handle bound to torch's current stream on one device."""

    def __init__(self, device="cuda"):
        if not torch.cuda.is_available():
            raise RuntimeError("spws needs a CUDA device; there is no CPU path")
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.handle = B_.Handle(torch.cuda.current_stream(self.device).cuda_stream)
        self._scratch = None

    def plan(self, expr, fmts, dtype, policy="auto", **options) -> B_.Plan:
        return B_.Plan(self.handle, expr, fmts, dtype, policy, **options)

    def exact_scratch_bytes(self, plan: B_.Plan, a: B_.TensorArrays, b: B_.TensorArrays, row_products: torch.Tensor | None = None) -> int:
        """Bytes the two passes really use for these operands (one sizing pass on the device; the
        result is remembered per plan and operand pair).  `row_products` (int64, one per row)
        receives the per-row product counts when given."""
        ptrs = lambda t: tuple(x.data_ptr() for x in list(t.pos) + list(t.crd) if x is not None)
        key = (ptrs(a), ptrs(b), tuple(a.n), tuple(b.n))
        cache = plan.__dict__.setdefault("_exact_bytes", {})
        if key in cache and row_products is None:
            return cache[key]
        own = plan.workspace_size_exact(a, b)
        sc = self.scratch(own)
        cache[key] = plan.workspace_size_exact(a, b, self._aligned_ptr(sc), own,
                                               row_products.data_ptr() if row_products is not None else None)
        return cache[key]

    def scratch(self, nbytes: int) -> torch.Tensor:
        if self._scratch is None or self._scratch.numel() < nbytes:
            self._scratch = None
            self._scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        return self._scratch

    @staticmethod
    def _aligned_ptr(t: torch.Tensor) -> int:
        return (t.data_ptr() + 255) & ~255

    # ------------------------------------------------------------------ SpGEMM
    def spgemm_symbolic(self, plan: B_.Plan, A: DeviceCSR, B: DeviceCSR):
        a, b = A.arrays(), B.arrays()
        nbytes = self.exact_scratch_bytes(plan, a, b)
        sc = self.scratch(nbytes)
        pos = torch.empty(A.nrows + 1, dtype=torch.int64, device=self.device)
        c = B_.csr_arrays(A.nrows, B.ncols, pos, None, None)
        plan.symbolic(a, b, c, self._aligned_ptr(sc), nbytes)
        return c, (a, b, sc, nbytes)

    def spgemm_numeric(self, plan: B_.Plan, c: B_.TensorArrays, state, crd=None, val=None) -> DeviceCSR:
        a, b, sc, nbytes = state
        nnz = c.n[1]
        vt = torch.float64 if plan.np_dtype == np.float64 else torch.float32
        c.crd[1] = crd if crd is not None else torch.empty(nnz, dtype=torch.int32, device=self.device)
        c.val = val if val is not None else torch.empty(nnz, dtype=vt, device=self.device)
        plan.numeric(a, b, c, self._aligned_ptr(sc), nbytes)
        return DeviceCSR(int(c.dims[0]), int(c.dims[1]), c.pos[1], c.crd[1][:nnz], c.val[:nnz])

    def gather_ceiling(self, plan: B_.Plan, c: B_.TensorArrays, state):
        """Runs the gather-only form of the dense numeric kernels after a symbolic pass; returns
        (sum of gathered column indices, sum of products) as Python numbers."""
        a, b, sc, nbytes = state[:4]
        sums = torch.zeros(2, dtype=torch.int64, device=self.device)
        plan.gather_ceiling(a, b, c, self._aligned_ptr(sc), nbytes, sums.data_ptr(), sums.data_ptr() + 8)
        torch.cuda.synchronize(self.device)
        return int(sums[0].item()), float(sums[1:].view(torch.float64).item())

    def spgemm(self, A: DeviceCSR, B: DeviceCSR, policy="auto", plan: B_.Plan | None = None, **options):
        """C = A*B in CSR; returns (C, stats)."""
        own = plan is None
        if own:
            dt = np.float64 if A.val.dtype == torch.float64 else np.float32
            plan = self.plan(EXPR_SPGEMM, (B_.SPWS_CSR,) * 3, dt, policy, **options)
        try:
            c, state = self.spgemm_symbolic(plan, A, B)
            C = self.spgemm_numeric(plan, c, state)
            return C, plan.get_stats()
        finally:
            if own:
                plan.close()

    # ------------------------------------------------------------------ outer-product SpGEMM
    def outer_symbolic(self, plan: B_.Plan, At: DeviceCSR, B: DeviceCSR):
        """Symbolic pass of C(i,j) = sum_k A(k,i) B(k,j); `At` holds A by its rows k (K x I)."""
        a, b = At.arrays(), B.arrays()
        nbytes = plan.workspace_size(a, b)          # counts the products on the device
        sc = self.scratch(nbytes)
        pos = torch.empty(At.ncols + 1, dtype=torch.int64, device=self.device)
        c = B_.csr_arrays(At.ncols, B.ncols, pos, None, None)
        plan.symbolic(a, b, c, self._aligned_ptr(sc), nbytes)
        return c, (a, b, sc, nbytes)

    def spgemm_outer(self, At: DeviceCSR, B: DeviceCSR, policy="auto", plan: B_.Plan | None = None, **options):
        """C = A^T-stored-by-rows times B through a second-order workspace; returns (C, stats)."""
        own = plan is None
        if own:
            dt = np.float64 if At.val.dtype == torch.float64 else np.float32
            plan = self.plan(EXPR_OUTER, (B_.SPWS_CSR,) * 3, dt, policy, **options)
        try:
            c, state = self.outer_symbolic(plan, At, B)
            C = self.spgemm_numeric(plan, c, state)
            return C, plan.get_stats()
        finally:
            if own:
                plan.close()

    # ------------------------------------------------------------------ higher-order scatters, COO result
    def scatter_coo(self, expr: str, T: DeviceCSF3, C: DeviceCSR, D: DeviceCSR | None = None, policy="auto", **options):
        """One of the higher-order scatters (EXPR_SPTTM, EXPR_SPTTM_I, EXPR_SPMTTKRP): CSF tensor
        times one or two CSR matrices, sparse result in coordinate form.  Returns
        (crd [nnz, order] int32, val [nnz], stats)."""
        dt = np.float64 if T.val.dtype == torch.float64 else np.float32
        fmts = (B_.SPWS_COO, B_.SPWS_CSF3, B_.SPWS_CSR) + ((B_.SPWS_CSR,) if D is not None else ())
        plan = self.plan(expr, fmts, dt, policy, **options)
        try:
            t, c = T.arrays(), C.arrays()
            d = D.arrays() if D is not None else None
            nbytes = plan.workspace_size(t, c, d)
            sc = self.scratch(nbytes)
            if expr == EXPR_SPMTTKRP:
                order, dims = 2, (T.dims[2], C.ncols, 0)
            elif expr == EXPR_SPTTM:
                order, dims = 3, (T.dims[1], T.dims[2], C.ncols)
            else:
                order, dims = 3, (T.dims[0], T.dims[2], C.ncols)
            out = B_.TensorArrays(order, dims, [None, None, None], [None, None, None], None, [0, 0, 0])
            nnz = plan.symbolic(t, c, out, self._aligned_ptr(sc), nbytes, D=d)[0]
            crd = [torch.empty(nnz, dtype=torch.int32, device=self.device) for _ in range(order)]
            out.crd = crd + [None] * (3 - order)
            out.val = torch.empty(nnz, dtype=T.val.dtype, device=self.device)
            out.n = [nnz, 0, 0]
            plan.numeric(t, c, out, self._aligned_ptr(sc), nbytes, D=d)
            return torch.stack(crd, dim=1) if nnz else torch.empty((0, order), dtype=torch.int32, device=self.device), out.val, plan.get_stats()
        finally:
            plan.close()

    # ------------------------------------------------------------------ TTM
    def ttm_symbolic(self, plan: B_.Plan, A: DeviceCSF3, B: DeviceCSR):
        """Symbolic pass of the 3-tensor form: allocates C's upper levels (bounded by A's) and returns
        (C arrays with sizes filled in, state for ttm_numeric)."""
        a, b = A.arrays(), B.arrays()
        nbytes = self.exact_scratch_bytes(plan, a, b)
        sc = self.scratch(nbytes)
        n_i, n_ij = a.n[0], a.n[1]
        i64, i32, dev = torch.int64, torch.int32, self.device
        pos0 = torch.empty(2, dtype=i64, device=dev)
        crd0 = torch.empty(n_i, dtype=i32, device=dev)
        pos1 = torch.empty(n_i + 1, dtype=i64, device=dev)
        crd1 = torch.empty(n_ij, dtype=i32, device=dev)
        pos2 = torch.empty(n_ij + 1, dtype=i64, device=dev)
        c = B_.TensorArrays(3, (A.dims[0], A.dims[1], B.ncols), [pos0, pos1, pos2], [crd0, crd1, None], None,
                            [n_i, n_ij, 0])
        sizes = plan.symbolic(a, b, c, self._aligned_ptr(sc), nbytes)
        return c, (a, b, sc, nbytes, sizes)

    def ttm_numeric(self, plan: B_.Plan, c: B_.TensorArrays, state, crd=None, val=None) -> DeviceCSF3:
        a, b, sc, nbytes, sizes = state
        nnz = sizes[2]
        vt = torch.float64 if plan.np_dtype == np.float64 else torch.float32
        c.crd[2] = crd if crd is not None else torch.empty(nnz, dtype=torch.int32, device=self.device)
        c.val = val if val is not None else torch.empty(nnz, dtype=vt, device=self.device)
        plan.numeric(a, b, c, self._aligned_ptr(sc), nbytes)
        return DeviceCSF3(c.dims, c.pos[0], c.crd[0][:sizes[0]], c.pos[1][:sizes[0] + 1], c.crd[1][:sizes[1]],
                          c.pos[2][:sizes[1] + 1], c.crd[2][:nnz], c.val[:nnz])

    def ttm(self, A: DeviceCSF3, B: DeviceCSR, policy="auto", plan: B_.Plan | None = None, **options):
        """C(i,j,l) = sum_k A(i,j,k) B(k,l) with A, C in CSF; returns (C, stats)."""
        own = plan is None
        if own:
            dt = np.float64 if A.val.dtype == torch.float64 else np.float32
            plan = self.plan(EXPR_TTM, (B_.SPWS_CSF3, B_.SPWS_CSF3, B_.SPWS_CSR), dt, policy, **options)
        try:
            c, state = self.ttm_symbolic(plan, A, B)
            C = self.ttm_numeric(plan, c, state)
            return C, plan.get_stats()
        finally:
            if own:
                plan.close()
