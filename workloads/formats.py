"""Host containers for the level formats the path reads and writes (paper Fig. 4, Sec. 2.1).

CSR  = ({Dense, Compressed}, {i, k}):  pos[m+1] (int64), crd[nnz] (int32), val[nnz].
CSF3 = ({Compressed, Compressed, Compressed}, {i, j, k}): three compressed levels
       pos0[2], crd0[n_i], pos1[n_i+1], crd1[n_ij], pos2[n_ij+1], crd2[nnz], val[nnz];
       no level stores an empty fibre.

Canonical form: zero-based coordinates, strictly increasing inside every row / fibre.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class CSR:
    nrows: int
    ncols: int
    pos: np.ndarray   # int64 [nrows+1]
    crd: np.ndarray   # int32 [nnz]
    val: np.ndarray   # float32/float64 [nnz]

    @property
    def nnz(self) -> int:
        return int(self.pos[-1])

    def to_dense(self) -> np.ndarray:
        d = np.zeros((self.nrows, self.ncols), dtype=np.float64)
        rows = np.repeat(np.arange(self.nrows), np.diff(self.pos))
        np.add.at(d, (rows, self.crd), self.val.astype(np.float64))
        return d

    def pattern_dense(self) -> np.ndarray:
        d = np.zeros((self.nrows, self.ncols), dtype=bool)
        rows = np.repeat(np.arange(self.nrows), np.diff(self.pos))
        d[rows, self.crd] = True
        return d

    def transpose(self) -> "CSR":
        rows = np.repeat(np.arange(self.nrows, dtype=np.int64), np.diff(self.pos))
        order = np.lexsort((rows, self.crd))
        counts = np.bincount(self.crd, minlength=self.ncols)
        pos = np.zeros(self.ncols + 1, dtype=np.int64)
        np.cumsum(counts, out=pos[1:])
        return CSR(self.ncols, self.nrows, pos, rows[order].astype(np.int32), self.val[order].copy())

    def row_block(self, r0: int, r1: int) -> "CSR":
        """Rows [r0, r1) as a CSR of their own (same column space)."""
        p0, p1 = int(self.pos[r0]), int(self.pos[r1])
        return CSR(r1 - r0, self.ncols, (self.pos[r0:r1 + 1] - p0).astype(np.int64),
                   self.crd[p0:p1].copy(), self.val[p0:p1].copy())

    @staticmethod
    def from_dense(d: np.ndarray, dtype=np.float64, keep_mask: np.ndarray | None = None) -> "CSR":
        mask = (d != 0) if keep_mask is None else keep_mask
        m, n = d.shape
        counts = mask.sum(axis=1)
        pos = np.zeros(m + 1, dtype=np.int64)
        np.cumsum(counts, out=pos[1:])
        r, c = np.nonzero(mask)
        return CSR(m, n, pos, c.astype(np.int32), d[r, c].astype(dtype))

    @staticmethod
    def from_coo(m: int, n: int, rows, cols, vals, dtype=np.float64) -> "CSR":
        """Build from COO triples whose (row, col) pairs are already unique."""
        rows = np.asarray(rows, dtype=np.int64)
        cols = np.asarray(cols, dtype=np.int64)
        vals = np.asarray(vals)
        order = np.lexsort((cols, rows))
        counts = np.bincount(rows, minlength=m)
        pos = np.zeros(m + 1, dtype=np.int64)
        np.cumsum(counts, out=pos[1:])
        return CSR(m, n, pos, cols[order].astype(np.int32), vals[order].astype(dtype))


@dataclass
class CSF3:
    dims: tuple          # (I, J, K)
    pos0: np.ndarray     # int64 [2]
    crd0: np.ndarray     # int32 [n_i]
    pos1: np.ndarray     # int64 [n_i+1]
    crd1: np.ndarray     # int32 [n_ij]
    pos2: np.ndarray     # int64 [n_ij+1]
    crd2: np.ndarray     # int32 [nnz]
    val: np.ndarray

    @property
    def nnz(self) -> int:
        return int(self.pos2[-1])

    @property
    def n_i(self) -> int:
        return int(self.crd0.shape[0])

    @property
    def n_ij(self) -> int:
        return int(self.crd1.shape[0])

    def to_coo(self):
        i_of_ij = np.repeat(self.crd0, np.diff(self.pos1))
        i = np.repeat(i_of_ij, np.diff(self.pos2))
        j = np.repeat(self.crd1, np.diff(self.pos2))
        return i.astype(np.int64), j.astype(np.int64), self.crd2.astype(np.int64), self.val

    def to_dense(self) -> np.ndarray:
        d = np.zeros(self.dims, dtype=np.float64)
        i, j, k, v = self.to_coo()
        np.add.at(d, (i, j, k), v.astype(np.float64))
        return d

    def fibres_as_csr(self) -> CSR:
        """The (i,j) fibres as the rows of a CSR matrix (n_ij x K); shares the arrays."""
        return CSR(self.n_ij, int(self.dims[2]), self.pos2, self.crd2, self.val)

    @staticmethod
    def from_coo(dims, i, j, k, vals, dtype=np.float64) -> "CSF3":
        """Build from COO triples with unique (i,j,k)."""
        i = np.asarray(i, dtype=np.int64)
        j = np.asarray(j, dtype=np.int64)
        k = np.asarray(k, dtype=np.int64)
        vals = np.asarray(vals)
        order = np.lexsort((k, j, i))
        i, j, k, vals = i[order], j[order], k[order], vals[order]
        nnz = i.shape[0]
        if nnz == 0:
            z = np.zeros(0, dtype=np.int32)
            return CSF3(tuple(dims), np.zeros(2, np.int64), z, np.zeros(1, np.int64), z.copy(),
                        np.zeros(1, np.int64), z.copy(), np.zeros(0, dtype=dtype))
        new_ij = np.ones(nnz, dtype=bool)
        new_ij[1:] = (i[1:] != i[:-1]) | (j[1:] != j[:-1])
        ij_start = np.nonzero(new_ij)[0]
        pos2 = np.append(ij_start, nnz).astype(np.int64)
        crd1 = j[ij_start].astype(np.int32)
        i_of_ij = i[ij_start]
        new_i = np.ones(i_of_ij.shape[0], dtype=bool)
        new_i[1:] = i_of_ij[1:] != i_of_ij[:-1]
        i_start = np.nonzero(new_i)[0]
        pos1 = np.append(i_start, i_of_ij.shape[0]).astype(np.int64)
        crd0 = i_of_ij[i_start].astype(np.int32)
        pos0 = np.array([0, crd0.shape[0]], dtype=np.int64)
        return CSF3(tuple(dims), pos0, crd0, pos1, crd1, pos2, k.astype(np.int32), vals.astype(dtype))


def _level_is_canonical(pos: np.ndarray, crd: np.ndarray, dim: int, allow_empty: bool) -> bool:
    if pos.ndim != 1 or pos.shape[0] < 1 or pos[0] != 0 or pos[-1] != crd.shape[0]:
        return False
    lens = np.diff(pos)
    if (lens < 0).any() or (not allow_empty and (lens == 0).any()):
        return False
    if crd.shape[0] == 0:
        return True
    if crd.min() < 0 or crd.max() >= dim:
        return False
    inc = np.ones(crd.shape[0], dtype=bool)
    inc[1:] = crd[1:] > crd[:-1]
    starts = pos[:-1][lens > 0]
    inc[starts] = True
    return bool(inc.all())


def csr_is_canonical(a: CSR) -> bool:
    if a.pos.shape[0] != a.nrows + 1:
        return False
    return _level_is_canonical(a.pos, a.crd, a.ncols, allow_empty=True)


def csf3_is_canonical(t: CSF3) -> bool:
    if t.pos0.shape[0] != 2 or t.pos1.shape[0] != t.n_i + 1 or t.pos2.shape[0] != t.n_ij + 1:
        return False
    return (_level_is_canonical(t.pos0, t.crd0, t.dims[0], True)
            and _level_is_canonical(t.pos1, t.crd1, t.dims[1], False)
            and _level_is_canonical(t.pos2, t.crd2, t.dims[2], False))
