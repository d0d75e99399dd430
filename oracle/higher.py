"""TEST INFRASTRUCTURE ONLY -- oracle of the paper's higher-order scatters (Sec. 7.3).

Plain definitions, one Python loop nest each in the loop order the paper writes, every product
accumulated into a dictionary keyed by the output coordinate (the map-per-result workspace),
emitted in lexicographic coordinate order.  For small operands only.

  spttm     : A(i,j,l) = sum_k  B(k,i,j) * C(k,l)          loops k -> i -> j -> l
  spttm_i   : A(k,j,l) = sum_i  B(k,i,j) * C(i,l)          loops k -> i -> j -> l
  spmttkrp  : A(i,j)   = sum_kl B(k,l,i) * C(k,j) * D(l,j) loops k -> l -> i -> j

B is a CSF 3-tensor stored in the order its indices are written; C and D are CSR.  An output
entry exists when at least one product lands on it (a sum that happens to be 0.0 is kept).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np


@dataclass
class CooResult:
    crd: np.ndarray        # int64 [nnz, order], rows sorted lexicographically, unique
    val: np.ndarray        # float64: sum in loop order, multiply then add
    val_ref: np.ndarray    # float64: exactly rounded sum of the exactly rounded products' doubles (math.fsum)
    abs: np.ndarray        # float64: sum of |product|
    products: int

    @property
    def nnz(self) -> int:
        return int(self.crd.shape[0])


def _emit(acc: dict, order: int, products: int) -> CooResult:
    keys = sorted(acc)
    crd = np.array(keys, dtype=np.int64).reshape(len(keys), order)
    val = np.array([acc[k][0] for k in keys], dtype=np.float64)
    ref = np.array([math.fsum(acc[k][1]) for k in keys], dtype=np.float64)
    ab = np.array([math.fsum(abs(x) for x in acc[k][1]) for k in keys], dtype=np.float64)
    return CooResult(crd, val, ref, ab, products)


def _add(acc: dict, key, prod: float):
    cell = acc.get(key)
    if cell is None:
        acc[key] = [0.0 + prod, [prod]]
    else:
        cell[0] += prod
        cell[1].append(prod)


def _entries(T):
    """(c0, c1, c2, value) of a CSF 3-tensor in storage order."""
    for s in range(T.n_i):
        for f in range(int(T.pos1[s]), int(T.pos1[s + 1])):
            for e in range(int(T.pos2[f]), int(T.pos2[f + 1])):
                yield int(T.crd0[s]), int(T.crd1[f]), int(T.crd2[e]), float(T.val[e])


def _row(M, r):
    s, e = int(M.pos[r]), int(M.pos[r + 1])
    return M.crd[s:e], M.val[s:e]


def spttm(B, C) -> CooResult:
    acc, n = {}, 0
    for k, i, j, b in _entries(B):
        cols, vals = _row(C, k)
        for l, c in zip(cols, vals):
            _add(acc, (i, j, int(l)), b * float(c))
            n += 1
    return _emit(acc, 3, n)


def spttm_i(B, C) -> CooResult:
    acc, n = {}, 0
    for k, i, j, b in _entries(B):
        cols, vals = _row(C, i)
        for l, c in zip(cols, vals):
            _add(acc, (k, j, int(l)), b * float(c))
            n += 1
    return _emit(acc, 3, n)


def spmttkrp(B, C, D) -> CooResult:
    acc, n = {}, 0
    for k, l, i, b in _entries(B):
        ccols, cvals = _row(C, k)
        dcols, dvals = _row(D, l)
        d_at = {int(j): float(v) for j, v in zip(dcols, dvals)}
        for j, c in zip(ccols, cvals):
            d = d_at.get(int(j))
            if d is None:
                continue
            _add(acc, (i, int(j)), (b * float(c)) * d)
            n += 1
    return _emit(acc, 2, n)
