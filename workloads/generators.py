"""Seeded generators for the five benchmark configurations and for small test operands.

Recipes (all draws come from numpy's Philox bit generator keyed by the seed, single stream,
so the output does not depend on thread count):

* uniform rows   : every row gets exactly `d` distinct columns drawn uniformly; rows that drew
                   a repeated column are redrawn until none repeats; columns sorted per row.
* R-MAT          : `edge_factor * 2**scale` edges; each of the `scale` levels picks a quadrant
                   with probabilities (a, b, c, d) = (row bit 0/col bit 0, 0/1, 1/0, 1/1); no
                   noise, no vertex permutation, directed, self loops kept; duplicate edges are
                   removed; values are drawn after de-duplication.
* 27-point stencil: grid point (x, y, z) -> row x + n*(y + n*z); neighbours at offsets
                   {-1,0,1}^3 that stay inside the grid.
* uniform CSF    : `nnz` distinct linear coordinates in [0, I*J*K) drawn uniformly (collisions
                   redrawn), sorted, split into (i, j, k).

The SuiteSparse / FROSTT files the paper measures on are not used; these inputs stand in for
them.
"""
from __future__ import annotations

import numpy as np

from .formats import CSR, CSF3

CONFIG_NAMES = ("uniform8", "rmat18", "stencil64", "wide26", "ttm4096")


def _rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream)]))


def _values(rng: np.random.Generator, n: int, lo: float, hi: float, dtype) -> np.ndarray:
    out = np.empty(n, dtype=dtype)
    step = 1 << 24
    for s in range(0, n, step):
        e = min(n, s + step)
        out[s:e] = (lo + (hi - lo) * rng.random(e - s)).astype(dtype)
    return out


def uniform_rows_csr(nrows: int, ncols: int, d: int, seed: int, lo=-1.0, hi=1.0,
                     dtype=np.float64, stream: int = 0) -> CSR:
    """Exactly `d` distinct uniformly drawn columns in every row."""
    assert d <= ncols
    rng = _rng(seed, stream)
    crd = np.empty((nrows, d), dtype=np.int32)
    step = max(1, (1 << 24) // max(d, 1))
    for s in range(0, nrows, step):
        e = min(nrows, s + step)
        blk = rng.integers(0, ncols, size=(e - s, d), dtype=np.int32)
        blk.sort(axis=1)
        rounds = 0
        while d > 1:
            bad = np.nonzero((blk[:, 1:] == blk[:, :-1]).any(axis=1))[0]
            if bad.size == 0:
                break
            rounds += 1
            if rounds > 64:
                # d is close to ncols: redrawing would go on for ever; take the first d of a
                # random permutation of the columns instead
                redo = np.argsort(rng.random((bad.size, ncols)), axis=1)[:, :d].astype(np.int32)
            else:
                redo = rng.integers(0, ncols, size=(bad.size, d), dtype=np.int32)
            redo.sort(axis=1)
            blk[bad] = redo
        crd[s:e] = blk
    pos = np.arange(nrows + 1, dtype=np.int64) * d
    val = _values(rng, nrows * d, lo, hi, dtype)
    return CSR(nrows, ncols, pos, crd.reshape(-1), val)


def rmat_csr(scale: int, edge_factor: int, seed: int, abcd=(0.57, 0.19, 0.19, 0.05),
             lo=-1.0, hi=1.0, dtype=np.float64) -> CSR:
    rng = _rng(seed)
    n = 1 << scale
    ne = edge_factor * n
    a, b, c, _ = abcd
    rows = np.zeros(ne, dtype=np.int64)
    cols = np.zeros(ne, dtype=np.int64)
    for _level in range(scale):
        r = rng.random(ne)
        rbit = r >= (a + b)
        cbit = ((r >= a) & (r < a + b)) | (r >= a + b + c)
        rows = (rows << 1) | rbit
        cols = (cols << 1) | cbit
    key = np.unique((rows << scale) | cols)
    rows = key >> scale
    cols = key & (n - 1)
    counts = np.bincount(rows, minlength=n)
    pos = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(counts, out=pos[1:])
    val = _values(rng, key.shape[0], lo, hi, dtype)
    return CSR(n, n, pos, cols.astype(np.int32), val)


def stencil27_csr(n: int, seed: int, lo=0.5, hi=1.5, dtype=np.float64, ones: bool = False) -> CSR:
    rng = _rng(seed)
    g = np.arange(n, dtype=np.int64)
    z, y, x = np.meshgrid(g, g, g, indexing="ij")
    x, y, z = x.reshape(-1), y.reshape(-1), z.reshape(-1)
    N = n ** 3
    cols = np.full((N, 27), -1, dtype=np.int64)
    s = 0
    for dz in (-1, 0, 1):          # ascending column order: z major, then y, then x
        for dy in (-1, 0, 1):
            for dx in (-1, 0, 1):
                ok = ((x + dx >= 0) & (x + dx < n) & (y + dy >= 0) & (y + dy < n)
                      & (z + dz >= 0) & (z + dz < n))
                cols[ok, s] = ((x + dx) + n * ((y + dy) + n * (z + dz)))[ok]
                s += 1
    mask = cols >= 0
    counts = mask.sum(axis=1)
    pos = np.zeros(N + 1, dtype=np.int64)
    np.cumsum(counts, out=pos[1:])
    crd = cols[mask].astype(np.int32)
    nnz = crd.shape[0]
    val = np.ones(nnz, dtype=dtype) if ones else _values(rng, nnz, lo, hi, dtype)
    return CSR(N, N, pos, crd, val)


def uniform_csf3(dims, nnz: int, seed: int, lo=-1.0, hi=1.0, dtype=np.float64) -> CSF3:
    rng = _rng(seed)
    I, J, K = (int(d) for d in dims)
    total = I * J * K
    assert nnz <= total
    lin = np.unique(rng.integers(0, total, size=nnz, dtype=np.int64))
    while lin.shape[0] < nnz:
        extra = rng.integers(0, total, size=nnz - lin.shape[0], dtype=np.int64)
        lin = np.unique(np.concatenate([lin, extra]))
    i = lin // (J * K)
    j = (lin // K) % J
    k = lin % K
    val = _values(rng, nnz, lo, hi, dtype)
    return CSF3.from_coo((I, J, K), i, j, k, val, dtype=dtype)


def random_csr(nrows: int, ncols: int, density: float, seed: int, lo=-1.0, hi=1.0,
               dtype=np.float64, empty_row_frac: float = 0.0) -> CSR:
    """Bernoulli(density) pattern for small test operands; optionally blanks whole rows."""
    rng = _rng(seed)
    mask = rng.random((nrows, ncols)) < density
    if empty_row_frac > 0:
        mask[rng.random(nrows) < empty_row_frac, :] = False
    d = np.where(mask, lo + (hi - lo) * rng.random((nrows, ncols)), 0.0)
    return CSR.from_dense(d, dtype=dtype, keep_mask=mask)


def crossover_operands(I: int, K: int, J: int, live_k: int, per_k: int, seed: int, dtype=np.float64):
    """Operands of the dense-versus-sparse workspace sweeps (Sec. 7.2): `live_k` of the K
    coordinates of the contracted index are non-empty (drawn uniformly, distinct); each of them
    has `per_k` entries at distinct uniform positions in A (rows i) and in B (columns j).
    Returns (At, B): At is A by its rows k (K x I, CSR), B is K x J (CSR); values uniform in [-1,1]."""
    rng = _rng(seed)
    live = np.sort(rng.choice(K, size=live_k, replace=False))

    def side(width, stream_seed):
        r = _rng(stream_seed)
        n = min(per_k, width)
        crd = np.empty((live_k, n), dtype=np.int32)
        for x in range(live_k):
            crd[x] = np.sort(r.choice(width, size=n, replace=False))
        counts = np.zeros(K, dtype=np.int64)
        counts[live] = n
        pos = np.zeros(K + 1, dtype=np.int64)
        np.cumsum(counts, out=pos[1:])
        return CSR(K, width, pos, crd.reshape(-1), _values(r, live_k * n, -1.0, 1.0, dtype))

    return side(I, seed * 7919 + 1), side(J, seed * 7919 + 2)


def config_inputs(name: str, seed: int = 1, reduced: bool = False) -> dict:
    """Operands of one benchmark configuration.

    Returns {"kind": "spgemm"|"ttm", "A": ..., "B": ..., "dtype": np.dtype, "name": ...}.
    `reduced=True` keeps the shape of the structure but shrinks it so a CPU check runs in
    seconds (the column space of "wide26" stays 2**26).
    """
    if name == "uniform8":
        A = uniform_rows_csr(2048, 2048, 8, seed)
        return dict(kind="spgemm", A=A, B=A, dtype=np.float64, name=name)
    if name == "rmat18":
        A = rmat_csr(12 if reduced else 18, 16, seed)
        return dict(kind="spgemm", A=A, B=A, dtype=np.float64, name=name)
    if name == "stencil64":
        A = stencil27_csr(12 if reduced else 64, seed)
        return dict(kind="spgemm", A=A, B=A, dtype=np.float64, name=name)
    if name == "wide26":
        k = (1 << 14) if reduced else (1 << 26)
        m = (1 << 10) if reduced else (1 << 16)
        A = uniform_rows_csr(m, k, 4, seed, dtype=np.float32, stream=0)
        B = uniform_rows_csr(k, 1 << 26, 4, seed, dtype=np.float32, stream=1)
        return dict(kind="spgemm", A=A, B=B, dtype=np.float32, name=name)
    if name == "ttm4096":
        d = 256 if reduced else 4096
        nnz = (1 << 13) if reduced else (1 << 21)
        A = uniform_csf3((d, d, d), nnz, seed)
        B = uniform_rows_csr(d, d, 8, seed + 1000)
        return dict(kind="ttm", A=A, B=B, dtype=np.float64, name=name)
    # same recipes at other sizes (profiling captures need a smaller case): "rmat16", "stencil40"
    if name.startswith("rmat") and name[4:].isdigit():
        A = rmat_csr(int(name[4:]), 16, seed)
        return dict(kind="spgemm", A=A, B=A, dtype=np.float64, name=name)
    if name.startswith("stencil") and name[7:].isdigit():
        A = stencil27_csr(int(name[7:]), seed)
        return dict(kind="spgemm", A=A, B=A, dtype=np.float64, name=name)
    raise ValueError(f"unknown config {name!r}; choose from {CONFIG_NAMES}")
