"""Pins for the CPU oracle: hand-worked cases, brute force, closed forms, invariants, a library
cross-check and the step-by-step Algorithm 1 restatements.  None of these retype the oracle's
own loop; each would fail for a plausible slip in it (dropped term, wrong index, transposed
operand, lost duplicate, pruned zero, unsorted row).
"""
import os

import numpy as np
import pytest
import scipy.sparse as sp

from helpers import GOLDEN, read_hand_case, rows_of
from workloads import (CSR, CSF3, csr_is_canonical, csf3_is_canonical, random_csr, rmat_csr,
                       stencil27_csr, uniform_rows_csr, uniform_csf3, config_inputs)


def dense_of(res, ncols):
    d = np.zeros((res.pos.shape[0] - 1, ncols))
    d[rows_of(res.pos), res.crd] = res.val_ref
    return d


def check_sorted_unique(pos, crd):
    inc = np.ones(crd.shape[0], dtype=bool)
    inc[1:] = crd[1:] > crd[:-1]
    inc[pos[:-1][np.diff(pos) > 0]] = True
    assert inc.all()


# ---------------------------------------------------------------- hand-worked cases
@pytest.mark.parametrize("name", ["hand_dedupe_4x4.txt", "hand_cancel_4x4.txt", "hand_rect_3x5x4.txt"])
def test_hand_cases(oracle_mod, name):
    A, B, cr, cc, cv, products = read_hand_case(name)
    res = oracle_mod.spgemm(A, B)
    assert np.array_equal(rows_of(res.pos), cr)
    assert np.array_equal(res.crd, cc)
    assert np.array_equal(res.val, cv)          # small integers / halves: exact
    assert np.array_equal(res.val_ref, cv)
    assert np.array_equal(res.products, products)


def test_cancelled_entry_is_kept(oracle_mod):
    A, B, cr, cc, cv, _ = read_hand_case("hand_cancel_4x4.txt")
    res = oracle_mod.spgemm(A, B)
    hit = (rows_of(res.pos) == 1) & (res.crd == 3)
    assert hit.sum() == 1 and res.val[hit][0] == 0.0
    assert res.abs[hit][0] == 6.0               # |2*1.5| + |-3*1|


# ---------------------------------------------------------------- brute force, tiny
def test_exhaustive_2x2_and_3x3_patterns(oracle_mod):
    """All 256 pairs of 2x2 0/1 matrices and all 512 x 512 pairs of 3x3 ones, each size run as one
    block-diagonal problem; expected = integer matmul of the patterns."""
    for n in (2, 3):
        codes = np.arange(1 << (n * n))
        ca, cb = np.meshgrid(codes, codes, indexing="ij")
        ca, cb = ca.reshape(-1), cb.reshape(-1)
        bits = np.arange(n * n)
        Ad = ((ca[:, None] >> bits) & 1).reshape(-1, n, n)
        Bd = ((cb[:, None] >> bits) & 1).reshape(-1, n, n)
        Cd = Ad @ Bd                                  # exact small integers
        nb = Ad.shape[0]

        def blockdiag(X):
            b, r, c = np.nonzero(X)
            return CSR.from_coo(nb * n, nb * n, b * n + r, b * n + c, X[b, r, c].astype(float))

        res = oracle_mod.spgemm(blockdiag(Ad), blockdiag(Bd))
        b, r, c = np.nonzero(Cd)                      # 0/1 inputs: no cancellation
        assert np.array_equal(rows_of(res.pos), b * n + r)
        assert np.array_equal(res.crd, b * n + c)
        assert np.array_equal(res.val, Cd[b, r, c].astype(float))


@pytest.mark.parametrize("m,k,n,dens,seed", [(1, 1, 1, 1.0, 0), (5, 7, 3, 0.5, 1), (16, 16, 16, 0.2, 2),
                                             (33, 64, 47, 0.1, 3), (64, 64, 64, 0.3, 4), (64, 20, 64, 0.9, 5),
                                             (8, 8, 8, 0.0, 6)])
def test_bruteforce_dense(oracle_mod, m, k, n, dens, seed):
    A = random_csr(m, k, dens, seed, empty_row_frac=0.2)
    B = random_csr(k, n, dens, seed + 100, empty_row_frac=0.2)
    res = oracle_mod.spgemm(A, B)
    # structure = boolean product of the structures (integer matmul of patterns)
    pat = (A.pattern_dense().astype(np.int64) @ B.pattern_dense().astype(np.int64)) > 0
    got = np.zeros((m, n), dtype=bool)
    got[rows_of(res.pos), res.crd] = True
    assert np.array_equal(got, pat)
    assert res.nnz == pat.sum()
    check_sorted_unique(res.pos, res.crd)
    # values: triple loop in a different order (j outer, k inner) via a dense product
    Ad, Bd = A.to_dense(), B.to_dense()
    ref = np.einsum("ik,kj->ij", Ad, Bd)
    scale = np.abs(Ad) @ np.abs(Bd)
    for v in (res.val, res.val_ref):
        d = np.zeros((m, n))
        d[rows_of(res.pos), res.crd] = v
        assert (np.abs(d - ref) <= 1e-14 * scale + 1e-300).all()
    dabs = np.zeros((m, n))
    dabs[rows_of(res.pos), res.crd] = res.abs
    assert np.allclose(dabs, scale * pat, rtol=1e-13, atol=0)
    # products per row = sum over A's entries of the length of the B row they pick
    blen = np.diff(B.pos)
    exp = np.array([blen[A.crd[A.pos[i]:A.pos[i + 1]]].sum() for i in range(m)], dtype=np.int64)
    assert np.array_equal(res.products, exp)


# ---------------------------------------------------------------- closed forms
def _stencil_forms():
    rows = []
    with open(os.path.join(GOLDEN, "stencil_closed_forms.txt")) as f:
        for line in f:
            if line.startswith("n "):
                rows.append(tuple(int(t) for t in line.split()[1:]))
    return rows


@pytest.mark.parametrize("form", [r for r in _stencil_forms() if r[0] <= 12])
def test_stencil_closed_forms(oracle_mod, form):
    n, nnzA, P, nnzC, span = form
    A = stencil27_csr(n, 0, ones=True)
    assert A.nnz == nnzA == (3 * n - 2) ** 3
    res = oracle_mod.spgemm(A, A)
    assert res.products.sum() == P == (9 * n - 10) ** 3
    assert res.nnz == nnzC == (5 * n - 6) ** 3
    c = n // 2
    i = c + n * (c + n * c)                              # an interior grid point
    seg = slice(res.pos[i], res.pos[i + 1])
    assert res.products[i] == 729 and res.pos[i + 1] - res.pos[i] == 125
    assert res.crd[seg][-1] - res.crd[seg][0] + 1 == span
    # all-ones values: C = kron(T2, T2, T2), T2 = square of the 1-D tridiagonal pattern
    T = (np.abs(np.subtract.outer(np.arange(n), np.arange(n))) <= 1).astype(float)
    T2 = T @ T
    assert list(T2[c, c - 2:c + 3]) == [1, 2, 3, 2, 1]
    rr = rows_of(res.pos)
    x, y, z = rr % n, (rr // n) % n, rr // (n * n)
    xx, yy, zz = res.crd % n, (res.crd // n) % n, res.crd // (n * n)
    assert np.array_equal(res.val, T2[x, xx] * T2[y, yy] * T2[z, zz])


def test_full_size_stencil_generator_counts():
    n, nnzA, _, _, _ = [r for r in _stencil_forms() if r[0] == 64][0]
    A = stencil27_csr(64, 1)
    assert A.nnz == nnzA and csr_is_canonical(A)
    assert A.val.min() >= 0.5 and A.val.max() <= 1.5


def test_uniform_and_wide_closed_forms(oracle_mod):
    c = config_inputs("uniform8")
    res = oracle_mod.spgemm(c["A"], c["B"])
    assert res.products.sum() == 2048 * 64 and (res.products == 64).all()
    w = config_inputs("wide26", reduced=True)
    res = oracle_mod.spgemm(w["A"], w["B"])
    assert (res.products == 16).all()
    assert res.crd.max() < (1 << 26) and res.crd.max() > (1 << 24)   # really spread over 2^26 columns


# ---------------------------------------------------------------- invariants
def test_identity_and_permutation(oracle_mod):
    A = random_csr(40, 40, 0.15, 11, empty_row_frac=0.1)
    eye = CSR.from_coo(40, 40, np.arange(40), np.arange(40), np.ones(40))
    res = oracle_mod.spgemm(A, eye)
    assert np.array_equal(res.pos, A.pos) and np.array_equal(res.crd, A.crd) and np.array_equal(res.val, A.val)
    res = oracle_mod.spgemm(eye, A)
    assert np.array_equal(res.pos, A.pos) and np.array_equal(res.crd, A.crd) and np.array_equal(res.val, A.val)
    perm = np.random.default_rng(3).permutation(40)
    Pm = CSR.from_coo(40, 40, np.arange(40), perm, np.ones(40))      # row r of P*A = row perm[r] of A
    res = oracle_mod.spgemm(Pm, A)
    for r in range(40):
        s, t = slice(res.pos[r], res.pos[r + 1]), slice(A.pos[perm[r]], A.pos[perm[r] + 1])
        assert np.array_equal(res.crd[s], A.crd[t]) and np.array_equal(res.val[s], A.val[t])


def test_transpose_identity(oracle_mod):
    A = random_csr(30, 50, 0.1, 21)
    B = random_csr(50, 20, 0.15, 22)
    C = oracle_mod.spgemm(A, B)
    Ct = oracle_mod.spgemm(B.transpose(), A.transpose())
    Cm = CSR(30, 20, C.pos, C.crd, C.val_ref).transpose()
    assert np.array_equal(Cm.pos, Ct.pos) and np.array_equal(Cm.crd, Ct.crd)
    assert np.allclose(Cm.val, Ct.val_ref, rtol=1e-14, atol=1e-300)


@pytest.mark.parametrize("cfg", ["uniform8", "rmat18", "stencil64", "wide26"])
def test_row_sums_identity_on_reduced_configs(oracle_mod, cfg):
    """C*1 = A*(B*1): a value check that never forms C any other way."""
    c = config_inputs(cfg, reduced=True)
    A, B = c["A"], c["B"]
    res = oracle_mod.spgemm(A, B, threads=2)
    b1 = np.add.reduceat(np.append(B.val.astype(np.float64), 0.0), np.minimum(B.pos[:-1], B.nnz)) * (np.diff(B.pos) > 0)
    picked = b1[A.crd] * A.val.astype(np.float64)
    ab1 = np.bincount(rows_of(A.pos), weights=picked, minlength=A.nrows)
    c1 = np.bincount(rows_of(res.pos), weights=res.val_ref, minlength=A.nrows)
    scale = np.bincount(rows_of(res.pos), weights=res.abs, minlength=A.nrows)
    assert (np.abs(c1 - ab1) <= 1e-13 * scale + 1e-300).all()
    check_sorted_unique(res.pos, res.crd)


# ---------------------------------------------------------------- library cross-check
@pytest.mark.parametrize("cfg", ["uniform8", "rmat18", "stencil64", "wide26"])
def test_against_scipy_on_reduced_configs(oracle_mod, cfg):
    c = config_inputs(cfg, reduced=True)
    A, B = c["A"], c["B"]
    res = oracle_mod.spgemm(A, B)
    # scipy drops nothing here as long as values do not cancel to exact zero; compare patterns
    # with all-ones values (so no cancellation) and values with the real ones.
    ones = lambda M: sp.csr_matrix((np.ones(M.nnz), M.crd, M.pos), shape=(M.nrows, M.ncols))
    real = lambda M: sp.csr_matrix((M.val.astype(np.float64), M.crd, M.pos), shape=(M.nrows, M.ncols))
    S = (ones(A) @ ones(B)).tocsr()
    S.sort_indices()
    assert np.array_equal(S.indptr, res.pos) and np.array_equal(S.indices, res.crd)
    V = (real(A) @ real(B)).tocsr()
    V.sort_indices()
    got = sp.csr_matrix((res.val_ref, res.crd, res.pos), shape=V.shape)
    diff = abs(got - V)
    bound = sp.csr_matrix((res.abs, res.crd, res.pos), shape=V.shape) * 1e-13
    assert (diff - bound).max() <= 1e-300


def test_row_subset_and_threads_agree(oracle_mod):
    A = rmat_csr(10, 8, 5)
    full = oracle_mod.spgemm(A, A)
    par = oracle_mod.spgemm(A, A, threads=4)
    for f in ("pos", "crd", "val", "val_ref", "abs", "products"):
        assert np.array_equal(getattr(full, f), getattr(par, f))
    rows = np.array([700, 3, 3, 512, 0, 1023])
    sub = oracle_mod.spgemm(A, A, rows=rows)
    for t, r in enumerate(rows):
        s, u = slice(sub.pos[t], sub.pos[t + 1]), slice(full.pos[r], full.pos[r + 1])
        assert np.array_equal(sub.crd[s], full.crd[u]) and np.array_equal(sub.val[s], full.val[u])
        assert sub.products[t] == full.products[r]


# ---------------------------------------------------------------- Algorithm 1 restatements
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_algorithm1_rowwise_any_capacity(oracle_mod, seed):
    A = random_csr(24, 30, 0.2, seed, empty_row_frac=0.1)
    B = random_csr(30, 26, 0.25, seed + 50)
    ref = oracle_mod.spgemm(A, B)
    P = int(ref.products.max())
    for cap in (1, 2, 3, 7, P, P + 1):
        got = oracle_mod.ism_rowwise(A, B, cap)
        assert np.array_equal(got.pos, ref.pos) and np.array_equal(got.crd, ref.crd)
        assert (np.abs(got.val - ref.val_ref) <= 1e-14 * ref.abs).all()
    # small integers: any capacity gives exactly the same sums, so a component that the
    # full-flush-reinsert protocol lost or counted twice would show
    Ai = CSR(A.nrows, A.ncols, A.pos, A.crd, np.round(A.val * 8))
    Bi = CSR(B.nrows, B.ncols, B.pos, B.crd, np.round(B.val * 8))
    ref = oracle_mod.spgemm(Ai, Bi)
    for cap in (1, 2, 3, 5):
        assert np.array_equal(oracle_mod.ism_rowwise(Ai, Bi, cap).val, ref.val)


@pytest.mark.parametrize("seed", [0, 1])
def test_algorithm1_outer_product_order(oracle_mod, seed):
    """Sum over k of outer products, second-order workspace, COO->CSR compress: the paper's
    running example computes the same matrix as the row-wise definition."""
    A = random_csr(20, 17, 0.25, seed + 7, empty_row_frac=0.15)
    B = random_csr(17, 23, 0.25, seed + 70, empty_row_frac=0.15)
    ref = oracle_mod.spgemm(A, B)
    total = int(ref.products.sum())
    for cap in (1, 2, 3, 16, total, total + 1):
        got = oracle_mod.ism_outer(A, B, cap)
        assert np.array_equal(got.pos, ref.pos) and np.array_equal(got.crd, ref.crd)
        assert (np.abs(got.val - ref.val_ref) <= 1e-14 * ref.abs).all()
    A, B, cr, cc, cv, _ = read_hand_case("hand_dedupe_4x4.txt")
    got = oracle_mod.ism_outer(A, B, 2)
    assert np.array_equal(rows_of(got.pos), cr) and np.array_equal(got.crd, cc) and np.array_equal(got.val, cv)


# ---------------------------------------------------------------- TTM
@pytest.mark.parametrize("dims,nnz,seed", [((4, 5, 6), 30, 0), ((8, 8, 8), 100, 1), ((3, 9, 16), 60, 2), ((16, 16, 16), 500, 3)])
def test_ttm_against_dense_einsum(oracle_mod, dims, nnz, seed):
    A = uniform_csf3(dims, nnz, seed)
    B = random_csr(dims[2], 7, 0.4, seed + 5, empty_row_frac=0.3)
    assert csf3_is_canonical(A)
    res = oracle_mod.ttm(A, B)
    ref = np.einsum("ijk,kl->ijl", A.to_dense(), B.to_dense())
    pat = np.einsum("ijk,kl->ijl", (A.to_dense() != 0).astype(np.int64), B.pattern_dense().astype(np.int64)) > 0
    C = CSF3(dims[:2] + (7,), res.pos0, res.crd0, res.pos1, res.crd1, res.pos2, res.crd2, res.val_ref)
    assert csf3_is_canonical(C)                 # sorted, unique, no empty fibre at any level
    i, j, l, v = C.to_coo()
    got = np.zeros(pat.shape, dtype=bool)
    got[i, j, l] = True
    assert np.array_equal(got, pat)
    assert np.allclose(C.to_dense(), ref, rtol=1e-13, atol=1e-15)


def test_ttm_drops_empty_fibres_and_slices(oracle_mod):
    # B rows 1 and 2 are empty.  Fibre (0,0) uses only k=1 -> dropped; slice i=1 uses only k in {1,2} -> dropped.
    A = CSF3.from_coo((3, 3, 4), [0, 0, 1, 1, 2], [0, 2, 0, 1, 1], [1, 0, 1, 2, 3], [1.0, 2.0, 3.0, 4.0, 5.0])
    B = CSR.from_coo(4, 5, [0, 0, 3], [4, 1, 2], [10.0, 20.0, 30.0])
    res = oracle_mod.ttm(A, B)
    assert list(res.crd0) == [0, 2] and list(res.pos1) == [0, 1, 2]
    assert list(res.crd1) == [2, 1] and list(res.pos2) == [0, 2, 3]
    assert list(res.crd2) == [1, 4, 2] and list(res.val) == [40.0, 20.0, 150.0]
    assert list(res.products) == [0, 2, 0, 0, 1]


def test_ttm_is_spgemm_on_fibres(oracle_mod):
    c = config_inputs("ttm4096", reduced=True)
    A, B = c["A"], c["B"]
    res = oracle_mod.ttm(A, B)
    flat = oracle_mod.spgemm(A.fibres_as_csr(), B)
    assert np.array_equal(res.crd2, flat.crd) and np.array_equal(res.val, flat.val)
    # every B row has 8 entries, so no fibre disappears and the upper levels are A's
    assert np.array_equal(res.crd0, A.crd0) and np.array_equal(res.pos1, A.pos1) and np.array_equal(res.crd1, A.crd1)
    assert res.products.sum() == 8 * A.nnz


# ---------------------------------------------------------------- generators
def test_generators_are_canonical_and_seeded():
    for cfg in ("uniform8", "rmat18", "stencil64", "wide26"):
        a = config_inputs(cfg, seed=3, reduced=True)
        b = config_inputs(cfg, seed=3, reduced=True)
        assert csr_is_canonical(a["A"]) and csr_is_canonical(a["B"])
        assert np.array_equal(a["A"].crd, b["A"].crd) and np.array_equal(a["A"].val, b["A"].val)
    u = uniform_rows_csr(500, 64, 8, 9)
    assert (np.diff(u.pos) == 8).all() and csr_is_canonical(u)
    r = rmat_csr(10, 16, 2)
    deg = np.diff(r.pos)
    assert deg.max() > 20 * np.median(deg[deg > 0])     # skewed degrees
    assert r.val.min() >= -1 and r.val.max() <= 1


# ---------------------------------------------------------------- higher-order scatters (Sec. 7.3)
def _dense_coo(d):
    idx = np.argwhere(d != 0)
    return idx, d[tuple(idx.T)]


@pytest.mark.parametrize("dims,nnz,seed", [((4, 5, 6), 30, 1), ((7, 3, 8), 60, 2), ((9, 9, 9), 200, 3)])
def test_higher_order_scatters_against_dense_einsum(oracle_mod, dims, nnz, seed):
    """Each of the three expressions against numpy's einsum on dense copies: structure = where the
    boolean einsum of the patterns is true, values within rounding of the dense result."""
    from workloads import uniform_csf3
    B = uniform_csf3(dims, nnz, seed)
    Bd = B.to_dense()
    L = 7
    cases = [
        ("spttm", oracle_mod.spttm, "kij,kl->ijl", [random_csr(dims[0], L, 0.4, seed + 10, empty_row_frac=0.2)]),
        ("spttm_i", oracle_mod.spttm_i, "kij,il->kjl", [random_csr(dims[1], L, 0.4, seed + 11, empty_row_frac=0.2)]),
        ("spmttkrp", oracle_mod.spmttkrp, "kli,kj,lj->ij", [random_csr(dims[0], L, 0.5, seed + 12), random_csr(dims[1], L, 0.5, seed + 13)]),
    ]
    for name, fn, spec, mats in cases:
        res = fn(B, *mats)
        dense = [m.to_dense() for m in mats]
        want = np.einsum(spec, Bd, *dense)
        pat = np.einsum(spec, (Bd != 0).astype(np.int64), *[(m.pattern_dense()).astype(np.int64) for m in mats]) > 0
        got_pat = np.zeros(want.shape, dtype=bool)
        got_pat[tuple(res.crd.T)] = True
        assert np.array_equal(got_pat, pat), name
        assert res.nnz == pat.sum(), name
        # sorted lexicographically and unique
        order = np.lexsort(tuple(res.crd.T[::-1]))
        assert np.array_equal(order, np.arange(res.nnz)), name
        scale = np.einsum(spec, np.abs(Bd), *[np.abs(x) for x in dense])
        for v in (res.val, res.val_ref):
            d = np.zeros(want.shape)
            d[tuple(res.crd.T)] = v
            assert (np.abs(d - want) <= 1e-13 * scale + 1e-300).all(), name
        dab = np.zeros(want.shape)
        dab[tuple(res.crd.T)] = res.abs
        assert np.allclose(dab, scale * pat, rtol=1e-12, atol=0), name
        assert res.products == int(np.einsum(spec, (Bd != 0).astype(np.int64), *[(m.pattern_dense()).astype(np.int64) for m in mats]).sum()), name


def test_higher_order_hand_case(oracle_mod):
    """B(k,i,j) with three entries, worked by hand.
    SpTTM  A(i,j,l) = B(k,i,j) C(k,l):   B(0,1,2)=2, B(1,1,2)=3, B(1,0,0)=5; C(0,1)=10, C(1,1)=100, C(1,3)=7
        -> A(0,0,1)=500, A(0,0,3)=35, A(1,2,1)=2*10+3*100=320, A(1,2,3)=21
    SpTTM-I A(k,j,l) = B(k,i,j) C(i,l) with the same C read as C(i,l):
        -> k=0: B(0,1,2)*C(1,:) -> A(0,2,1)=200, A(0,2,3)=14; k=1: B(1,0,0)*C(0,:) -> A(1,0,1)=50; B(1,1,2)*C(1,:) -> A(1,2,1)=300, A(1,2,3)=21
    SpMTTKRP A(i,j) = B(k,l,i) C(k,j) D(l,j) with B read as B(k,l,i), D = C:
        B(0,1,2): C(0,:)={1:10}, D(1,:)={1:100,3:7} -> A(2,1)=2*10*100=2000
        B(1,0,0): C(1,:)={1:100,3:7}, D(0,:)={1:10} -> A(0,1)=5*100*10=5000
        B(1,1,2): C(1,:), D(1,:) -> A(2,1)+=3*100*100=30000, A(2,3)=3*7*7=147
    """
    from workloads import CSF3
    B = CSF3.from_coo((2, 2, 3), [0, 1, 1], [1, 1, 0], [2, 2, 0], [2.0, 3.0, 5.0])
    C = CSR.from_coo(2, 4, [0, 1, 1], [1, 1, 3], [10.0, 100.0, 7.0])
    r = oracle_mod.spttm(B, C)
    assert r.crd.tolist() == [[0, 0, 1], [0, 0, 3], [1, 2, 1], [1, 2, 3]] and r.val.tolist() == [500.0, 35.0, 320.0, 21.0]
    assert r.products == 5
    r = oracle_mod.spttm_i(B, C)
    assert r.crd.tolist() == [[0, 2, 1], [0, 2, 3], [1, 0, 1], [1, 2, 1], [1, 2, 3]]
    assert r.val.tolist() == [200.0, 14.0, 50.0, 300.0, 21.0]
    r = oracle_mod.spmttkrp(B, C, C)
    assert r.crd.tolist() == [[0, 1], [2, 1], [2, 3]] and r.val.tolist() == [5000.0, 32000.0, 147.0]
    assert r.products == 4
